// Fused context kernel, variant 6: temperature 1 compiled out = 0, JSD bound = 1, top-k thresholds = 1.
#define LANTERN_VARIANT_TONE false
#define LANTERN_VARIANT_JSD true
#define LANTERN_VARIANT_TOPK true
#define LANTERN_VARIANT_NAME launch_context_v6
#include "verify_context_variant.cuh"
