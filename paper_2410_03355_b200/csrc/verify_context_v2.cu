// Fused context kernel, variant 2: temperature 1 compiled out = 0, JSD bound = 1, top-k thresholds = 0.
#define LANTERN_VARIANT_TONE false
#define LANTERN_VARIANT_JSD true
#define LANTERN_VARIANT_TOPK false
#define LANTERN_VARIANT_NAME launch_context_v2
#include "verify_context_variant.cuh"
