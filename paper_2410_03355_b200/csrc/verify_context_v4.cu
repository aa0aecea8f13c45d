// Fused context kernel, variant 4: temperature 1 compiled out = 0, JSD bound = 0, top-k thresholds = 1.
#define LANTERN_VARIANT_TONE false
#define LANTERN_VARIANT_JSD false
#define LANTERN_VARIANT_TOPK true
#define LANTERN_VARIANT_NAME launch_context_v4
#include "verify_context_variant.cuh"
