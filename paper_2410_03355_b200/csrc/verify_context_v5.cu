// Fused context kernel, variant 5: temperature 1 compiled out = 1, JSD bound = 0, top-k thresholds = 1.
#define LANTERN_VARIANT_TONE true
#define LANTERN_VARIANT_JSD false
#define LANTERN_VARIANT_TOPK true
#define LANTERN_VARIANT_NAME launch_context_v5
#include "verify_context_variant.cuh"
