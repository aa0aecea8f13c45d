// Fused context kernel, variant 7: temperature 1 compiled out = 1, JSD bound = 1, top-k thresholds = 1.
#define LANTERN_VARIANT_TONE true
#define LANTERN_VARIANT_JSD true
#define LANTERN_VARIANT_TOPK true
#define LANTERN_VARIANT_NAME launch_context_v7
#include "verify_context_variant.cuh"
