// Fused context kernel, variant 1: temperature 1 compiled out = 1, JSD bound = 0, top-k thresholds = 0.
#define LANTERN_VARIANT_TONE true
#define LANTERN_VARIANT_JSD false
#define LANTERN_VARIANT_TOPK false
#define LANTERN_VARIANT_NAME launch_context_v1
#include "verify_context_variant.cuh"
