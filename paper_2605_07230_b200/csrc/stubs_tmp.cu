#include "cascade_internal.h"
int launch_tree_attn_bf16(cascade_ctx*, const cascade_tree*, const __nv_bfloat16*, const __nv_bfloat16*, const __nv_bfloat16*, int, const int32_t*, const __nv_bfloat16*, const __nv_bfloat16*, __nv_bfloat16*, float, cudaStream_t) { return CASCADE_ERR_UNSUPPORTED_SHAPE; }
