// Launch side of the tensor-core scan over a quantised cache (see rap_attn_q8_kernel.cuh).
#include "rap_internal.h"

rap_status rap_launch_attn_q8_mma(rap_ctx* ctx, const rap_attn_args& a, int n_split_req, cudaStream_t st) {
  (void)ctx; (void)a; (void)n_split_req; (void)st;
  return RAP_EUNSUPPORTED;
}
