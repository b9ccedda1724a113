// tcgen05 projection GEMM (bf16 in, fp32 accumulate in tensor memory).
#include "rap_internal.h"

rap_status rap_launch_proj_tc(rap_ctx* ctx, const rap_proj_args& a, int* ksplit_out, cudaStream_t st) {
  (void)ctx; (void)a; (void)ksplit_out; (void)st;
  return RAP_EUNSUPPORTED;   // the caller falls back to the CUDA-core GEMM
}
