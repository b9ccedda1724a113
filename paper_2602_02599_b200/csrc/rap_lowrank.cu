// Low-rank comparator: latent K cache rebuilt to full width and rotated at every step.
#include "rap_internal.h"

rap_status rap_launch_lowrank_attn(rap_ctx* ctx, const rap_lowrank_args& a, cudaStream_t st) {
  (void)ctx; (void)a; (void)st;
  return RAP_EUNSUPPORTED;
}
