// Host side of the C ABI: context life cycle, argument validation, table construction
// (Algorithm 2, selection step, Eq. 6, Eq. 3) and the per-layer decode loop.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <new>
#include <numeric>

#include "rap_internal.h"

namespace {

bool desc_ok(const rap_model_desc& d) {
  if (d.n_layers < 1 || d.hidden < 1 || d.n_q_heads < 1 || d.n_kv_heads < 1) return false;
  if (d.head_dim < 2 || (d.head_dim & 1) || d.head_dim > 256) return false;
  if (d.n_q_heads % d.n_kv_heads) return false;
  if (d.n_q_heads / d.n_kv_heads > RAP_MAX_GROUP) return false;
  if (!(d.rope_theta > 1.0) || !std::isfinite(d.rope_theta)) return false;
  if (d.pairing != RAP_PAIR_HALF && d.pairing != RAP_PAIR_ADJACENT) return false;
  if (d.dtype != RAP_F32 && d.dtype != RAP_BF16) return false;
  if (d.max_batch < 1 || d.max_rows < 1) return false;
  if ((d.hidden * rap_elem_bytes(d.dtype)) % 16) return false;   // rows of X / W~ stay 16-byte aligned
  return true;
}

void free_all(rap_ctx* c) {
  if (c->d_status) cudaFree(c->d_status);
  if (c->d_attn_ws) cudaFree(c->d_attn_ws);
  if (c->d_unit_cnt) cudaFree(c->d_unit_cnt);
  if (c->d_proj_ws) cudaFree(c->d_proj_ws);
  if (c->d_proj_cnt) cudaFree(c->d_proj_cnt);
  if (c->d_stage_x) cudaFree(c->d_stage_x);
  if (c->d_stage_out) cudaFree(c->d_stage_out);
  if (c->d_stage_q) cudaFree(c->d_stage_q);
  if (c->d_oproj_x) cudaFree(c->d_oproj_x);
  if (c->d_pf_v) cudaFree(c->d_pf_v);
  if (c->d_lr_k) cudaFree(c->d_lr_k);
  if (c->d_lr_cs) cudaFree(c->d_lr_cs);
  if (c->h_tables) cudaFreeHost(c->h_tables);
  if (c->copy_in) cudaStreamDestroy((cudaStream_t)c->copy_in);
  if (c->copy_out) cudaStreamDestroy((cudaStream_t)c->copy_out);
  if (c->ev_in) cudaEventDestroy((cudaEvent_t)c->ev_in);
  if (c->ev_mid) cudaEventDestroy((cudaEvent_t)c->ev_mid);
  for (cudaEvent_t e : c->prof_ev) cudaEventDestroy(e);
}

}  // namespace

extern "C" {

const char* rap_status_string(rap_status s) {
  switch (s) {
    case RAP_OK: return "RAP_OK";
    case RAP_EINVAL: return "RAP_EINVAL: invalid argument";
    case RAP_ESHAPE: return "RAP_ESHAPE: shape outside what the context was created for";
    case RAP_ECAPACITY: return "RAP_ECAPACITY: cache capacity exceeded";
    case RAP_EALIGN: return "RAP_EALIGN: pointer not 16-byte aligned or S_cap not a multiple of 8";
    case RAP_EUNSUPPORTED: return "RAP_EUNSUPPORTED: not implemented in this build";
    case RAP_ECUDA: return "RAP_ECUDA: CUDA runtime error";
    case RAP_ETIMEOUT: return "RAP_ETIMEOUT: bounded device wait gave up";
    case RAP_ESTATE: return "RAP_ESTATE: rap_build_tables has not run on this context";
    case RAP_EBOUNDS: return "RAP_EBOUNDS: an index check of the bounds-checking build failed";
  }
  return "unknown rap_status";
}

const char* rap_last_cuda_error(const rap_ctx* ctx) { return ctx ? ctx->cuda_error.c_str() : ""; }

int64_t rap_kernel_launch_count(const rap_ctx* ctx) { return ctx ? ctx->launches : 0; }

rap_status rap_set_attn_variant(rap_ctx* ctx, int32_t variant) {
  if (!ctx || variant < 0 || variant > 4) return RAP_EINVAL;
  ctx->attn_variant = variant;
  return RAP_OK;
}

rap_status rap_debug_claim_scan_workspace(rap_ctx* ctx, int64_t n_floats) {
  if (!ctx || n_floats < 0) return RAP_EINVAL;
  ctx->dbg_ws_floats = n_floats;
  return RAP_OK;
}

rap_status rap_debug_arm_wait_timeout(rap_ctx* ctx) {
  if (!ctx) return RAP_EINVAL;
  ctx->dbg_arm_timeout = 1;
  return RAP_OK;
}

rap_status rap_debug_set_scan_pieces(rap_ctx* ctx, int32_t piece_tiles, int32_t frac_x256) {
  if (!ctx || piece_tiles < -1 || frac_x256 < 0 || frac_x256 > 256) return RAP_EINVAL;
  ctx->dbg_dyn_piece = piece_tiles;
  ctx->dbg_dyn_frac = frac_x256;
  return RAP_OK;
}

rap_status rap_set_proj_variant(rap_ctx* ctx, int32_t variant) {
  if (!ctx || variant < 0 || variant > 1) return RAP_EINVAL;
  ctx->proj_variant = variant;
  return RAP_OK;
}

rap_status rap_retained_counts(double rho, int32_t head_dim, int32_t* n_pairs, int32_t* n_vch) {
  if (!n_pairs || !n_vch || !(rho > 0.0) || rho > 1.0 || head_dim < 2 || (head_dim & 1)) return RAP_EINVAL;
  *n_pairs = (int32_t)std::floor(rho * (double)(head_dim / 2) + 0.5);
  *n_vch = (int32_t)std::floor(rho * (double)head_dim + 0.5);
  return RAP_OK;
}

size_t rap_cache_elem_offset(int32_t n_kv_heads, int32_t S_cap, int32_t W, int32_t b, int32_t h,
                             int32_t pos, int32_t c) {
  return (((size_t)b * (size_t)n_kv_heads + (size_t)h) * (size_t)S_cap + (size_t)pos) * (size_t)W + (size_t)c;
}

rap_status rap_budget_alloc(int32_t n_layers, int32_t n_kv_heads, int32_t head_dim, const double* k_pair_scores,
                            double rho, int32_t* n_pairs, int32_t* n_vch) {
  if (!k_pair_scores || !n_pairs || !n_vch || n_layers < 1 || n_kv_heads < 1 || head_dim < 2 || (head_dim & 1) ||
      !(rho > 0.0) || rho > 1.0)
    return RAP_EINVAL;
  const int L = n_layers, P = head_dim / 2;
  const size_t per_layer = (size_t)n_kv_heads * P;
  std::vector<double> sigma(L);
  for (int l = 0; l < L; ++l) {
    double s = 0.0;
    for (size_t i = 0; i < per_layer; ++i) {
      const double v = k_pair_scores[(size_t)l * per_layer + i];
      if (!std::isfinite(v) || v < 0.0) return RAP_EINVAL;
      s += v;
    }
    sigma[l] = s / (double)per_layer;
  }
  long total = (long)std::floor(rho * (double)P * (double)L + 0.5);
  total = std::min<long>(std::max<long>(total, L), (long)P * L);
  // water-filling: layers whose proportional share leaves [1, P] are pinned to the bound, the rest re-share
  std::vector<int> pinned(L, 0);
  std::vector<double> target(L, 0.0);
  for (;;) {
    long rest = total;
    double ssum = 0.0;
    int n_free = 0;
    for (int l = 0; l < L; ++l) {
      if (pinned[l]) rest -= pinned[l];
      else { ssum += sigma[l]; ++n_free; }
    }
    if (n_free == 0) break;
    bool over = false, under = false;
    for (int l = 0; l < L; ++l) {
      if (pinned[l]) continue;
      target[l] = ssum > 0.0 ? (double)rest * sigma[l] / ssum : (double)rest / (double)n_free;
      over |= target[l] > (double)P;
      under |= target[l] < 1.0;
    }
    if (over) {
      for (int l = 0; l < L; ++l) if (!pinned[l] && target[l] > (double)P) pinned[l] = P;
    } else if (under) {
      for (int l = 0; l < L; ++l) if (!pinned[l] && target[l] < 1.0) pinned[l] = 1;
    } else {
      break;
    }
  }
  std::vector<int> free_layers;
  long have = 0;
  for (int l = 0; l < L; ++l) {
    if (pinned[l]) n_pairs[l] = pinned[l];
    else { n_pairs[l] = (int32_t)std::floor(target[l]); free_layers.push_back(l); }
    have += n_pairs[l];
  }
  // the units lost to flooring go to the largest fractional parts (ties: lower layer)
  std::stable_sort(free_layers.begin(), free_layers.end(), [&](int a, int b) {
    return (target[a] - std::floor(target[a])) > (target[b] - std::floor(target[b]));
  });
  long missing = total - have;
  for (size_t i = 0, spins = 0; missing > 0 && !free_layers.empty() && spins < 4 * free_layers.size() + (size_t)total; ++i, ++spins) {
    const int l = free_layers[i % free_layers.size()];
    if (n_pairs[l] < P) { ++n_pairs[l]; --missing; }
  }
  for (int l = 0; l < L; ++l) n_vch[l] = 2 * n_pairs[l];
  return RAP_OK;
}

rap_status rap_create(const rap_model_desc* desc, rap_ctx** out) {
  if (!desc || !out) return RAP_EINVAL;
  *out = nullptr;
  if (!desc_ok(*desc)) return RAP_EINVAL;
  rap_ctx* c = new (std::nothrow) rap_ctx();
  if (!c) return RAP_EINVAL;
  c->desc = *desc;
  c->n_pairs.assign(desc->n_layers, 0);
  c->n_vch.assign(desc->n_layers, 0);
  // From here on errors are reported through a context the caller can inspect and destroy.
  *out = c;
  RAP_CUDA_TRY(c, cudaGetDevice(&c->device));
  cudaDeviceProp prop;
  RAP_CUDA_TRY(c, cudaGetDeviceProperties(&prop, c->device));
  if (prop.major != 10) {
    c->cuda_error = "device is not sm_100 (B200) -- this library carries sm_100a code only";
    return RAP_ECUDA;
  }
  c->sm_count = prop.multiProcessorCount;
  const rap_model_desc& d = c->desc;
  const size_t e = rap_elem_bytes(d.dtype);
  size_t n_out_max = (size_t)(d.n_q_heads + 2 * d.n_kv_heads) * d.head_dim;
  if ((size_t)d.hidden > n_out_max) n_out_max = d.hidden;       // the workspace also serves rap_out_proj
  c->attn_ws_bytes = (size_t)d.max_batch * d.n_q_heads * RAP_MAX_SPLIT * (size_t)(d.head_dim + 2) * sizeof(float);
  // full-size fp32 results for any row count, plus room for reduction splits on decode-sized calls
  {
    const size_t small_rows = d.max_rows < 256 ? d.max_rows : 256;
    const size_t a = (size_t)d.max_rows * n_out_max * sizeof(float);
    const size_t b = small_rows * n_out_max * sizeof(float) * RAP_MAX_KSPLIT;
    c->proj_ws_bytes = a > b ? a : b;
  }
  c->stage_x_bytes = (size_t)d.n_layers * d.max_batch * d.hidden * e;
  c->stage_out_bytes = (size_t)d.n_layers * d.max_batch * d.n_q_heads * d.head_dim * sizeof(float);
  RAP_CUDA_TRY(c, cudaMalloc(&c->d_status, 2 * sizeof(int32_t)));
  RAP_CUDA_TRY(c, cudaMemset(c->d_status, 0, 2 * sizeof(int32_t)));
  RAP_CUDA_TRY(c, cudaMalloc(&c->d_attn_ws, c->attn_ws_bytes));
  // two sets of unit arrival counters, then the two piece counters of the scans that hand out their last tiles at run time
  RAP_CUDA_TRY(c, cudaMalloc(&c->d_unit_cnt, (2 * (size_t)d.max_batch * d.n_kv_heads + 2) * sizeof(int32_t)));
  RAP_CUDA_TRY(c, cudaMemset(c->d_unit_cnt, 0, (2 * (size_t)d.max_batch * d.n_kv_heads + 2) * sizeof(int32_t)));
  RAP_CUDA_TRY(c, cudaMalloc(&c->d_proj_ws, c->proj_ws_bytes));
  c->proj_cnt_n = 4 * (int)((n_out_max + 127) / 128);
  RAP_CUDA_TRY(c, cudaMalloc(&c->d_proj_cnt, 2 * (size_t)c->proj_cnt_n * sizeof(int32_t)));
  RAP_CUDA_TRY(c, cudaMemset(c->d_proj_cnt, 0, 2 * (size_t)c->proj_cnt_n * sizeof(int32_t)));
  RAP_CUDA_TRY(c, cudaMalloc(&c->d_stage_x, c->stage_x_bytes));
  RAP_CUDA_TRY(c, cudaMalloc(&c->d_stage_out, c->stage_out_bytes));
  RAP_CUDA_TRY(c, cudaMalloc(&c->d_stage_q, (size_t)d.max_batch * d.n_q_heads * d.head_dim * e));
  RAP_CUDA_TRY(c, cudaMalloc(&c->d_oproj_x, (size_t)d.max_batch * d.n_q_heads * d.head_dim * sizeof(__nv_bfloat16)));
  const size_t units = (size_t)d.n_layers * d.n_kv_heads;
  c->h_tables_bytes = units * ((size_t)(d.head_dim / 2 + 2 * d.head_dim) * sizeof(int32_t) +
                               (size_t)(d.head_dim / 2) * sizeof(double));
  RAP_CUDA_TRY(c, cudaMallocHost(&c->h_tables, c->h_tables_bytes));
  {   // copy streams and events of rap_decode_step_host
    cudaStream_t s1, s2;
    cudaEvent_t e1, e2;
    RAP_CUDA_TRY(c, cudaStreamCreateWithFlags(&s1, cudaStreamNonBlocking));
    c->copy_in = s1;
    RAP_CUDA_TRY(c, cudaStreamCreateWithFlags(&s2, cudaStreamNonBlocking));
    c->copy_out = s2;
    RAP_CUDA_TRY(c, cudaEventCreateWithFlags(&e1, cudaEventDisableTiming));
    c->ev_in = e1;
    RAP_CUDA_TRY(c, cudaEventCreateWithFlags(&e2, cudaEventDisableTiming));
    c->ev_mid = e2;
  }
  return RAP_OK;
}

rap_status rap_destroy(rap_ctx* ctx) {
  if (!ctx) return RAP_EINVAL;
  if (ctx->tables_inflight) cudaStreamSynchronize((cudaStream_t)ctx->tables_stream);
  free_all(ctx);
  delete ctx;
  return RAP_OK;
}

// kc / rope_layer are NULL for an all-rotary model
// Shared by the three table builders.  Per layer the first R dims of a head are rotary (pairs inside that block,
// frequency theta^(-2i/R)) and Pr of the P kept pair slots hold rotated pairs; the other slots hold 2 (P - Pr)
// channels of the unrotated dims R..D-1 with frequency zero.  rap_build_tables: R = D, Pr = P everywhere;
// the hybrid form: R = 0, Pr = 0 on layers without RoPE; the partial form: R and Pr per layer from the caller.
// pair_freq (NULL, or [L][D/2]): the model's own frequency of every original pair, used instead of theta^(-2i/D).
static rap_status build_tables_impl(rap_ctx* ctx, const double* ks, const double* kc, const double* vs,
                                    const double* pair_freq, const int32_t* rope_layer, const int32_t* rot_dims, const int32_t* n_rot_pairs,
                                    const int32_t* n_pairs, const int32_t* n_vch,
                                    int32_t* d_k_pair_idx, int32_t* d_k_dim_idx, int32_t* d_v_idx, double* d_inv_freq,
                                    void* stream) {
  if (!ctx || !ks || !vs || !n_pairs || !n_vch || !d_k_pair_idx || !d_k_dim_idx || !d_v_idx || !d_inv_freq)
    return RAP_EINVAL;
  if (!rap_aligned16(d_k_pair_idx) || !rap_aligned16(d_k_dim_idx) || !rap_aligned16(d_v_idx) ||
      !rap_aligned16(d_inv_freq))
    return RAP_EALIGN;
  const rap_model_desc& d = ctx->desc;
  const int L = d.n_layers, H = d.n_kv_heads, D = d.head_dim, half = D / 2;
  std::vector<int> rot(L), prot(L);
  for (int l = 0; l < L; ++l) {
    if (n_pairs[l] < 1 || n_pairs[l] > half || n_vch[l] < 1 || n_vch[l] > D) return RAP_EINVAL;
    rot[l] = rot_dims ? rot_dims[l] : (rope_layer && !rope_layer[l]) ? 0 : D;
    prot[l] = rot_dims ? n_rot_pairs[l] : (rope_layer && !rope_layer[l]) ? 0 : n_pairs[l];
    const int chans = 2 * (n_pairs[l] - prot[l]);
    if (rot[l] < 0 || rot[l] > D || (rot[l] & 1) || prot[l] < 0 || prot[l] > rot[l] / 2 || chans < 0 ||
        chans > D - rot[l] || (chans > 0 && !kc))
      return RAP_EINVAL;
  }
  const size_t units = (size_t)L * H;
  for (size_t i = 0; i < units * half; ++i) if (std::isnan(ks[i])) return RAP_EINVAL;
  for (size_t i = 0; i < units * D; ++i) if (std::isnan(vs[i])) return RAP_EINVAL;
  if (kc) for (size_t i = 0; i < units * D; ++i) if (std::isnan(kc[i])) return RAP_EINVAL;
  if (pair_freq) for (size_t i = 0; i < (size_t)L * half; ++i) if (!std::isfinite(pair_freq[i])) return RAP_EINVAL;
  cudaStream_t st = (cudaStream_t)stream;
  if (ctx->tables_inflight) {
    RAP_CUDA_TRY(ctx, cudaStreamSynchronize((cudaStream_t)ctx->tables_stream));
    ctx->tables_inflight = false;
  }
  double* h_freq = (double*)ctx->h_tables;          // doubles first so they stay 8-byte aligned
  int32_t* h_pair = (int32_t*)(h_freq + units * half);
  int32_t* h_dim = h_pair + units * half;
  int32_t* h_v = h_dim + units * D;
  std::fill(h_pair, h_pair + units * half, -1);
  std::fill(h_dim, h_dim + units * D, -1);
  std::fill(h_v, h_v + units * D, -1);
  std::fill(h_freq, h_freq + units * half, 0.0);

  std::vector<int32_t> order;
  auto top_k = [&order](const double* s, int n, int k, int32_t* dst) {
    order.resize(n);
    std::iota(order.begin(), order.end(), 0);
    // larger score first; equal scores keep the lower index first
    std::stable_sort(order.begin(), order.end(), [s](int32_t a, int32_t b) { return s[a] > s[b]; });
    std::sort(order.begin(), order.begin() + k);
    std::copy(order.begin(), order.begin() + k, dst);
  };
  for (int l = 0; l < L; ++l) {
    const int P = n_pairs[l], dv = n_vch[l];
    for (int h = 0; h < H; ++h) {
      const size_t u = (size_t)l * H + h;
      const int R = rot[l], Pr = prot[l];
      int32_t* pr = h_pair + u * half;
      if (Pr > 0) top_k(ks + u * half, R / 2, Pr, pr);
      for (int c = 0; c < Pr; ++c) {
        const int i = pr[c];
        if (d.pairing == RAP_PAIR_HALF) {
          h_dim[u * D + 2 * c] = i;
          h_dim[u * D + 2 * c + 1] = i + R / 2;
        } else {
          h_dim[u * D + 2 * c] = 2 * i;
          h_dim[u * D + 2 * c + 1] = 2 * i + 1;
        }
        h_freq[u * half + c] = pair_freq ? pair_freq[(size_t)l * half + i] : std::pow(d.rope_theta, -2.0 * (double)i / (double)R);
      }
      if (P > Pr) {
        // unrotated dims: plain channel pruning; their slots keep frequency zero (identity rotation)
        int32_t* ch = h_dim + u * D + 2 * Pr;
        top_k(kc + u * D + R, D - R, 2 * (P - Pr), ch);
        for (int c = 0; c < 2 * (P - Pr); ++c) ch[c] += R;
      }
      top_k(vs + u * D, D, dv, h_v + u * D);
    }
  }
  RAP_CUDA_TRY(ctx, cudaMemcpyAsync(d_k_pair_idx, h_pair, units * half * sizeof(int32_t), cudaMemcpyHostToDevice, st));
  RAP_CUDA_TRY(ctx, cudaMemcpyAsync(d_k_dim_idx, h_dim, units * D * sizeof(int32_t), cudaMemcpyHostToDevice, st));
  RAP_CUDA_TRY(ctx, cudaMemcpyAsync(d_v_idx, h_v, units * D * sizeof(int32_t), cudaMemcpyHostToDevice, st));
  RAP_CUDA_TRY(ctx, cudaMemcpyAsync(d_inv_freq, h_freq, units * half * sizeof(double), cudaMemcpyHostToDevice, st));
  ctx->tables_inflight = true;
  ctx->tables_stream = stream;
  for (int l = 0; l < L; ++l) {
    ctx->n_pairs[l] = n_pairs[l];
    ctx->n_vch[l] = n_vch[l];
  }
  ctx->tables_built = true;
  return RAP_OK;
}

rap_status rap_build_tables(rap_ctx* ctx, const double* ks, const double* vs, const int32_t* n_pairs,
                            const int32_t* n_vch, int32_t* d_k_pair_idx, int32_t* d_k_dim_idx,
                            int32_t* d_v_idx, double* d_inv_freq, void* stream) {
  return build_tables_impl(ctx, ks, nullptr, vs, nullptr, nullptr, nullptr, nullptr, n_pairs, n_vch, d_k_pair_idx, d_k_dim_idx, d_v_idx,
                           d_inv_freq, stream);
}

rap_status rap_build_tables_freq(rap_ctx* ctx, const double* ks, const double* vs, const double* pair_freq,
                                 const int32_t* n_pairs, const int32_t* n_vch, int32_t* d_k_pair_idx,
                                 int32_t* d_k_dim_idx, int32_t* d_v_idx, double* d_inv_freq, void* stream) {
  if (!pair_freq) return RAP_EINVAL;
  return build_tables_impl(ctx, ks, nullptr, vs, pair_freq, nullptr, nullptr, nullptr, n_pairs, n_vch, d_k_pair_idx, d_k_dim_idx,
                           d_v_idx, d_inv_freq, stream);
}

rap_status rap_build_tables_hybrid(rap_ctx* ctx, const double* ks, const double* kc, const double* vs,
                                   const int32_t* rope_layer, const int32_t* n_pairs, const int32_t* n_vch,
                                   int32_t* d_k_pair_idx, int32_t* d_k_dim_idx, int32_t* d_v_idx, double* d_inv_freq,
                                   void* stream) {
  if (!kc || !rope_layer) return RAP_EINVAL;
  return build_tables_impl(ctx, ks, kc, vs, nullptr, rope_layer, nullptr, nullptr, n_pairs, n_vch, d_k_pair_idx, d_k_dim_idx,
                           d_v_idx, d_inv_freq, stream);
}

rap_status rap_build_tables_partial(rap_ctx* ctx, const double* ks, const double* kc, const double* vs,
                                    const int32_t* rot_dims, const int32_t* n_rot_pairs, const int32_t* n_pairs,
                                    const int32_t* n_vch, int32_t* d_k_pair_idx, int32_t* d_k_dim_idx,
                                    int32_t* d_v_idx, double* d_inv_freq, void* stream) {
  if (!kc || !rot_dims || !n_rot_pairs) return RAP_EINVAL;
  return build_tables_impl(ctx, ks, kc, vs, nullptr, nullptr, rot_dims, n_rot_pairs, n_pairs, n_vch, d_k_pair_idx, d_k_dim_idx,
                           d_v_idx, d_inv_freq, stream);
}

rap_status rap_pack_weights(rap_ctx* ctx, int32_t layer, const void* d_wq, const void* d_wk, const void* d_wv,
                            const int32_t* d_k_dim_idx, const int32_t* d_v_idx, void* d_w_qkv,
                            const void* d_bq, const void* d_bk, const void* d_bv, void* d_bias, void* stream) {
  if (!ctx || !d_wq || !d_wk || !d_wv || !d_k_dim_idx || !d_v_idx || !d_w_qkv) return RAP_EINVAL;
  if (!ctx->tables_built) return RAP_ESTATE;
  if (layer < 0 || layer >= ctx->desc.n_layers) return RAP_EINVAL;
  const bool any_b = d_bq || d_bk || d_bv || d_bias, all_b = d_bq && d_bk && d_bv && d_bias;
  if (any_b && !all_b) return RAP_EINVAL;
  if (!rap_aligned16(d_wq) || !rap_aligned16(d_wk) || !rap_aligned16(d_wv) || !rap_aligned16(d_w_qkv))
    return RAP_EALIGN;
  return rap_launch_pack(ctx, layer, d_wq, d_wk, d_wv, d_k_dim_idx, d_v_idx, d_w_qkv, d_bq, d_bk, d_bv,
                         d_bias, (cudaStream_t)stream);
}

rap_status rap_pack_wo(rap_ctx* ctx, int32_t layer, const void* d_wo, const int32_t* d_v_idx, void* d_wo_tilde,
                       void* stream) {
  if (!ctx || !d_wo || !d_v_idx || !d_wo_tilde) return RAP_EINVAL;
  if (!ctx->tables_built) return RAP_ESTATE;
  if (layer < 0 || layer >= ctx->desc.n_layers) return RAP_EINVAL;
  if (!rap_aligned16(d_wo) || !rap_aligned16(d_wo_tilde) || !rap_aligned16(d_v_idx)) return RAP_EALIGN;
  return rap_launch_pack_wo(ctx, layer, d_wo, d_v_idx, d_wo_tilde, (cudaStream_t)stream);
}

rap_status rap_out_proj(rap_ctx* ctx, int32_t layer, int32_t T, const float* d_attn_out, const void* d_wo_tilde,
                        void* d_y, void* stream) {
  if (!ctx || !d_attn_out || !d_wo_tilde || !d_y) return RAP_EINVAL;
  if (!ctx->tables_built) return RAP_ESTATE;
  if (layer < 0 || layer >= ctx->desc.n_layers || T < 0) return RAP_EINVAL;
  if (T > ctx->desc.max_batch) return RAP_ESHAPE;
  if (!rap_aligned16(d_attn_out) || !rap_aligned16(d_wo_tilde) || !rap_aligned16(d_y)) return RAP_EALIGN;
  if (T == 0) return RAP_OK;
  return rap_launch_out_proj(ctx, layer, T, d_attn_out, d_wo_tilde, d_y, (cudaStream_t)stream);
}

rap_status rap_qkv_rope_append(rap_ctx* ctx, int32_t layer, int32_t T, const void* d_x, const void* d_w_qkv,
                               const void* d_bias, const int32_t* d_seq_id, const int32_t* d_pos,
                               const int32_t* d_slot, int32_t h_slot_max, const double* d_inv_freq,
                               void* d_q_out, void* d_k_cache, void* d_v_cache, int32_t B_cache,
                               int32_t S_cap, void* stream) {
  if (!ctx || !d_x || !d_w_qkv || !d_seq_id || !d_pos || !d_slot || !d_inv_freq || !d_q_out || !d_k_cache ||
      !d_v_cache)
    return RAP_EINVAL;
  if (!ctx->tables_built) return RAP_ESTATE;
  const rap_model_desc& d = ctx->desc;
  if (layer < 0 || layer >= d.n_layers || T < 0 || B_cache < 1 || S_cap < 1) return RAP_EINVAL;
  if (T > d.max_rows) return RAP_ESHAPE;
  if (S_cap % 8) return RAP_EALIGN;
  if (h_slot_max < 0) return RAP_EINVAL;
  if (h_slot_max >= S_cap) return RAP_ECAPACITY;
  if (!rap_aligned16(d_x) || !rap_aligned16(d_w_qkv) || !rap_aligned16(d_q_out) || !rap_aligned16(d_k_cache) ||
      !rap_aligned16(d_v_cache) || !rap_aligned16(d_inv_freq) || (d_bias && !rap_aligned16(d_bias)))
    return RAP_EALIGN;
  if (T == 0) return RAP_OK;
  rap_proj_args a;
  a.x = d_x; a.w = d_w_qkv; a.bias = d_bias;
  a.seq_id = d_seq_id; a.pos = d_pos; a.slot = d_slot;
  a.inv_freq = d_inv_freq + (size_t)layer * d.n_kv_heads * (d.head_dim / 2);
  a.q_out = d_q_out; a.k_cache = d_k_cache; a.v_cache = d_v_cache;
  a.T = T; a.hidden = d.hidden; a.Hq = d.n_q_heads; a.Hkv = d.n_kv_heads;
  a.P2 = 2 * ctx->n_pairs[layer]; a.dv = ctx->n_vch[layer]; a.half_dim = d.head_dim / 2;
  a.B_cache = B_cache; a.S_cap = S_cap; a.dtype = d.dtype;
  return rap_launch_qkv_rope_append(ctx, a, (cudaStream_t)stream);
}

rap_status rap_decode_attn(rap_ctx* ctx, int32_t layer, int32_t B, const void* d_q, const void* d_k_cache,
                           const void* d_v_cache, int32_t S_cap, const int32_t* d_seq_len,
                           int32_t h_seq_len_max, int32_t n_split, float* d_out, void* stream) {
  if (!ctx || !d_q || !d_k_cache || !d_v_cache || !d_seq_len || !d_out) return RAP_EINVAL;
  if (!ctx->tables_built) return RAP_ESTATE;
  const rap_model_desc& d = ctx->desc;
  if (layer < 0 || layer >= d.n_layers || B < 0 || S_cap < 1 || n_split < 0 || h_seq_len_max < 0) return RAP_EINVAL;
  if (B > d.max_batch || n_split > RAP_MAX_SPLIT) return RAP_ESHAPE;
  if (S_cap % 8) return RAP_EALIGN;
  if (h_seq_len_max > S_cap) return RAP_ECAPACITY;
  if (!rap_aligned16(d_q) || !rap_aligned16(d_k_cache) || !rap_aligned16(d_v_cache) || !rap_aligned16(d_out) ||
      !rap_aligned16(d_seq_len))
    return RAP_EALIGN;
  if (B == 0) return RAP_OK;
  rap_attn_args a;
  a.q = d_q; a.k = d_k_cache; a.v = d_v_cache; a.seq_len = d_seq_len; a.len_add = 0;
  a.B = B; a.Hq = d.n_q_heads; a.Hkv = d.n_kv_heads; a.P2 = 2 * ctx->n_pairs[layer]; a.dv = ctx->n_vch[layer];
  a.S_cap = S_cap; a.head_dim = d.head_dim; a.dtype = d.dtype; a.n_split = n_split; a.h_len_max = h_seq_len_max;
  a.out = d_out;
  return rap_launch_attn(ctx, a, (cudaStream_t)stream);
}

size_t rap_q8_row_bytes(int32_t W) { return W < 1 ? 0 : ((size_t)W + 2 + 3) / 4 * 4; }

rap_status rap_quantize_rows(rap_ctx* ctx, int32_t dtype_in, int64_t n_rows, int32_t W, const void* d_rows, void* d_q8,
                             void* stream) {
  if (!ctx || !d_rows || !d_q8) return RAP_EINVAL;
  if ((dtype_in != RAP_F32 && dtype_in != RAP_BF16) || n_rows < 0 || W < 1 || W > 65535) return RAP_EINVAL;
  if (!rap_aligned16(d_rows) || !rap_aligned16(d_q8)) return RAP_EALIGN;
  if (n_rows == 0) return RAP_OK;
  if ((n_rows + 7) / 8 > 0x7fffffffLL) return RAP_ESHAPE;
  return rap_launch_quantize_rows(ctx, dtype_in, n_rows, W, d_rows, d_q8, (cudaStream_t)stream);
}

rap_status rap_qkv_rope_append_q8(rap_ctx* ctx, int32_t layer, int32_t T, const void* d_x, const void* d_w_qkv,
                                  const void* d_bias, const int32_t* d_seq_id, const int32_t* d_pos, const int32_t* d_slot,
                                  int32_t h_slot_max, const double* d_inv_freq, void* d_q_out, void* d_k8, void* d_v8,
                                  int32_t B_cache, int32_t S_cap, void* stream) {
  if (!ctx || !d_x || !d_w_qkv || !d_seq_id || !d_pos || !d_slot || !d_inv_freq || !d_q_out || !d_k8 || !d_v8)
    return RAP_EINVAL;
  if (!ctx->tables_built) return RAP_ESTATE;
  const rap_model_desc& d = ctx->desc;
  if (layer < 0 || layer >= d.n_layers || T < 0 || B_cache < 1 || S_cap < 1) return RAP_EINVAL;
  if (T > d.max_rows) return RAP_ESHAPE;
  if (S_cap % 8) return RAP_EALIGN;
  if (h_slot_max < 0) return RAP_EINVAL;
  if (h_slot_max >= S_cap) return RAP_ECAPACITY;
  if (d.head_dim > 256) return RAP_EUNSUPPORTED;
  if (!rap_aligned16(d_x) || !rap_aligned16(d_w_qkv) || !rap_aligned16(d_q_out) || !rap_aligned16(d_k8) ||
      !rap_aligned16(d_v8) || !rap_aligned16(d_inv_freq) || (d_bias && !rap_aligned16(d_bias)))
    return RAP_EALIGN;
  if (T == 0) return RAP_OK;
  rap_proj_args a;
  a.x = d_x; a.w = d_w_qkv; a.bias = d_bias;
  a.seq_id = d_seq_id; a.pos = d_pos; a.slot = d_slot;
  a.inv_freq = d_inv_freq + (size_t)layer * d.n_kv_heads * (d.head_dim / 2);
  a.q_out = d_q_out; a.k_cache = d_k8; a.v_cache = d_v8;
  a.T = T; a.hidden = d.hidden; a.Hq = d.n_q_heads; a.Hkv = d.n_kv_heads;
  a.P2 = 2 * ctx->n_pairs[layer]; a.dv = ctx->n_vch[layer]; a.half_dim = d.head_dim / 2;
  a.B_cache = B_cache; a.S_cap = S_cap; a.dtype = d.dtype;
  return rap_launch_qkv_rope_append_q8(ctx, a, (cudaStream_t)stream);
}

rap_status rap_decode_attn_q8(rap_ctx* ctx, int32_t layer, int32_t B, const void* d_q, const void* d_k8, const void* d_v8,
                              int32_t S_cap, const int32_t* d_seq_len, int32_t h_seq_len_max, int32_t n_split, float* d_out,
                              void* stream) {
  if (!ctx || !d_q || !d_k8 || !d_v8 || !d_seq_len || !d_out) return RAP_EINVAL;
  if (!ctx->tables_built) return RAP_ESTATE;
  const rap_model_desc& d = ctx->desc;
  if (layer < 0 || layer >= d.n_layers || B < 0 || S_cap < 1 || n_split < 0 || h_seq_len_max < 0) return RAP_EINVAL;
  if (B > d.max_batch || n_split > RAP_MAX_SPLIT) return RAP_ESHAPE;
  if (S_cap % 8) return RAP_EALIGN;
  if (h_seq_len_max > S_cap) return RAP_ECAPACITY;
  if (!rap_aligned16(d_q) || !rap_aligned16(d_k8) || !rap_aligned16(d_v8) || !rap_aligned16(d_out) || !rap_aligned16(d_seq_len))
    return RAP_EALIGN;
  if (B == 0) return RAP_OK;
  rap_attn_args a;
  a.q = d_q; a.k = d_k8; a.v = d_v8; a.seq_len = d_seq_len; a.len_add = 0;
  a.B = B; a.Hq = d.n_q_heads; a.Hkv = d.n_kv_heads; a.P2 = 2 * ctx->n_pairs[layer]; a.dv = ctx->n_vch[layer];
  a.S_cap = S_cap; a.head_dim = d.head_dim; a.dtype = d.dtype; a.n_split = n_split; a.h_len_max = h_seq_len_max;
  a.out = d_out;
  return rap_launch_attn_q8(ctx, a, (cudaStream_t)stream);
}

rap_status rap_decode_step_q8(rap_ctx* ctx, int32_t B, const void* d_x, const void* const* h_w_qkv, const void* const* h_bias,
                              const double* d_inv_freq, void* const* h_k8, void* const* h_v8, int32_t S_cap,
                              int32_t* d_seq_len, int32_t h_seq_len_max, int32_t n_split, void* d_q_scratch, float* d_out,
                              size_t out_layer_stride, int32_t advance, void* stream) {
  if (!ctx || !d_x || !h_w_qkv || !d_inv_freq || !h_k8 || !h_v8 || !d_seq_len || !d_q_scratch || !d_out) return RAP_EINVAL;
  if (!ctx->tables_built) return RAP_ESTATE;
  const rap_model_desc& d = ctx->desc;
  if (B < 0 || S_cap < 1 || n_split < 0 || h_seq_len_max < 0) return RAP_EINVAL;
  if (B > d.max_batch || B > d.max_rows || n_split > RAP_MAX_SPLIT) return RAP_ESHAPE;
  if (S_cap % 8) return RAP_EALIGN;
  if (h_seq_len_max >= S_cap) return RAP_ECAPACITY;
  if (d.head_dim > 256) return RAP_EUNSUPPORTED;
  if (!rap_aligned16(d_x) || !rap_aligned16(d_inv_freq) || !rap_aligned16(d_seq_len) || !rap_aligned16(d_q_scratch) ||
      !rap_aligned16(d_out) || (out_layer_stride % 4))
    return RAP_EALIGN;
  for (int l = 0; l < d.n_layers; ++l) {
    if (!h_w_qkv[l] || !h_k8[l] || !h_v8[l]) return RAP_EINVAL;
    if (out_layer_stride < (size_t)B * d.n_q_heads * ctx->n_vch[l]) return RAP_ESHAPE;
    if (!rap_aligned16(h_w_qkv[l]) || !rap_aligned16(h_k8[l]) || !rap_aligned16(h_v8[l]) ||
        (h_bias && h_bias[l] && !rap_aligned16(h_bias[l])))
      return RAP_EALIGN;
  }
  if (B == 0) return RAP_OK;
  cudaStream_t st = (cudaStream_t)stream;
  const size_t e = rap_elem_bytes(d.dtype);
  for (int l = 0; l < d.n_layers; ++l) {
    rap_proj_args p;
    p.x = (const char*)d_x + (size_t)l * B * d.hidden * e;
    p.w = h_w_qkv[l]; p.bias = h_bias ? h_bias[l] : nullptr;
    p.seq_id = nullptr; p.pos = d_seq_len; p.slot = nullptr;   // decode mode: row r = sequence r at pos = slot = len
    p.inv_freq = d_inv_freq + (size_t)l * d.n_kv_heads * (d.head_dim / 2);
    p.q_out = d_q_scratch; p.k_cache = h_k8[l]; p.v_cache = h_v8[l];
    p.T = B; p.hidden = d.hidden; p.Hq = d.n_q_heads; p.Hkv = d.n_kv_heads;
    p.P2 = 2 * ctx->n_pairs[l]; p.dv = ctx->n_vch[l]; p.half_dim = d.head_dim / 2;
    p.B_cache = B; p.S_cap = S_cap; p.dtype = d.dtype;
    p.pdl = l > 0 ? 1 : 0;     // the GEMM of layer l may stream its weights while the scan of layer l - 1 drains
    rap_status s = rap_launch_qkv_rope_append_q8(ctx, p, st);
    if (s != RAP_OK) return s;
    rap_attn_args a;
    a.q = d_q_scratch; a.k = h_k8[l]; a.v = h_v8[l]; a.seq_len = d_seq_len; a.len_add = 1;
    a.B = B; a.Hq = d.n_q_heads; a.Hkv = d.n_kv_heads; a.P2 = p.P2; a.dv = p.dv; a.S_cap = S_cap;
    a.head_dim = d.head_dim; a.dtype = d.dtype; a.n_split = n_split; a.h_len_max = h_seq_len_max + 1;
    a.out = d_out + (size_t)l * out_layer_stride;
    a.pdl = 1;
    s = rap_launch_attn_q8(ctx, a, st);
    if (s != RAP_OK) return s;
  }
  if (advance) return rap_launch_advance(ctx, d_seq_len, B, st);
  return RAP_OK;
}

rap_status rap_prefill_attn(rap_ctx* ctx, int32_t layer, int32_t B, int32_t T, const void* d_q, const void* d_k_cache,
                            const void* d_v_cache, int32_t S_cap, const int32_t* d_start, int32_t h_start_max,
                            float* d_out, void* stream) {
  if (!ctx || !d_q || !d_k_cache || !d_v_cache || !d_start || !d_out) return RAP_EINVAL;
  if (!ctx->tables_built) return RAP_ESTATE;
  const rap_model_desc& d = ctx->desc;
  if (layer < 0 || layer >= d.n_layers || B < 0 || T < 0 || S_cap < 1 || h_start_max < 0) return RAP_EINVAL;
  if (B > d.max_batch) return RAP_ESHAPE;
  if (S_cap % 8) return RAP_EALIGN;
  if ((long long)h_start_max + T > S_cap) return RAP_ECAPACITY;
  if (!rap_aligned16(d_q) || !rap_aligned16(d_k_cache) || !rap_aligned16(d_v_cache) || !rap_aligned16(d_out) ||
      !rap_aligned16(d_start))
    return RAP_EALIGN;
  if (B == 0 || T == 0) return RAP_OK;
  return rap_launch_prefill_attn(ctx, B, T, d_q, d_k_cache, d_v_cache, 2 * ctx->n_pairs[layer], ctx->n_vch[layer], S_cap,
                                 d_start, d_out, (cudaStream_t)stream);
}

// argument checks of a decode step (everything but launching it)
static rap_status decode_step_check(rap_ctx* ctx, int32_t B, const void* d_x, const void* const* h_w_qkv,
                                    const void* const* h_bias, const double* d_inv_freq, void* const* h_k_cache,
                                    void* const* h_v_cache, int32_t S_cap, int32_t* d_seq_len, int32_t h_seq_len_max,
                                    int32_t n_split, void* d_q_scratch, float* d_out, size_t out_layer_stride) {
  if (!ctx || !d_x || !h_w_qkv || !d_inv_freq || !h_k_cache || !h_v_cache || !d_seq_len || !d_q_scratch || !d_out)
    return RAP_EINVAL;
  if (!ctx->tables_built) return RAP_ESTATE;
  const rap_model_desc& d = ctx->desc;
  if (B < 0 || S_cap < 1 || n_split < 0 || h_seq_len_max < 0) return RAP_EINVAL;
  if (B > d.max_batch || B > d.max_rows || n_split > RAP_MAX_SPLIT) return RAP_ESHAPE;
  if (S_cap % 8) return RAP_EALIGN;
  if (h_seq_len_max >= S_cap) return RAP_ECAPACITY;
  if (!rap_aligned16(d_x) || !rap_aligned16(d_inv_freq) || !rap_aligned16(d_seq_len) || !rap_aligned16(d_q_scratch) ||
      !rap_aligned16(d_out) || (out_layer_stride % 4))
    return RAP_EALIGN;
  for (int l = 0; l < d.n_layers; ++l) {
    if (!h_w_qkv[l] || !h_k_cache[l] || !h_v_cache[l]) return RAP_EINVAL;
    if (out_layer_stride < (size_t)B * d.n_q_heads * ctx->n_vch[l]) return RAP_ESHAPE;
    if (!rap_aligned16(h_w_qkv[l]) || !rap_aligned16(h_k_cache[l]) || !rap_aligned16(h_v_cache[l]) ||
        (h_bias && h_bias[l] && !rap_aligned16(h_bias[l])))
      return RAP_EALIGN;
  }
  return RAP_OK;
}

// layers [l0, l1) of a decode step whose arguments have been checked
static rap_status decode_layers(rap_ctx* ctx, int l0, int l1, int32_t B, const void* d_x, const void* const* h_w_qkv,
                                const void* const* h_bias, const double* d_inv_freq, void* const* h_k_cache,
                                void* const* h_v_cache, int32_t S_cap, int32_t* d_seq_len, int32_t h_seq_len_max,
                                int32_t n_split, void* d_q_scratch, float* d_out, size_t out_layer_stride, cudaStream_t st) {
  const rap_model_desc& d = ctx->desc;
  const size_t e = rap_elem_bytes(d.dtype);
  for (int l = l0; l < l1; ++l) {
    const bool timed = 2 * (ctx->prof_pairs + 1) <= (int)ctx->prof_ev.size();   // events around this layer's attention
    rap_proj_args p;
    p.x = (const char*)d_x + (size_t)l * B * d.hidden * e;
    p.w = h_w_qkv[l]; p.bias = h_bias ? h_bias[l] : nullptr;
    p.seq_id = nullptr; p.pos = d_seq_len; p.slot = nullptr;   // decode mode: row r = sequence r at pos = slot = len
    p.inv_freq = d_inv_freq + (size_t)l * d.n_kv_heads * (d.head_dim / 2);
    p.q_out = d_q_scratch; p.k_cache = h_k_cache[l]; p.v_cache = h_v_cache[l];
    p.T = B; p.hidden = d.hidden; p.Hq = d.n_q_heads; p.Hkv = d.n_kv_heads;
    p.P2 = 2 * ctx->n_pairs[l]; p.dv = ctx->n_vch[l]; p.half_dim = d.head_dim / 2;
    p.B_cache = B; p.S_cap = S_cap; p.dtype = d.dtype;
    // Inside a run of layers the library knows what precedes each launch: from the run's second layer on the
    // projection follows an attention launch that does not touch what the projection reads, so it may start
    // streaming its weights while that launch drains (the first projection follows caller work or a copy, and waits).
    p.pdl = (l > l0 && !timed) ? 1 : 0;
    rap_status s = rap_launch_qkv_rope_append(ctx, p, st);
    if (s != RAP_OK) return s;
    rap_attn_args a;
    a.q = d_q_scratch; a.k = h_k_cache[l]; a.v = h_v_cache[l]; a.seq_len = d_seq_len; a.len_add = 1;
    a.B = B; a.Hq = d.n_q_heads; a.Hkv = d.n_kv_heads; a.P2 = p.P2; a.dv = p.dv; a.S_cap = S_cap;
    a.head_dim = d.head_dim; a.dtype = d.dtype; a.n_split = n_split; a.h_len_max = h_seq_len_max + 1;
    a.out = d_out + (size_t)l * out_layer_stride;
    a.pdl = timed ? 0 : 1;
    if (timed) RAP_CUDA_TRY(ctx, cudaEventRecord(ctx->prof_ev[2 * ctx->prof_pairs], st));
    s = rap_launch_attn(ctx, a, st);
    if (s != RAP_OK) return s;
    if (timed) {
      RAP_CUDA_TRY(ctx, cudaEventRecord(ctx->prof_ev[2 * ctx->prof_pairs + 1], st));
      ctx->prof_pairs++;
    }
  }
  return RAP_OK;
}

rap_status rap_decode_step(rap_ctx* ctx, int32_t B, const void* d_x, const void* const* h_w_qkv,
                           const void* const* h_bias, const double* d_inv_freq, void* const* h_k_cache,
                           void* const* h_v_cache, int32_t S_cap, int32_t* d_seq_len, int32_t h_seq_len_max,
                           int32_t n_split, void* d_q_scratch, float* d_out, size_t out_layer_stride,
                           int32_t advance, void* stream) {
  rap_status s = decode_step_check(ctx, B, d_x, h_w_qkv, h_bias, d_inv_freq, h_k_cache, h_v_cache, S_cap, d_seq_len,
                                   h_seq_len_max, n_split, d_q_scratch, d_out, out_layer_stride);
  if (s != RAP_OK || B == 0) return s;
  cudaStream_t st = (cudaStream_t)stream;
  s = decode_layers(ctx, 0, ctx->desc.n_layers, B, d_x, h_w_qkv, h_bias, d_inv_freq, h_k_cache, h_v_cache, S_cap, d_seq_len,
                    h_seq_len_max, n_split, d_q_scratch, d_out, out_layer_stride, st);
  if (s != RAP_OK) return s;
  if (advance) return rap_launch_advance(ctx, d_seq_len, B, st);
  return RAP_OK;
}

rap_status rap_decode_step_host(rap_ctx* ctx, int32_t B, const void* h_x, const void* const* h_w_qkv,
                                const void* const* h_bias, const double* d_inv_freq, void* const* h_k_cache,
                                void* const* h_v_cache, int32_t S_cap, int32_t* d_seq_len, int32_t h_seq_len_max,
                                int32_t n_split, float* h_out, size_t out_layer_stride, int32_t advance,
                                void* stream) {
  if (!ctx || !h_x || !h_out) return RAP_EINVAL;
  const rap_model_desc& d = ctx->desc;
  if (B < 0) return RAP_EINVAL;
  if (B > d.max_batch) return RAP_ESHAPE;
  if (out_layer_stride > (size_t)d.max_batch * d.n_q_heads * d.head_dim) return RAP_ESHAPE;
  cudaStream_t st = (cudaStream_t)stream;
  const size_t xb = (size_t)d.n_layers * B * d.hidden * rap_elem_bytes(d.dtype);
  const size_t ob = (size_t)d.n_layers * out_layer_stride * sizeof(float);
  if (B == 0) return RAP_OK;
  rap_status s = decode_step_check(ctx, B, ctx->d_stage_x, h_w_qkv, h_bias, d_inv_freq, h_k_cache, h_v_cache, S_cap, d_seq_len,
                                   h_seq_len_max, n_split, ctx->d_stage_q, ctx->d_stage_out, out_layer_stride);
  if (s != RAP_OK) return s;
  const int L = d.n_layers;
  const size_t x_layer = (size_t)B * d.hidden * rap_elem_bytes(d.dtype), o_layer = out_layer_stride * sizeof(float);
  auto layers = [&](int l0, int l1) {
    return decode_layers(ctx, l0, l1, B, ctx->d_stage_x, h_w_qkv, h_bias, d_inv_freq, h_k_cache, h_v_cache, S_cap, d_seq_len,
                         h_seq_len_max, n_split, ctx->d_stage_q, ctx->d_stage_out, out_layer_stride, st);
  };
  if (L < 4) {       // short stacks: copy in, run, copy out
    RAP_CUDA_TRY(ctx, cudaMemcpyAsync(ctx->d_stage_x, h_x, xb, cudaMemcpyHostToDevice, st));
    if ((s = layers(0, L)) != RAP_OK) return s;
    if (advance && (s = rap_launch_advance(ctx, d_seq_len, B, st)) != RAP_OK) return s;
    RAP_CUDA_TRY(ctx, cudaMemcpyAsync(h_out, ctx->d_stage_out, ob, cudaMemcpyDeviceToHost, st));
    RAP_CUDA_TRY(ctx, cudaStreamSynchronize(st));
    return RAP_OK;
  }
  // The copies overlap the layers.  Only layer 0's inputs are copied ahead of it on the caller's stream; the rest
  // arrive on a second stream while layer 0 runs (layer 0's copy is issued first: a copy engine serves copies in
  // the order they were issued).  The outputs leave in three pieces: layers [0, L/2) on a third stream while the
  // second half runs, [L/2, L-1) while the last layer runs, the last layer's on the caller's stream.  The staging
  // buffers are free when a call starts: the previous call synchronized every stream that touched them.
  cudaStream_t cin = (cudaStream_t)ctx->copy_in, cout = (cudaStream_t)ctx->copy_out;
  const char* hx = (const char*)h_x;
  RAP_CUDA_TRY(ctx, cudaMemcpyAsync(ctx->d_stage_x, hx, x_layer, cudaMemcpyHostToDevice, st));
  RAP_CUDA_TRY(ctx, cudaMemcpyAsync((char*)ctx->d_stage_x + x_layer, hx + x_layer, xb - x_layer, cudaMemcpyHostToDevice, cin));
  RAP_CUDA_TRY(ctx, cudaEventRecord((cudaEvent_t)ctx->ev_in, cin));
  if ((s = layers(0, 1)) != RAP_OK) return s;
  RAP_CUDA_TRY(ctx, cudaStreamWaitEvent(st, (cudaEvent_t)ctx->ev_in, 0));
  const int cut[3] = {0, L / 2, L - 1};
  for (int c = 0; c < 2; ++c) {
    if ((s = layers(c == 0 ? 1 : cut[c], cut[c + 1])) != RAP_OK) return s;
    RAP_CUDA_TRY(ctx, cudaEventRecord((cudaEvent_t)ctx->ev_mid, st));
    RAP_CUDA_TRY(ctx, cudaStreamWaitEvent(cout, (cudaEvent_t)ctx->ev_mid, 0));
    RAP_CUDA_TRY(ctx, cudaMemcpyAsync((char*)h_out + (size_t)cut[c] * o_layer, (const char*)ctx->d_stage_out + (size_t)cut[c] * o_layer,
                                      (size_t)(cut[c + 1] - cut[c]) * o_layer, cudaMemcpyDeviceToHost, cout));
  }
  if ((s = layers(L - 1, L)) != RAP_OK) return s;
  if (advance && (s = rap_launch_advance(ctx, d_seq_len, B, st)) != RAP_OK) return s;
  RAP_CUDA_TRY(ctx, cudaMemcpyAsync((char*)h_out + (size_t)(L - 1) * o_layer, (const char*)ctx->d_stage_out + (size_t)(L - 1) * o_layer,
                                    o_layer, cudaMemcpyDeviceToHost, st));
  RAP_CUDA_TRY(ctx, cudaStreamSynchronize(st));
  RAP_CUDA_TRY(ctx, cudaStreamSynchronize(cout));
  return RAP_OK;
}

rap_status rap_lowrank_decode_attn(rap_ctx* ctx, int32_t B, int32_t r, int32_t d_v, const void* d_q_full,
                                   const void* d_k_latent, const void* d_bk, const void* d_v_cache, int32_t S_cap,
                                   const int32_t* d_seq_len, int32_t h_seq_len_max, int32_t n_split, float* d_out,
                                   void* stream) {
  if (!ctx || !d_q_full || !d_k_latent || !d_bk || !d_v_cache || !d_seq_len || !d_out) return RAP_EINVAL;
  const rap_model_desc& d = ctx->desc;
  if (B < 0 || r < 1 || r > d.head_dim || d_v < 1 || d_v > d.head_dim || S_cap < 1 || n_split < 0 ||
      h_seq_len_max < 0)
    return RAP_EINVAL;
  if (B > d.max_batch || n_split > RAP_MAX_SPLIT) return RAP_ESHAPE;
  if (S_cap % 8) return RAP_EALIGN;
  if (h_seq_len_max > S_cap) return RAP_ECAPACITY;
  if (!rap_aligned16(d_q_full) || !rap_aligned16(d_k_latent) || !rap_aligned16(d_bk) || !rap_aligned16(d_v_cache) ||
      !rap_aligned16(d_out) || !rap_aligned16(d_seq_len))
    return RAP_EALIGN;
  if (B == 0) return RAP_OK;
  rap_lowrank_args a;
  a.q_full = d_q_full; a.k_latent = d_k_latent; a.bk = d_bk; a.v = d_v_cache; a.seq_len = d_seq_len;
  a.B = B; a.Hq = d.n_q_heads; a.Hkv = d.n_kv_heads; a.r = r; a.dv = d_v; a.S_cap = S_cap;
  a.head_dim = d.head_dim; a.dtype = d.dtype; a.pairing = d.pairing; a.rope_theta = d.rope_theta;
  a.n_split = n_split; a.h_len_max = h_seq_len_max; a.out = d_out;
  return rap_launch_lowrank_attn(ctx, a, (cudaStream_t)stream);
}

rap_status rap_profile_attn(rap_ctx* ctx, int32_t capacity) {
  if (!ctx || capacity < 0) return RAP_EINVAL;
  for (cudaEvent_t e : ctx->prof_ev) cudaEventDestroy(e);
  ctx->prof_ev.clear();
  ctx->prof_pairs = 0;
  for (int i = 0; i < 2 * capacity; ++i) {
    cudaEvent_t e;
    RAP_CUDA_TRY(ctx, cudaEventCreate(&e));
    ctx->prof_ev.push_back(e);
  }
  return RAP_OK;
}

rap_status rap_profile_attn_read(rap_ctx* ctx, float* ms_sum, int32_t* n_calls) {
  if (!ctx || !ms_sum || !n_calls) return RAP_EINVAL;
  float sum = 0.f;
  for (int i = 0; i < ctx->prof_pairs; ++i) {
    float ms = 0.f;
    RAP_CUDA_TRY(ctx, cudaEventSynchronize(ctx->prof_ev[2 * i + 1]));
    RAP_CUDA_TRY(ctx, cudaEventElapsedTime(&ms, ctx->prof_ev[2 * i], ctx->prof_ev[2 * i + 1]));
    sum += ms;
  }
  *ms_sum = sum;
  *n_calls = ctx->prof_pairs;
  ctx->prof_pairs = 0;
  return RAP_OK;
}

rap_status rap_get_last_device_status(rap_ctx* ctx, int32_t* code, int32_t* detail, void* stream) {
  if (!ctx || !code || !detail) return RAP_EINVAL;
  int32_t h[2] = {0, 0};
  cudaStream_t st = (cudaStream_t)stream;
  RAP_CUDA_TRY(ctx, cudaMemcpyAsync(h, ctx->d_status, sizeof(h), cudaMemcpyDeviceToHost, st));
  RAP_CUDA_TRY(ctx, cudaMemsetAsync(ctx->d_status, 0, sizeof(h), st));
  RAP_CUDA_TRY(ctx, cudaStreamSynchronize(st));
  if (h[0] != 0) {   // a kernel that gave up may have left arrival counters behind (the next launches clear them too)
    const rap_model_desc& d = ctx->desc;
    RAP_CUDA_TRY(ctx, cudaMemsetAsync(ctx->d_unit_cnt, 0, (2 * (size_t)d.max_batch * d.n_kv_heads + 2) * sizeof(int32_t), st));
    RAP_CUDA_TRY(ctx, cudaMemsetAsync(ctx->d_proj_cnt, 0, 2 * (size_t)ctx->proj_cnt_n * sizeof(int32_t), st));
    RAP_CUDA_TRY(ctx, cudaStreamSynchronize(st));
  }
  *code = h[0];
  *detail = h[1];
  return RAP_OK;
}

}  // extern "C"
