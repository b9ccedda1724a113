// Split-KV decode attention over the reduced dims (Eq. 2 restricted to the retained pairs and
// channels, Eq. 7; softmax scale 1/sqrt(D) with the ORIGINAL head_dim).
//
// This file holds the shape-generic scan kernel (any 2P, d_v', fp32 or bf16), the split
// combine kernel and the launch heuristics.  The bandwidth-tuned bf16 scans live in
// rap_attn_scan.cu (specialised per head shape) and rap_attn_fast.cu (run-time shape);
// rap_launch_attn picks them when their shape rules hold.
//
// Partial results of split s for (b, g) live in the context workspace as d_v' accumulators
// followed by (m, l): m = running max of the base-2 logits, l = sum 2^(s - m).
#include <math.h>

#include <mutex>

#include "rap_internal.h"

rap_status rap_launch_attn_fast(rap_ctx* ctx, const rap_attn_args& a, int n_split, cudaStream_t st);
rap_status rap_launch_attn_scan(rap_ctx* ctx, const rap_attn_args& a, int n_split, cudaStream_t st);
rap_status rap_launch_attn_mma(rap_ctx* ctx, const rap_attn_args& a, int n_split, cudaStream_t st);

namespace {

constexpr int GEN_TILE = 64;      // positions per tile
constexpr int GEN_THREADS = 256;  // >= largest d_v' (head_dim <= 256)

template <typename T> __device__ __forceinline__ float ld(const T* p);
template <> __device__ __forceinline__ float ld<float>(const float* p) { return *p; }
template <> __device__ __forceinline__ float ld<__nv_bfloat16>(const __nv_bfloat16* p) { return __bfloat162float(*p); }

template <typename T>
__global__ void __launch_bounds__(GEN_THREADS)
attn_generic_kernel(const T* __restrict__ q, const T* __restrict__ kc, const T* __restrict__ vc,
                    const int32_t* __restrict__ seq_len, int len_add, int Hq, int Hkv, int P2, int dv, int S_cap,
                    float qscale, int n_split, float* __restrict__ ws) {
  extern __shared__ float smem[];
  const int G = Hq / Hkv;
  float* q_s = smem;                  // [G][P2]   pre-scaled by log2(e)/sqrt(D)
  float* s_s = q_s + G * P2;          // [G][GEN_TILE]
  float* alpha_s = s_s + G * GEN_TILE;  // [G]
  const int split = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  int len = seq_len[b] + len_add;
  len = min(max(len, 0), S_cap);
  const int n_tiles = (len + GEN_TILE - 1) / GEN_TILE;
  const int tps = (n_tiles + n_split - 1) / n_split;
  const int tile_begin = split * tps, tile_end = min(n_tiles, tile_begin + tps);

  for (int i = tid; i < G * P2; i += GEN_THREADS) {
    const int g = i / P2, d = i - g * P2;
    q_s[i] = ld<T>(q + ((size_t)b * Hq + h * G + g) * P2 + d) * qscale;
  }
  const T* kb = kc + ((size_t)b * Hkv + h) * (size_t)S_cap * P2;
  const T* vb = vc + ((size_t)b * Hkv + h) * (size_t)S_cap * dv;
  float m_run = -INFINITY, l_run = 0.f;   // meaningful in warp g < G (all lanes hold the same value)
  float acc[RAP_MAX_GROUP];
#pragma unroll
  for (int g = 0; g < RAP_MAX_GROUP; ++g) acc[g] = 0.f;
  __syncthreads();

  for (int tile = tile_begin; tile < tile_end; ++tile) {
    const int j0 = tile * GEN_TILE;
    const int nj = min(GEN_TILE, len - j0);
    // logits: one warp per position, lanes over dims
    for (int j = warp; j < nj; j += GEN_THREADS / 32) {
      const T* kr = kb + (size_t)(j0 + j) * P2;
      float part[RAP_MAX_GROUP];
#pragma unroll
      for (int g = 0; g < RAP_MAX_GROUP; ++g) part[g] = 0.f;
      for (int d = lane; d < P2; d += 32) {
        const float kv = ld<T>(kr + d);
#pragma unroll
        for (int g = 0; g < RAP_MAX_GROUP; ++g)
          if (g < G) part[g] = fmaf(kv, q_s[g * P2 + d], part[g]);
      }
#pragma unroll
      for (int g = 0; g < RAP_MAX_GROUP; ++g) {
        if (g < G) {
          float v = part[g];
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
          if (lane == 0) s_s[g * GEN_TILE + j] = v;
        }
      }
    }
    __syncthreads();
    // online softmax: warp g owns head g
    if (warp < G) {
      const int g = warp;
      float mx = -INFINITY;
      for (int j = lane; j < nj; j += 32) mx = fmaxf(mx, s_s[g * GEN_TILE + j]);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      const float m_new = fmaxf(m_run, mx);
      float sum = 0.f;
      for (int j = lane; j < nj; j += 32) {
        const float p = exp2f(s_s[g * GEN_TILE + j] - m_new);
        s_s[g * GEN_TILE + j] = p;
        sum += p;
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
      const float alpha = exp2f(m_run - m_new);   // first tile: 2^(-inf) = 0
      l_run = l_run * alpha + sum;
      m_run = m_new;
      if (lane == 0) alpha_s[g] = alpha;
    }
    __syncthreads();
    // weighted sum: one thread per retained V channel
    if (tid < dv) {
#pragma unroll
      for (int g = 0; g < RAP_MAX_GROUP; ++g)
        if (g < G) acc[g] *= alpha_s[g];
      for (int j = 0; j < nj; ++j) {
        const float vv = ld<T>(vb + (size_t)(j0 + j) * dv + tid);
#pragma unroll
        for (int g = 0; g < RAP_MAX_GROUP; ++g)
          if (g < G) acc[g] = fmaf(s_s[g * GEN_TILE + j], vv, acc[g]);
      }
    }
    __syncthreads();
  }
  // partials: ws[((b*Hq + gq) * n_split + split)][dv + 2]
#pragma unroll
  for (int g = 0; g < RAP_MAX_GROUP; ++g) {
    if (g < G) {
      float* dst = ws + (((size_t)b * Hq + h * G + g) * n_split + split) * (size_t)(dv + 2);
      if (tid < dv) dst[tid] = acc[g];
      if (warp == g && lane == 0) {
        dst[dv] = m_run;
        dst[dv + 1] = l_run;
      }
    }
  }
}

// out[b][g][c] = sum_s 2^(m_s - M) acc_s[c] / sum_s 2^(m_s - M) l_s ; empty splits have l = 0.
__global__ void attn_combine_kernel(const float* __restrict__ ws, int n_split, int dv, float* __restrict__ out) {
  const size_t bg = blockIdx.x;
  const float* base = ws + bg * n_split * (size_t)(dv + 2);
  float M = -INFINITY;
  for (int s = 0; s < n_split; ++s) {
    const float l = base[(size_t)s * (dv + 2) + dv + 1];
    if (l > 0.f) M = fmaxf(M, base[(size_t)s * (dv + 2) + dv]);
  }
  float den = 0.f;
  for (int s = 0; s < n_split; ++s) {
    const float l = base[(size_t)s * (dv + 2) + dv + 1];
    if (l > 0.f) den += exp2f(base[(size_t)s * (dv + 2) + dv] - M) * l;
  }
  for (int c = threadIdx.x; c < dv; c += blockDim.x) {
    float num = 0.f;
    for (int s = 0; s < n_split; ++s) {
      const float l = base[(size_t)s * (dv + 2) + dv + 1];
      if (l > 0.f) num += exp2f(base[(size_t)s * (dv + 2) + dv] - M) * base[(size_t)s * (dv + 2) + c];
    }
    out[bg * dv + c] = den > 0.f ? num / den : 0.f;
  }
}

}  // namespace

// Number of sequence splits: enough CTAs to fill the GPU a few times over, but no split shorter
// than a handful of tiles.
static int choose_split(const rap_ctx* ctx, const rap_attn_args& a, int tile, int ctas_per_sm, int min_tiles) {
  const int units = a.B * a.Hkv;
  const int n_tiles = (a.h_len_max + tile - 1) / tile;
  const int want = ctx->sm_count * ctas_per_sm * 2;
  int ns = (want + units - 1) / units;
  const int cap = n_tiles / min_tiles > 0 ? n_tiles / min_tiles : 1;
  if (ns > cap) ns = cap;
  if (ns > RAP_MAX_SPLIT) ns = RAP_MAX_SPLIT;
  if (ns < 1) ns = 1;
  return ns;
}

rap_status rap_launch_attn(rap_ctx* ctx, const rap_attn_args& a, cudaStream_t st) {
  const int G = a.Hq / a.Hkv;
  if (a.dtype == RAP_BF16 && ctx->attn_variant != 1) {
    // shape-specialised scans (mma.sync, then FP32 pipes), then the shape-generic bf16 scan, then the fully
    // generic kernel
    if (ctx->attn_variant == 4) return rap_launch_attn_mma(ctx, a, a.n_split, st);
    if (ctx->attn_variant == 0) {
      const rap_status s = rap_launch_attn_mma(ctx, a, a.n_split, st);
      if (s != RAP_EUNSUPPORTED) return s;
    }
    if (ctx->attn_variant == 0 || ctx->attn_variant == 3) {
      const rap_status s = rap_launch_attn_scan(ctx, a, a.n_split, st);
      if (s != RAP_EUNSUPPORTED) return s;
    }
    const rap_status s = rap_launch_attn_fast(ctx, a, a.n_split, st);
    if (s != RAP_EUNSUPPORTED) return s;
  }
  if (a.B > 65535 || a.Hkv > 65535) return RAP_ESHAPE;   // grid.z / grid.y of the generic scan
  const int n_split = a.n_split > 0 ? a.n_split : choose_split(ctx, a, GEN_TILE, 4, 4);
  const float qscale = (float)(1.4426950408889634 / sqrt((double)a.head_dim));
  const size_t smem = (size_t)(G * a.P2 + G * GEN_TILE + G) * sizeof(float);
  dim3 grid(n_split, a.Hkv, a.B);
  if (a.dtype == RAP_F32)
    attn_generic_kernel<float><<<grid, GEN_THREADS, smem, st>>>((const float*)a.q, (const float*)a.k,
                                                                (const float*)a.v, a.seq_len, a.len_add, a.Hq, a.Hkv,
                                                                a.P2, a.dv, a.S_cap, qscale, n_split, ctx->d_attn_ws);
  else
    attn_generic_kernel<__nv_bfloat16><<<grid, GEN_THREADS, smem, st>>>(
        (const __nv_bfloat16*)a.q, (const __nv_bfloat16*)a.k, (const __nv_bfloat16*)a.v, a.seq_len, a.len_add, a.Hq,
        a.Hkv, a.P2, a.dv, a.S_cap, qscale, n_split, ctx->d_attn_ws);
  ctx->launches++;
  RAP_CUDA_TRY(ctx, cudaGetLastError());
  attn_combine_kernel<<<a.B * a.Hq, 128, 0, st>>>(ctx->d_attn_ws, n_split, a.dv, a.out);
  ctx->launches++;
  RAP_CUDA_TRY(ctx, cudaGetLastError());
  return RAP_OK;
}

// ---- allocation-free variant ---------------------------------------------------------------
// Split-KV partials of rap_decode_attn_noalloc live in this file-scope array instead of a
// context workspace (RAP_NOALLOC_WS_FLOATS floats = 4 MiB, the limit rap.h documents).  Every GPU that loads
// the library reserves it until the process exits.
static __device__ __align__(256) float g_noalloc_ws[RAP_NOALLOC_WS_FLOATS];

namespace {
constexpr int NOALLOC_MAX_DEVICES = 64;
std::mutex g_noalloc_mu;
float* g_noalloc_addr[NOALLOC_MAX_DEVICES];   // device address of g_noalloc_ws, per device ordinal

// In host code `g_noalloc_ws` names a host-side shadow, not device memory; the address a kernel
// may use comes from cudaGetSymbolAddress, asked once per device with that device current.
cudaError_t noalloc_ws_address(float** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= NOALLOC_MAX_DEVICES) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_noalloc_mu);
  if (!g_noalloc_addr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_noalloc_ws);
    if (e != cudaSuccess) return e;
    g_noalloc_addr[dev] = static_cast<float*>(p);
  }
  *out = g_noalloc_addr[dev];
  return cudaSuccess;
}
}  // namespace

extern "C" rap_status rap_decode_attn_noalloc(int32_t dtype, int32_t B, int32_t n_q_heads, int32_t n_kv_heads,
                                              int32_t head_dim, int32_t n_pairs, int32_t n_vch, const void* d_q,
                                              const void* d_k_cache, const void* d_v_cache, int32_t S_cap,
                                              const int32_t* d_seq_len, int32_t h_seq_len_max, int32_t n_split,
                                              float* d_out, void* stream) {
  if (!d_q || !d_k_cache || !d_v_cache || !d_seq_len || !d_out) return RAP_EINVAL;
  if (dtype != RAP_F32 && dtype != RAP_BF16) return RAP_EINVAL;
  if (B < 0 || n_q_heads < 1 || n_kv_heads < 1 || n_q_heads % n_kv_heads || head_dim < 2 || (head_dim & 1) ||
      head_dim > GEN_THREADS || n_pairs < 1 || n_pairs > head_dim / 2 || n_vch < 1 || n_vch > head_dim ||
      S_cap < 1 || n_split < 0 || h_seq_len_max < 0)
    return RAP_EINVAL;
  const int G = n_q_heads / n_kv_heads;
  if (G > RAP_MAX_GROUP || n_split > RAP_MAX_SPLIT) return RAP_ESHAPE;
  if (B > 65535 || n_kv_heads > 65535) return RAP_ESHAPE;   // grid.z / grid.y of the scan
  if (S_cap % 8) return RAP_EALIGN;
  if (h_seq_len_max > S_cap) return RAP_ECAPACITY;
  if (!rap_aligned16(d_q) || !rap_aligned16(d_k_cache) || !rap_aligned16(d_v_cache) || !rap_aligned16(d_out) ||
      !rap_aligned16(d_seq_len))
    return RAP_EALIGN;
  if (B == 0) return RAP_OK;
  // the partials of one split: B * H_q rows of d_v' accumulators + (m, l)
  const size_t per_split = (size_t)B * n_q_heads * (size_t)(n_vch + 2);
  if (per_split > RAP_NOALLOC_WS_FLOATS) return RAP_ESHAPE;
  const int fit = (int)(RAP_NOALLOC_WS_FLOATS / per_split);
  int ns = n_split;
  if (ns == 0) {
    // a few CTAs per SM, splits of at least four tiles, and no more than the static array holds
    const int n_tiles = (h_seq_len_max + GEN_TILE - 1) / GEN_TILE;
    ns = (1024 + B * n_kv_heads - 1) / (B * n_kv_heads);
    if (ns > n_tiles / 4) ns = n_tiles / 4;
    if (ns > RAP_MAX_SPLIT) ns = RAP_MAX_SPLIT;
    if (ns > fit) ns = fit;
    if (ns < 1) ns = 1;
  } else if (ns > fit) {
    return RAP_ESHAPE;
  }
  float* ws = nullptr;
  if (noalloc_ws_address(&ws) != cudaSuccess) return RAP_ECUDA;
  cudaStream_t st = (cudaStream_t)stream;
  const int P2 = 2 * n_pairs;
  const float qscale = (float)(1.4426950408889634 / sqrt((double)head_dim));
  const size_t smem = (size_t)(G * P2 + G * GEN_TILE + G) * sizeof(float);
  dim3 grid(ns, n_kv_heads, B);
  if (dtype == RAP_F32)
    attn_generic_kernel<float><<<grid, GEN_THREADS, smem, st>>>((const float*)d_q, (const float*)d_k_cache,
                                                                (const float*)d_v_cache, d_seq_len, 0, n_q_heads,
                                                                n_kv_heads, P2, n_vch, S_cap, qscale, ns, ws);
  else
    attn_generic_kernel<__nv_bfloat16><<<grid, GEN_THREADS, smem, st>>>(
        (const __nv_bfloat16*)d_q, (const __nv_bfloat16*)d_k_cache, (const __nv_bfloat16*)d_v_cache, d_seq_len, 0,
        n_q_heads, n_kv_heads, P2, n_vch, S_cap, qscale, ns, ws);
  if (cudaGetLastError() != cudaSuccess) return RAP_ECUDA;
  attn_combine_kernel<<<B * n_q_heads, 128, 0, st>>>(ws, ns, n_vch, d_out);
  if (cudaGetLastError() != cudaSuccess) return RAP_ECUDA;
  return RAP_OK;
}
