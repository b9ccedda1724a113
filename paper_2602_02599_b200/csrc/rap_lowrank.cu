// Low-rank comparator (Section 3: a weight-side low-rank method caches the latent X A_k and must
// rebuild K = latent B_k, then rotate it at full width, at EVERY decode step).  Measurement-only
// counterpart of rap_decode_attn at equal cached dims: same split-KV structure, same V side, but
// every tile of latents [64][r] is first expanded to [64][D] with B_k[h] ([r][D]) and rotated with
// the standard RoPE table theta^(-2i/D) at positions j0 .. j0+63 before the logits are taken with
// the full-width, already rotated query.
//
// One CTA per (split, KV head, sequence), 256 threads:
//   expand:  thread (column d = tid % D', row set) accumulates rows in fp32 from shared B_k and latents
//   rotate:  thread per (row, pair): fp64 angle, fp64 sincos, fp32 rotation, in place
//   logits / softmax / PV: as in the shape-generic scan (one warp per position, warp g owns head g,
//   one thread per V channel).
// Partials go to the context workspace and are merged by the combine kernel below.
#include <math.h>

#include "rap_internal.h"

namespace {

constexpr int LR_TILE = 64;
constexpr int LR_THREADS = 256;
constexpr int LR_SMEM_MAX = 227 * 1024;   // the dynamic shared-memory limit is raised once, to the device maximum

template <typename T> __device__ __forceinline__ float ldf(const T* p);
template <> __device__ __forceinline__ float ldf<float>(const float* p) { return *p; }
template <> __device__ __forceinline__ float ldf<__nv_bfloat16>(const __nv_bfloat16* p) { return __bfloat162float(*p); }

template <typename T>
__global__ void __launch_bounds__(LR_THREADS)
lowrank_attn_kernel(const T* __restrict__ q_full, const T* __restrict__ k_latent, const T* __restrict__ bk,
                    const T* __restrict__ vc, const int32_t* __restrict__ seq_len, int Hq, int Hkv, int r, int dv,
                    int D, int S_cap, int pairing, double rope_theta, float qscale, int n_split,
                    float* __restrict__ ws) {
  extern __shared__ __align__(16) unsigned char lr_smem[];
  const int G = Hq / Hkv, half = D / 2, KS = D + 1;
  double* freq_s = reinterpret_cast<double*>(lr_smem);            // [D/2]
  float* bk_s = reinterpret_cast<float*>(freq_s + half);          // [r][D]
  float* lat_s = bk_s + r * D;                                    // [LR_TILE][r]
  float* kf_s = lat_s + LR_TILE * r;                              // [LR_TILE][D + 1]
  float* q_s = kf_s + LR_TILE * KS;                               // [G][D] pre-scaled by log2(e)/sqrt(D)
  float* s_s = q_s + G * D;                                       // [G][LR_TILE]
  float* alpha_s = s_s + G * LR_TILE;                             // [G]
  const int split = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  int len = seq_len[b];
  len = min(max(len, 0), S_cap);
  const int n_tiles = (len + LR_TILE - 1) / LR_TILE;
  const int tps = (n_tiles + n_split - 1) / n_split;
  const int tile_begin = split * tps, tile_end = min(n_tiles, tile_begin + tps);

  for (int i = tid; i < half; i += LR_THREADS) freq_s[i] = pow(rope_theta, -2.0 * (double)i / (double)D);
  for (int i = tid; i < r * D; i += LR_THREADS) bk_s[i] = ldf<T>(bk + (size_t)h * r * D + i);
  for (int i = tid; i < G * D; i += LR_THREADS) {
    const int g = i / D, d = i - g * D;
    q_s[i] = ldf<T>(q_full + ((size_t)b * Hq + h * G + g) * D + d) * qscale;
  }
  const T* lb = k_latent + ((size_t)b * Hkv + h) * (size_t)S_cap * r;
  const T* vb = vc + ((size_t)b * Hkv + h) * (size_t)S_cap * dv;
  float m_run = -INFINITY, l_run = 0.f;
  float acc[RAP_MAX_GROUP];
#pragma unroll
  for (int g = 0; g < RAP_MAX_GROUP; ++g) acc[g] = 0.f;
  __syncthreads();

  for (int tile = tile_begin; tile < tile_end; ++tile) {
    const int j0 = tile * LR_TILE;
    const int nj = min(LR_TILE, len - j0);
    // stage the latent rows of the tile
    for (int i = tid; i < nj * r; i += LR_THREADS) lat_s[i] = ldf<T>(lb + (size_t)j0 * r + i);
    __syncthreads();
    // expand: K_full[j][d] = sum_c latent[j][c] * B_k[c][d]
    for (int o = tid; o < nj * D; o += LR_THREADS) {
      const int j = o / D, d = o - j * D;
      float a = 0.f;
      for (int c = 0; c < r; ++c) a = fmaf(lat_s[j * r + c], bk_s[c * D + d], a);
      kf_s[j * KS + d] = a;
    }
    __syncthreads();
    // rotate pair i of row j at position j0 + j (Eq. 3, full table)
    for (int o = tid; o < nj * half; o += LR_THREADS) {
      const int j = o / half, i = o - j * half;
      const int d0 = pairing == RAP_PAIR_HALF ? i : 2 * i;
      const int d1 = pairing == RAP_PAIR_HALF ? i + half : 2 * i + 1;
      double sn, cs;
      sincos((double)(j0 + j) * freq_s[i], &sn, &cs);
      const float cf = (float)cs, sf = (float)sn;
      const float x = kf_s[j * KS + d0], y = kf_s[j * KS + d1];
      kf_s[j * KS + d0] = x * cf - y * sf;
      kf_s[j * KS + d1] = x * sf + y * cf;
    }
    __syncthreads();
    // logits: one warp per position, lanes over the D dims
    for (int j = warp; j < nj; j += LR_THREADS / 32) {
      float part[RAP_MAX_GROUP];
#pragma unroll
      for (int g = 0; g < RAP_MAX_GROUP; ++g) part[g] = 0.f;
      for (int d = lane; d < D; d += 32) {
        const float kv = kf_s[j * KS + d];
#pragma unroll
        for (int g = 0; g < RAP_MAX_GROUP; ++g)
          if (g < G) part[g] = fmaf(kv, q_s[g * D + d], part[g]);
      }
#pragma unroll
      for (int g = 0; g < RAP_MAX_GROUP; ++g) {
        if (g < G) {
          float v = part[g];
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
          if (lane == 0) s_s[g * LR_TILE + j] = v;
        }
      }
    }
    __syncthreads();
    if (warp < G) {
      const int g = warp;
      float mx = -INFINITY;
      for (int j = lane; j < nj; j += 32) mx = fmaxf(mx, s_s[g * LR_TILE + j]);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      const float m_new = fmaxf(m_run, mx);
      float sum = 0.f;
      for (int j = lane; j < nj; j += 32) {
        const float pj = exp2f(s_s[g * LR_TILE + j] - m_new);
        s_s[g * LR_TILE + j] = pj;
        sum += pj;
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
      const float alpha = exp2f(m_run - m_new);
      l_run = l_run * alpha + sum;
      m_run = m_new;
      if (lane == 0) alpha_s[g] = alpha;
    }
    __syncthreads();
    if (tid < dv) {
#pragma unroll
      for (int g = 0; g < RAP_MAX_GROUP; ++g)
        if (g < G) acc[g] *= alpha_s[g];
      for (int j = 0; j < nj; ++j) {
        const float vv = ldf<T>(vb + (size_t)(j0 + j) * dv + tid);
#pragma unroll
        for (int g = 0; g < RAP_MAX_GROUP; ++g)
          if (g < G) acc[g] = fmaf(s_s[g * LR_TILE + j], vv, acc[g]);
      }
    }
    __syncthreads();
  }
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

__global__ void lowrank_combine_kernel(const float* __restrict__ ws, int n_split, int dv, float* __restrict__ out) {
  const size_t bg = blockIdx.x;
  const float* base = ws + bg * n_split * (size_t)(dv + 2);
  float M = -INFINITY;
  for (int s = 0; s < n_split; ++s)
    if (base[(size_t)s * (dv + 2) + dv + 1] > 0.f) M = fmaxf(M, base[(size_t)s * (dv + 2) + dv]);
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

rap_status rap_launch_lowrank_fast(rap_ctx* ctx, const rap_lowrank_args& a, cudaStream_t st);

rap_status rap_launch_lowrank_attn(rap_ctx* ctx, const rap_lowrank_args& a, cudaStream_t st) {
  if (ctx->attn_variant == 0) {   // tensor-core rebuild + shape-specialised scan when the shape allows
    const rap_status f = rap_launch_lowrank_fast(ctx, a, st);
    if (f != RAP_EUNSUPPORTED) return f;
  }
  const int G = a.Hq / a.Hkv, D = a.head_dim;
  if (a.dv > LR_THREADS) return RAP_EUNSUPPORTED;
  int n_split = a.n_split;
  if (n_split <= 0) {
    const int n_tiles = (a.h_len_max + LR_TILE - 1) / LR_TILE;
    n_split = (4 * ctx->sm_count + a.B * a.Hkv - 1) / (a.B * a.Hkv);
    if (n_split > n_tiles / 4) n_split = n_tiles / 4;
    if (n_split > RAP_MAX_SPLIT) n_split = RAP_MAX_SPLIT;
    if (n_split < 1) n_split = 1;
  }
  const size_t smem = (size_t)(D / 2) * sizeof(double) +
                      (size_t)(a.r * D + LR_TILE * a.r + LR_TILE * (D + 1) + G * D + G * LR_TILE + G) * sizeof(float);
  if (smem > (size_t)LR_SMEM_MAX) return RAP_EUNSUPPORTED;
  const float qscale = (float)(1.4426950408889634 / sqrt((double)D));
  dim3 grid(n_split, a.Hkv, a.B);
  if (a.dtype == RAP_F32) {
    RAP_CUDA_TRY(ctx, rap_raise_smem(ctx, lowrank_attn_kernel<float>, LR_SMEM_MAX));
    lowrank_attn_kernel<float><<<grid, LR_THREADS, smem, st>>>(
        (const float*)a.q_full, (const float*)a.k_latent, (const float*)a.bk, (const float*)a.v, a.seq_len, a.Hq, a.Hkv,
        a.r, a.dv, D, a.S_cap, a.pairing, a.rope_theta, qscale, n_split, ctx->d_attn_ws);
  } else {
    RAP_CUDA_TRY(ctx, rap_raise_smem(ctx, lowrank_attn_kernel<__nv_bfloat16>, LR_SMEM_MAX));
    lowrank_attn_kernel<__nv_bfloat16><<<grid, LR_THREADS, smem, st>>>(
        (const __nv_bfloat16*)a.q_full, (const __nv_bfloat16*)a.k_latent, (const __nv_bfloat16*)a.bk,
        (const __nv_bfloat16*)a.v, a.seq_len, a.Hq, a.Hkv, a.r, a.dv, D, a.S_cap, a.pairing, a.rope_theta, qscale,
        n_split, ctx->d_attn_ws);
  }
  ctx->launches++;
  RAP_CUDA_TRY(ctx, cudaGetLastError());
  lowrank_combine_kernel<<<a.B * a.Hq, 128, 0, st>>>(ctx->d_attn_ws, n_split, a.dv, a.out);
  ctx->launches++;
  RAP_CUDA_TRY(ctx, cudaGetLastError());
  return RAP_OK;
}
