// Pruned QKV projection (Eq. 1 on the reduced widths), index-aware RoPE on the retained
// pairs (Eq. 3 with each pair's original frequency) and append into the compact cache.
//
// Decode-sized bf16 calls (T <= 32) run as ONE kernel: the tcgen05 GEMM of rap_proj_tc.cu with this epilogue
// fused in.  Every other call takes two stages on the caller's stream:
//   1. a GEMM  Y[ks][t][n] = sum_{k in split ks} X[t][k] * W~[n][k]   (fp32 results in the
//      context workspace; ks = reduction split so that weight streaming can use every SM),
//   2. an epilogue that sums the splits, adds the bias, rotates q~/k~ pairs, rounds once to the
//      storage dtype and scatters q~ / K row / V row.
// This file holds the CUDA-core GEMM that works for every shape and dtype, the epilogue, the
// offline weight gather and the sequence-length bump.  The tcgen05 GEMM lives in
// rap_proj_tc.cu and is selected by rap_launch_qkv_rope_append when its shape rules hold.
#include "rap_internal.h"

rap_status rap_launch_proj_tc(rap_ctx* ctx, const rap_proj_args& a, int* ksplit_out, cudaStream_t st);
rap_status rap_launch_proj_fused(rap_ctx* ctx, const rap_proj_args& a, cudaStream_t st);
rap_status rap_launch_gemm_tc(rap_ctx* ctx, const void* x, const void* w, int T, int K, int N, int* ksplit_out,
                              cudaStream_t st, int pdl);

namespace {

template <typename T> struct Vec16;
template <> struct Vec16<float> { static constexpr int N = 4; };
template <> struct Vec16<__nv_bfloat16> { static constexpr int N = 8; };

template <typename T> __device__ __forceinline__ void load16(const T* p, float* f);
template <> __device__ __forceinline__ void load16<float>(const float* p, float* f) {
  const float4 v = *reinterpret_cast<const float4*>(p);
  f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w;
}
template <> __device__ __forceinline__ void load16<__nv_bfloat16>(const __nv_bfloat16* p, float* f) {
  const uint4 v = *reinterpret_cast<const uint4*>(p);
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    f[2 * i] = __uint_as_float(w[i] << 16);
    f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}

// One warp per weight row n, TT token rows per block pass.  hidden * sizeof(T) is a multiple of 16.
constexpr int PROJ_TT = 8;
constexpr int PROJ_WARPS = 8;

template <typename T>
__global__ void __launch_bounds__(PROJ_WARPS * 32)
proj_generic_kernel(const T* __restrict__ x, const T* __restrict__ w, float* __restrict__ y, int Trows, int hidden,
                    int n_out) {
  constexpr int V = Vec16<T>::N;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n = blockIdx.x * PROJ_WARPS + warp;
  const int t0 = blockIdx.y * PROJ_TT;
  if (n >= n_out) return;
  float acc[PROJ_TT];
#pragma unroll
  for (int i = 0; i < PROJ_TT; ++i) acc[i] = 0.f;
  const T* wr = w + (size_t)n * hidden;
  for (int k = lane * V; k < hidden; k += 32 * V) {
    float wf[V];
    load16<T>(wr + k, wf);
#pragma unroll
    for (int i = 0; i < PROJ_TT; ++i) {
      if (t0 + i < Trows) {
        float xf[V];
        load16<T>(x + (size_t)(t0 + i) * hidden + k, xf);
#pragma unroll
        for (int j = 0; j < V; ++j) acc[i] = fmaf(wf[j], xf[j], acc[i]);
      }
    }
  }
#pragma unroll
  for (int i = 0; i < PROJ_TT; ++i) {
    float v = acc[i];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if (lane == 0 && t0 + i < Trows) y[(size_t)(t0 + i) * n_out + n] = v;
  }
}

template <typename T> __device__ __forceinline__ T to_storage(float v);
template <> __device__ __forceinline__ float to_storage<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 to_storage<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }
template <typename T> __device__ __forceinline__ float from_storage(T v);
template <> __device__ __forceinline__ float from_storage<float>(float v) { return v; }
template <> __device__ __forceinline__ float from_storage<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

// One thread per (row t, item): items are the H_kv * P retained pairs (c-th pair of KV head h) followed by
// the H_kv * d_v' value channels.  A pair item evaluates the angle pos * inv_freq[h][c] once (fp64) and
// rotates the k pair of head h and the q pairs of its G query heads with it.  y holds `ksplit` partial
// results, each [T][n_out].
template <typename T>
__global__ void rope_append_kernel(const float* __restrict__ y, int ksplit, const T* __restrict__ bias,
                                   const int32_t* __restrict__ seq_id, const int32_t* __restrict__ pos,
                                   const int32_t* __restrict__ slot, const double* __restrict__ inv_freq,
                                   T* __restrict__ q_out, T* __restrict__ k_cache, T* __restrict__ v_cache, int Trows,
                                   int Hq, int Hkv, int P2, int dv, int half_dim, int B_cache, int S_cap,
                                   int32_t* __restrict__ status) {
  const int P = P2 >> 1;
  const int n_pair_items = Hkv * P;
  const int n_items = n_pair_items + Hkv * dv;
  const int n_out = (Hq + Hkv) * P2 + Hkv * dv;
  const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (gid >= (long long)Trows * n_items) return;
  const int t = (int)(gid / n_items);
  const int item = (int)(gid - (long long)t * n_items);
  const int p = pos[t];
  const int sq = seq_id ? seq_id[t] : t;
  const int sl = slot ? slot[t] : p;
  const bool row_ok = (sq >= 0 && sq < B_cache && sl >= 0 && sl < S_cap);
  if (!row_ok && item == 0) {
    atomicCAS(&status[0], 0, (int)RAP_ECAPACITY);
    status[1] = t;
  }
  const size_t split_stride = (size_t)Trows * n_out;
  const float* yr = y + (size_t)t * n_out;
  if (item < n_pair_items) {
    const int h = item / P, c = item - h * P;
    const int G = Hq / Hkv;
    // angle and its reduction to [-pi, pi] in fp64 (positions reach 1e5: an fp32 angle would be off by 1e-2 rad),
    // sine and cosine of the reduced angle in fp32 (about 2e-7 absolute)
    const double ang = (double)p * inv_freq[h * half_dim + c];
    const double turns = rint(ang * 0.15915494309189535);                        // 1 / (2 pi)
    const double red = fma(-turns, 2.4492935982947064e-16, fma(-turns, 6.283185307179586, ang));   // 2 pi = hi + lo
    float sf, cf;
    sincosf((float)red, &sf, &cf);
    for (int j = 0; j <= G; ++j) {          // j < G: query head h*G + j; j == G: the key head itself
      const int head = j < G ? h * G + j : Hq + h;
      const int col = head * P2 + 2 * c;
      float a = 0.f, b = 0.f;
      for (int s = 0; s < ksplit; ++s) {
        a += yr[s * split_stride + col];          // (rows of y are only 4-byte aligned when n_out is odd)
        b += yr[s * split_stride + col + 1];
      }
      if (bias) { a += from_storage<T>(bias[col]); b += from_storage<T>(bias[col + 1]); }
      // one rounded product and one fused multiply-add each, spelled out: every kernel that rotates (this one, the
      // one-launch projection, the quantising epilogue) rounds the same way, whatever the compiler would contract
      const float ra = fmaf(-b, sf, __fmul_rn(a, cf));
      const float rb = fmaf(a, sf, __fmul_rn(b, cf));
      if (j < G) {
        T* dst = q_out + ((size_t)t * Hq + head) * P2 + 2 * c;
        dst[0] = to_storage<T>(ra);
        dst[1] = to_storage<T>(rb);
      } else if (row_ok) {
        T* dst = k_cache + (((size_t)sq * Hkv + h) * S_cap + sl) * P2 + 2 * c;
        dst[0] = to_storage<T>(ra);
        dst[1] = to_storage<T>(rb);
      }
    }
  } else if (row_ok) {
    const int vi = item - n_pair_items;
    const int h = vi / dv, c = vi - h * dv;
    const int col = (Hq + Hkv) * P2 + vi;
    float a = 0.f;
    for (int s = 0; s < ksplit; ++s) a += yr[s * split_stride + col];
    if (bias) a += from_storage<T>(bias[col]);
    v_cache[(((size_t)sq * Hkv + h) * S_cap + sl) * dv + c] = to_storage<T>(a);
  }
}

// Offline row gather: W~_qkv row n <- the dense row RAPIndex / v_idx points at (16-byte chunks).
__global__ void pack_rows_kernel(const uint4* __restrict__ wq, const uint4* __restrict__ wk, const uint4* __restrict__ wv,
                                 const int32_t* __restrict__ k_dim_idx, const int32_t* __restrict__ v_idx,
                                 uint4* __restrict__ dst, int Hq, int Hkv, int D, int P2, int dv, int row_chunks) {
  const int n = blockIdx.x;
  const int G = Hq / Hkv;
  const uint4* src;
  if (n < Hq * P2) {
    const int g = n / P2, r = n - g * P2;
    src = wq + (size_t)(g * D + k_dim_idx[(g / G) * D + r]) * row_chunks;
  } else if (n < (Hq + Hkv) * P2) {
    const int m = n - Hq * P2, h = m / P2, r = m - h * P2;
    src = wk + (size_t)(h * D + k_dim_idx[h * D + r]) * row_chunks;
  } else {
    const int m = n - (Hq + Hkv) * P2, h = m / dv, r = m - h * dv;
    src = wv + (size_t)(h * D + v_idx[h * D + r]) * row_chunks;
  }
  uint4* d = dst + (size_t)n * row_chunks;
  for (int i = threadIdx.x; i < row_chunks; i += blockDim.x) d[i] = src[i];
}

template <typename T>
__global__ void pack_bias_kernel(const T* __restrict__ bq, const T* __restrict__ bk, const T* __restrict__ bv,
                                 const int32_t* __restrict__ k_dim_idx, const int32_t* __restrict__ v_idx,
                                 T* __restrict__ dst, int Hq, int Hkv, int D, int P2, int dv) {
  const int n = blockIdx.x * blockDim.x + threadIdx.x;
  const int n_out = (Hq + Hkv) * P2 + Hkv * dv;
  if (n >= n_out) return;
  const int G = Hq / Hkv;
  if (n < Hq * P2) {
    const int g = n / P2, r = n - g * P2;
    dst[n] = bq[g * D + k_dim_idx[(g / G) * D + r]];
  } else if (n < (Hq + Hkv) * P2) {
    const int m = n - Hq * P2, h = m / P2, r = m - h * P2;
    dst[n] = bk[h * D + k_dim_idx[h * D + r]];
  } else {
    const int m = n - (Hq + Hkv) * P2, h = m / dv, r = m - h * dv;
    dst[n] = bv[h * D + v_idx[h * D + r]];
  }
}

// Offline column gather of the output projection (Algorithm 1: W~_o = E_v W_o): dst[n][g*dv + c] =
// src[n][g*D + v_idx[g/G][c]], one block per output row n.
template <typename T>
__global__ void pack_wo_kernel(const T* __restrict__ wo, const int32_t* __restrict__ v_idx, T* __restrict__ dst, int Hq,
                               int Hkv, int D, int dv) {
  const int n = blockIdx.x, G = Hq / Hkv;
  const T* src = wo + (size_t)n * Hq * D;
  T* d = dst + (size_t)n * Hq * dv;
  for (int i = threadIdx.x; i < Hq * dv; i += blockDim.x) {
    const int g = i / dv, c = i - g * dv;
    d[i] = src[g * D + v_idx[(g / G) * D + c]];
  }
}

__global__ void cast_bf16_kernel(const float* __restrict__ src, __nv_bfloat16* __restrict__ dst, size_t n) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");     // a GEMM launched behind this may start its prologue
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) dst[i] = __float2bfloat16_rn(src[i]);
}

// y[i] = storage( sum over the reduction splits of ws[ks][i] )
template <typename T>
__global__ void sum_splits_kernel(const float* __restrict__ ws, int ksplit, size_t n, T* __restrict__ y) {
  // (launched behind the GEMM with programmatic serialization in rap_out_proj: the partial results are awaited here)
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  float a = 0.f;
  for (int s = 0; s < ksplit; ++s) a += ws[(size_t)s * n + i];
  y[i] = to_storage<T>(a);
}

__global__ void advance_kernel(int32_t* seq_len, int B) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b < B) seq_len[b] += 1;
}

template <typename T>
rap_status run_generic(rap_ctx* ctx, const rap_proj_args& a, int n_out, cudaStream_t st) {
  dim3 grid((n_out + PROJ_WARPS - 1) / PROJ_WARPS, (a.T + PROJ_TT - 1) / PROJ_TT);
  proj_generic_kernel<T><<<grid, PROJ_WARPS * 32, 0, st>>>((const T*)a.x, (const T*)a.w, ctx->d_proj_ws, a.T,
                                                           a.hidden, n_out);
  ctx->launches++;
  RAP_CUDA_TRY(ctx, cudaGetLastError());
  return RAP_OK;
}

template <typename T>
rap_status run_epilogue(rap_ctx* ctx, const rap_proj_args& a, int ksplit, cudaStream_t st) {
  const int P = a.P2 / 2;
  const long long total = (long long)a.T * (a.Hkv * P + a.Hkv * a.dv);
  const int threads = 256;
  const unsigned blocks = (unsigned)((total + threads - 1) / threads);
  rope_append_kernel<T><<<blocks, threads, 0, st>>>(ctx->d_proj_ws, ksplit, (const T*)a.bias, a.seq_id, a.pos, a.slot,
                                                    a.inv_freq, (T*)a.q_out, (T*)a.k_cache, (T*)a.v_cache, a.T, a.Hq,
                                                    a.Hkv, a.P2, a.dv, a.half_dim, a.B_cache, a.S_cap, ctx->d_status);
  ctx->launches++;
  RAP_CUDA_TRY(ctx, cudaGetLastError());
  return RAP_OK;
}

}  // namespace

rap_status rap_launch_qkv_rope_append(rap_ctx* ctx, const rap_proj_args& a, cudaStream_t st) {
  const int n_out = (a.Hq + a.Hkv) * a.P2 + a.Hkv * a.dv;
  int ksplit = 1;
  rap_status s = RAP_EUNSUPPORTED;
  if (a.dtype == RAP_BF16 && ctx->proj_variant != 1) {      // decode-sized calls: one launch, epilogue fused in
    s = rap_launch_proj_fused(ctx, a, st);
    if (s != RAP_EUNSUPPORTED) return s;
  }
  if (a.dtype == RAP_BF16) s = rap_launch_proj_tc(ctx, a, &ksplit, st);
  if (s == RAP_EUNSUPPORTED) {
    ksplit = 1;
    s = a.dtype == RAP_F32 ? run_generic<float>(ctx, a, n_out, st) : run_generic<__nv_bfloat16>(ctx, a, n_out, st);
  }
  if (s != RAP_OK) return s;
  return a.dtype == RAP_F32 ? run_epilogue<float>(ctx, a, ksplit, st) : run_epilogue<__nv_bfloat16>(ctx, a, ksplit, st);
}

// Y[T][n_out] (fp32, context workspace, one split) with the CUDA-core GEMM: any dtype and shape.
rap_status rap_launch_proj_generic(rap_ctx* ctx, const rap_proj_args& a, cudaStream_t st) {
  const int n_out = (a.Hq + a.Hkv) * a.P2 + a.Hkv * a.dv;
  return a.dtype == RAP_F32 ? run_generic<float>(ctx, a, n_out, st) : run_generic<__nv_bfloat16>(ctx, a, n_out, st);
}

rap_status rap_launch_pack(rap_ctx* ctx, int32_t layer, const void* wq, const void* wk, const void* wv,
                           const int32_t* k_dim_idx, const int32_t* v_idx, void* w_qkv, const void* bq,
                           const void* bk, const void* bv, void* bias, cudaStream_t st) {
  const rap_model_desc& d = ctx->desc;
  const int P2 = 2 * ctx->n_pairs[layer], dv = ctx->n_vch[layer], D = d.head_dim;
  const int n_out = (d.n_q_heads + d.n_kv_heads) * P2 + d.n_kv_heads * dv;
  const int row_chunks = d.hidden * rap_elem_bytes(d.dtype) / 16;
  const int32_t* kd = k_dim_idx + (size_t)layer * d.n_kv_heads * D;
  const int32_t* vi = v_idx + (size_t)layer * d.n_kv_heads * D;
  pack_rows_kernel<<<n_out, 128, 0, st>>>((const uint4*)wq, (const uint4*)wk, (const uint4*)wv, kd, vi,
                                          (uint4*)w_qkv, d.n_q_heads, d.n_kv_heads, D, P2, dv, row_chunks);
  ctx->launches++;
  RAP_CUDA_TRY(ctx, cudaGetLastError());
  if (bias) {
    const int blocks = (n_out + 255) / 256;
    if (d.dtype == RAP_F32)
      pack_bias_kernel<float><<<blocks, 256, 0, st>>>((const float*)bq, (const float*)bk, (const float*)bv, kd, vi,
                                                      (float*)bias, d.n_q_heads, d.n_kv_heads, D, P2, dv);
    else
      pack_bias_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>((const __nv_bfloat16*)bq, (const __nv_bfloat16*)bk,
                                                              (const __nv_bfloat16*)bv, kd, vi, (__nv_bfloat16*)bias,
                                                              d.n_q_heads, d.n_kv_heads, D, P2, dv);
    ctx->launches++;
    RAP_CUDA_TRY(ctx, cudaGetLastError());
  }
  return RAP_OK;
}

rap_status rap_launch_advance(rap_ctx* ctx, int32_t* seq_len, int32_t B, cudaStream_t st) {
  advance_kernel<<<(B + 127) / 128, 128, 0, st>>>(seq_len, B);
  ctx->launches++;
  RAP_CUDA_TRY(ctx, cudaGetLastError());
  return RAP_OK;
}

rap_status rap_launch_pack_wo(rap_ctx* ctx, int32_t layer, const void* wo, const int32_t* v_idx, void* dst, cudaStream_t st) {
  const rap_model_desc& d = ctx->desc;
  const int dv = ctx->n_vch[layer], D = d.head_dim;
  const int32_t* vi = v_idx + (size_t)layer * d.n_kv_heads * D;
  if (d.dtype == RAP_F32)
    pack_wo_kernel<float><<<d.hidden, 256, 0, st>>>((const float*)wo, vi, (float*)dst, d.n_q_heads, d.n_kv_heads, D, dv);
  else
    pack_wo_kernel<__nv_bfloat16><<<d.hidden, 256, 0, st>>>((const __nv_bfloat16*)wo, vi, (__nv_bfloat16*)dst,
                                                            d.n_q_heads, d.n_kv_heads, D, dv);
  ctx->launches++;
  RAP_CUDA_TRY(ctx, cudaGetLastError());
  return RAP_OK;
}

// y[T][hidden] = attn_out[T][Hq*dv] (fp32) * W~_o[hidden][Hq*dv]^T, result in the storage dtype
rap_status rap_launch_out_proj(rap_ctx* ctx, int32_t layer, int32_t T, const float* attn_out, const void* wo_tilde,
                               void* y, cudaStream_t st) {
  const rap_model_desc& d = ctx->desc;
  const int K = d.n_q_heads * ctx->n_vch[layer], N = d.hidden;
  const size_t n = (size_t)T * N;
  if ((size_t)T * N * sizeof(float) > ctx->proj_ws_bytes) return RAP_ESHAPE;
  int ksplit = 1;
  if (d.dtype == RAP_BF16) {
    const size_t nx = (size_t)T * K;
    cast_bf16_kernel<<<(unsigned)((nx + 255) / 256), 256, 0, st>>>(attn_out, (__nv_bfloat16*)ctx->d_oproj_x, nx);
    ctx->launches++;
    RAP_CUDA_TRY(ctx, cudaGetLastError());
    // the three launches are chained with programmatic serialization: the GEMM's prologue and first weight tiles
    // overlap the cast, the split sum is resident and waiting when the GEMM ends
    rap_status s = rap_launch_gemm_tc(ctx, ctx->d_oproj_x, wo_tilde, T, K, N, &ksplit, st, 2);
    if (s == RAP_EUNSUPPORTED) {
      if ((K * 2) % 16) return RAP_EUNSUPPORTED;
      ksplit = 1;
      dim3 grid((N + PROJ_WARPS - 1) / PROJ_WARPS, (T + PROJ_TT - 1) / PROJ_TT);
      proj_generic_kernel<__nv_bfloat16><<<grid, PROJ_WARPS * 32, 0, st>>>(
          (const __nv_bfloat16*)ctx->d_oproj_x, (const __nv_bfloat16*)wo_tilde, ctx->d_proj_ws, T, K, N);
      ctx->launches++;
      RAP_CUDA_TRY(ctx, cudaGetLastError());
    } else if (s != RAP_OK) {
      return s;
    }
    {
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3((unsigned)((n + 255) / 256), 1, 1);
      cfg.blockDim = dim3(256, 1, 1);
      cfg.stream = st;
      cudaLaunchAttribute attr[1];
      attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
      attr[0].val.programmaticStreamSerializationAllowed = 1;
      cfg.attrs = attr;
      cfg.numAttrs = 1;
      RAP_CUDA_TRY(ctx, cudaLaunchKernelEx(&cfg, sum_splits_kernel<__nv_bfloat16>, (const float*)ctx->d_proj_ws, ksplit, n,
                                           (__nv_bfloat16*)y));
    }
  } else {
    if ((K * 4) % 16) return RAP_EUNSUPPORTED;
    dim3 grid((N + PROJ_WARPS - 1) / PROJ_WARPS, (T + PROJ_TT - 1) / PROJ_TT);
    proj_generic_kernel<float><<<grid, PROJ_WARPS * 32, 0, st>>>(attn_out, (const float*)wo_tilde, ctx->d_proj_ws, T, K, N);
    ctx->launches++;
    RAP_CUDA_TRY(ctx, cudaGetLastError());
    sum_splits_kernel<float><<<(unsigned)((n + 255) / 256), 256, 0, st>>>(ctx->d_proj_ws, 1, n, (float*)y);
  }
  ctx->launches++;
  RAP_CUDA_TRY(ctx, cudaGetLastError());
  return RAP_OK;
}
