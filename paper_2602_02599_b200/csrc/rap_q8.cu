// Composition of the pruned cache with 8-bit cache quantisation (the paper calls pruning the cache width and
// lowering the bit-width of what is cached orthogonal, and composes pruning with a plain symmetric round-to-nearest
// quantiser).  The reading taken here: every compact cache row keeps int8 codes in [-127, 127] and one scale,
//     s = bf16(max|x| / 127),   c_i = clip(rint(x_i / s), -127, 127),   x_i ~ c_i s,
// decided in fp32.  A quantised row of width W occupies rap_q8_row_bytes(W) = (W + 2) rounded up to 4 bytes: the
// codes, padding, and the bf16 scale in the last two bytes, so a block of rows is one contiguous byte range that
// carries its scales along.  A code is stored as the unsigned byte c + 128 (1 .. 255): that byte under the high byte
// 0x64 is the fp16 number 1152 + c, which is how the tensor-core scan turns codes into MMA operands without a
// conversion instruction.
//
// This file holds the quantiser (rap_quantize_rows), the RoPE / append epilogue that quantises the new K and V rows
// straight from their fp32 values (rap_qkv_rope_append_q8; the projection GEMM is the one of rap_qkv_rope_append),
// and the shape-generic split-KV attention over a quantised cache with its combine step (rap_decode_attn_q8 for
// head shapes without a specialised scan, and the cross-check of the specialised one).
#include <math.h>

#include "rap_internal.h"

rap_status rap_launch_proj_tc(rap_ctx* ctx, const rap_proj_args& a, int* ksplit_out, cudaStream_t st);
rap_status rap_launch_proj_generic(rap_ctx* ctx, const rap_proj_args& a, cudaStream_t st);
rap_status rap_launch_attn_q8_mma(rap_ctx* ctx, const rap_attn_args& a, int n_split, cudaStream_t st);

namespace {

__device__ __forceinline__ float q8_ld(const float* p) { return *p; }
__device__ __forceinline__ float q8_ld(const __nv_bfloat16* p) { return __bfloat162float(*p); }
__device__ __forceinline__ void q8_st(float* p, float v) { *p = v; }
__device__ __forceinline__ void q8_st(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
// the scale of a row with largest magnitude amax, as stored (a bf16 number) -- fp32 division, one rounding to bf16
__device__ __forceinline__ float q8_scale(float amax) { return __bfloat162float(__float2bfloat16_rn(__fdiv_rn(amax, 127.0f))); }
// the stored byte of x under scale s: code + 128
__device__ __forceinline__ unsigned char q8_code(float x, float s) {
  if (!(s > 0.f)) return 128;
  const float c = rintf(__fdiv_rn(x, s));
  return (unsigned char)(128 + (int)fminf(fmaxf(c, -127.f), 127.f));
}
__device__ __forceinline__ float q8_value(unsigned char byte) { return (float)((int)byte - 128); }
// codes are written by the lanes that own them; lane 0 adds the padding and the scale
__device__ __forceinline__ void q8_finish_row(unsigned char* row, int W, int row_bytes, float s, int lane) {
  if (lane == 0) {
    for (int i = W; i < row_bytes - 2; ++i) row[i] = 0;
    *reinterpret_cast<__nv_bfloat16*>(row + row_bytes - 2) = __float2bfloat16_rn(s);     // exact: s is a bf16 number
  }
}

// One warp per row: src [n_rows][W] (fp32 or bf16), dst [n_rows][row_bytes].
template <typename T>
__global__ void __launch_bounds__(256) quantize_rows_kernel(const T* __restrict__ src, unsigned char* __restrict__ dst,
                                                            long long n_rows, int W, int row_bytes) {
  const long long row = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= n_rows) return;
  const T* x = src + row * W;
  float amax = 0.f;
  for (int i = lane; i < W; i += 32) amax = fmaxf(amax, fabsf(q8_ld(x + i)));
  const float s = q8_scale(warp_max(amax));
  unsigned char* d = dst + row * row_bytes;
  for (int i = lane; i < W; i += 32) d[i] = q8_code(q8_ld(x + i), s);
  q8_finish_row(d, W, row_bytes, s, lane);
}

// RoPE / append epilogue with quantisation.  One warp per (row t, item): items are the H_q query heads (rotated,
// rounded to the storage dtype, written to q_out as in the unquantised path), then the H_kv key heads (rotated in
// fp32, quantised, appended), then the H_kv value heads (quantised, appended).  y holds `ksplit` partial results,
// each [T][n_out].  P <= 128, d_v' <= 256: a lane keeps at most four pairs / eight channels.
template <typename T>
__global__ void __launch_bounds__(256)
rope_append_q8_kernel(const float* __restrict__ y, int ksplit, const T* __restrict__ bias, const int32_t* __restrict__ seq_id,
                      const int32_t* __restrict__ pos, const int32_t* __restrict__ slot, const double* __restrict__ inv_freq,
                      T* __restrict__ q_out, unsigned char* __restrict__ k8, unsigned char* __restrict__ v8, int Trows, int Hq,
                      int Hkv, int P2, int dv, int half_dim, int B_cache, int S_cap, int k_row_bytes, int v_row_bytes,
                      int32_t* __restrict__ status) {
  // launched behind the GEMM with programmatic serialization inside a decode step: nothing above this line touches
  // memory; the GEMM's results (and, through the GEMM, the end of the scan before it) are awaited here
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int items = Hq + 2 * Hkv;
  const long long wid = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (wid >= (long long)Trows * items) return;
  const int t = (int)(wid / items), item = (int)(wid - (long long)t * items);
  const int P = P2 >> 1, G = Hq / Hkv;
  const int n_out = (Hq + Hkv) * P2 + Hkv * dv;
  const int p = pos[t];
  const int sq = seq_id ? seq_id[t] : t;
  const int sl = slot ? slot[t] : p;
  const bool row_ok = (sq >= 0 && sq < B_cache && sl >= 0 && sl < S_cap);
  if (!row_ok && item == 0 && lane == 0) {
    atomicCAS(&status[0], 0, (int)RAP_ECAPACITY);
    status[1] = t;
  }
  const size_t split_stride = (size_t)Trows * n_out;
  const float* yr = y + (size_t)t * n_out;
  if (item < Hq + Hkv) {
    const bool is_q = item < Hq;
    const int h = is_q ? item / G : item - Hq;                 // KV head whose frequencies apply
    const int col0 = item * P2;                                // q heads, then k heads: item * 2P either way
    float ra[4], rb[4];
    float amax = 0.f;
    // every partial of this lane's pairs first (independent loads), then the sums in split order and the bias
    float pa[4][RAP_MAX_KSPLIT], pb[4][RAP_MAX_KSPLIT];
#pragma unroll
    for (int k = 0; k < 4; ++k)
#pragma unroll
      for (int s = 0; s < RAP_MAX_KSPLIT; ++s) {
        const int c = lane + 32 * k;
        const bool on = c < P && s < ksplit;
        pa[k][s] = on ? yr[s * split_stride + col0 + 2 * c] : 0.f;
        pb[k][s] = on ? yr[s * split_stride + col0 + 2 * c + 1] : 0.f;
      }
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int c = lane + 32 * k;
      ra[k] = rb[k] = 0.f;
      if (c < P) {
        // fp64 angle and reduction to [-pi, pi], fp32 sine and cosine of the reduced angle (as in the unquantised path)
        const double ang = (double)p * inv_freq[h * half_dim + c];
        const double turns = rint(ang * 0.15915494309189535);
        const double red = fma(-turns, 2.4492935982947064e-16, fma(-turns, 6.283185307179586, ang));
        float sf, cf;
        sincosf((float)red, &sf, &cf);
        float a = 0.f, b = 0.f;
#pragma unroll
        for (int s = 0; s < RAP_MAX_KSPLIT; ++s)
          if (s < ksplit) { a += pa[k][s]; b += pb[k][s]; }
        if (bias) { a += q8_ld(bias + col0 + 2 * c); b += q8_ld(bias + col0 + 2 * c + 1); }
        ra[k] = fmaf(-b, sf, __fmul_rn(a, cf));          // the same roundings as the unquantised kernels
        rb[k] = fmaf(a, sf, __fmul_rn(b, cf));
        amax = fmaxf(amax, fmaxf(fabsf(ra[k]), fabsf(rb[k])));
      }
    }
    if (is_q) {
      T* dst = q_out + ((size_t)t * Hq + item) * P2;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int c = lane + 32 * k;
        if (c < P) {
          q8_st(dst + 2 * c, ra[k]);
          q8_st(dst + 2 * c + 1, rb[k]);
        }
      }
    } else if (row_ok) {
      const float s = q8_scale(warp_max(amax));
      unsigned char* d = k8 + (((size_t)sq * Hkv + h) * S_cap + sl) * (size_t)k_row_bytes;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int c = lane + 32 * k;
        if (c < P) {
          d[2 * c] = q8_code(ra[k], s);
          d[2 * c + 1] = q8_code(rb[k], s);
        }
      }
      q8_finish_row(d, P2, k_row_bytes, s, lane);
    }
  } else if (row_ok) {
    const int h = item - Hq - Hkv;
    const int col0 = (Hq + Hkv) * P2 + h * dv;
    float v[8];
    float amax = 0.f;
    float pv[8][RAP_MAX_KSPLIT];
#pragma unroll
    for (int k = 0; k < 8; ++k)
#pragma unroll
      for (int s = 0; s < RAP_MAX_KSPLIT; ++s) pv[k][s] = (lane + 32 * k < dv && s < ksplit) ? yr[s * split_stride + col0 + lane + 32 * k] : 0.f;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const int c = lane + 32 * k;
      float a = 0.f;
#pragma unroll
      for (int s = 0; s < RAP_MAX_KSPLIT; ++s)
        if (s < ksplit) a += pv[k][s];
      if (bias && c < dv) a += q8_ld(bias + col0 + c);
      v[k] = c < dv ? a : 0.f;
      amax = fmaxf(amax, fabsf(v[k]));
    }
    const float s = q8_scale(warp_max(amax));
    unsigned char* d = v8 + (((size_t)sq * Hkv + h) * S_cap + sl) * (size_t)v_row_bytes;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const int c = lane + 32 * k;
      if (c < dv) d[c] = q8_code(v[k], s);
    }
    q8_finish_row(d, dv, v_row_bytes, s, lane);
  }
}

// ---- shape-generic split-KV attention over a quantised cache ------------------------------------------------------
constexpr int Q8G_TILE = 64;
constexpr int Q8G_THREADS = 256;

template <typename T>
__global__ void __launch_bounds__(Q8G_THREADS)
attn_q8_generic_kernel(const T* __restrict__ q, const unsigned char* __restrict__ k8, const unsigned char* __restrict__ v8,
                       const int32_t* __restrict__ seq_len, int len_add, int Hq, int Hkv, int P2, int dv, int S_cap,
                       int k_row_bytes, int v_row_bytes, float qscale, int n_split, float* __restrict__ ws) {
  extern __shared__ float smem[];
  const int G = Hq / Hkv;
  float* q_s = smem;                      // [G][P2] pre-scaled by log2(e)/sqrt(D)
  float* s_s = q_s + G * P2;              // [G][TILE] logits, then weights
  float* vs_s = s_s + G * Q8G_TILE;       // [TILE] V scales of the tile
  float* alpha_s = vs_s + Q8G_TILE;       // [G]
  const int split = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  int len = seq_len[b] + len_add;
  len = min(max(len, 0), S_cap);
  const int n_tiles = (len + Q8G_TILE - 1) / Q8G_TILE;
  const int tps = (n_tiles + n_split - 1) / n_split;
  const int tile_begin = split * tps, tile_end = min(n_tiles, tile_begin + tps);
  for (int i = tid; i < G * P2; i += Q8G_THREADS) {
    const int g = i / P2, d = i - g * P2;
    q_s[i] = q8_ld(q + ((size_t)b * Hq + h * G + g) * P2 + d) * qscale;
  }
  const unsigned char* kb = k8 + ((size_t)b * Hkv + h) * (size_t)S_cap * k_row_bytes;
  const unsigned char* vb = v8 + ((size_t)b * Hkv + h) * (size_t)S_cap * v_row_bytes;
  float m_run = -INFINITY, l_run = 0.f;
  float acc[RAP_MAX_GROUP];
#pragma unroll
  for (int g = 0; g < RAP_MAX_GROUP; ++g) acc[g] = 0.f;
  __syncthreads();
  for (int tile = tile_begin; tile < tile_end; ++tile) {
    const int j0 = tile * Q8G_TILE;
    const int nj = min(Q8G_TILE, len - j0);
    for (int j = warp; j < nj; j += Q8G_THREADS / 32) {
      const unsigned char* kr = kb + (size_t)(j0 + j) * k_row_bytes;
      const float ks = __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(kr + k_row_bytes - 2));
      float part[RAP_MAX_GROUP];
#pragma unroll
      for (int g = 0; g < RAP_MAX_GROUP; ++g) part[g] = 0.f;
      for (int d = lane; d < P2; d += 32) {
        const float kv = q8_value(kr[d]);
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
          if (lane == 0) s_s[g * Q8G_TILE + j] = v * ks;
        }
      }
      if (lane == 0) vs_s[j] = __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(vb + (size_t)(j0 + j) * v_row_bytes + v_row_bytes - 2));
    }
    __syncthreads();
    if (warp < G) {
      const int g = warp;
      float mx = -INFINITY;
      for (int j = lane; j < nj; j += 32) mx = fmaxf(mx, s_s[g * Q8G_TILE + j]);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      const float m_new = fmaxf(m_run, mx);
      float sum = 0.f;
      for (int j = lane; j < nj; j += 32) {
        const float pw = exp2f(s_s[g * Q8G_TILE + j] - m_new);
        s_s[g * Q8G_TILE + j] = pw;
        sum += pw;
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
        const float vv = q8_value(vb[(size_t)(j0 + j) * v_row_bytes + tid]) * vs_s[j];
#pragma unroll
        for (int g = 0; g < RAP_MAX_GROUP; ++g)
          if (g < G) acc[g] = fmaf(s_s[g * Q8G_TILE + j], vv, acc[g]);
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

// out[b][g][c] = sum_s 2^(m_s - M) acc_s[c] / sum_s 2^(m_s - M) l_s ; empty splits have l = 0.
__global__ void attn_q8_combine_kernel(const float* __restrict__ ws, int n_split, int dv, float* __restrict__ out) {
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

rap_status rap_launch_quantize_rows(rap_ctx* ctx, int32_t dtype_in, long long n_rows, int W, const void* src, void* dst,
                                    cudaStream_t st) {
  const int rb = (int)rap_q8_row_bytes(W);
  const unsigned blocks = (unsigned)((n_rows + 7) / 8);
  if (dtype_in == RAP_F32)
    quantize_rows_kernel<float><<<blocks, 256, 0, st>>>((const float*)src, (unsigned char*)dst, n_rows, W, rb);
  else
    quantize_rows_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>((const __nv_bfloat16*)src, (unsigned char*)dst, n_rows, W, rb);
  ctx->launches++;
  RAP_CUDA_TRY(ctx, cudaGetLastError());
  return RAP_OK;
}

// a.k_cache / a.v_cache are the quantised caches of this layer
rap_status rap_launch_qkv_rope_append_q8(rap_ctx* ctx, const rap_proj_args& a, cudaStream_t st) {
  int ksplit = 1;
  rap_status s = RAP_EUNSUPPORTED;
  if (a.dtype == RAP_BF16) s = rap_launch_proj_tc(ctx, a, &ksplit, st);
  if (s == RAP_EUNSUPPORTED) {
    ksplit = 1;
    s = rap_launch_proj_generic(ctx, a, st);
  }
  if (s != RAP_OK) return s;
  const long long warps = (long long)a.T * (a.Hq + 2 * a.Hkv);
  const unsigned blocks = (unsigned)((warps + 7) / 8);
  const int krb = (int)rap_q8_row_bytes(a.P2), vrb = (int)rap_q8_row_bytes(a.dv);
  // inside a decode step (a.pdl): launched behind the tcgen05 GEMM with programmatic serialization, so that its launch
  // overlaps the GEMM's tail; the kernel waits for the GEMM before it touches memory (the CUDA-core GEMM of the other
  // path never triggers early, which makes the attribute a no-op there)
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(blocks, 1, 1);
  cfg.blockDim = dim3(256, 1, 1);
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = a.pdl ? 1 : 0;
  const float* y = ctx->d_proj_ws;
  unsigned char* k8 = (unsigned char*)a.k_cache;
  unsigned char* v8 = (unsigned char*)a.v_cache;
  if (a.dtype == RAP_F32)
    RAP_CUDA_TRY(ctx, cudaLaunchKernelEx(&cfg, rope_append_q8_kernel<float>, y, ksplit, (const float*)a.bias, a.seq_id, a.pos,
                                         a.slot, a.inv_freq, (float*)a.q_out, k8, v8, a.T, a.Hq, a.Hkv, a.P2, a.dv,
                                         a.half_dim, a.B_cache, a.S_cap, krb, vrb, ctx->d_status));
  else
    RAP_CUDA_TRY(ctx, cudaLaunchKernelEx(&cfg, rope_append_q8_kernel<__nv_bfloat16>, y, ksplit, (const __nv_bfloat16*)a.bias,
                                         a.seq_id, a.pos, a.slot, a.inv_freq, (__nv_bfloat16*)a.q_out, k8, v8, a.T, a.Hq, a.Hkv,
                                         a.P2, a.dv, a.half_dim, a.B_cache, a.S_cap, krb, vrb, ctx->d_status));
  ctx->launches++;
  return RAP_OK;
}

// a.k / a.v are the quantised caches; a.q has the storage dtype
rap_status rap_launch_attn_q8(rap_ctx* ctx, const rap_attn_args& a, cudaStream_t st) {
  if (a.dtype == RAP_BF16 && ctx->attn_variant != 1) {
    const rap_status s = rap_launch_attn_q8_mma(ctx, a, a.n_split, st);
    if (s != RAP_EUNSUPPORTED || ctx->attn_variant == 4) return s;
  }
  if (a.B > 65535 || a.Hkv > 65535) return RAP_ESHAPE;
  const int G = a.Hq / a.Hkv;
  int n_split = a.n_split;
  if (n_split <= 0) {      // a few CTAs per SM, splits of at least four tiles
    const int n_tiles = (a.h_len_max + Q8G_TILE - 1) / Q8G_TILE;
    n_split = (8 * ctx->sm_count + a.B * a.Hkv - 1) / (a.B * a.Hkv);
    if (n_split > n_tiles / 4) n_split = n_tiles / 4;
    if (n_split > RAP_MAX_SPLIT) n_split = RAP_MAX_SPLIT;
    if (n_split < 1) n_split = 1;
  }
  const float qscale = (float)(1.4426950408889634 / sqrt((double)a.head_dim));
  const size_t smem = (size_t)(G * a.P2 + G * Q8G_TILE + Q8G_TILE + G) * sizeof(float);
  const int krb = (int)rap_q8_row_bytes(a.P2), vrb = (int)rap_q8_row_bytes(a.dv);
  dim3 grid(n_split, a.Hkv, a.B);
  if (a.dtype == RAP_F32)
    attn_q8_generic_kernel<float><<<grid, Q8G_THREADS, smem, st>>>((const float*)a.q, (const unsigned char*)a.k,
                                                                   (const unsigned char*)a.v, a.seq_len, a.len_add, a.Hq,
                                                                   a.Hkv, a.P2, a.dv, a.S_cap, krb, vrb, qscale, n_split,
                                                                   ctx->d_attn_ws);
  else
    attn_q8_generic_kernel<__nv_bfloat16><<<grid, Q8G_THREADS, smem, st>>>(
        (const __nv_bfloat16*)a.q, (const unsigned char*)a.k, (const unsigned char*)a.v, a.seq_len, a.len_add, a.Hq, a.Hkv,
        a.P2, a.dv, a.S_cap, krb, vrb, qscale, n_split, ctx->d_attn_ws);
  ctx->launches++;
  RAP_CUDA_TRY(ctx, cudaGetLastError());
  attn_q8_combine_kernel<<<a.B * a.Hq, 128, 0, st>>>(ctx->d_attn_ws, n_split, a.dv, a.out);
  ctx->launches++;
  RAP_CUDA_TRY(ctx, cudaGetLastError());
  return RAP_OK;
}
