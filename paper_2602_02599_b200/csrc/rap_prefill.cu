// Causal attention of a block of T new tokens per sequence over the reduced dims (Eq. 2 for every t
// of the block, on 2P retained K dims and d_v' retained V channels, scale 1/sqrt(D)): the prefill-side
// counterpart of rap_decode_attn.  Here the path IS a dense contraction (2 T^2 (2P + d_v') flops per
// head against T (2P + d_v') cache elements), so it runs on the tensor cores: warp-level
// mma.sync.m16n8k16 (bf16 in, fp32 accumulate) in the flash-attention arrangement --
//   CTA = 64 queries of one query head (4 warps x 16 rows), looping over 64-key tiles up to the causal
//   limit; S = Q K^T in registers, online softmax per row (quad shuffles), P re-used from the S
//   accumulators as the A operand of O += P V.
// K and V rows are dense-packed with widths that are not multiples of 16 bytes, so the tiles are
// staged row by row with 4-byte cp.async into rows padded to a conflict-free, 16-byte aligned stride
// (double buffered); rows past the sequence's end are zero-filled by the copy itself.  Fragments then
// come from ldmatrix (K as stored, V transposed on the fly).  Odd d_v' (2-byte aligned rows) takes a
// plain 16-bit staging loop.
#include <math.h>

#include "rap_internal.h"

namespace {

constexpr int PF_BM = 64, PF_BN = 64, PF_THREADS = 128;

__device__ __forceinline__ uint32_t pf_smem(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void cp_async4(uint32_t dst, const void* src, int src_bytes) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void ldsm4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm4_t(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float pf_ex2(float x) {      // 2^x, one instruction; 2^(-inf) = 0
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pf_pack(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}

struct PfParams {
  const __nv_bfloat16* q;     // [B][T][Hq][P2]
  const __nv_bfloat16* k;     // [B][Hkv][S_cap][P2]
  const __nv_bfloat16* v;     // [B][Hkv][S_cap][dv]
  const int32_t* start;       // rows cached before the block, per sequence
  float* out;                 // [B][T][Hq][dv]
  int T, Hq, Hkv, P2, dv, S_cap;
  float qscale;               // log2(e) / sqrt(D)
};

// KD = k-steps of Q K^T (ceil(2P / 16)), NV = n-tiles of P V (ceil(d_v' / 8), even)
template <int KD, int NV>
__global__ void __launch_bounds__(PF_THREADS) prefill_attn_kernel(const PfParams p) {
  constexpr int KSTR = KD * 16 + 8;      // smem row stride of K tiles (bf16): 16-byte aligned, conflict-free for ldmatrix
  constexpr int VSTR = NV * 8 + 8;
  constexpr int K_TILE = PF_BN * KSTR, V_TILE = PF_BN * VSTR;
  extern __shared__ __align__(16) unsigned char pf_smem_raw[];
  __nv_bfloat16* ks = reinterpret_cast<__nv_bfloat16*>(pf_smem_raw);             // [2][64][KSTR]
  __nv_bfloat16* vs = ks + 2 * K_TILE;                                           // [2][64][VSTR]
  const int qb = blockIdx.x, g = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int gid = lane >> 2, tq = lane & 3;
  const int h = g / (p.Hq / p.Hkv);
  const int start = min(max(p.start[b], 0), p.S_cap - p.T);
  const int n_valid = start + p.T;                                 // cache rows of this sequence
  const int q0 = qb * PF_BM;
  const int last_pos = start + min(p.T, q0 + PF_BM) - 1;           // last key any query of this block may see
  const int n_tiles = last_pos / PF_BN + 1;
  const __nv_bfloat16* kg = p.k + ((size_t)b * p.Hkv + h) * (size_t)p.S_cap * p.P2;
  const __nv_bfloat16* vg = p.v + ((size_t)b * p.Hkv + h) * (size_t)p.S_cap * p.dv;

  // zero the pad columns once: the copies never touch them, the MMAs read them
  for (int i = tid; i < 2 * K_TILE; i += PF_THREADS) ks[i] = __float2bfloat16(0.f);
  for (int i = tid; i < 2 * V_TILE; i += PF_THREADS) vs[i] = __float2bfloat16(0.f);
  __syncthreads();

  const int kw = p.P2 / 2, vw = p.dv / 2;            // 4-byte words per row (P2 is even)
  const bool v_odd = (p.dv & 1) != 0;
  auto load_tile = [&](int tile, int buf) {
    const int j0 = tile * PF_BN;
    __nv_bfloat16* kd = ks + buf * K_TILE;
    __nv_bfloat16* vd = vs + buf * V_TILE;
    // one row per warp and pass, lanes over the row's 4-byte words: no index divisions in the copy loop
    for (int r = warp; r < PF_BN; r += PF_THREADS / 32) {
      const bool ok = j0 + r < n_valid;
      const int bytes = ok ? 4 : 0;
      const __nv_bfloat16* ksrc = kg + (size_t)(ok ? j0 + r : 0) * p.P2;
      const uint32_t kdst = pf_smem(kd + r * KSTR);
      for (int w = lane; w < kw; w += 32) cp_async4(kdst + 4 * w, ksrc + 2 * w, bytes);
      if (!v_odd) {
        const __nv_bfloat16* vsrc = vg + (size_t)(ok ? j0 + r : 0) * p.dv;
        const uint32_t vdst = pf_smem(vd + r * VSTR);
        for (int w = lane; w < vw; w += 32) cp_async4(vdst + 4 * w, vsrc + 2 * w, bytes);
      } else {   // rows are only 2-byte aligned: element-wise staging
        const __nv_bfloat16* vsrc = vg + (size_t)(j0 + r) * p.dv;
        for (int c = lane; c < p.dv; c += 32) vd[r * VSTR + c] = ok ? vsrc[c] : __float2bfloat16(0.f);
      }
    }
    cp_commit();
  };

  // ---- Q fragments of this warp's 16 rows, straight from global (row r = q0 + 16 warp + gid, + 8) ----
  uint32_t qa[KD][4];
  {
    const int t0 = q0 + 16 * warp + gid, t1 = t0 + 8;
    const __nv_bfloat16* r0 = p.q + (((size_t)b * p.T + min(t0, p.T - 1)) * p.Hq + g) * p.P2;
    const __nv_bfloat16* r1 = p.q + (((size_t)b * p.T + min(t1, p.T - 1)) * p.Hq + g) * p.P2;
#pragma unroll
    for (int ksx = 0; ksx < KD; ++ksx) {
      const int d0 = ksx * 16 + 2 * tq, d1 = d0 + 8;
      qa[ksx][0] = (t0 < p.T && d0 < p.P2) ? *reinterpret_cast<const uint32_t*>(r0 + d0) : 0u;
      qa[ksx][1] = (t1 < p.T && d0 < p.P2) ? *reinterpret_cast<const uint32_t*>(r1 + d0) : 0u;
      qa[ksx][2] = (t0 < p.T && d1 < p.P2) ? *reinterpret_cast<const uint32_t*>(r0 + d1) : 0u;
      qa[ksx][3] = (t1 < p.T && d1 < p.P2) ? *reinterpret_cast<const uint32_t*>(r1 + d1) : 0u;
    }
  }
  const int pos0 = start + q0 + 16 * warp + gid, pos1 = pos0 + 8;   // cache rows of this thread's two queries

  float o[NV][4];
#pragma unroll
  for (int n = 0; n < NV; ++n)
#pragma unroll
    for (int e = 0; e < 4; ++e) o[n][e] = 0.f;
  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;

  load_tile(0, 0);
  for (int tile = 0; tile < n_tiles; ++tile) {
    const int buf = tile & 1;
    if (tile + 1 < n_tiles) {
      load_tile(tile + 1, buf ^ 1);
      cp_wait<1>();
    } else {
      cp_wait<0>();
    }
    __syncthreads();
    const uint32_t kbase = pf_smem(ks + buf * K_TILE), vbase = pf_smem(vs + buf * V_TILE);
    // ---- S = Q K^T: 8 key n-tiles of 8, KD k-steps; ldmatrix.x4 gives b0, b1 of two key tiles ----------
    float s[8][4];
#pragma unroll
    for (int n = 0; n < 8; ++n)
#pragma unroll
      for (int e = 0; e < 4; ++e) s[n][e] = 0.f;
#pragma unroll
    for (int ksx = 0; ksx < KD; ++ksx) {
#pragma unroll
      for (int np = 0; np < 4; ++np) {
        // matrices: (keys 16np..+7, dims k0..+7), (same keys, dims k0+8..), (keys 16np+8.., k0..), (keys 16np+8.., k0+8..)
        const int row = 16 * np + (lane & 7) + ((lane >> 4) << 3);
        const int col = ksx * 16 + (((lane >> 3) & 1) << 3);
        uint32_t bfr[4];
        ldsm4(bfr, kbase + (uint32_t)(row * KSTR + col) * 2);
        mma16816(s[2 * np], qa[ksx], bfr[0], bfr[1]);
        mma16816(s[2 * np + 1], qa[ksx], bfr[2], bfr[3]);
      }
    }
    // ---- scale, causal mask, online softmax (rows gid and gid + 8 of the warp's 16) -------------------
    const int j0 = tile * PF_BN;
    float mx0 = -INFINITY, mx1 = -INFINITY;
    const bool diagonal = j0 + PF_BN - 1 > start + q0 + 16 * warp;   // some key of the tile lies past this warp's first query
    if (diagonal) {
#pragma unroll
      for (int n = 0; n < 8; ++n) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int key = j0 + 8 * n + 2 * tq + (e & 1);
          const int pos = (e < 2) ? pos0 : pos1;
          const float v = key <= pos ? s[n][e] * p.qscale : -INFINITY;
          s[n][e] = v;
          if (e < 2) mx0 = fmaxf(mx0, v); else mx1 = fmaxf(mx1, v);
        }
      }
    } else {
#pragma unroll
      for (int n = 0; n < 8; ++n) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          s[n][e] *= p.qscale;
          if (e < 2) mx0 = fmaxf(mx0, s[n][e]); else mx1 = fmaxf(mx1, s[n][e]);
        }
      }
    }
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
    const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);
    // a row that has seen no allowed key yet keeps m = -inf: use 0 as its reference so that 2^(-inf - 0) = 0
    const float r0 = mn0 == -INFINITY ? 0.f : mn0, r1 = mn1 == -INFINITY ? 0.f : mn1;
    const float a0 = pf_ex2(m0 - r0), a1 = pf_ex2(m1 - r1);
    m0 = mn0; m1 = mn1;
    float sum0 = 0.f, sum1 = 0.f;
    uint32_t pa[4][4];                         // P as A fragments: k-step kk covers keys 16kk .. 16kk+15
#pragma unroll
    for (int n = 0; n < 8; ++n) {
      const float p00 = pf_ex2(s[n][0] - r0), p01 = pf_ex2(s[n][1] - r0);
      const float p10 = pf_ex2(s[n][2] - r1), p11 = pf_ex2(s[n][3] - r1);
      sum0 += p00 + p01;
      sum1 += p10 + p11;
      pa[n >> 1][(n & 1) * 2 + 0] = pf_pack(p00, p01);
      pa[n >> 1][(n & 1) * 2 + 1] = pf_pack(p10, p11);
    }
    l0 = l0 * a0 + sum0;
    l1 = l1 * a1 + sum1;
#pragma unroll
    for (int n = 0; n < NV; ++n) {
      o[n][0] *= a0; o[n][1] *= a0; o[n][2] *= a1; o[n][3] *= a1;
    }
    // ---- O += P V: 4 k-steps of 16 keys, NV channel tiles; ldmatrix.trans turns V rows into B fragments ---
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {
#pragma unroll
      for (int np = 0; np < NV / 2; ++np) {
        // matrices: (keys 16kk..+7, ch 16np..+7), (keys 16kk+8.., same ch), (keys 16kk.., ch 16np+8..), (keys 16kk+8.., ch 16np+8..)
        const int row = 16 * kk + (lane & 7) + (((lane >> 3) & 1) << 3);
        const int col = 16 * np + ((lane >> 4) << 3);
        uint32_t bfr[4];
        ldsm4_t(bfr, vbase + (uint32_t)(row * VSTR + col) * 2);
        mma16816(o[2 * np], pa[kk], bfr[0], bfr[1]);
        mma16816(o[2 * np + 1], pa[kk], bfr[2], bfr[3]);
      }
    }
    __syncthreads();          // this buffer is refilled by the copy issued in the next iteration
  }
  // ---- normalise and store (sum over the quad first) ----------------------------------------------------
  l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
  l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
  const float i0 = l0 > 0.f ? 1.f / l0 : 0.f, i1 = l1 > 0.f ? 1.f / l1 : 0.f;
  const int t0 = q0 + 16 * warp + gid, t1 = t0 + 8;
#pragma unroll
  for (int n = 0; n < NV; ++n) {
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int c = 8 * n + 2 * tq + (e & 1);
      const int t = e < 2 ? t0 : t1;
      if (t < p.T && c < p.dv) p.out[(((size_t)b * p.T + t) * p.Hq + g) * p.dv + c] = o[n][e] * (e < 2 ? i0 : i1);
    }
  }
}

template <int KD, int NV>
rap_status launch_prefill(rap_ctx* ctx, const PfParams& p, int B, cudaStream_t st) {
  const size_t smem = (size_t)2 * PF_BN * ((KD * 16 + 8) + (NV * 8 + 8)) * sizeof(__nv_bfloat16);
  RAP_CUDA_TRY(ctx, rap_raise_smem(ctx, prefill_attn_kernel<KD, NV>, (int)smem));
  dim3 grid((p.T + PF_BM - 1) / PF_BM, p.Hq, B);
  prefill_attn_kernel<KD, NV><<<grid, PF_THREADS, smem, st>>>(p);
  ctx->launches++;
  RAP_CUDA_TRY(ctx, cudaGetLastError());
  return RAP_OK;
}

}  // namespace

rap_status rap_launch_prefill_attn_tc(rap_ctx* ctx, int B, int T, const void* q, const void* k, const void* v, int P2,
                                      int dv, int S_cap, const int32_t* start, float* out, cudaStream_t st);

rap_status rap_launch_prefill_attn(rap_ctx* ctx, int B, int T, const void* q, const void* k, const void* v, int P2,
                                   int dv, int S_cap, const int32_t* start, float* out, cudaStream_t st) {
  if (ctx->attn_variant == 0) {   // tcgen05 kernel first; this file's mma.sync kernel is the fallback / cross-check
    const rap_status s = rap_launch_prefill_attn_tc(ctx, B, T, q, k, v, P2, dv, S_cap, start, out, st);
    if (s != RAP_EUNSUPPORTED) return s;
  }
  const rap_model_desc& d = ctx->desc;
  if (d.dtype != RAP_BF16 || P2 > 128 || dv > 128) return RAP_EUNSUPPORTED;
  PfParams p;
  p.q = (const __nv_bfloat16*)q; p.k = (const __nv_bfloat16*)k; p.v = (const __nv_bfloat16*)v; p.start = start; p.out = out;
  p.T = T; p.Hq = d.n_q_heads; p.Hkv = d.n_kv_heads; p.P2 = P2; p.dv = dv; p.S_cap = S_cap;
  p.qscale = (float)(1.4426950408889634 / sqrt((double)d.head_dim));
  const int kd = (P2 + 15) / 16, nv = ((dv + 15) / 16) * 2;
  if (kd <= 4 && nv <= 8) return launch_prefill<4, 8>(ctx, p, B, st);
  if (kd <= 6 && nv <= 12) return launch_prefill<6, 12>(ctx, p, B, st);
  if (kd <= 7 && nv <= 14) return launch_prefill<7, 14>(ctx, p, B, st);
  return launch_prefill<8, 16>(ctx, p, B, st);
}
