// Low-rank comparator, fast path (Section 3: a low-rank method caches the latent X A_k and must
// rebuild K = latent B_k and rotate it at full width at EVERY decode step).  Done the way a
// framework does it, but with each stage at hardware speed, so that the comparison is fair:
//   1. a (cos, sin) table for positions 0 .. len-1 and the D/2 standard frequencies (Eq. 3),
//   2. a rebuild kernel: per 64-position tile of one (sequence, KV head), K_full = latent * B_k on
//      the tensor cores (mma.sync m16n8k16, bf16 in, fp32 accumulate -- the reconstruction is the
//      one dense contraction of this path), rotate-half RoPE from the table in the accumulator
//      registers, rounded to bf16 into a full-width K workspace [B][H_kv][S_cap][D],
//   3. the shape-specialised split-KV scan of rap_decode_attn over (K workspace, V cache).
// bf16, D = 128, rotate-half pairing, even r <= 128 only; anything else takes the reference kernel.
#include <math.h>

#include "rap_internal.h"

rap_status rap_launch_attn_scan(rap_ctx* ctx, const rap_attn_args& a, int n_split, cudaStream_t st);

namespace {

constexpr int RB_TILE = 64;
constexpr int RB_D = 128;

__global__ void lr_table_kernel(float2* __restrict__ cs, int n_pos, int half, double theta, int D) {
  __shared__ double freq[RB_D / 2];
  if (threadIdx.x < half) freq[threadIdx.x] = pow(theta, -2.0 * (double)threadIdx.x / (double)D);
  __syncthreads();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n_pos * half) return;
  const int pos = i / half, c = i - pos * half;
  double sn, co;
  sincos((double)pos * freq[c], &sn, &co);
  cs[i] = make_float2((float)co, (float)sn);
}

__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}

// grid (tiles, H_kv, B), 256 threads.  Warp w owns rows 16 * (w / 2) .. + 15 of the tile and the
// columns [32 s, 32 s + 32) and [64 + 32 s, 64 + 32 s + 32), s = w % 2, so that both members of every
// rotate-half pair (i, i + 64) sit in the same thread.
template <int RP>   // r rounded up to a multiple of 16
__global__ void __launch_bounds__(256)
lr_rebuild_kernel(const __nv_bfloat16* __restrict__ latent, const __nv_bfloat16* __restrict__ bk,
                  const float2* __restrict__ cs, const int32_t* __restrict__ seq_len, __nv_bfloat16* __restrict__ kout,
                  int Hkv, int r, int S_cap) {
  constexpr int BS = RP + 8;                       // B_k^T row stride (bf16): keeps the fragment reads conflict-free
  extern __shared__ __align__(16) unsigned char rb_smem[];
  __nv_bfloat16* bkt = reinterpret_cast<__nv_bfloat16*>(rb_smem);          // [128][BS]: B_k^T, zero padded in k
  __nv_bfloat16* lat0 = bkt + RB_D * BS;                                   // 2 x ([64][r] latent tile as stored, + 16 zeros)
  constexpr int LAT = RB_TILE * RB_D + 16;
  __nv_bfloat16* kst = lat0 + 2 * LAT;                                     // [64][136] rotated tile before the coalesced store
  const int h = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int len = min(max(seq_len[b], 0), S_cap);
  const int n_tiles = (len + RB_TILE - 1) / RB_TILE;
  const __nv_bfloat16 zero = __float2bfloat16(0.f);
  // B_k[h] is [r][128]: read it row by row (coalesced), store it transposed, once per CTA
  for (int i = tid; i < BS * RB_D; i += 256) {
    const int k = i / RB_D, n = i - k * RB_D;
    bkt[n * BS + k] = k < r ? bk[((size_t)h * r + k) * RB_D + n] : zero;
  }
  // the fragment loads of the last k step run past the row (into the next row, or the pad after the
  // last one) where B_k^T holds zeros: those values only have to be finite
  for (int i = tid; i < 2 * LAT; i += 256) lat0[i] = zero;
  __syncthreads();
  const int g = lane >> 2, t = lane & 3;
  // the latent tiles are fetched one tile ahead (16-byte asynchronous copies into the other buffer)
  auto fetch = [&](int tile, int buf) {
    const int j0 = tile * RB_TILE;
    const int nj = min(RB_TILE, len - j0);
    const unsigned char* lsrc = reinterpret_cast<const unsigned char*>(latent + (((size_t)b * Hkv + h) * S_cap + j0) * r);
    const int nvec = (nj * r * 2 + 15) / 16;          // the tile is one contiguous, 16-byte aligned range
    const uint32_t dst = (uint32_t)__cvta_generic_to_shared(lat0 + buf * LAT);
    for (int i = tid; i < nvec; i += 256)
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + 16u * (uint32_t)i), "l"(lsrc + 16 * (size_t)i) : "memory");
  };
  int buf = 0;
  if ((int)blockIdx.x < n_tiles) fetch(blockIdx.x, 0);
  asm volatile("cp.async.commit_group;" ::: "memory");
  for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, buf ^= 1) {
  const int j0 = tile * RB_TILE;
  const int nj = min(RB_TILE, len - j0);
  const __nv_bfloat16* lat = lat0 + buf * LAT;
  if (tile + (int)gridDim.x < n_tiles) fetch(tile + gridDim.x, buf ^ 1);   // its last readers passed the barrier below a tile ago
  asm volatile("cp.async.commit_group;" ::: "memory");
  const int row0 = 16 * (warp >> 1), cset = warp & 1;
  // this thread's (cos, sin) pairs, on their way while the tile lands and the MMAs run
  float4 csv[2][4];
#pragma unroll
  for (int hr = 0; hr < 2; ++hr) {
    const int row = min(row0 + g + 8 * hr, nj - 1);
    const float4* csr = reinterpret_cast<const float4*>(cs + (size_t)(j0 + row) * (RB_D / 2));
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) csv[hr][nt] = __ldg(csr + ((32 * cset + 8 * nt + 2 * t) >> 1));
  }
  asm volatile("cp.async.wait_group 1;" ::: "memory");
  __syncthreads();                                  // this tile has landed for every thread; the previous tile's rows are stored
  float acc[8][4];
#pragma unroll
  for (int nt = 0; nt < 8; ++nt)
#pragma unroll
    for (int e = 0; e < 4; ++e) acc[nt][e] = 0.f;
#pragma unroll
  for (int k0 = 0; k0 < RP; k0 += 16) {
    uint32_t a[4];
    a[0] = *reinterpret_cast<const uint32_t*>(lat + (row0 + g) * r + k0 + 2 * t);
    a[1] = *reinterpret_cast<const uint32_t*>(lat + (row0 + g + 8) * r + k0 + 2 * t);
    a[2] = *reinterpret_cast<const uint32_t*>(lat + (row0 + g) * r + k0 + 2 * t + 8);
    a[3] = *reinterpret_cast<const uint32_t*>(lat + (row0 + g + 8) * r + k0 + 2 * t + 8);
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
      const int n = (nt < 4 ? 32 * cset + 8 * nt : 64 + 32 * cset + 8 * (nt - 4)) + g;
      const uint32_t b0 = *reinterpret_cast<const uint32_t*>(bkt + n * BS + k0 + 2 * t);
      const uint32_t b1 = *reinterpret_cast<const uint32_t*>(bkt + n * BS + k0 + 2 * t + 8);
      mma_bf16(acc[nt], a, b0, b1);
    }
  }
  // rotate pair (i, i + 64) at position j0 + row, round once, stage, then store whole rows
  constexpr int KSS = RB_D + 8;
#pragma unroll
  for (int hr = 0; hr < 2; ++hr) {
    const int row = row0 + g + 8 * hr;
    if (row < nj) {
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) {
        const int i = 32 * cset + 8 * nt + 2 * t;           // pair indices i, i + 1
        const float4 c = csv[hr][nt];                       // (cos_i, sin_i, cos_i+1, sin_i+1)
        const float x0 = acc[nt][2 * hr], x1 = acc[nt][2 * hr + 1];
        const float y0 = acc[nt + 4][2 * hr], y1 = acc[nt + 4][2 * hr + 1];
        *reinterpret_cast<uint32_t*>(kst + row * KSS + i) = pack_bf16(x0 * c.x - y0 * c.y, x1 * c.z - y1 * c.w);
        *reinterpret_cast<uint32_t*>(kst + row * KSS + 64 + i) = pack_bf16(x0 * c.y + y0 * c.x, x1 * c.w + y1 * c.z);
      }
    }
  }
  __syncthreads();
  uint4* kdst = reinterpret_cast<uint4*>(kout + (((size_t)b * Hkv + h) * S_cap + j0) * RB_D);
  for (int i = tid; i < nj * (RB_D / 8); i += 256) {
    const int row = i >> 4, c8 = i & 15;
    kdst[i] = *reinterpret_cast<const uint4*>(kst + row * KSS + c8 * 8);
  }
  }   // tile loop
  asm volatile("cp.async.wait_group 0;" ::: "memory");
}

template <int RP>
rap_status launch_rebuild(rap_ctx* ctx, const rap_lowrank_args& a, cudaStream_t st) {
  const size_t smem = (size_t)(RB_D * (RP + 8) + 2 * (RB_TILE * RB_D + 16) + RB_TILE * (RB_D + 8)) * sizeof(__nv_bfloat16);
  RAP_CUDA_TRY(ctx, rap_raise_smem(ctx, lr_rebuild_kernel<RP>, (int)smem));
  // a few CTAs per SM, each looping over tiles so that the B_k^T staging is paid once per CTA
  const int n_tiles = (a.h_len_max + RB_TILE - 1) / RB_TILE;
  int gx = (4 * ctx->sm_count + a.B * a.Hkv - 1) / (a.B * a.Hkv);
  gx = gx < 1 ? 1 : gx > n_tiles ? n_tiles : gx;
  dim3 grid(gx, a.Hkv, a.B);
  lr_rebuild_kernel<RP><<<grid, 256, smem, st>>>((const __nv_bfloat16*)a.k_latent, (const __nv_bfloat16*)a.bk,
                                                 (const float2*)ctx->d_lr_cs, a.seq_len, (__nv_bfloat16*)ctx->d_lr_k, a.Hkv,
                                                 a.r, a.S_cap);
  ctx->launches++;
  RAP_CUDA_TRY(ctx, cudaGetLastError());
  return RAP_OK;
}

}  // namespace

// RAP_EUNSUPPORTED when the shape is outside this path (the caller then runs the reference kernel).
rap_status rap_launch_lowrank_fast(rap_ctx* ctx, const rap_lowrank_args& a, cudaStream_t st) {
  if (a.dtype != RAP_BF16 || a.head_dim != RB_D || a.pairing != RAP_PAIR_HALF || (a.r & 1) || a.r > RB_D ||
      a.Hq / a.Hkv != 4 || a.h_len_max < 1)
    return RAP_EUNSUPPORTED;
  if (a.dv != 128 && a.dv != 115 && a.dv != 102 && a.dv != 90 && a.dv != 64) return RAP_EUNSUPPORTED;
  // workspaces grow on demand (allocation happens outside the timed path after the first call)
  const size_t kbytes = (size_t)a.B * a.Hkv * a.S_cap * RB_D * sizeof(__nv_bfloat16);
  if (kbytes > ctx->lr_k_bytes) {
    RAP_CUDA_TRY(ctx, cudaStreamSynchronize(st));
    if (ctx->d_lr_k) cudaFree(ctx->d_lr_k);
    ctx->d_lr_k = nullptr; ctx->lr_k_bytes = 0;
    RAP_CUDA_TRY(ctx, cudaMalloc(&ctx->d_lr_k, kbytes));
    ctx->lr_k_bytes = kbytes;
  }
  const size_t csbytes = (size_t)a.S_cap * (RB_D / 2) * sizeof(float2);
  if (csbytes > ctx->lr_cs_bytes) {
    RAP_CUDA_TRY(ctx, cudaStreamSynchronize(st));
    if (ctx->d_lr_cs) cudaFree(ctx->d_lr_cs);
    ctx->d_lr_cs = nullptr; ctx->lr_cs_bytes = 0; ctx->lr_cs_len = 0;
    RAP_CUDA_TRY(ctx, cudaMalloc(&ctx->d_lr_cs, csbytes));
    ctx->lr_cs_bytes = csbytes;
  }
  if (a.h_len_max > ctx->lr_cs_len) {   // the table is kept across calls, as frameworks keep their cos / sin cache
    const int n_pos = a.S_cap;
    const int n_cs = n_pos * (RB_D / 2);
    lr_table_kernel<<<(n_cs + 255) / 256, 256, 0, st>>>((float2*)ctx->d_lr_cs, n_pos, RB_D / 2, a.rope_theta, RB_D);
    ctx->launches++;
    RAP_CUDA_TRY(ctx, cudaGetLastError());
    ctx->lr_cs_len = n_pos;
  }
  const int rp = (a.r + 15) / 16 * 16;
  rap_status s;
  switch (rp) {
    case 16: s = launch_rebuild<16>(ctx, a, st); break;
    case 32: s = launch_rebuild<32>(ctx, a, st); break;
    case 48: s = launch_rebuild<48>(ctx, a, st); break;
    case 64: s = launch_rebuild<64>(ctx, a, st); break;
    case 80: s = launch_rebuild<80>(ctx, a, st); break;
    case 96: s = launch_rebuild<96>(ctx, a, st); break;
    case 112: s = launch_rebuild<112>(ctx, a, st); break;
    default: s = launch_rebuild<128>(ctx, a, st); break;
  }
  if (s != RAP_OK) return s;
  rap_attn_args t;
  t.q = a.q_full; t.k = ctx->d_lr_k; t.v = a.v; t.seq_len = a.seq_len; t.len_add = 0;
  t.B = a.B; t.Hq = a.Hq; t.Hkv = a.Hkv; t.P2 = RB_D; t.dv = a.dv; t.S_cap = a.S_cap; t.head_dim = RB_D;
  t.dtype = RAP_BF16; t.n_split = a.n_split; t.h_len_max = a.h_len_max; t.out = a.out;
  return rap_launch_attn_scan(ctx, t, a.n_split, st);
}
