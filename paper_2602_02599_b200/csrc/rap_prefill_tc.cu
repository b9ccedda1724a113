// tcgen05 version of rap_prefill_attn: causal attention of a block of T new tokens per sequence over the
// reduced dims (Eq. 2 for every t of the block; 2P retained K dims, d_v' retained V channels, scale
// 1/sqrt(D)).  One CTA handles 128 queries of one query head and walks 128-key tiles up to the causal limit:
//   S      = Q K^T      tcgen05.mma (M = 128 queries, N = 128 keys, K = 2P in steps of 16), accumulator in TMEM
//   P      = 2^(S - m)  one thread per query row reads its S row from TMEM (tcgen05.ld), applies the causal
//                       mask and a lazy running maximum, and writes P as bf16 into shared memory
//   O_tile = P V        tcgen05.mma (N = d_v' rounded up to 32, K = 128 keys), fresh accumulator per tile;
//                       the row's thread then folds O_tile into its register accumulator with the rescale
//                       factor, so tensor memory never has to be rewritten.
// Cache rows are not multiples of 16 bytes, so TMA tensor maps cannot describe them: all threads stage the
// tiles by hand into the K-major, 128-byte-swizzled layout the MMA descriptors expect (Q and K as stored, V
// transposed to [channel][key]); rows past the sequence end and pad columns are zeros.  Stages of one tile
// run one after the other (no double buffering yet).  Every mbarrier wait is bounded.
#include <math.h>

#include "rap_internal.h"

namespace {

constexpr int PT_BM = 128, PT_BN = 128, PT_THREADS = 160;       // warps 0-3: rows / softmax, warp 4: MMA issue
constexpr int PT_TILE_BYTES = 2 * 128 * 128;                     // two 64-element atom columns of 128 rows
constexpr uint32_t PT_WAIT_LIMIT = 1u << 21;

__device__ __forceinline__ uint32_t pt_smem(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void pt_mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ bool pt_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool pt_wait(uint32_t bar, uint32_t parity) {
  for (uint32_t i = 0; i < PT_WAIT_LIMIT; ++i)
    if (pt_try_wait(bar, parity)) return true;
  return false;
}
// K-major operand tile, 128-byte swizzle: 8-row groups 1024 bytes apart (see rap_proj_tc.cu)
__device__ __forceinline__ uint64_t pt_desc(uint32_t addr) {
  const uint32_t lo = ((addr & 0x3FFFFu) >> 4) | (1u << 16);
  const uint32_t hi = (1024u >> 4) | (1u << 14) | (2u << 29);
  return ((uint64_t)hi << 32) | lo;
}
__device__ __forceinline__ void pt_mma(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc)
      : "memory");
}
__device__ __forceinline__ void pt_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void pt_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ float pt_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// byte offset of element (row, col) of a K-major bf16 tile of `rows` rows: 64-column atom columns, rows of
// 128 bytes whose 16-byte chunks are XORed with row % 8
__device__ __forceinline__ uint32_t pt_off(int row, int col, int rows) {
  const int ac = col >> 6, c = col & 63;
  return (uint32_t)(ac * rows * 128 + (row >> 3) * 1024 + (row & 7) * 128 + ((((c >> 3) ^ (row & 7))) << 4) + ((c & 7) << 1));
}

struct PtParams {
  const __nv_bfloat16* q;     // [B][T][Hq][P2]
  const __nv_bfloat16* k;     // [B][Hkv][S_cap][P2]
  const __nv_bfloat16* v;     // [B][Hkv][S_cap][dv]
  const int32_t* start;
  float* out;                 // [B][T][Hq][dv]
  int32_t* status;
  int T, Hq, Hkv, P2, dv, S_cap;
  float qscale;               // log2(e) / sqrt(D)
};

// DK = k-steps of Q K^T (ceil(2P / 16)); NVP = d_v' rounded up to a multiple of 32 (N of the second MMA)
template <int DK, int NVP>
__global__ void __launch_bounds__(PT_THREADS, 2) prefill_tc_kernel(const PtParams p) {
  extern __shared__ unsigned char pt_raw[];
  unsigned char* smem = pt_raw + ((1024u - (pt_smem(pt_raw) & 1023u)) & 1023u);
  unsigned char* q_s = smem;                         // [128 queries][<=128 dims]
  unsigned char* k_s = q_s + PT_TILE_BYTES;          // [128 keys][<=128 dims]
  unsigned char* v_s = k_s + PT_TILE_BYTES;          // [NVP channels][128 keys]   (V transposed)
  unsigned char* p_s = k_s;                          // [128 queries][128 keys]: reuses the K tile, which the
                                                     // first MMA has finished reading when P is written
  const uint32_t bar_s = pt_smem(v_s + PT_TILE_BYTES), bar_o = bar_s + 8;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(v_s + PT_TILE_BYTES + 16);

  const int qb = blockIdx.x, g = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int h = g / (p.Hq / p.Hkv);
  const int start = min(max(p.start[b], 0), p.S_cap - p.T);
  const int n_valid = start + p.T;
  const int q0 = qb * PT_BM;
  const int last_pos = start + min(p.T, q0 + PT_BM) - 1;
  const int n_tiles = last_pos / PT_BN + 1;
  const __nv_bfloat16* kg = p.k + ((size_t)b * p.Hkv + h) * (size_t)p.S_cap * p.P2;
  const __nv_bfloat16* vg = p.v + ((size_t)b * p.Hkv + h) * (size_t)p.S_cap * p.dv;

  if (tid == 0) {
    pt_mbar_init(bar_s, 1);
    pt_mbar_init(bar_o, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 4) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(pt_smem(tmem_slot)), "r"(256)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // zero all four tiles once (pad columns and pad channel rows are never written again), then stage Q
  for (int i = tid; i < 3 * PT_TILE_BYTES / 16; i += PT_THREADS) reinterpret_cast<uint4*>(smem)[i] = make_uint4(0, 0, 0, 0);
  __syncthreads();
  const int kw = p.P2 >> 1;                          // 4-byte words per q / K row
  for (int r = warp; r < PT_BM; r += PT_THREADS / 32) {
    const int t = q0 + r;
    if (t < p.T) {
      const uint32_t* src = reinterpret_cast<const uint32_t*>(p.q + (((size_t)b * p.T + t) * p.Hq + g) * p.P2);
      for (int w = lane; w < kw; w += 32) *reinterpret_cast<uint32_t*>(q_s + pt_off(r, 2 * w, PT_BM)) = src[w];
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_s = *tmem_slot, tmem_o = tmem_s + 128;
  constexpr uint32_t IDESC_S = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(PT_BN >> 3) << 17) | ((uint32_t)(PT_BM >> 4) << 24);
  constexpr uint32_t IDESC_O = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(NVP >> 3) << 17) | ((uint32_t)(PT_BM >> 4) << 24);

  const int row = tid;                               // warps 0-3: query row = TMEM lane
  const int pos = start + q0 + row;                  // cache row of this thread's query
  float o[NVP];
#pragma unroll
  for (int c = 0; c < NVP; ++c) o[c] = 0.f;
  float m_ref = -1.0e30f, l_run = 0.f;
  bool timed_out = false;
  uint32_t phase = 0;

  for (int tile = 0; tile < n_tiles; ++tile) {
    const int j0 = tile * PT_BN;
    // ---- stage K (as stored) and V (transposed); rows past the end become zeros ------------------------
    // K: 4-byte cp.async straight to the swizzled position (zero fill past the end), all in flight at once;
    // V: eight rows per pass so that eight independent loads are in flight before the transposed stores
    for (int r = warp; r < PT_BN; r += PT_THREADS / 32) {
      const bool ok = j0 + r < n_valid;
      const __nv_bfloat16* ksrc = kg + (size_t)(ok ? j0 + r : 0) * p.P2;
      for (int w = lane; w < kw; w += 32)
        asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(pt_smem(k_s + pt_off(r, 2 * w, PT_BN))),
                     "l"(ksrc + 2 * w), "r"(ok ? 4 : 0)
                     : "memory");
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    for (int r0 = 8 * warp; r0 < PT_BN; r0 += 8 * (PT_THREADS / 32)) {
      for (int c = lane; c < p.dv; c += 32) {
        __nv_bfloat16 vals[8];
#pragma unroll
        for (int i = 0; i < 8; ++i)
          vals[i] = j0 + r0 + i < n_valid ? vg[(size_t)(j0 + r0 + i) * p.dv + c] : __float2bfloat16(0.f);
        // rows r0 .. r0+7 of channel c are one 16-byte chunk of the transposed tile
        *reinterpret_cast<uint4*>(v_s + pt_off(c, r0, NVP)) = *reinterpret_cast<const uint4*>(vals);
      }
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> tensor-core (async proxy) reads
    __syncthreads();
    // ---- S = Q K^T ----------------------------------------------------------------------------------------
    if (warp == 4 && lane == 0) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
      for (int ks = 0; ks < DK; ++ks) {
        const uint32_t o2 = (uint32_t)((ks >> 2) * PT_BM * 128 + (ks & 3) * 32);
        pt_mma(tmem_s, pt_desc(pt_smem(q_s) + o2), pt_desc(pt_smem(k_s) + o2), IDESC_S, ks > 0 ? 1u : 0u);
      }
      pt_commit(bar_s);
    }
    float alpha = 1.f;
    if (warp < 4) {
      if (!pt_wait(bar_s, phase)) timed_out = true;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t trow = tmem_s + ((uint32_t)(warp * 32) << 16);
      // pass 1: the row's maximum over the allowed keys of the tile
      float mx = -INFINITY;
#pragma unroll 1
      for (int c0 = 0; c0 < PT_BN; c0 += 32) {
        uint32_t r[32];
        pt_ld32(trow + c0, r);
#pragma unroll
        for (int j = 0; j < 32; ++j)
          if (j0 + c0 + j <= pos) mx = fmaxf(mx, __uint_as_float(r[j]) * p.qscale);
      }
      if (mx > m_ref + 8.f) {          // lazy reference maximum: p stays <= 2^8
        alpha = pt_ex2(m_ref - mx);    // first time: 2^(-1e30 - mx) = 0
        m_ref = mx;
        l_run *= alpha;
      }
      // pass 2: p = 2^(s - m_ref), bf16, into the A-operand layout (this thread's row, 16 chunks of 8 keys)
#pragma unroll 1
      for (int c0 = 0; c0 < PT_BN; c0 += 32) {
        uint32_t r[32];
        pt_ld32(trow + c0, r);
        uint32_t pk[16];
#pragma unroll
        for (int j = 0; j < 32; j += 2) {
          const float p0 = j0 + c0 + j <= pos ? pt_ex2(__uint_as_float(r[j]) * p.qscale - m_ref) : 0.f;
          const float p1 = j0 + c0 + j + 1 <= pos ? pt_ex2(__uint_as_float(r[j + 1]) * p.qscale - m_ref) : 0.f;
          const __nv_bfloat162 v2 = __floats2bfloat162_rn(p0, p1);
          // the row sum uses the rounded values the second MMA will see
          l_run += __bfloat162float(v2.x) + __bfloat162float(v2.y);
          pk[j >> 1] = *reinterpret_cast<const uint32_t*>(&v2);
        }
#pragma unroll
        for (int ch = 0; ch < 4; ++ch)
          *reinterpret_cast<uint4*>(p_s + pt_off(row, c0 + 8 * ch, PT_BM)) =
              make_uint4(pk[4 * ch], pk[4 * ch + 1], pk[4 * ch + 2], pk[4 * ch + 3]);
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    }
    if (__syncthreads_or(timed_out)) { timed_out = true; break; }
    // ---- O_tile = P V -----------------------------------------------------------------------------------------
    if (warp == 4 && lane == 0) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
      for (int ks = 0; ks < PT_BN / 16; ++ks) {
        const uint32_t oa = (uint32_t)((ks >> 2) * PT_BM * 128 + (ks & 3) * 32);
        const uint32_t ob = (uint32_t)((ks >> 2) * NVP * 128 + (ks & 3) * 32);
        pt_mma(tmem_o, pt_desc(pt_smem(p_s) + oa), pt_desc(pt_smem(v_s) + ob), IDESC_O, ks > 0 ? 1u : 0u);
      }
      pt_commit(bar_o);
    }
    // everybody waits for the second MMA: the next tile's staging overwrites what it reads
    if (!pt_wait(bar_o, phase)) timed_out = true;
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (warp < 4) {
      const uint32_t trow = tmem_o + ((uint32_t)(warp * 32) << 16);
#pragma unroll
      for (int c0 = 0; c0 < NVP; c0 += 32) {
        uint32_t r[32];
        pt_ld32(trow + c0, r);
#pragma unroll
        for (int j = 0; j < 32; ++j) o[c0 + j] = o[c0 + j] * alpha + __uint_as_float(r[j]);
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    }
    phase ^= 1u;
    if (__syncthreads_or(timed_out)) { timed_out = true; break; }
  }

  if (timed_out && tid == 0) {
    atomicCAS(&p.status[0], 0, (int)RAP_ETIMEOUT);
    p.status[1] = 0x60000000 | (blockIdx.x & 0xffffff);
  }
  if (warp < 4 && !timed_out) {
    const int t = q0 + row;
    if (t < p.T) {
      const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
      float* dst = p.out + (((size_t)b * p.T + t) * p.Hq + g) * p.dv;
#pragma unroll
      for (int c = 0; c < NVP; ++c)
        if (c < p.dv) dst[c] = o[c] * inv;
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 4) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_s), "r"(256) : "memory");
  }
}

template <int DK, int NVP>
rap_status launch_pt(rap_ctx* ctx, const PtParams& p, int B, cudaStream_t st) {
  const int smem = 3 * PT_TILE_BYTES + 64 + 1024;
  RAP_CUDA_TRY(ctx, rap_raise_smem(ctx, prefill_tc_kernel<DK, NVP>, smem));
  dim3 grid((p.T + PT_BM - 1) / PT_BM, p.Hq, B);
  prefill_tc_kernel<DK, NVP><<<grid, PT_THREADS, smem, st>>>(p);
  ctx->launches++;
  RAP_CUDA_TRY(ctx, cudaGetLastError());
  return RAP_OK;
}

}  // namespace

// RAP_EUNSUPPORTED for shapes this kernel is not instantiated for (the caller then takes the mma.sync kernel)
rap_status rap_launch_prefill_attn_tc(rap_ctx* ctx, int B, int T, const void* q, const void* k, const void* v, int P2,
                                      int dv, int S_cap, const int32_t* start, float* out, cudaStream_t st) {
  const rap_model_desc& d = ctx->desc;
  if (d.dtype != RAP_BF16 || P2 > 128 || dv > 128 || (P2 & 1)) return RAP_EUNSUPPORTED;
  PtParams p;
  p.q = (const __nv_bfloat16*)q; p.k = (const __nv_bfloat16*)k; p.v = (const __nv_bfloat16*)v; p.start = start; p.out = out;
  p.status = ctx->d_status;
  p.T = T; p.Hq = d.n_q_heads; p.Hkv = d.n_kv_heads; p.P2 = P2; p.dv = dv; p.S_cap = S_cap;
  p.qscale = (float)(1.4426950408889634 / sqrt((double)d.head_dim));
  const int dk = (P2 + 15) / 16, nvp = (dv + 31) / 32 * 32;
  if (dk <= 4 && nvp <= 64) return launch_pt<4, 64>(ctx, p, B, st);
  if (dk <= 6 && nvp <= 96) return launch_pt<6, 96>(ctx, p, B, st);
  return launch_pt<8, 128>(ctx, p, B, st);
}
