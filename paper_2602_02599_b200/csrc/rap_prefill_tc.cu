// tcgen05 version of rap_prefill_attn: causal attention of a block of T new tokens per sequence over the
// reduced dims (Eq. 2 for every t of the block; 2P retained K dims, d_v' retained V channels, scale
// 1/sqrt(D)).  One CTA (one per SM, 448 threads) handles 256 consecutive queries of one query head as two query
// tiles A and B of 128, and walks 64-key tiles up to each tile's causal limit:
//   S_X    = Q_X K^T    tcgen05.mma (M = 128 queries, N = 64 keys, K = 2P in steps of 16), accumulator in TMEM,
//                       double buffered per query tile: S of key tile t + 1 is issued before P of t is waited for
//   P_X    = 2^(S - m)  softmax warp group X (warps 0-3: A, 4-7: B), one thread per query row: the S row in
//                       registers with one TMEM round trip, causal mask only on the tiles that reach the diagonal,
//                       lazy running maximum, P as packed bf16 back into tensor memory over the S columns it
//                       came from
//   O_X   += P_X V      tcgen05.mma with A = P in tensor memory (N = d_v' rounded up to 32, K = 64 keys),
//                       accumulating in TMEM across the key tiles; a warp rescales its 32 accumulator rows
//                       (tcgen05.ld / st) only in the rare tile where the lazy maximum moved.
// Where the N of the second MMA has a spare column (d_v' below its multiple of 32: every pruned shape), that column of
// every staged V tile holds the constant one, so the tensor core accumulates the row sum of the weights next to O --
// from the very bf16 weights it multiplies, rescaled with O when the maximum moves -- and the softmax threads keep no
// sum at all (LSUM; a third of their instructions per weight otherwise).
// While one group runs its softmax the tensor core works for the other, and a staged K / V tile serves 256 queries.
// Cache rows are not multiples of 16 bytes, so TMA tensor maps cannot describe them: four producer warps (10-11: K,
// 12-13: V) stage the tiles by hand (4-byte cp.async) into rings of five buffers each, in the 128-byte-swizzled
// layouts the MMA descriptors expect (K as stored = K-major; V as stored = the N-major form of the B operand, so
// nothing is transposed); rows past the sequence end and pad columns are zeros.  The copies' completion arrives on
// the buffer's mbarrier by itself; the consumer issues the proxy fence.  The roles meet only on mbarriers; every wait
// is bounded and gives up early once another role has given up.  Lane 0 of warp 8 issues the MMAs of query tile A,
// lane 0 of warp 9 those of B.
#include <math.h>

#include "rap_internal.h"

namespace {

constexpr int P2_KT = 64;                              // keys per tile
constexpr int P2_THREADS = 448;
constexpr int P2_STAGES = 5;                           // K buffers and V buffers
constexpr int P2_Q_BYTES = 2 * 128 * 128;              // [128 queries][<=128 dims]: two 64-element atom columns
constexpr int P2_KV_BYTES = 2 * P2_KT * 128;           // [64 keys][<=128 dims or channels]
constexpr int P2_TAIL = 320;                           // mbarriers, TMEM address, give-up flag
constexpr int P2_SMEM = 2 * P2_Q_BYTES + 2 * P2_STAGES * P2_KV_BYTES + P2_TAIL;
constexpr uint32_t PT_WAIT_HINT_NS = 20000;      // a parked probe returns at the phase change or after this long
constexpr uint32_t PT_WAIT_LIMIT = 1u << 15;    // probes before a wait gives up (well under a second)

__device__ __forceinline__ uint32_t pt_smem(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void pt_mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
// one probe of the barrier's phase; the hardware may park the thread for up to PT_WAIT_HINT_NS before it answers
__device__ __forceinline__ bool pt_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity), "r"(PT_WAIT_HINT_NS) : "memory");
  return ok != 0;
}
// one probe that never parks the thread
__device__ __forceinline__ bool pt_test_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// tcgen05.mma with shared-memory operand descriptors given as (low word, high word).  K-major operand tile, 128-byte
// swizzle, 8-row groups 1024 bytes apart (see rap_proj_tc.cu): the high word is the same for every operand here; the
// low word carries the start address (in 16-byte units, 14 bits) and the leading offset (bits 16-29), so walking a
// ring or the k-steps of a tile is one 32-bit add on it.  pt_mma_ts2: A in tensor memory (row = lane, two bf16 K
// elements per 32-bit column).
__device__ __forceinline__ void pt_mma2(uint32_t tmem_d, uint32_t a_lo, uint32_t b_lo, uint32_t hi, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
      "mov.b64 da, {%1, %3};\n\t"
      "mov.b64 db, {%2, %3};\n\t"
      "setp.ne.b32 p, %5, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p;\n\t}" ::"r"(tmem_d),
      "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc), "r"(acc)
      : "memory");
}
__device__ __forceinline__ void pt_mma_ts2(uint32_t tmem_d, uint32_t tmem_a, uint32_t b_lo, uint32_t hi, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 db;\n\t"
      "mov.b64 db, {%2, %3};\n\t"
      "setp.ne.b32 p, %5, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %4, p;\n\t}" ::"r"(tmem_d),
      "r"(tmem_a), "r"(b_lo), "r"(hi), "r"(idesc), "r"(acc)
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
__device__ __forceinline__ void pt_ld32_nowait(uint32_t taddr, uint32_t (&r)[32]) {
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
}
__device__ __forceinline__ uint32_t pt_ld1(uint32_t taddr) {     // one column of this warp's 32 lanes
  uint32_t r;
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];" : "=r"(r) : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
  return r;
}
__device__ __forceinline__ void pt_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
      "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]),
      "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]),
      "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
// 4-byte cp.async; the first src_bytes come from memory, the rest of the copy is zero-filled
__device__ __forceinline__ void pt_cp4(uint32_t dst, const void* src, int src_bytes) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
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

// N-major operand tile (B = V as stored, [key][channel]), 128-byte swizzle: an atom is 8 keys x 64 channels
// (key rows of 128 bytes, 16-byte chunks XORed with key % 8); atoms of consecutive 8-key groups are 1024 bytes
// apart (stride offset), the two 64-channel atom columns of a 64-key tile 8 KB apart (leading offset: bits 16-29 of
// the descriptor's low word).
// Byte offset inside a 64-row tile row of its byte e: 64-element (128-byte) atom columns 8 KB apart, 16-byte chunks
// XORed with row % 8 (the layout is the same for the K-major K tile and the N-major V tile).
__device__ __forceinline__ uint32_t pt_swz2(int e, int r7) {
  const int w = e >> 2;
  return (uint32_t)(((w >> 5) << 13) + ((((w & 31) >> 2) ^ r7) << 4) + ((w & 3) << 2));
}
struct PtParams {
  const __nv_bfloat16* q;     // [B][T][Hq][P2]
  const __nv_bfloat16* k;     // [B][Hkv][S_cap][P2]
  const __nv_bfloat16* v;     // [B][Hkv][S_cap][dv]
  const int32_t* start;
  float* out;                 // [B][T][Hq][dv]
  int32_t* status;
  int T, Hq, Hkv, P2, dv, S_cap;
  int vs;                     // elements between V rows: d_v', or d_v' + 1 when the rows were copied to an even length
  float qscale;               // log2(e) / sqrt(D)
};

// Odd d_v': V rows are only 2-byte aligned, which rules out the 4-byte asynchronous copies of the staging.  The rows
// the block can see (start + T per sequence) are first copied to rows of d_v' + 1 elements (the last one zero): a
// few MB against the GB the attention itself moves through the SMs.
__global__ void __launch_bounds__(256) prefill_repack_v_kernel(const __nv_bfloat16* __restrict__ v, __nv_bfloat16* __restrict__ dst,
                                                               const int32_t* __restrict__ start, int T, int Hkv, int dv,
                                                               int S_cap) {
  const int unit = blockIdx.y, b = unit / Hkv;
  const int n = min(max(start[b], 0), S_cap - T) + T;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int row = blockIdx.x * 8 + warp; row < n; row += gridDim.x * 8) {
    const __nv_bfloat16* src = v + ((size_t)unit * S_cap + row) * dv;
    __nv_bfloat16* d = dst + ((size_t)unit * S_cap + row) * (dv + 1);
    for (int c = lane; c <= dv; c += 32) d[c] = c < dv ? src[c] : __float2bfloat16(0.f);
  }
}

// DK = k-steps of Q K^T (ceil(2P / 16)); NVP = d_v' rounded up to a multiple of 32 (N of the second MMA)
// LSUM: column p.vs (< NVP) of every V tile is the constant one and the row sums come out of the second MMA
template <int DK, int NVP, bool LSUM>
__global__ void __launch_bounds__(P2_THREADS, 1) prefill_tc_kernel(const PtParams p) {
  extern __shared__ unsigned char pt_raw[];
  unsigned char* smem = pt_raw + ((1024u - (pt_smem(pt_raw) & 1023u)) & 1023u);
  unsigned char* q_s = smem;                                   // Q_A, Q_B
  unsigned char* k_s = q_s + 2 * P2_Q_BYTES;                   // ring of K tiles
  unsigned char* v_s = k_s + P2_STAGES * P2_KV_BYTES;          // ring of V tiles (N-major)
  unsigned char* tail = v_s + P2_STAGES * P2_KV_BYTES;
  const uint32_t bar_fk = pt_smem(tail), bar_ek = bar_fk + 8 * P2_STAGES, bar_fv = bar_ek + 8 * P2_STAGES,
                 bar_ev = bar_fv + 8 * P2_STAGES, bar_s = bar_ev + 8 * P2_STAGES /* [X][2] */, bar_p = bar_s + 32 /* [X][2] */,
                 bar_o = bar_p + 32 /* [X] */, bar_end = bar_o + 16 /* [X] */;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tail + 32 * P2_STAGES + 96);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tail + 32 * P2_STAGES + 100);
  static_assert(32 * P2_STAGES + 104 <= P2_TAIL, "barriers and flags fit the tail");

  // the blocks with the most key tiles (the last queries) are dispatched first, the short ones fill the tail
  const int qb = (int)gridDim.z - 1 - (int)blockIdx.z, g = blockIdx.x, b = blockIdx.y;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int h = g / (p.Hq / p.Hkv);
  const int start = min(max(p.start[b], 0), p.S_cap - p.T);
  const int n_valid = start + p.T;
  const int q0 = qb * 256;
  // key tiles each query tile needs (tile B may lie wholly past the block)
  int nt[2];
#pragma unroll
  for (int X = 0; X < 2; ++X) {
    const int q0x = q0 + 128 * X;
    nt[X] = q0x < p.T ? (start + min(p.T, q0x + 128) - 1) / P2_KT + 1 : 0;
  }
  const int n_max = max(nt[0], nt[1]);
  const __nv_bfloat16* kg = p.k + ((size_t)b * p.Hkv + h) * (size_t)p.S_cap * p.P2;
  const __nv_bfloat16* vg = p.v + ((size_t)b * p.Hkv + h) * (size_t)p.S_cap * p.vs;

  if (tid == 0) {
    for (int i = 0; i < P2_STAGES; ++i) {
      pt_mbar_init(bar_fk + 8 * i, 64);
      pt_mbar_init(bar_ek + 8 * i, 2);               // both MMA-issuing lanes release a buffer
      pt_mbar_init(bar_fv + 8 * i, 64);
      pt_mbar_init(bar_ev + 8 * i, 2);
    }
    for (int i = 0; i < 4; ++i) {
      pt_mbar_init(bar_s + 8 * i, 1);
      // "P written" has one barrier per S buffer: the softmax may be a tile ahead of the lane that waits for it, and
      // with a single barrier two completed phases would look like none
      pt_mbar_init(bar_p + 8 * i, 128);
    }
    for (int X = 0; X < 2; ++X) pt_mbar_init(bar_o + 8 * X, 1);
    pt_mbar_init(bar_end, 1);
    pt_mbar_init(bar_end + 8, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 8) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(pt_smem(tmem_slot)), "r"(512)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // zero every tile once (pad columns and pad channel rows are never written again), then stage Q_A and Q_B
  for (int i = tid; i < (P2_SMEM - P2_TAIL) / 16; i += P2_THREADS) reinterpret_cast<uint4*>(smem)[i] = make_uint4(0, 0, 0, 0);
  __syncthreads();
  if constexpr (LSUM) {
    // the ones column: channel p.vs of all 64 key rows of every V buffer (the producers never write that element)
    for (int i = tid; i < P2_STAGES * P2_KT; i += P2_THREADS) {
      const int buf = i / P2_KT, r = i - buf * P2_KT, c = p.vs;
      unsigned char* e = v_s + buf * P2_KV_BYTES + r * 128 + pt_swz2(4 * (c >> 1), r & 7) + 2 * (c & 1);
      *reinterpret_cast<__nv_bfloat16*>(e) = __float2bfloat16(1.0f);
    }
  }
  const int kw = p.P2 >> 1;                          // 4-byte words per q / K row
  {
    // a warp takes rows warp, warp + 14, ...; the loads of ten rows are in flight before the first store (one round
    // trip to memory per batch instead of one per row)
    constexpr int NWARP = P2_THREADS / 32, QB = 10;
    const size_t q_row = (size_t)p.Hq * p.P2 / 2;    // words between consecutive queries of one head
    const uint32_t* qsrc = reinterpret_cast<const uint32_t*>(p.q + (((size_t)b * p.T + q0) * p.Hq + g) * p.P2);
#pragma unroll 1
    for (int r0 = warp; r0 < 256; r0 += NWARP * QB) {
      uint32_t qv[QB][2];
#pragma unroll
      for (int u = 0; u < QB; ++u) {
        const int r = r0 + NWARP * u;
        const bool ok = r < 256 && q0 + r < p.T;
#pragma unroll
        for (int sl = 0; sl < 2; ++sl) {
          const int w = lane + 32 * sl;
          qv[u][sl] = (ok && w < kw) ? __ldg(qsrc + (size_t)r * q_row + w) : 0u;
        }
      }
#pragma unroll
      for (int u = 0; u < QB; ++u) {
        const int r = r0 + NWARP * u;
        if (r < 256 && q0 + r < p.T) {
          unsigned char* qd = q_s + (r >> 7) * P2_Q_BYTES;
#pragma unroll
          for (int sl = 0; sl < 2; ++sl) {
            const int w = lane + 32 * sl;
            if (w < kw) *reinterpret_cast<uint32_t*>(qd + pt_off(r & 127, 2 * w, 128)) = qv[u][sl];
          }
        }
      }
    }
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;             // S_X(t): columns 128 X + 64 (t & 1); O_X: columns 256 + 128 X
  constexpr uint32_t IDESC_S = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(P2_KT >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
  constexpr uint32_t IDESC_O = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(NVP >> 3) << 17) |
                               ((uint32_t)(128 >> 4) << 24);
  auto wait = [&](uint32_t bar, uint32_t parity) -> bool {
    if (pt_test_wait(bar, parity)) return true;        // the usual case: the phase is long over (a parking probe costs ~250 cycles even then)
    for (uint32_t i = 0; i < PT_WAIT_LIMIT; ++i) {
      if (pt_try_wait(bar, parity)) return true;
      if ((i & 15u) == 15u && *abort_flag) return false;
    }
    *abort_flag = 1;
    return false;
  };

  float l_run = 0.f;
  const int X = (warp >> 2) & 1;                     // softmax group = query tile
  const int row = (warp & 3) * 32 + lane;
  const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
  const uint32_t tmem_o = tmem_base + 256 + 128 * X;
  if (warp >= 10) {
    // ================= producers: warps 10-11 stage K, warps 12-13 stage V, in order, tiles of 64 rows =================
    const bool is_v = warp >= 12;
    const int pw = (warp - 10) & 1;
    const int rowlen = is_v ? p.vs : p.P2;            // even in both cases
    const unsigned char* src0 = reinterpret_cast<const unsigned char*>(is_v ? vg : kg);
    unsigned char* ring = is_v ? v_s : k_s;
    const uint32_t bar_f = is_v ? bar_fv : bar_fk, bar_e = is_v ? bar_ev : bar_ek;
    uint32_t swz[4][2];
    int nb[2];                                        // this lane's words of a row: 4 bytes each, or none
#pragma unroll
    for (int sl = 0; sl < 2; ++sl) {
      const int w = lane + 32 * sl;
      nb[sl] = 2 * rowlen - 4 * w >= 4 ? 4 : 0;
#pragma unroll
      for (int c = 0; c < 4; ++c) swz[c][sl] = pt_swz2(4 * w, (pw + 2 * c) & 7);
    }
    int stg = 0, use = 0;
    for (int tile = 0; tile < n_max; ++tile) {
      const int j0 = tile * P2_KT;
      if (use > 0 && !wait(bar_e + 8 * stg, (use - 1) & 1)) break;
      const uint32_t du = pt_smem(ring + stg * P2_KV_BYTES);
      const int rows_ok = min(P2_KT, n_valid - j0);
      const unsigned char* tsrc = src0 + (size_t)j0 * (size_t)(2 * rowlen);
      if (rows_ok == P2_KT) {
        // a full tile (all but the last one of a sequence): no predicates, running pointers
        const unsigned char* sp = tsrc + (size_t)pw * (size_t)(2 * rowlen) + 4 * lane;
        uint32_t db = du + (uint32_t)pw * 128u;
        const bool one = nb[0] > 0, two = nb[1] > 0;
#pragma unroll 4
        for (int i = 0; i < P2_KT / 2; ++i) {
          if (one) pt_cp4(db + swz[i & 3][0], sp, 4);
          if (two) pt_cp4(db + swz[i & 3][1], sp + 128, 4);
          sp += 4 * rowlen;                            // two rows on
          db += 256;
        }
      } else {
#pragma unroll 4
        for (int i = 0; i < P2_KT / 2; ++i) {
          const int r = pw + 2 * i;
          const bool ok = r < rows_ok;                 // rows past the end: zero fill, nothing is read
          const uint32_t* src = reinterpret_cast<const uint32_t*>(tsrc + (size_t)(ok ? r : 0) * (size_t)(2 * rowlen));
          const uint32_t rb = du + (uint32_t)r * 128u;
          if (nb[0] > 0) pt_cp4(rb + swz[i & 3][0], src + lane, ok ? 4 : 0);
          if (nb[1] > 0) pt_cp4(rb + swz[i & 3][1], src + lane + 32, ok ? 4 : 0);
        }
      }
      // the arrival is triggered by the completion of this thread's copies: go on to the next tile
      asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar_f + 8 * stg) : "memory");
      if (++stg == P2_STAGES) { stg = 0; ++use; }
    }
  } else if (warp >= 8) {
    // ================= MMA issue: lane 0 of warp 8 for query tile A, of warp 9 for query tile B =================
    // Two issuing lanes halve the serial chain of waits, fences, descriptors and commits per key tile.  A buffer of
    // the K / V rings is free when both lanes have committed past it; a lane whose tile needs no more keys keeps
    // arriving in step (after the buffer was filled), so the phases stay aligned.
    if (lane == 0) {
      const int Y = warp - 8, n_y = nt[Y];
      const uint32_t tmem_sy = tmem_base + 128u * (uint32_t)Y, tmem_oy = tmem_base + 256u + 128u * (uint32_t)Y;
      // This lane's instructions are the serial part of a key tile, so everything that does not change is worked out
      // here: the descriptors' high word, the low words of Q's k-steps, of the first K and V buffers; ring positions
      // and phases are counters, not divisions.
      constexpr uint32_t DESC_HI = (1024u >> 4) | (1u << 14) | (2u << 29);
      constexpr uint32_t BUF16 = (uint32_t)P2_KV_BYTES >> 4;
      uint32_t q_lo[DK];
#pragma unroll
      for (int ks = 0; ks < DK; ++ks)
        q_lo[ks] = (((pt_smem(q_s + Y * P2_Q_BYTES) + (uint32_t)((ks >> 2) * 16384 + (ks & 3) * 32)) & 0x3FFFFu) >> 4) | (1u << 16);
      const uint32_t k_lo0 = ((pt_smem(k_s) & 0x3FFFFu) >> 4) | (1u << 16);
      const uint32_t v_lo0 = ((pt_smem(v_s) & 0x3FFFFu) >> 4) | ((8192u >> 4) << 16);
      auto issue_s = [&](uint32_t kbuf, uint32_t sbuf) {     // S into buffer sbuf from K buffer kbuf
        const uint32_t kb = k_lo0 + kbuf * BUF16, td = tmem_sy + 64u * sbuf;
#pragma unroll
        for (int ks = 0; ks < DK; ++ks)
          pt_mma2(td, q_lo[ks], kb + (uint32_t)(((ks >> 2) * 8192 + (ks & 3) * 32) >> 4), DESC_HI, IDESC_S, ks > 0 ? 1u : 0u);
        pt_commit(bar_s + 8 * (2 * Y + sbuf));
      };
      auto release = [&](uint32_t bar, bool issued) {   // after MMAs: when they complete; otherwise at once
        if (issued) pt_commit(bar);
        else asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
      };
      bool ok = wait(bar_fk, 0);
      if (ok) {
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (n_y > 0) issue_s(0, 0);
        release(bar_ek, n_y > 0);
      }
      uint32_t kbuf = 1, kpar = 0;       // ring position and phase of K tile + 1
      uint32_t vbuf = 0, vpar = 0;       // of V tile
      for (int tile = 0; ok && tile < n_max; ++tile) {
        const uint32_t sb = (uint32_t)tile & 1u;
        if (tile + 1 < n_max) {
          if (!wait(bar_fk + 8 * kbuf, kpar)) { ok = false; break; }
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          if (tile + 1 < n_y) issue_s(kbuf, sb ^ 1u);
          release(bar_ek + 8 * kbuf, tile + 1 < n_y);
          if (++kbuf == P2_STAGES) { kbuf = 0; kpar ^= 1u; }
        }
        if (!wait(bar_fv + 8 * vbuf, vpar)) { ok = false; break; }
        if (tile < n_y) {
          if (!wait(bar_p + 8 * (2 * Y + sb), (uint32_t)(tile >> 1) & 1u)) { ok = false; break; }
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t vb = v_lo0 + vbuf * BUF16, ta = tmem_sy + 64u * sb;
#pragma unroll
          for (int ks = 0; ks < P2_KT / 16; ++ks)   // A = P in tensor memory, over the S columns it was computed from
            pt_mma_ts2(tmem_oy, ta + 8u * (uint32_t)ks, vb + (uint32_t)(ks * 2048 >> 4), DESC_HI, IDESC_O,
                       (tile > 0 || ks > 0) ? 1u : 0u);
          pt_commit(bar_o + 8 * Y);
        }
        release(bar_ev + 8 * vbuf, tile < n_y);
        if (++vbuf == P2_STAGES) { vbuf = 0; vpar ^= 1u; }
      }
      // every MMA issued above has completed before tensor memory is released
      pt_commit(bar_end + 8 * Y);
      wait(bar_end + 8 * Y, 0);
    }
    __syncwarp();
  } else {
    // ================= softmax group X: one thread per query row of tile X =================
    const int q0x = q0 + 128 * X;
    const int pos = start + q0x + row;
    const int n_my = nt[X];
    float m_ref = -1.0e30f;
    bool rows_ok = true;
    for (int tile = 0; tile < n_my; ++tile) {
      const int j0 = tile * P2_KT;
      const uint32_t trow = tmem_base + 128u * (uint32_t)X + 64u * (uint32_t)(tile & 1) + lane_off;
      if (!__all_sync(0xffffffffu, wait(bar_s + 8 * (2 * X + (tile & 1)), (tile >> 1) & 1))) { rows_ok = false; break; }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      uint32_t r[64];
      pt_ld32_nowait(trow, *reinterpret_cast<uint32_t(*)[32]>(r));
      pt_ld32_nowait(trow + 32, *reinterpret_cast<uint32_t(*)[32]>(r + 32));
      asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
      const bool interior = j0 + P2_KT - 1 <= start + q0x;   // no key of the tile is masked for any row of the tile
      float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
      if (interior) {
#pragma unroll
        for (int j = 0; j < 64; ++j) mx4[j & 3] = fmaxf(mx4[j & 3], __uint_as_float(r[j]));
      } else {
#pragma unroll
        for (int j = 0; j < 64; ++j)
          if (j0 + j <= pos) mx4[j & 3] = fmaxf(mx4[j & 3], __uint_as_float(r[j]));
      }
      const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * p.qscale;
      float alpha = 1.f;
      if (mx > m_ref + 8.f) {          // lazy reference maximum: p stays <= 2^8
        alpha = pt_ex2(m_ref - mx);
        m_ref = mx;
        l_run *= alpha;
      }
      const float nm = -m_ref;
      float ls[4] = {0.f, 0.f, 0.f, 0.f};
      if (interior) {
        // no mask
        // two logits per packed FMA, two weights per packed add
        uint64_t qs2, nm2, l2[4] = {0ull, 0ull, 0ull, 0ull};
        asm("mov.b64 %0, {%1, %1};" : "=l"(qs2) : "f"(p.qscale));
        asm("mov.b64 %0, {%1, %1};" : "=l"(nm2) : "f"(nm));
#pragma unroll
        for (int j = 0; j < 64; j += 2) {
          uint64_t s2, x2, p2;
          asm("mov.b64 %0, {%1, %2};" : "=l"(s2) : "r"(r[j]), "r"(r[j + 1]));
          asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(x2) : "l"(s2), "l"(qs2), "l"(nm2));
          float x0, x1;
          asm("mov.b64 {%0, %1}, %2;" : "=f"(x0), "=f"(x1) : "l"(x2));
          const float p0 = pt_ex2(x0), p1 = pt_ex2(x1);
          const __nv_bfloat162 v2 = __floats2bfloat162_rn(p0, p1);
          const uint32_t pk = *reinterpret_cast<const uint32_t*>(&v2);
          if constexpr (!LSUM) {
            // the row sum takes the rounded weights the second MMA will see (a one-hot row comes out exact)
            asm("mov.b64 %0, {%1, %2};" : "=l"(p2) : "r"(pk << 16), "r"(pk & 0xffff0000u));
            asm("add.rn.f32x2 %0, %1, %2;" : "=l"(l2[(j >> 1) & 3]) : "l"(l2[(j >> 1) & 3]), "l"(p2));
          }
          r[j >> 1] = pk;
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          float a0, a1;
          asm("mov.b64 {%0, %1}, %2;" : "=f"(a0), "=f"(a1) : "l"(l2[k]));
          ls[k] += a0 + a1;
        }
      } else {
        // diagonal tile: causal mask
#pragma unroll
        for (int j = 0; j < 64; j += 2) {
          float p0 = pt_ex2(fmaf(__uint_as_float(r[j]), p.qscale, nm));
          float p1 = pt_ex2(fmaf(__uint_as_float(r[j + 1]), p.qscale, nm));
          if (j0 + j > pos) p0 = 0.f;
          if (j0 + j + 1 > pos) p1 = 0.f;
          const __nv_bfloat162 v2 = __floats2bfloat162_rn(p0, p1);
          const uint32_t pk = *reinterpret_cast<const uint32_t*>(&v2);
          if constexpr (!LSUM) ls[(j >> 1) & 3] += __uint_as_float(pk << 16) + __uint_as_float(pk & 0xffff0000u);
          r[j >> 1] = pk;
        }
      }
      l_run += (ls[0] + ls[1]) + (ls[2] + ls[3]);
      if (tile > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {
        // rare: rescale this warp's accumulator rows in tensor memory, once the previous tile's update is in
        if (!__all_sync(0xffffffffu, wait(bar_o + 8 * X, (tile - 1) & 1))) { rows_ok = false; break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        {
#pragma unroll 1
          for (int c0 = 0; c0 < NVP; c0 += 32) {
            uint32_t oc[32];
            pt_ld32(tmem_o + lane_off + c0, oc);
#pragma unroll
            for (int j = 0; j < 32; ++j) oc[j] = __float_as_uint(__uint_as_float(oc[j]) * alpha);
            pt_st32(tmem_o + lane_off + c0, oc);
          }
          asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        }
      }
      // P (64 bf16 = 32 packed columns) goes back into tensor memory over the first half of the S columns it came
      // from: it is the A operand of the second MMA, and the next S into this buffer is issued after that MMA
      pt_st32(trow, *reinterpret_cast<uint32_t(*)[32]>(r));
      asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar_p + 8 * (2 * X + (tile & 1))) : "memory");
    }
    if (rows_ok && n_my > 0) __all_sync(0xffffffffu, wait(bar_o + 8 * X, (n_my - 1) & 1));
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  const bool timed_out = *abort_flag != 0;
  if (timed_out && tid == 0) {
    atomicCAS(&p.status[0], 0, (int)RAP_ETIMEOUT);
    p.status[1] = 0x60000000 | (qb & 0xffffff);
  }
  // The tiles are free now (every MMA has completed, every copy has landed).  A thread owns a query row in tensor
  // memory, but a row of the output is contiguous in global memory: the normalised rows go through shared memory
  // (rows of NVP + 1 floats: the row-per-thread stores hit 32 banks) and leave as whole rows, one warp per row.
  float* o_s = reinterpret_cast<float*>(smem);
  constexpr int OS = NVP + 1;
  static_assert(256 * OS * 4 <= P2_SMEM - P2_TAIL, "the output tile fits the freed tiles");
  if (warp < 8 && !timed_out && nt[X] > 0) {
    if constexpr (LSUM) l_run = __uint_as_float(pt_ld1(tmem_o + lane_off + (uint32_t)p.vs));
    const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
    float* orow = o_s + (size_t)(128 * X + row) * OS;
#pragma unroll 1
    for (int c0 = 0; c0 < NVP; c0 += 32) {
      uint32_t oc[32];
      pt_ld32(tmem_o + lane_off + c0, oc);
#pragma unroll
      for (int j = 0; j < 32; ++j) orow[c0 + j] = __uint_as_float(oc[j]) * inv;
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  }
  __syncthreads();
  if (!timed_out) {
    for (int r = warp; r < 256; r += P2_THREADS / 32) {
      const int t = q0 + r;
      if (t < p.T && nt[r >> 7] > 0) {
        float* dst = p.out + (((size_t)b * p.T + t) * p.Hq + g) * p.dv;
        const float* src = o_s + (size_t)r * OS;
        for (int c = lane; c < p.dv; c += 32) dst[c] = src[c];
      }
    }
  }
  if (warp == 8) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
  }
}

template <int DK, int NVP, bool LSUM>
rap_status launch_pt(rap_ctx* ctx, const PtParams& p, int B, cudaStream_t st) {
  const int smem = P2_SMEM + 1024;
  RAP_CUDA_TRY(ctx, rap_raise_smem(ctx, prefill_tc_kernel<DK, NVP, LSUM>, smem));
  dim3 grid(p.Hq, B, (p.T + 255) / 256);
  prefill_tc_kernel<DK, NVP, LSUM><<<grid, P2_THREADS, smem, st>>>(p);
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
  p.T = T; p.Hq = d.n_q_heads; p.Hkv = d.n_kv_heads; p.P2 = P2; p.dv = dv; p.S_cap = S_cap; p.vs = dv;
  p.qscale = (float)(1.4426950408889634 / sqrt((double)d.head_dim));
  if (dv & 1) {
    // rows of an odd length: copy what the block can see to rows of d_v' + 1 elements (workspace grown on demand;
    // the growth allocates, so the first call at a new size is not for a stream capture)
    const size_t need = (size_t)B * d.n_kv_heads * (size_t)S_cap * (size_t)(dv + 1) * sizeof(__nv_bfloat16);
    if (need > ctx->pf_v_bytes) {
      RAP_CUDA_TRY(ctx, cudaStreamSynchronize(st));
      if (ctx->d_pf_v) cudaFree(ctx->d_pf_v);
      ctx->d_pf_v = nullptr; ctx->pf_v_bytes = 0;
      RAP_CUDA_TRY(ctx, cudaMalloc(&ctx->d_pf_v, need));
      ctx->pf_v_bytes = need;
    }
    dim3 grid(64, B * d.n_kv_heads);
    prefill_repack_v_kernel<<<grid, 256, 0, st>>>(p.v, (__nv_bfloat16*)ctx->d_pf_v, start, T, d.n_kv_heads, dv, S_cap);
    ctx->launches++;
    RAP_CUDA_TRY(ctx, cudaGetLastError());
    p.v = (const __nv_bfloat16*)ctx->d_pf_v;
    p.vs = dv + 1;
  }
  // p.vs + 1 channels when the row sums ride along as a ones column (every shape but the ones that fill their last
  // 32-channel block: then the softmax threads keep the sums)
  const int dk = (P2 + 15) / 16, nvp = (p.vs + 1 + 31) / 32 * 32;
  if (dk <= 4 && nvp <= 64) return launch_pt<4, 64, true>(ctx, p, B, st);
  if (dk <= 4 && nvp <= 96) return launch_pt<4, 96, true>(ctx, p, B, st);
  if (dk <= 6 && nvp <= 96) return launch_pt<6, 96, true>(ctx, p, B, st);
  if (dk <= 7 && nvp <= 128) return launch_pt<7, 128, true>(ctx, p, B, st);
  if (nvp <= 128) return launch_pt<8, 128, true>(ctx, p, B, st);
  return launch_pt<8, 128, false>(ctx, p, B, st);
}
