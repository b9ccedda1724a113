// tcgen05 projection GEMM of rap_qkv_rope_append (Eq. 1 on the reduced widths): bf16 in, fp32
// accumulate in tensor memory.
//
//   Y[ks][t][n] = sum_{k in split ks} X[t][k] * W~[n][k]
//
// computed "swap-AB": the weight rows sit on the MMA's M side (128 rows per CTA, the full
// tensor-memory lane range) and the tokens on its N side (32 / 64 / 128 / 256 per CTA), so that a
// decode-sized call (T <= 32) still issues full-height instructions and is bounded by streaming
// the weights from HBM, while a prefill-shaped call (T in the thousands) is a dense contraction.
// Both operands are K-major, staged by TMA (cp.async.bulk.tensor.2d, 128-byte swizzle, no
// multicast, OOB rows / columns read as zeros) into a ring of shared-memory stages.
//
// The kernel is persistent (one CTA per SM walks a list of work items = row tile x token tile x reduction
// split); the accumulator is double buffered in tensor memory so the epilogue of one item overlaps the
// MMAs of the next.  Roles inside one CTA of 192 threads:
//   warp 0   producer: one lane waits for a free stage, arms its mbarrier with the byte count
//            and issues the two tensor copies (W tile 128 x 64, X tile TN x 64);
//   warp 1   allocates TN tensor-memory columns; one lane waits for a full stage and issues four
//            tcgen05.mma (K = 16 each) on shared-memory descriptors, then tcgen05.commit frees the
//            stage; a last commit signals the accumulator;
//   warps 2-5 epilogue: tcgen05.ld of the warp's 32 lanes x 32 columns, coalesced fp32 stores to
//            the workspace (consecutive lanes = consecutive output features n).
// A reduction split lets a decode-sized call use every SM.  For calls of more than 32 rows the RoPE / append
// epilogue kernel (rap_proj.cu) sums the splits.  For decode-sized calls (T <= 32) the epilogue is fused in
// (FUSED = true): every epilogue warp owns 32 weight rows of its CTA's row tile; it stores its partial, and the warp
// that delivers the last split of those 32 rows (an arrival counter per row tile and warp quarter) sums the
// splits from L2, adds the bias, rotates the retained pairs (the partner of a row is the adjacent row, i.e. the
// adjacent lane), rounds once and scatters q~ / K row / V row -- no second launch, no second pass.  The sine and
// cosine of a lane's rows are computed while the warp would otherwise wait for the accumulator.  The fused kernel
// also takes part in programmatic dependent launch: it lets its successor start early and waits for its
// predecessor only before it writes q~ and the cache rows (its weight streaming overlaps the predecessor's tail).
// Every mbarrier wait is bounded; a wait that gives up records RAP_ETIMEOUT in the device status word and the
// CTA winds down.
#include <cuda.h>

#include <string.h>

#include <mutex>

#include "rap_internal.h"

namespace {

constexpr int TC_BM = 128;              // weight rows per CTA = MMA M
constexpr int TC_BK = 64;               // bf16 elements per stage along K = one 128-byte swizzle row
constexpr int TC_THREADS = 192;
constexpr int TC_A_BYTES = TC_BM * TC_BK * 2;
constexpr int TC_SMEM_TILES = 196608;   // bytes of the stage ring at most
constexpr uint32_t TC_WAIT_LIMIT = 1u << 21;

template <int TN>
struct TcCfg {
  static constexpr int B_BYTES = TN * TC_BK * 2;
  static constexpr int STAGE = TC_A_BYTES + B_BYTES;            // multiples of 1024: descriptors need no base offset
  static constexpr int NS_RAW = TC_SMEM_TILES / STAGE;
  static constexpr int NS = NS_RAW > 8 ? 8 : NS_RAW;
  static constexpr int OFF_BARS = NS * STAGE;                   // full[NS], empty[NS], acc_full[2], acc_empty[2], tmem slot
  static constexpr int SMEM = OFF_BARS + (2 * NS + 5) * 8 + 1024;   // + slack to align the ring to 1024 bytes
  // fused epilogue: per epilogue warp [16][32] (cos, sin) pairs and [32][32] summed results
  static constexpr int OFF_FUSED = (OFF_BARS + (2 * NS + 5) * 8 + 15) & ~15;
  static constexpr int FUSED_WARP_BYTES = 16 * 32 * 8 + 32 * 32 * 4;
  static constexpr int SMEM_FUSED = OFF_FUSED + 4 * FUSED_WARP_BYTES + 1024;
  // instruction descriptor: fp32 accumulate, bf16 x bf16, both K-major, N = TN, M = 128
  static constexpr uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(TN >> 3) << 17) | ((uint32_t)(TC_BM >> 4) << 24);
};

__device__ __forceinline__ uint32_t tc_smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void tc_mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void tc_mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool tc_mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool tc_mbar_wait(uint32_t bar, uint32_t parity) {
  {   // first a probe that never parks the thread: try_wait may, and then costs a few hundred cycles even when the phase is over
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    if (ok) return true;
  }
  for (uint32_t i = 0; i < TC_WAIT_LIMIT; ++i)
    if (tc_mbar_try_wait(bar, parity)) return true;
  return false;
}
// 2-D tiled tensor copy global -> this CTA's shared memory (no multicast); x = element index along K
__device__ __forceinline__ void tc_tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
      "l"(map), "r"(x), "r"(y), "r"(bar)
      : "memory");
}
// shared-memory matrix descriptor of a K-major tile stored as 128-byte rows with the 128-byte
// swizzle: 8-row groups are 1024 bytes apart (stride offset), leading offset unused (1)
__device__ __forceinline__ uint64_t tc_smem_desc(uint32_t addr) {
  const uint32_t lo = ((addr & 0x3FFFFu) >> 4) | (1u << 16);
  const uint32_t hi = (1024u >> 4) | (1u << 14) | (2u << 29);   // stride offset, descriptor version 1, SWIZZLE_128B
  return ((uint64_t)hi << 32) | lo;
}
__device__ __forceinline__ void tc_mma(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&r)[32]) {
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

struct TcParams {
  float* y;            // [ksplit][T][n_out]
  int32_t* status;
  int T, n_out, nkb_total, nkb_per_split;
  int row_tiles, tok_tiles, n_work;     // work items = row tiles x token tiles x reduction splits
  int wait_x;          // x is written by the previous kernel in the stream (programmatic launch): wait for it before x is read
};

// What the fused RoPE / append epilogue needs beyond the GEMM (decode-sized calls, one token tile).
struct TcFused {
  const __nv_bfloat16* bias;                 // [n_out] or nullptr
  const int32_t* seq_id;                     // nullptr: row t belongs to sequence t
  const int32_t* pos;
  const int32_t* slot;                       // nullptr: slot = pos
  const double* inv_freq;                    // this layer's [H_kv][half_dim]
  __nv_bfloat16* q_out;
  __nv_bfloat16* k_cache;
  __nv_bfloat16* v_cache;
  int32_t* cnt;                              // [row_tiles][4] split arrivals of this launch (zero on entry, zero on exit)
  int32_t* cnt_other;                        // the set the previous launch used: cleared here in case that launch gave up
  int n_cnt;
  int ksplit, Hq, Hkv, P2, dv, half_dim, B_cache, S_cap;
};

__device__ __forceinline__ void tc_pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void tc_pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__device__ __forceinline__ void tc_mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

// Persistent: CTA c takes work items c, c + gridDim.x, ...  The stage ring runs on across items, and the
// accumulator is double buffered in tensor memory (2 x TN columns) so that the epilogue of one item
// overlaps the MMAs of the next.
template <int TN, bool FUSED>
__global__ void __launch_bounds__(TC_THREADS, 1)
proj_tc_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_x, const TcParams p,
               const TcFused f) {
  using C = TcCfg<TN>;
  static_assert(!FUSED || TN == 32, "the fused epilogue holds one 32-token chunk per lane");
  extern __shared__ unsigned char tc_smem_raw[];
  // the swizzled tiles and their descriptors want a 1024-byte aligned ring
  unsigned char* smem = tc_smem_raw + ((1024u - (tc_smem_u32(tc_smem_raw) & 1023u)) & 1023u);
  const uint32_t ring = tc_smem_u32(smem);
  const uint32_t full0 = ring + C::OFF_BARS, empty0 = full0 + 8 * C::NS;
  const uint32_t acc_full0 = empty0 + 8 * C::NS, acc_empty0 = acc_full0 + 16;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + C::OFF_BARS + (2 * C::NS + 4) * 8);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < C::NS; ++s) {
      tc_mbar_init(full0 + 8 * s, 1);
      tc_mbar_init(empty0 + 8 * s, 1);
    }
    for (int s = 0; s < 2; ++s) {
      tc_mbar_init(acc_full0 + 8 * s, 1);
      tc_mbar_init(acc_empty0 + 8 * s, 4);      // one arrival per epilogue warp
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {   // tensor-memory columns for two accumulators (power of two >= 32)
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tc_smem_u32(tmem_slot)),
                 "r"(2 * TN)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_d = *tmem_slot;
  bool timed_out = false;
  tc_pdl_launch_dependents();        // the next kernel in the stream may start its own prologue
  if constexpr (FUSED) {
    if (blockIdx.x == 0)             // counters a predecessor that gave up may have left behind
      for (int i = threadIdx.x; i < f.n_cnt; i += TC_THREADS) f.cnt_other[i] = 0;
  }

  // work item w -> (token tile, row tile, split); token tiles vary fastest so that the CTAs working at the
  // same time share a weight tile through L2
  auto decode = [&](int w, int& n0, int& t0, int& ks, int& kb0, int& nkb) {
    const int tt = w % p.tok_tiles, rest = w / p.tok_tiles;
    const int rt = rest % p.row_tiles;
    ks = rest / p.row_tiles;
    n0 = rt * TC_BM;
    t0 = tt * TN;
    kb0 = ks * p.nkb_per_split;
    nkb = max(0, min(p.nkb_per_split, p.nkb_total - kb0));
  };

  if (warp == 0) {
    if (lane == 0) {
      uint32_t kbg = 0;      // k-blocks issued so far: position in the ring
      int pre = 0;           // k-blocks of the first item already issued
      if (p.wait_x) {
        // The weights do not depend on the previous kernel: the first ring-full of W tiles goes out before the wait,
        // the x tiles of those stages after it (the stages are empty on the first lap).
        int n0, t0, ks, kb0, nkb = 0;
        if ((int)blockIdx.x < p.n_work) decode(blockIdx.x, n0, t0, ks, kb0, nkb);
        pre = nkb < C::NS ? nkb : C::NS;
        for (int kb = 0; kb < pre; ++kb) {
          tc_mbar_expect_tx(full0 + 8 * kb, C::STAGE);
          tc_tma_load_2d(ring + kb * C::STAGE, &map_w, (kb0 + kb) * TC_BK, n0, full0 + 8 * kb);
        }
        tc_pdl_wait();
        for (int kb = 0; kb < pre; ++kb)
          tc_tma_load_2d(ring + kb * C::STAGE + TC_A_BYTES, &map_x, (kb0 + kb) * TC_BK, t0, full0 + 8 * kb);
        kbg = (uint32_t)pre;
      }
      for (int w = blockIdx.x; w < p.n_work && !timed_out; w += gridDim.x) {
        int n0, t0, ks, kb0, nkb;
        decode(w, n0, t0, ks, kb0, nkb);
        for (int kb = (w == (int)blockIdx.x ? pre : 0); kb < nkb; ++kb, ++kbg) {
          const uint32_t s = kbg % C::NS, ph = (kbg / C::NS) & 1u;
          if (!tc_mbar_wait(empty0 + 8 * s, ph ^ 1u)) { timed_out = true; break; }   // first lap passes at once
          const uint32_t a = ring + s * C::STAGE, b = a + TC_A_BYTES;
          tc_mbar_expect_tx(full0 + 8 * s, C::STAGE);
          tc_tma_load_2d(a, &map_w, (kb0 + kb) * TC_BK, n0, full0 + 8 * s);
          tc_tma_load_2d(b, &map_x, (kb0 + kb) * TC_BK, t0, full0 + 8 * s);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      uint32_t kbg = 0, it = 0;    // it: items with work so far -> accumulator buffer and its phase
      for (int w = blockIdx.x; w < p.n_work && !timed_out; w += gridDim.x) {
        int n0, t0, ks, kb0, nkb;
        decode(w, n0, t0, ks, kb0, nkb);
        if (nkb == 0) continue;
        const uint32_t buf = it & 1u, use = it >> 1;
        if (!tc_mbar_wait(acc_empty0 + 8 * buf, (use & 1u) ^ 1u)) { timed_out = true; break; }   // epilogue done with it
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        for (int kb = 0; kb < nkb; ++kb, ++kbg) {
          const uint32_t s = kbg % C::NS, ph = (kbg / C::NS) & 1u;
          if (!tc_mbar_wait(full0 + 8 * s, ph)) { timed_out = true; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint64_t adesc = tc_smem_desc(ring + s * C::STAGE);
          const uint64_t bdesc = tc_smem_desc(ring + s * C::STAGE + TC_A_BYTES);
#pragma unroll
          for (int kk = 0; kk < TC_BK / 16; ++kk)   // 16 bf16 = 32 bytes = 2 descriptor address units per step
            tc_mma(tmem_d + buf * TN, adesc + 2 * kk, bdesc + 2 * kk, C::IDESC, (kb | kk) != 0 ? 1u : 0u);
          tc_commit(empty0 + 8 * s);     // arrives when the MMAs above have read the stage
        }
        if (timed_out) break;
        tc_commit(acc_full0 + 8 * buf);
        ++it;
      }
    }
  } else {
    // epilogue: this warp reads tensor-memory lanes 32 * (warp % 4) .. + 31 = weight rows of the tile
    const int quarter = warp & 3;
    uint32_t it = 0;
    for (int w = blockIdx.x; w < p.n_work; w += gridDim.x) {
      int n0, t0, ks, kb0, nkb;
      decode(w, n0, t0, ks, kb0, nkb);
      const int n = n0 + quarter * 32 + lane;
      const uint32_t buf = it & 1u, use = it >> 1;

      // fused epilogue, part 1 (while the MMAs of this item run): what this lane's weight row is, where its results
      // go, and the sine and cosine of its pair -- each lane of a pair evaluates half of the tokens (the even lane
      // 0..15, the odd lane 16..31) into shared memory.  The loops of the fused epilogue are kept rolled: a warp runs
      // this code once, so its cost is the instruction fetch as much as the arithmetic.
      int kind = 2;                            // 0: q row, 1: k row, 2: v row (or past the end)
      __nv_bfloat16* dst = nullptr;            // q~: element of token 0; K / V: element of cache row 0 of this lane's head
      int row_w = 0;                           // K / V: row width in elements
      float2* cs_w = nullptr;                  // [16][32] (cos, sin): entry [j][l] belongs to token j + 16 (l & 1) of lane l's pair
      float* vs_w = nullptr;                   // [32][32] summed results, token-major
      float bias = 0.f;
      int my_row = -1;                         // lane t: cache row of token t over all sequences, for head 0; -1 = skip the row
      bool bad_row = false;                    // lane t: token t names a sequence or a slot that is not there
      if constexpr (FUSED) {
        if (n < p.n_out && f.bias) bias = __bfloat162float(f.bias[n]);
        if (lane < p.T) {
          const int sq = f.seq_id ? f.seq_id[lane] : lane;
          const int sl = f.slot ? f.slot[lane] : f.pos[lane];
          if (sq >= 0 && sq < f.B_cache && sl >= 0 && sl < f.S_cap) my_row = sq * f.Hkv * f.S_cap + sl;   // fits: checked on the host
          else bad_row = true;
        }
        unsigned char* fw = smem + C::OFF_FUSED + quarter * C::FUSED_WARP_BYTES;
        cs_w = reinterpret_cast<float2*>(fw);
        vs_w = reinterpret_cast<float*>(fw + 16 * 32 * 8);
        const int nq = f.Hq * f.P2, nk = f.Hkv * f.P2;
        int head = 0, r = 0;
        if (n < nq) { kind = 0; head = n / f.P2; r = n - head * f.P2; }
        else if (n < nq + nk) { kind = 1; head = (n - nq) / f.P2; r = n - nq - head * f.P2; }
        else if (n < p.n_out) { head = (n - nq - nk) / f.dv; r = n - nq - nk - head * f.dv; }
        const int hkv = kind == 0 ? head / (f.Hq / f.Hkv) : head;
        const double freq = kind < 2 ? f.inv_freq[hkv * f.half_dim + (r >> 1)] : 0.0;
        if (kind == 0) dst = f.q_out + (size_t)head * f.P2 + r;
        else if (kind == 1) { dst = f.k_cache + (size_t)head * f.S_cap * f.P2 + r; row_w = f.P2; }
        else { dst = f.v_cache + (size_t)head * f.S_cap * f.dv + r; row_w = f.dv; }
#pragma unroll 1
        for (int j = 0; j < 16; ++j) {
          const int t = j + 16 * (lane & 1);
          float c = 1.f, sn = 0.f;
          if (t < p.T && freq != 0.0) {
            // fp64 angle and reduction to [-pi, pi] (positions reach 1e5 and more), fp32 sine and cosine of the rest
            const double ang = (double)f.pos[t] * freq;
            const double turns = rint(ang * 0.15915494309189535);
            const double red = fma(-turns, 2.4492935982947064e-16, fma(-turns, 6.283185307179586, ang));
            sincosf((float)red, &sn, &c);
          }
          cs_w[j * 32 + lane] = make_float2(c, sn);
        }
        __syncwarp();
      }

      bool ready = true;
      if (nkb > 0) {
        ready = __all_sync(0xffffffffu, !timed_out && tc_mbar_wait(acc_full0 + 8 * buf, use & 1u));
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (!ready) timed_out = true;
      }
      float* ybase = p.y + (size_t)ks * p.T * p.n_out;
#pragma unroll 1
      for (int c0 = 0; c0 < TN; c0 += 32) {
        if (t0 + c0 >= p.T) break;             // columns past the last token hold zero-filled rows
        uint32_t r32[32];
        if (nkb > 0 && ready) {
          tc_ld32(tmem_d + buf * TN + ((uint32_t)(quarter * 32) << 16) + (uint32_t)c0, r32);
          asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        } else {
#pragma unroll
          for (int j = 0; j < 32; ++j) r32[j] = 0u;
        }
        if (n < p.n_out) {
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const int t = t0 + c0 + j;
            if (t < p.T) ybase[(size_t)t * p.n_out + n] = __uint_as_float(r32[j]);
          }
        }
      }
      if (nkb > 0) {
        if (ready) {
          asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
          __syncwarp();
          if (lane == 0) tc_mbar_arrive(acc_empty0 + 8 * buf);    // this warp has drained the accumulator
        }
        ++it;
      }

      if constexpr (FUSED) {
        // fused epilogue, part 2: count this warp's partial in; the warp that brings the last one finishes the rows.
        // A warp that timed out does not count itself in, so the rows are never finished from a missing partial.
        int last = 0;
        if (ready) {
          __threadfence();                       // the partial is visible before the arrival is
          __syncwarp();
          const int slot_c = (n0 / TC_BM) * 4 + quarter;
          if (lane == 0) last = atomicAdd(&f.cnt[slot_c], 1) == f.ksplit - 1;
          last = __shfl_sync(0xffffffffu, last, 0);
          if (last) {
            __threadfence();
            tc_pdl_wait();                       // the previous kernel in the stream may still read q~
            const size_t split_stride = (size_t)p.T * p.n_out;
            const bool in_range = n < p.n_out;
            // sum the splits.  Every batch of loads is one round trip through a memory system that other CTAs are
            // still saturating (microseconds, not hundreds of nanoseconds), so a batch covers all tokens and four
            // splits: 128 independent loads for the usual split counts
            {
              float v[32];
#pragma unroll
              for (int t = 0; t < 32; ++t) v[t] = 0.f;
#pragma unroll 1
              for (int s0 = 0; s0 < f.ksplit; s0 += 4) {
                float part[4][32];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                  const float* src = p.y + (size_t)(s0 + u) * split_stride + n;
                  const bool on = s0 + u < f.ksplit && in_range &&
                                  RAP_BOUNDS((size_t)(s0 + u) * split_stride + (size_t)(p.T - 1) * p.n_out + n,
                                             (size_t)f.ksplit * split_stride, p.status, 0x301);
#pragma unroll
                  for (int t = 0; t < 32; ++t) part[u][t] = (on && t < p.T) ? __ldcg(src + (size_t)t * p.n_out) : 0.f;
                }
#pragma unroll
                for (int u = 0; u < 4; ++u)
#pragma unroll
                  for (int t = 0; t < 32; ++t) v[t] += part[u][t];
              }
#pragma unroll
              for (int t = 0; t < 32; ++t) vs_w[t * 32 + lane] = v[t] + bias;     // splits in order, then the bias
            }
            if (bad_row && n0 == 0 && quarter == 0) {    // reported once per launch: by the warp that owns weight row 0
              atomicCAS(&p.status[0], 0, (int)RAP_ECAPACITY);
              p.status[1] = lane;
            }
            __syncwarp();
            const size_t q_stride = (size_t)f.Hq * f.P2;
            const int cs_lane = (lane & ~1);
#pragma unroll 4
            for (int t = 0; t < p.T; ++t) {
              if (!RAP_BOUNDS(t, 32, p.status, 0x304)) break;     // (the staging buffers hold 32 tokens)
              const float mine = vs_w[t * 32 + lane], other = vs_w[t * 32 + (lane ^ 1)];
              const float2 cs = cs_w[(t & 15) * 32 + (cs_lane | (t >> 4))];
              const int row = __shfl_sync(0xffffffffu, my_row, t);
              // pair (a, b) on lanes (even, odd):  a' = a cos - b sin,  b' = a sin + b cos
              const float rot = (lane & 1) ? fmaf(other, cs.y, __fmul_rn(mine, cs.x)) : fmaf(-other, cs.y, __fmul_rn(mine, cs.x));
              const __nv_bfloat16 o = __float2bfloat16_rn(kind == 2 ? mine : rot);
              if (in_range) {
                if (kind == 0) {
                  if (RAP_BOUNDS((dst - f.q_out) + (long long)(t * q_stride), (long long)p.T * (long long)q_stride, p.status, 0x302))
                    dst[t * q_stride] = o;
                } else if (row >= 0) {                             // a row whose sequence or slot is out of range is skipped
                  if (RAP_BOUNDS((dst - (kind == 1 ? f.k_cache : f.v_cache)) + (long long)row * row_w,
                                 (long long)f.B_cache * f.Hkv * f.S_cap * row_w, p.status, 0x303))
                    dst[(size_t)row * row_w] = o;
                }
              }
            }
            if (lane == 0) f.cnt[slot_c] = 0;      // ready for the next launch that uses this set
          }
        }
      }
    }
  }
  if (timed_out && lane == 0) {
    atomicCAS(&p.status[0], 0, (int)RAP_ETIMEOUT);
    p.status[1] = 0x50000000 | (warp << 24) | (blockIdx.x & 0xffffff);
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_d), "r"(2 * TN) : "memory");
  }
  // The plain form writes nothing its predecessor in the stream reads, so it never had to wait for it; but a kernel
  // launched behind this one with programmatic serialization only waits for THIS kernel: by not ending before the
  // predecessor has, this kernel's completion stands for both.
  if constexpr (!FUSED) tc_pdl_wait();
}

typedef CUresult (*encode_tiled_t)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

encode_tiled_t get_encode_fn() {
  static encode_tiled_t fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<encode_tiled_t>(p);
  });
  return fn;
}

// [rows][cols] bf16 row-major -> tiles of box_rows x 64 elements, 128-byte swizzle, zero fill outside
bool make_map(rap_ctx* ctx, CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  static_assert(sizeof(CUtensorMap) == 128, "tensor map size");
  for (const rap_ctx::MapSlot& m : ctx->tmaps)
    if (m.base == base && m.rows == rows && m.cols == cols && m.box == box_rows) {
      memcpy(map, m.map, sizeof(CUtensorMap));
      return true;
    }
  encode_tiled_t fn = get_encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {cols * 2};
  const cuuint32_t box[2] = {TC_BK, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  if (fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return false;
  rap_ctx::MapSlot slot;
  slot.base = base; slot.rows = rows; slot.cols = cols; slot.box = box_rows;
  memcpy(slot.map, map, sizeof(CUtensorMap));
  if (ctx->tmaps.size() < 256) {
    ctx->tmaps.push_back(slot);
  } else {
    ctx->tmaps[ctx->tmap_next] = slot;
    ctx->tmap_next = (ctx->tmap_next + 1) % 256;
  }
  return true;
}

// pdl: launch with programmatic stream serialization.  The plain GEMM reads X and W and writes only the projection
// workspace, none of which the kernel before it in a decode step (an attention scan) touches, so it may run alongside
// that kernel's tail without waiting for it; the epilogue kernel after it is launched normally and waits for both.
template <int TN>
rap_status launch_tc(rap_ctx* ctx, const CUtensorMap& mw, const CUtensorMap& mx, const TcParams& p, dim3 grid,
                     cudaStream_t st, int pdl) {
  RAP_CUDA_TRY(ctx, rap_raise_smem(ctx, proj_tc_kernel<TN, false>, TcCfg<TN>::SMEM));
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(TC_THREADS, 1, 1);
  cfg.dynamicSmemBytes = TcCfg<TN>::SMEM;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  RAP_CUDA_TRY(ctx, cudaLaunchKernelEx(&cfg, proj_tc_kernel<TN, false>, mw, mx, p, TcFused{}));
  ctx->launches++;
  return RAP_OK;
}

// Work split of one GEMM call: token tile width, reduction splits (enough CTAs for every SM on decode-sized
// calls, within the workspace, no empty split) and the work-item counts.
bool plan_gemm(const rap_ctx* ctx, int T, int K, int N, int* tn_out, int* ksplit_out, TcParams* p) {
  const int tn = T <= 32 ? 32 : T <= 64 ? 64 : T <= 128 ? 128 : 256;
  const int row_tiles = (N + TC_BM - 1) / TC_BM, tok_tiles = (T + tn - 1) / tn;
  const int nkb = (K + TC_BK - 1) / TC_BK;
  int ksplit = ctx->sm_count / (row_tiles * tok_tiles);
  if (ksplit > RAP_MAX_KSPLIT) ksplit = RAP_MAX_KSPLIT;
  if (ksplit > nkb / 4) ksplit = nkb / 4;
  while (ksplit > 1 && (size_t)ksplit * T * N * sizeof(float) > ctx->proj_ws_bytes) --ksplit;
  if (ksplit < 1) ksplit = 1;
  const int per = (nkb + ksplit - 1) / ksplit;
  ksplit = (nkb + per - 1) / per;          // no empty split
  if ((size_t)ksplit * T * N * sizeof(float) > ctx->proj_ws_bytes) return false;
  p->y = ctx->d_proj_ws; p->status = ctx->d_status; p->T = T; p->n_out = N; p->nkb_total = nkb; p->nkb_per_split = per;
  p->row_tiles = row_tiles; p->tok_tiles = tok_tiles; p->n_work = row_tiles * tok_tiles * ksplit;
  p->wait_x = 0;
  *tn_out = tn;
  *ksplit_out = ksplit;
  return true;
}

}  // namespace

bool rap_tensor_map_bf16(rap_ctx* ctx, void* map128, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  return make_map(ctx, reinterpret_cast<CUtensorMap*>(map128), base, rows, cols, box_rows);
}

// Y[ks][T][N] (fp32, context workspace) = X[T][K] * W[N][K]^T, bf16 operands, K split over work items.
// pdl: 0 = ordinary launch; 1 = programmatic stream serialization, x does not depend on the previous kernel in the
// stream; 2 = the same, and x is what that kernel writes (the first weight tiles still go out before the wait)
rap_status rap_launch_gemm_tc(rap_ctx* ctx, const void* x, const void* w, int T, int K, int N, int* ksplit_out,
                              cudaStream_t st, int pdl) {
  if (T < 1 || (K % 8) != 0) return RAP_EUNSUPPORTED;     // tensor-map rows must be multiples of 16 bytes
  TcParams p;
  int tn = 0, ksplit = 1;
  if (!plan_gemm(ctx, T, K, N, &tn, &ksplit, &p)) return RAP_EUNSUPPORTED;
  CUtensorMap mw, mx;
  if (!make_map(ctx, &mw, w, (uint64_t)N, (uint64_t)K, TC_BM)) return RAP_EUNSUPPORTED;
  if (!make_map(ctx, &mx, x, (uint64_t)T, (uint64_t)K, (uint32_t)tn)) return RAP_EUNSUPPORTED;
  dim3 grid(p.n_work < ctx->sm_count ? p.n_work : ctx->sm_count, 1, 1);
  *ksplit_out = ksplit;
  p.wait_x = pdl == 2 ? 1 : 0;
  switch (tn) {
    case 32: return launch_tc<32>(ctx, mw, mx, p, grid, st, pdl);
    case 64: return launch_tc<64>(ctx, mw, mx, p, grid, st, pdl);
    case 128: return launch_tc<128>(ctx, mw, mx, p, grid, st, pdl);
    default: return launch_tc<256>(ctx, mw, mx, p, grid, st, pdl);
  }
}

rap_status rap_launch_proj_tc(rap_ctx* ctx, const rap_proj_args& a, int* ksplit_out, cudaStream_t st) {
  if (a.dtype != RAP_BF16) return RAP_EUNSUPPORTED;
  const int n_out = (a.Hq + a.Hkv) * a.P2 + a.Hkv * a.dv;
  return rap_launch_gemm_tc(ctx, a.x, a.w, a.T, a.hidden, n_out, ksplit_out, st, a.pdl);
}

// Decode-sized rap_qkv_rope_append in ONE launch: the tcgen05 GEMM with the RoPE / append epilogue fused in.
// RAP_EUNSUPPORTED when the call is not decode-sized (T > 32) or not bf16; the caller then takes the two-stage path.
// a.pdl != 0 launches the kernel with programmatic stream serialization (its weight streaming may overlap the tail
// of the previous kernel in the stream; it waits for that kernel before it writes q~ or the cache rows).
rap_status rap_launch_proj_fused(rap_ctx* ctx, const rap_proj_args& a, cudaStream_t st) {
  if (a.dtype != RAP_BF16 || a.T < 1 || a.T > 32 || (a.hidden % 8) != 0 || (a.P2 & 1)) return RAP_EUNSUPPORTED;
  const int n_out = (a.Hq + a.Hkv) * a.P2 + a.Hkv * a.dv;
  TcParams p;
  int tn = 0, ksplit = 1;
  if (!plan_gemm(ctx, a.T, a.hidden, n_out, &tn, &ksplit, &p) || tn != 32 || p.tok_tiles != 1) return RAP_EUNSUPPORTED;
  if (4 * p.row_tiles > ctx->proj_cnt_n) return RAP_EUNSUPPORTED;
  if ((long long)a.B_cache * a.Hkv * a.S_cap >= (1LL << 31)) return RAP_EUNSUPPORTED;   // cache row indices are 32-bit in the epilogue
  CUtensorMap mw, mx;
  if (!make_map(ctx, &mw, a.w, (uint64_t)n_out, (uint64_t)a.hidden, TC_BM)) return RAP_EUNSUPPORTED;
  if (!make_map(ctx, &mx, a.x, (uint64_t)a.T, (uint64_t)a.hidden, 32u)) return RAP_EUNSUPPORTED;
  TcFused f;
  f.bias = (const __nv_bfloat16*)a.bias; f.seq_id = a.seq_id; f.pos = a.pos; f.slot = a.slot; f.inv_freq = a.inv_freq;
  f.q_out = (__nv_bfloat16*)a.q_out; f.k_cache = (__nv_bfloat16*)a.k_cache; f.v_cache = (__nv_bfloat16*)a.v_cache;
  const int set = (int)(ctx->proj_epoch++ & 1u);       // two counter sets take turns; each launch clears the other one
  f.cnt = ctx->d_proj_cnt + set * ctx->proj_cnt_n;
  f.cnt_other = ctx->d_proj_cnt + (set ^ 1) * ctx->proj_cnt_n;
  f.n_cnt = ctx->proj_cnt_n;
  f.ksplit = ksplit; f.Hq = a.Hq; f.Hkv = a.Hkv; f.P2 = a.P2; f.dv = a.dv; f.half_dim = a.half_dim;
  f.B_cache = a.B_cache; f.S_cap = a.S_cap;
  RAP_CUDA_TRY(ctx, rap_raise_smem(ctx, proj_tc_kernel<32, true>, TcCfg<32>::SMEM_FUSED));
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(p.n_work < ctx->sm_count ? p.n_work : ctx->sm_count, 1, 1);
  cfg.blockDim = dim3(TC_THREADS, 1, 1);
  cfg.dynamicSmemBytes = TcCfg<32>::SMEM_FUSED;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = a.pdl ? 1 : 0;
  RAP_CUDA_TRY(ctx, cudaLaunchKernelEx(&cfg, proj_tc_kernel<32, true>, mw, mx, p, f));
  ctx->launches++;
  return RAP_OK;
}
