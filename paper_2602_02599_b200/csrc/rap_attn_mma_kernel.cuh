// Split-KV decode scan with the two small contractions of Eq. 2 on warp-level tensor-core instructions
// (mma.sync m16n8k16, bf16 in, fp32 accumulate), for rap_decode_attn on the retained dims (Eq. 7, scale
// 1/sqrt(D)).
//
// The scan stays bound by HBM: every cache byte is read once.  What the tensor-core form buys is issue
// slots and energy -- a handful of warp instructions per cache position instead of a few dozen on the
// FP32 pipes -- so that the SMs idle behind the copy engine instead of sharing the power budget with it,
// and the time no longer depends on the group size G (the G query heads of a KV head sit on the M axis of
// both contractions, padded to 16).
//
// Every warp is its own pipeline; there is no CTA-wide barrier inside the scan.
//   * A CTA takes tiles of 32 * NW positions of one (sequence, KV head) unit (the same balanced plan as the
//     FP32 scan); warp w owns the 32-row block [32 w, 32 w + 32) of each tile, with a private ring of
//     NSTG stages that its lane 0 fills with bulk async copies (K block and V block are contiguous byte
//     ranges of the dense-packed cache; completion is counted in bytes on the stage's mbarrier).
//   * S^T = q K^T:  A = q (heads x dims, from registers, loaded once per unit), B = K read straight from the
//     block with 32-bit shared loads (thread (g, t) of the fragment layout wants K[row(g)][dims 2t, 2t+1],
//     which is one stored word), 16 dims per step; the last step is shifted back into the row and its
//     overlap meets zeroed q.  The 8 columns of an n-tile are 8 rows spread over the block so that the
//     loads hit distinct banks for the row strides of the pruned shapes.
//   * softmax in the accumulator layout: thread (g, t) holds head g's logits of 8 rows.  The reference
//     maximum is lazy (raised only when a logit exceeds it by more than 8), the row sum stays per thread.
//   * O += P V:  A = P (the logit accumulators, already in the A layout), B = V: a fragment register holds
//     the same channel of two rows, so two 32-bit loads (two rows, channels c, c+1) and two byte permutes
//     give the B registers of an even-channel and an odd-channel n-tile.  Odd d_v' (rows only 2-byte
//     aligned): the odd rows of a block take the neighbouring aligned words instead.
//   * Rows of exactly 128 or 256 bytes (P = 32, 64 with d_v' = 64, 128: the unpruned cache and rho = 0.5) would
//     put every row on the same banks.  For them the blocks come in through tensor maps instead
//     (cp.async.bulk.tensor.2d, boxes of 32 rows x 128 bytes, 128-byte swizzle, no multicast): the 16-byte
//     chunk c of row r lands at chunk c ^ (r % 8), which spreads the fragment loads over all banks at no
//     extra instruction (the swizzled offsets are per-thread constants).
//   * At the end of a unit the warps merge (maximum, scaled sums) through shared memory and the CTA writes
//     one partial; the CTA that delivers a unit's last partial merges the unit (as in the FP32 scan).
// P enters the second contraction as two bf16 operands, the rounded value and the rounding remainder (two
// MMAs per tile on the same V fragments), so the weights carry about 17 bits; the row sum uses the fp32 values.
// Every mbarrier wait is bounded: on timeout the CTA records RAP_ETIMEOUT and leaves.
#pragma once
#include <cuda.h>

#include "rap_attn_common.cuh"

namespace {

#ifndef RAP_MMA_NW
#define RAP_MMA_NW 4
#endif
#ifndef RAP_MMA_NSTG
#define RAP_MMA_NSTG 2
#endif
#ifndef RAP_MMA_PSPLIT
#define RAP_MMA_PSPLIT 1     // 1: P = bf16 head + bf16 remainder (two MMAs per tile); 0: bf16 head only
#endif

constexpr float MMA_LAZY_SLACK = 8.f;
constexpr int MMA_BR = 32;                      // rows per warp block

template <int G, int WK, int DV>
struct MmaCfg {
  static_assert(G >= 1 && G <= 8, "the query heads of a KV head sit on 8 fragment rows");
  static_assert(WK >= 8 && DV >= 16, "one full k-step / channel block");
  static constexpr int NKS = (WK + 7) / 8;                    // k-steps of 16 dims (8 words)
  static constexpr int NCB = (DV + 15) / 16;                  // blocks of 16 channels
  static constexpr bool VODD = (DV & 1) != 0;
  static constexpr int CB_LAST = VODD ? DV - 15 : DV - 16;    // first channel of the last block (even)
  static constexpr int CW = CB_LAST + 16;                     // channel slots (odd d_v': one phantom channel)
  // row step between the 8 columns of an n-tile: K-word stride * step = 4 * odd puts them on distinct banks
  static constexpr int RS_K = (WK % 2) ? 4 : (WK % 4) ? 2 : 1;
  static constexpr int RS = (VODD && RS_K == 1) ? 2 : RS_K;   // odd d_v' wants row pairs of one parity
  // tensor-map staging with the 128-byte swizzle: panels of 32 rows x 128 bytes
  static constexpr bool TMA = (WK % 32) == 0 && (DV % 64) == 0;
  static constexpr int NKP = WK / 32, NVP = DV / 64;          // panels per K / V block (TMA only)
  static constexpr int K_BYTES = MMA_BR * WK * 4, V_BYTES = MMA_BR * DV * 2;
  static constexpr int STAGE_BYTES = TMA ? K_BYTES + V_BYTES : cround(K_BYTES + V_BYTES + 16, 128);
  static constexpr int STAGE_ALIGN = TMA ? 1024 : 128;
  static constexpr int NSTG = RAP_MMA_NSTG;
  static constexpr int RED_BYTES_1 = G * CW * 4;              // per warp
  static constexpr int MERGE_BYTES = (G * RAP_MAX_SPLIT + 8) * 4;
  static constexpr int OFF_RED = 512;
  static constexpr int fits(int nw) {
    const int red = nw * RED_BYTES_1 > MERGE_BYTES ? nw * RED_BYTES_1 : MERGE_BYTES;
    return cround(OFF_RED + red, STAGE_ALIGN) + nw * NSTG * STAGE_BYTES + (TMA ? 1024 : 0);
  }
  static constexpr int NW = fits(RAP_MMA_NW) <= SMEM_BUDGET ? RAP_MMA_NW
                            : fits(3) <= SMEM_BUDGET        ? 3
                            : fits(2) <= SMEM_BUDGET        ? 2
                                                            : 1;
  static constexpr int RED_BYTES = NW * RED_BYTES_1 > MERGE_BYTES ? NW * RED_BYTES_1 : MERGE_BYTES;
  static constexpr int OFF_STAGE = cround(OFF_RED + RED_BYTES, STAGE_ALIGN);
  static constexpr int SMEM = OFF_STAGE + NW * NSTG * STAGE_BYTES + (TMA ? 1024 : 0);   // slack to align the base
  static constexpr int THREADS = NW * 32;
  static constexpr int ST = NW * MMA_BR;                      // positions per CTA tile
  static_assert(SMEM <= SMEM_BUDGET, "ring does not fit");
  static_assert(NW * NSTG * 8 + NW * 64 <= OFF_RED - 16, "barriers and merge scalars sit below the reduction buffer");
  // row of column n of n-tile t inside the warp's block
  static __device__ __forceinline__ constexpr int row(int t, int n) { return RS * n + (t % RS) + 8 * RS * (t / RS); }
};

__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1) {
  // rows 8..15 of A (registers a1, a3) are the padding of the head axis: zero
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %5}, {%7, %8}, {%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(0u), "r"(a2), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float mma_ex2(float x) {      // 2^x, one instruction; 2^(-inf) = 0
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t mma_pack_bf16(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
// one box of a 2-D tensor map (x = element column, y = row) into this CTA's shared memory; no multicast
__device__ __forceinline__ void mma_tma_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
      "l"(map), "r"(x), "r"(y), "r"(bar)
      : "memory");
}
__device__ __forceinline__ uint32_t mma_prmt(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t r;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
  return r;
}

// DYN: the instantiation that can hand the last tiles of a launch out at run time (long launches; rap_scan_params)
template <int G, int WK, int DV, bool DYN>
__global__ void __launch_bounds__(MmaCfg<G, WK, DV>::THREADS, 2) attn_mma_kernel(const ScanParams p,
                                                                                 const __grid_constant__ CUtensorMap map_k,
                                                                                 const __grid_constant__ CUtensorMap map_v) {
  using C = MmaCfg<G, WK, DV>;
  constexpr int ST = C::ST, NW = C::NW, NSTG = C::NSTG, NKS = C::NKS, NCB = C::NCB, CW = C::CW;
  constexpr int THREADS = C::THREADS;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  // swizzled panels want a 1024-byte aligned base
  unsigned char* smem = C::TMA ? smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u) : smem_raw;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem);                        // [NW][NSTG]
  float* m_s = reinterpret_cast<float*>(smem + NW * NSTG * 8);               // [NW][8] reference maxima of the warps
  float* l_s = m_s + NW * 8;                                                 // [NW][8] scaled row sums
  float* red = reinterpret_cast<float*>(smem + C::OFF_RED);                  // [NW][G][CW]; later the merge weights
  int* s_flag = reinterpret_cast<int*>(smem + C::OFF_RED - 16);              // time-out seen by any warp
  int* s_last = s_flag + 1;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int gid = lane >> 2, tq = lane & 3;
  int b = 0, h = 0, len = 0, t_begin = 0, n_my = 0;
  float* ws_base = nullptr;
  size_t ws_head = 0;
  SkPlan plan;
  plan.T = 0; plan.nc = 0;
  int cur = 0, hi = 0, unit_start = 0;
  // Pieces claimed at run time (see rap_scan_params): the tiles [T_s, T) in n_dyn pieces of DC tiles; a piece's index
  // in tile order is the CTA's number for the part assigned up front, nc + j for run-time piece j
  int T_s = 0, n_dyn = 0, my_piece = (int)blockIdx.x;
  const int DC = p.dyn_piece;
  SkPlan splan;
  splan.T = 0; splan.nc = 0;
  bool shared_plan = false;
  int* const pref = reinterpret_cast<int*>(red);
  auto piece_of = [&](int tile) {
    if constexpr (DYN) return tile < T_s ? sk_cta_of(tile, splan) : splan.nc + (tile - T_s) / DC;
    else return sk_cta_of(tile, plan);
  };
  auto locate = [&](int tile) {      // the unit that holds this tile: b, h, unit_start
    int pb = 0;
    if (shared_plan) {
      b = sk_seq_of(pref, p.B, tile);
      pb = b > 0 ? pref[b - 1] : 0;
    } else {
      for (b = 0; b < p.B; ++b) {
        const int nb = sk_tiles_of(p.seq_len, b, p.len_add, p.S_cap, ST) * p.Hkv;
        if (tile < pb + nb) break;
        pb += nb;
      }
    }
    const int ntb = sk_tiles_of(p.seq_len, b, p.len_add, p.S_cap, ST);
    h = (tile - pb) / ntb;
    unit_start = pb + h * ntb;
  };
  if (p.balanced) {
    // the plan (reads the lengths only): computed by the first warp into the reduction buffer, which is free until
    // the first merge; batches too large for that buffer are planned by every thread on its own
    shared_plan = sk_plan_shared(p.seq_len, p.B, p.Hkv, p.len_add, p.S_cap, ST, (int)gridDim.x, pref, C::RED_BYTES / 4, &plan);
    if (!shared_plan) plan = sk_plan(p.seq_len, p.B, p.Hkv, p.len_add, p.S_cap, ST, (int)gridDim.x);
    T_s = plan.T;
    if (DYN && shared_plan && DC > 0 && plan.T > 0) {
      const int n_max = pref[C::RED_BYTES / 4 - 1];     // tiles of the longest sequence
      const int nd = (int)((long long)plan.T * p.dyn_frac_x256 / 256 / DC);
      const int ts = plan.T - nd * DC;
      // no unit may get more than RAP_MAX_SPLIT partials: pieces of either kind that can touch it, ragged ends included
      const int ncs = min(plan.nc, ts);                  // CTAs with a part assigned up front
      // ... and a piece must be small against a CTA's own part (the launcher judged by the longest sequence; a batch of
      // mostly short ones has far fewer tiles), unless the test hook chose the sizes
      const bool small_pieces = !p.dyn_guard || (long long)DC * plan.nc * 6 <= (long long)plan.T;
      if (nd > 0 && small_pieces && (ts == 0 ? 0LL : (long long)n_max * ncs / ts) + n_max / DC + 4 <= RAP_MAX_SPLIT) {
        n_dyn = nd;
        T_s = ts;
      }
    }
    splan.T = T_s;
    splan.nc = min(plan.nc, T_s);
    // Everything below reads q~ and the cache rows the previous kernel in the stream wrote, and writes what the next
    // one may depend on: wait for the predecessor first, and only then let the successor start (it may begin to
    // stream its weights while this scan runs, and waits for this kernel before it writes anything this one reads).
    pdl_wait();
    pdl_launch_dependents();
    if (blockIdx.x == 0) {   // sequences without any row are scanned by nobody: their output is zero
      for (int i = tid; i < p.B * p.Hkv; i += THREADS) p.unit_cnt_other[i] = 0;   // counters a launch that gave up left behind
      if (tid == 0) *p.dyn_next_other = 0;                                        // and the piece counter of the previous launch
      for (int bb = 0; bb < p.B; ++bb) {
        const bool empty = shared_plan ? pref[bb] == (bb > 0 ? pref[bb - 1] : 0)
                                       : sk_tiles_of(p.seq_len, bb, p.len_add, p.S_cap, ST) == 0;
        if (empty)
          for (int i = tid; i < p.Hq * DV; i += THREADS) p.out[(size_t)bb * p.Hq * DV + i] = 0.f;
      }
    }
    if ((int)blockIdx.x >= plan.nc) return;
    if constexpr (DYN) {
      if ((int)blockIdx.x < splan.nc) {
        cur = (int)((long long)blockIdx.x * T_s / splan.nc);
        hi = (int)((long long)(blockIdx.x + 1) * T_s / splan.nc);
      }
      if (cur < hi) {
        locate(cur);
      } else if (n_dyn == 0) {
        return;
      }
    } else {
      cur = (int)((long long)blockIdx.x * plan.T / plan.nc);
      hi = (int)((long long)(blockIdx.x + 1) * plan.T / plan.nc);
      if (cur >= hi) return;
      locate(cur);
    }
  } else {
    pdl_wait();
    pdl_launch_dependents();
    b = blockIdx.z;
    h = blockIdx.y;
  }
  const uint32_t bar0 = smem_u32(bars) + warp * NSTG * 8;                     // this warp's barriers
  unsigned char* wstage = smem + C::OFF_STAGE + warp * NSTG * C::STAGE_BYTES;   // this warp's ring
  const uint32_t wstage_u = smem_u32(wstage);
  if (tid == 0) {
    *s_flag = 0;
    for (int i = 0; i < NW * NSTG; ++i) mbar_init(smem_u32(bars) + 8 * i, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  // fragment addressing inside a block (words): K rows of this thread's n-tile columns
  int koff[4];
#pragma unroll
  for (int t = 0; t < 4; ++t) koff[t] = C::row(t, gid) * WK + tq;
  // swizzled panels (rows gid + 8 t, chunk c of the row at chunk c ^ gid): word offsets by chunk, the panel and
  // the n-tile are immediates
  int kx[8];
#pragma unroll
  for (int c = 0; c < 8; ++c) kx[c] = gid * 32 + ((c ^ gid) << 2) + tq;
  // V, swizzled: rows 2 tq + e + 8 t, word 8 (cb % 4) + gid of the panel row
  int vx[4][2];
#pragma unroll
  for (int cm = 0; cm < 4; ++cm)
#pragma unroll
    for (int e = 0; e < 2; ++e) vx[cm][e] = (2 * tq + e) * 32 + (((2 * cm + (gid >> 2)) ^ (2 * tq + e)) << 2) + (gid & 3);
  // V words of this thread's rows: row(t, 2 tq) of n-tile t, channel word gid (floor for odd rows of an odd d_v')
  int vofs[4];
#pragma unroll
  for (int t = 0; t < 4; ++t) vofs[t] = ((C::row(t, 2 * tq) * DV) >> 1) + gid;
  constexpr int VPAIR = C::RS * DV / 2;            // words from row(t, 2 tq) to row(t, 2 tq + 1) (RS * DV is even)
  bool dbg_done = false;       // the test hook of issue_block fires once, on the first block issued
  int st = 0;                  // ring position and phase of this warp, running on across units
  uint32_t parity = 0;
  bool timed_out = false;
  const float cs = p.qscale;   // log2(e) / sqrt(D)

  // claims the next of the pieces that are handed out at run time; false when none is left (every thread calls it)
  auto claim = [&]() -> bool {
    __syncthreads();                   // the merge scalars and the reduction buffer are free
    if (tid == 0) {
      const int got = atomicAdd(p.dyn_next, 1);
      *s_last = got;
      // Every CTA that takes part claims until it is refused once: n_dyn + nc claims per launch.  Whoever makes the
      // last one leaves the counter at zero for the next launch that uses it (a replayed CUDA graph may run two
      // launches in a row on the same counter, so clearing "the other one" at the start of a launch is not enough).
      if (got == n_dyn + plan.nc - 1) *p.dyn_next = 0;
    }
    __syncthreads();
    const int j = *s_last;
    if (j >= n_dyn) return false;
    my_piece = splan.nc + j;
    cur = T_s + j * DC;
    hi = cur + DC;
    SkPlan again;                      // the prefix of the plan once more: the reduction buffer held sums in between
    sk_plan_shared(p.seq_len, p.B, p.Hkv, p.len_add, p.S_cap, ST, (int)gridDim.x, pref, C::RED_BYTES / 4, &again);
    locate(cur);
    __syncthreads();                   // every thread has read the prefix before the buffer is reused
    return true;
  };
  if constexpr (DYN) {
    if (p.balanced && cur >= hi && !claim()) return;    // a CTA without a part assigned up front starts with a piece
  }

  for (;;) {   // one pass per segment (a single one unless the mode is balanced)
    int seg_tiles;
    {
      len = min(max(p.seq_len[b] + p.len_add, 0), p.S_cap);
      seg_tiles = (len + ST - 1) / ST;
      if (p.balanced) {
        t_begin = cur - unit_start;
        n_my = min(seg_tiles - t_begin, hi - cur);
        const int seg = my_piece - piece_of(unit_start);
        ws_head = (size_t)RAP_MAX_SPLIT * (DV + 2);
        ws_base = p.ws + (((size_t)b * p.Hq + (size_t)h * G) * RAP_MAX_SPLIT + seg) * (size_t)(DV + 2);
      } else {
        const int split = blockIdx.x;
        const int tps = (seg_tiles + p.n_split - 1) / p.n_split;
        t_begin = min(seg_tiles, split * tps);
        n_my = min(seg_tiles, t_begin + tps) - t_begin;
        ws_head = (size_t)p.n_split * (DV + 2);
        ws_base = p.ws + (((size_t)b * p.Hq + (size_t)h * G) * p.n_split + split) * (size_t)(DV + 2);
        if (n_my <= 0) {   // nothing to scan: neutral partials
          for (int i = tid; i < G * (DV + 2); i += THREADS) {
            const int g = i / (DV + 2), c = i - g * (DV + 2);
            ws_base[g * ws_head + c] = (c == DV) ? -INFINITY : 0.f;
          }
          return;
        }
      }
    }
    const size_t unit = (size_t)b * p.Hkv + h;
    const unsigned char* kg = p.k + unit * (size_t)p.S_cap * (size_t)(WK * 4);
    const unsigned char* vg = p.v + unit * (size_t)p.S_cap * (size_t)(DV * 2);
    const int len8 = (len + 7) & ~7;                  // rows a copy may touch: S_cap is a multiple of 8
    // this warp's blocks: rows [(t_begin + i) ST + 32 warp, + 32) for i < n_blk, those that hold a valid row
    const int row_w = t_begin * ST + MMA_BR * warp;
    const int n_blk = len > row_w ? min(n_my, (len - row_w + ST - 1) / ST) : 0;

    auto issue_block = [&](int i, int stg) {          // all lanes converged; lane 0 issues
      const int j0 = row_w + i * ST;
      const int rows = min(MMA_BR, len8 - j0);
      const uint32_t bar = bar0 + 8 * stg, dst = wstage_u + stg * C::STAGE_BYTES;
      const uint32_t kb = (uint32_t)rows * WK * 4, vb = (uint32_t)rows * DV * 2;
      if (lane == 0 && RAP_BOUNDS(j0 + rows - 1, p.S_cap, p.status, 0x102) && RAP_BOUNDS(stg, NSTG, p.status, 0x103) &&
          RAP_BOUNDS(rows - 1, MMA_BR, p.status, 0x104)) {
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // earlier generic writes (zero fill) come first
        if constexpr (C::TMA) {
          // whole boxes: rows past the end of the tensor are zero-filled, rows of a neighbouring unit are masked
          const int y = (int)unit * p.S_cap + j0;
          mbar_expect_tx(bar, C::STAGE_BYTES);
#pragma unroll
          for (int pn = 0; pn < C::NKP; ++pn) mma_tma_2d(dst + pn * 4096, &map_k, 64 * pn, y, bar);
#pragma unroll
          for (int pn = 0; pn < C::NVP; ++pn) mma_tma_2d(dst + C::K_BYTES + pn * 4096, &map_v, 64 * pn, y, bar);
        } else if (p.dbg_skip_copy && blockIdx.x == 0 && warp == 0 && !dbg_done) {
          // test hook: the stage is armed and nothing is copied into it, so the wait below runs out (nothing is in
          // flight for this stage when the CTA leaves)
          mbar_expect_tx(bar, kb + vb);
        } else {
          mbar_expect_tx(bar, kb + vb);
          bulk_g2s(dst, kg + (size_t)j0 * (WK * 4), kb, bar);
          bulk_g2s(dst + C::K_BYTES, vg + (size_t)j0 * (DV * 2), vb, bar);
        }
      }
      dbg_done = true;
    };
    {
      const int pre = min(n_blk, NSTG - 1);
      for (int i = 0; i < pre; ++i) issue_block(i, (st + i) % NSTG);
    }

    // ---- q as the A operand: head gid, words (8 ks + tq) and (8 ks + 4 + tq); zero for the padding heads ----
    uint32_t qa[NKS][2];
    {
      const uint32_t* qrow = p.q + ((size_t)b * p.Hq + (size_t)h * G + (gid < G ? gid : 0)) * WK;
#pragma unroll
      for (int ks = 0; ks < NKS; ++ks) {
        const int wb = ks < NKS - 1 ? 8 * ks : WK - 8;        // last step shifted back into the row
#pragma unroll
        for (int hlf = 0; hlf < 2; ++hlf) {
          const int w = wb + 4 * hlf + tq;
          const bool fresh = w >= 8 * ks;                      // not covered by an earlier step
          qa[ks][hlf] = (gid < G && fresh && RAP_BOUNDS(w, WK, p.status, 0x101)) ? qrow[w] : 0u;
        }
      }
    }
    float o[NCB][2][4];
#pragma unroll
    for (int cb = 0; cb < NCB; ++cb)
#pragma unroll
      for (int e = 0; e < 2; ++e)
#pragma unroll
        for (int r = 0; r < 4; ++r) o[cb][e][r] = 0.f;
    float m_ref = -INFINITY, l_thr = 0.f;

    for (int i = 0; i < n_blk; ++i) {
      if (i + NSTG - 1 < n_blk) issue_block(i + NSTG - 1, (st + NSTG - 1) % NSTG);
      if (!__all_sync(0xffffffffu, mbar_wait_bounded(bar0 + 8 * st, parity, p.wait_limit))) {   // warp-uniform verdict
        timed_out = true;
        break;
      }
      const unsigned char* stage = wstage + st * C::STAGE_BYTES;
      const uint32_t* kw = reinterpret_cast<const uint32_t*>(stage);
      const uint32_t* vw = reinterpret_cast<const uint32_t*>(stage + C::K_BYTES);
      const int nrows = len - (row_w + i * ST);      // valid rows of this block (>= 1)
      if (nrows < MMA_BR) {
        // last block of the sequence: rows >= nrows were not written by this sequence; zero their V so that
        // the second contraction meets 0 * 0 there
        if constexpr (C::TMA) {   // a row is 128 contiguous bytes of each panel, whatever the swizzle
          uint32_t* vz = reinterpret_cast<uint32_t*>(wstage + st * C::STAGE_BYTES + C::K_BYTES);
          for (int pn = 0; pn < C::NVP; ++pn)
            for (int x = nrows * 32 + lane; x < MMA_BR * 32; x += 32) vz[pn * 1024 + x] = 0u;
        } else {
          uint16_t* vz = reinterpret_cast<uint16_t*>(wstage + st * C::STAGE_BYTES + C::K_BYTES);
          for (int x = nrows * DV + lane; x < MMA_BR * DV; x += 32) vz[x] = 0;
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // before a later bulk copy into this stage
        __syncwarp();
      }

      // ---- S^T = q K^T: four n-tiles (8 rows each), NKS steps of 16 dims ----
      float s[4][4];
#pragma unroll
      for (int t = 0; t < 4; ++t) s[t][0] = s[t][1] = s[t][2] = s[t][3] = 0.f;
#pragma unroll
      for (int ks = 0; ks < NKS; ++ks) {
        const int wb = ks < NKS - 1 ? 8 * ks : WK - 8;
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          uint32_t b0, b1;
          if constexpr (C::TMA) {
            const int i0 = kx[(2 * ks) % 8] + (ks / 4) * 1024 + 256 * t, i1 = kx[(2 * ks + 1) % 8] + (ks / 4) * 1024 + 256 * t;
            b0 = RAP_BOUNDS(i0, C::K_BYTES / 4, p.status, 0x105) ? kw[i0] : 0u;
            b1 = RAP_BOUNDS(i1, C::K_BYTES / 4, p.status, 0x105) ? kw[i1] : 0u;
          } else {
            b0 = RAP_BOUNDS(koff[t] + wb, C::K_BYTES / 4, p.status, 0x106) ? kw[koff[t] + wb] : 0u;
            b1 = RAP_BOUNDS(koff[t] + wb + 4, C::K_BYTES / 4, p.status, 0x106) ? kw[koff[t] + wb + 4] : 0u;
          }
          mma_bf16(s[t], qa[ks][0], qa[ks][1], b0, b1);
        }
      }

      // ---- softmax on the accumulators: x = s log2(e)/sqrt(D) - m_ref for head gid, rows row(t, 2 tq + e) ----
      float x[4][2];
      bool raise = false;
#pragma unroll
      for (int t = 0; t < 4; ++t)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          x[t][e] = fmaf(s[t][e], cs, -m_ref);
          if (nrows < MMA_BR && C::row(t, 2 * tq + e) >= nrows) x[t][e] = -INFINITY;
          raise |= x[t][e] > MMA_LAZY_SLACK;
        }
      if (__any_sync(0xffffffffu, raise)) {
        float mx = -INFINITY;
#pragma unroll
        for (int t = 0; t < 4; ++t)
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const bool masked = nrows < MMA_BR && C::row(t, 2 * tq + e) >= nrows;
            x[t][e] = masked ? -INFINITY : s[t][e] * cs;
            mx = fmaxf(mx, x[t][e]);
          }
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        const float m_new = fmaxf(m_ref, mx);                  // finite: every block holds a valid row
        const float alpha = mma_ex2(m_ref - m_new);            // first block: 2^(-inf) = 0
        m_ref = m_new;
        l_thr *= alpha;
#pragma unroll
        for (int cb = 0; cb < NCB; ++cb)
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            o[cb][e][0] *= alpha;
            o[cb][e][1] *= alpha;
          }
#pragma unroll
        for (int t = 0; t < 4; ++t)
#pragma unroll
          for (int e = 0; e < 2; ++e) x[t][e] -= m_ref;
      }
      uint32_t pa[4], pl[4];
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        const float p0 = mma_ex2(x[t][0]), p1 = mma_ex2(x[t][1]);
        l_thr += p0 + p1;
        pa[t] = mma_pack_bf16(p0, p1);
        // what the rounding to bf16 dropped, as a second bf16 operand: P = head + remainder to about 2^-17
        pl[t] = RAP_MMA_PSPLIT ? mma_pack_bf16(p0 - __uint_as_float(pa[t] << 16), p1 - __uint_as_float(pa[t] & 0xffff0000u))
                               : 0u;
      }

      // ---- O += P V: two k-blocks of 16 rows (n-tiles 2 kb and 2 kb + 1), NCB blocks of 16 channels ----
      // (bounds-checking build: the fragment offsets do not depend on the data, so their largest value is checked
      // once per block against the words this stage holds behind the K block)
      bool v_ok = true;
      {
        constexpr int V_WORDS = (C::STAGE_BYTES - C::K_BYTES) / 4;
        const int cw_last = C::CB_LAST / 2;
        const int far = C::TMA ? vx[3][1] + ((NCB - 1) / 4) * 1024 + 256 * 3
                               : max(vofs[1], vofs[3]) + cw_last + VPAIR + (C::VODD ? 1 : 0);
        v_ok = RAP_BOUNDS(far, V_WORDS, p.status, 0x107);
      }
#pragma unroll
      for (int kb = 0; kb < 2 && v_ok; ++kb) {
        const uint32_t* v0 = vw + vofs[2 * kb];
        const uint32_t* v1 = vw + vofs[2 * kb + 1];
#pragma unroll
        for (int cb = 0; cb < NCB; ++cb) {
          const int cw = (cb < NCB - 1 ? 16 * cb : C::CB_LAST) / 2;
          uint32_t xa0, xb0;
          if constexpr (C::TMA) {
            xa0 = vw[vx[cb % 4][0] + (cb / 4) * 1024 + 256 * (2 * kb)];
            xb0 = vw[vx[cb % 4][1] + (cb / 4) * 1024 + 256 * (2 * kb)];
          } else {
            xa0 = v0[cw];
            xb0 = v0[cw + VPAIR];
          }
          const uint32_t be0 = mma_prmt(xa0, xb0, 0x5410u), bo0 = mma_prmt(xa0, xb0, 0x7632u);
          uint32_t be1, bo1;
          if constexpr (C::TMA) {
            const uint32_t xa1 = vw[vx[cb % 4][0] + (cb / 4) * 1024 + 256 * (2 * kb + 1)];
            const uint32_t xb1 = vw[vx[cb % 4][1] + (cb / 4) * 1024 + 256 * (2 * kb + 1)];
            be1 = mma_prmt(xa1, xb1, 0x5410u);
            bo1 = mma_prmt(xa1, xb1, 0x7632u);
          } else if constexpr (!C::VODD) {
            const uint32_t xa1 = v1[cw], xb1 = v1[cw + VPAIR];
            be1 = mma_prmt(xa1, xb1, 0x5410u);
            bo1 = mma_prmt(xa1, xb1, 0x7632u);
          } else {
            // odd rows of an odd d_v': the aligned word holds channels (c - 1, c), the next one (c + 1, c + 2)
            const uint32_t xa1 = v1[cw], xb1 = v1[cw + VPAIR], ya1 = v1[cw + 1], yb1 = v1[cw + VPAIR + 1];
            be1 = mma_prmt(xa1, xb1, 0x7632u);
            bo1 = mma_prmt(ya1, yb1, 0x5410u);
          }
          mma_bf16(o[cb][0], pa[2 * kb], pa[2 * kb + 1], be0, be1);
          mma_bf16(o[cb][1], pa[2 * kb], pa[2 * kb + 1], bo0, bo1);
          if (RAP_MMA_PSPLIT) {
            mma_bf16(o[cb][0], pl[2 * kb], pl[2 * kb + 1], be0, be1);
            mma_bf16(o[cb][1], pl[2 * kb], pl[2 * kb + 1], bo0, bo1);
          }
        }
      }
      __syncwarp();            // every lane is done with this stage before lane 0 refills it
      if (++st == NSTG) { st = 0; parity ^= 1u; }
    }

    // ---- merge the warps: common maximum per head, scaled sums ----
    l_thr += __shfl_xor_sync(0xffffffffu, l_thr, 1);
    l_thr += __shfl_xor_sync(0xffffffffu, l_thr, 2);
    if (timed_out && lane == 0) *s_flag = 1;
    if (tq == 0) m_s[warp * 8 + gid] = m_ref;
    __syncthreads();
    if (*s_flag) {
      if (tid == 0) {
        atomicCAS(&p.status[0], 0, (int)RAP_ETIMEOUT);
        p.status[1] = (b * p.Hkv + h) * RAP_MAX_SPLIT + (int)(blockIdx.x % RAP_MAX_SPLIT);
      }
      // give copies still in flight a bounded chance to land before the shared memory is released
      if (lane == 0)
        for (int sg = 0; sg < NSTG; ++sg) {
          mbar_wait_bounded(bar0 + 8 * sg, 0, p.wait_limit);
          mbar_wait_bounded(bar0 + 8 * sg, 1, p.wait_limit);
        }
      __syncthreads();
      return;
    }
    float m_all = -INFINITY;
#pragma unroll
    for (int w = 0; w < NW; ++w) m_all = fmaxf(m_all, m_s[w * 8 + gid]);
    const float f = m_ref == -INFINITY ? 0.f : mma_ex2(m_ref - m_all);   // a warp without a block contributes nothing
    if (tq == 0) l_s[warp * 8 + gid] = l_thr * f;
    if (gid < G && RAP_BOUNDS(((size_t)warp * G + gid) * CW + CW - 1, C::RED_BYTES / 4, p.status, 0x108)) {
      float* rr = red + ((size_t)warp * G + gid) * CW;
#pragma unroll
      for (int cb = 0; cb < NCB; ++cb) {
        const int c0 = (cb < NCB - 1 ? 16 * cb : C::CB_LAST) + 4 * tq;   // this thread's four channels of the block
        rr[c0] = o[cb][0][0] * f;
        rr[c0 + 1] = o[cb][1][0] * f;
        rr[c0 + 2] = o[cb][0][1] * f;
        rr[c0 + 3] = o[cb][1][1] * f;
      }
    }
    __syncthreads();
    const bool ws_ok = RAP_BOUNDS((ws_base - p.ws) + (long long)(G - 1) * ws_head + DV + 1, p.ws_floats, p.status, 0x109);
    for (int i = tid; i < G * DV && ws_ok; i += THREADS) {
      const int g = i / DV, c = i - g * DV;
      float sum = 0.f;
#pragma unroll
      for (int w = 0; w < NW; ++w) sum += red[((size_t)w * G + g) * CW + c];
      ws_base[g * ws_head + c] = sum;
    }
    if (tid < G && ws_ok) {
      float l = 0.f, mm = -INFINITY;
#pragma unroll
      for (int w = 0; w < NW; ++w) {
        l += l_s[w * 8 + tid];
        mm = fmaxf(mm, m_s[w * 8 + tid]);
      }
      ws_base[tid * ws_head + DV] = mm;
      ws_base[tid * ws_head + DV + 1] = l;
    }
    if (p.balanced) {
      // ---- the CTA that delivers a unit's last partial merges them (no separate combine launch) ----
      __threadfence();           // this CTA's partials are visible before its arrival is counted
      __syncthreads();
      const int first = piece_of(unit_start);
      const int nseg = piece_of(unit_start + seg_tiles - 1) - first + 1;
      const int u = b * p.Hkv + h;
      if (tid == 0) *s_last = RAP_BOUNDS(u, p.B * p.Hkv, p.status, 0x10a) && atomicAdd(&p.unit_cnt[u], 1) == nseg - 1;
      __syncthreads();
      if (*s_last) {
        __threadfence();
        const float* ub = p.ws + ((size_t)b * p.Hq + (size_t)h * G) * RAP_MAX_SPLIT * (size_t)(DV + 2);
        const bool m_ok = RAP_BOUNDS((ub - p.ws) + (long long)(G - 1) * ws_head + (long long)(nseg - 1) * (DV + 2) + DV + 1,
                                     p.ws_floats, p.status, 0x10b) &&
                          RAP_BOUNDS(((size_t)b * p.Hq + (size_t)h * G + G - 1) * DV + DV - 1, (size_t)p.B * p.Hq * DV, p.status, 0x10c);
        if (!m_ok) {
          // (bounds-checking build only) the unit's merge would leave its buffers: skipped and reported
        } else if (nseg <= 4) {
          // few partials (the usual case): every output thread loads the maxima, the sums and its own channel of all
          // partials at once -- one round trip through the memory system instead of two -- and weighs them itself
          for (int i = tid; i < G * DV; i += THREADS) {
            const int g = i / DV, c = i - g * DV;
            const float* gb = ub + (size_t)g * ws_head;
            float mv[4], lv[4], av[4];
#pragma unroll
            for (int sg = 0; sg < 4; ++sg) {
              const bool on = sg < nseg;
              lv[sg] = on ? __ldcg(gb + (size_t)sg * (DV + 2) + DV + 1) : 0.f;
              mv[sg] = on ? __ldcg(gb + (size_t)sg * (DV + 2) + DV) : -INFINITY;
              av[sg] = on ? __ldcg(gb + (size_t)sg * (DV + 2) + c) : 0.f;
            }
            float M = -INFINITY;
#pragma unroll
            for (int sg = 0; sg < 4; ++sg)
              if (lv[sg] > 0.f) M = fmaxf(M, mv[sg]);
            float den = 0.f, num = 0.f;
#pragma unroll
            for (int sg = 0; sg < 4; ++sg) {
              const float wk = lv[sg] > 0.f ? exp2f(mv[sg] - M) : 0.f;
              den += wk * lv[sg];
              num += wk * av[sg];
            }
            p.out[((size_t)b * p.Hq + (size_t)h * G + g) * DV + c] = den > 0.f ? num / den : 0.f;
          }
        } else {
          float* wgt = red;        // [G][RAP_MAX_SPLIT] segment weights, then G reciprocals of the denominators
          for (int g = warp; g < G; g += NW) {
            const float* gb = ub + (size_t)g * ws_head;
            float mv[2], lv[2];
  #pragma unroll
            for (int k = 0; k < 2; ++k) {
              const int sg = lane + 32 * k;
              lv[k] = sg < nseg ? __ldcg(gb + (size_t)sg * (DV + 2) + DV + 1) : 0.f;
              mv[k] = (sg < nseg && lv[k] > 0.f) ? __ldcg(gb + (size_t)sg * (DV + 2) + DV) : -INFINITY;
            }
            float M = fmaxf(mv[0], mv[1]);
  #pragma unroll
            for (int o2 = 16; o2 > 0; o2 >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o2));
            float den = 0.f;
  #pragma unroll
            for (int k = 0; k < 2; ++k) {
              const float wk = lv[k] > 0.f ? exp2f(mv[k] - M) : 0.f;
              wgt[g * RAP_MAX_SPLIT + lane + 32 * k] = wk;
              den += wk * lv[k];
            }
  #pragma unroll
            for (int o2 = 16; o2 > 0; o2 >>= 1) den += __shfl_xor_sync(0xffffffffu, den, o2);
            if (lane == 0) wgt[G * RAP_MAX_SPLIT + g] = den > 0.f ? 1.f / den : 0.f;
          }
          __syncthreads();
          for (int i = tid; i < G * DV; i += THREADS) {
            const int g = i / DV, c = i - g * DV;
            const float* gb = ub + (size_t)g * ws_head + c;
            float num = 0.f;
            for (int sg = 0; sg < nseg; ++sg) num += wgt[g * RAP_MAX_SPLIT + sg] * __ldcg(gb + (size_t)sg * (DV + 2));
            p.out[((size_t)b * p.Hq + (size_t)h * G + g) * DV + c] = num * wgt[G * RAP_MAX_SPLIT + g];
          }
        }
        if (tid == 0) p.unit_cnt[u] = 0;   // ready for the next call on this context
      }
    }
    // ---- next segment: the following unit, from its first tile ----
    if (!p.balanced) break;
    cur += n_my;
    if constexpr (DYN) {
      bool more = cur < hi;
      if (more) {
        unit_start += seg_tiles;
        if (++h == p.Hkv) {
          h = 0;
          do { ++b; } while (b < p.B && sk_tiles_of(p.seq_len, b, p.len_add, p.S_cap, ST) == 0);
          if (b >= p.B) more = false;
        }
      }
      if (!more) {
        // this piece is done: claim the next of the pieces that are handed out at run time, if there is one left
        if (n_dyn == 0 || !claim()) break;
      }
    } else {
      if (cur >= hi) break;
      unit_start += seg_tiles;
      if (++h == p.Hkv) {
        h = 0;
        do { ++b; } while (b < p.B && sk_tiles_of(p.seq_len, b, p.len_add, p.S_cap, ST) == 0);
        if (b >= p.B) break;
      }
    }
    __syncthreads();   // the reduction buffer and the merge scalars are reused by the next segment
  }   // segment loop
}

}  // namespace
