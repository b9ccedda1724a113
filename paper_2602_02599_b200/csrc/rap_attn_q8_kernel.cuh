// Split-KV decode scan over an 8-bit quantised cache (rap_decode_attn_q8): the tensor-core scan of
// rap_attn_mma_kernel.cuh with the cache rows stored as int8 codes plus one bf16 scale per row (codes, padding, scale
// in the last two bytes of a row of rap_q8_row_bytes(W) bytes).  Same work plan, per-warp copy pipelines, lazy online
// softmax and fused merge; what changes is how the operands reach the MMAs (mma.sync m16n8k16, fp16 in, fp32
// accumulate):
//   * a code c is stored as the byte u = c + 128 in [1, 255], and the bit pattern 0x6400 | u is the fp16 number
//     1024 + u = 1152 + c (fp16 has a step of one between 1024 and 2048): one byte permute turns two stored codes
//     into one operand register, a 32-bit word of four codes into two, without any integer-to-float conversion.
//   * which cache rows form an n-tile and which dims of a k-step sit on which MMA k-slot is free as long as both
//     operands agree: a thread's four k-slots of a step are the four bytes of ONE stored K word (one load per
//     n-tile and step), and column n of n-tile t is block row 4 n + t, which puts the 32 loads of a warp on 32
//     banks for rows of an odd number of words (and spreads the V loads of the four row pairs likewise).
//   * S^T = q K^T: q enters as fp16 (its bf16 values converted once per unit: exact but for values below the fp16
//     normal range), the K operand as 1152 + c.  The products are exact in fp32; the constant is taken out again on
//     the accumulators (1152 times the sum of the head's q, known per unit), and the row's K scale is applied to the
//     logit.  Six accumulation steps per logit: the detour through 1152 costs a few units of the last fp32 place.
//   * O += P V: the row's V scale is folded into the weight (p' = p s_V, fp16, eleven significant bits, so the
//     two-operand split of the bf16 scan is not needed); the V operand must be the centred code here -- thousands of
//     rows accumulate into one output, and a constant of 1152 per row would swallow the low bits of the sum -- so it
//     gets one more packed subtraction (1152 + c) - 1152 = c, exact.  A thread loads one 32-bit word (four channels)
//     from each of its four rows of a 16-row step and builds the operand registers of four 8-channel tiles from
//     them; which channels form a tile is free, so tile i of a 32-channel group holds channels 4 g + i.
//   * rows past the end of a sequence get weight zero and scale zero, so nothing has to be cleared in the stages.
// Every mbarrier wait is bounded: on timeout the CTA records RAP_ETIMEOUT and leaves.
#pragma once
#include <cuda_fp16.h>

#include "rap_attn_common.cuh"

namespace {

constexpr float Q8_LAZY_SLACK = 8.f;
constexpr int Q8_BR = 32;                       // rows per warp block
constexpr int Q8_NW = 4;                        // warps per CTA
constexpr int Q8_NSTG = 4;                      // stages per warp where they fit (rows are half as long as bf16 rows)

template <int G, int WK, int DV>
struct Q8Cfg {
  static_assert(G >= 1 && G <= 8, "the query heads of a KV head sit on 8 fragment rows");
  static_assert(WK >= 8 && DV >= 16, "one full k-step / channel block");
  static constexpr int NKS = (WK + 7) / 8;                    // k-steps of 16 dims
  static constexpr int NCG = (DV + 31) / 32;                  // groups of 32 channels
  static constexpr int CW = 32 * NCG;                         // channel slots of the reduction buffer
  static constexpr int KS = (2 * WK + 2 + 3) / 4 * 4;         // bytes of a quantised K row (codes, padding, bf16 scale)
  static constexpr int VS = (DV + 2 + 3) / 4 * 4;             // bytes of a quantised V row
  static constexpr int K_BYTES = Q8_BR * KS, V_BYTES = Q8_BR * VS;
  static constexpr int STAGE_BYTES = cround(K_BYTES + V_BYTES + 32, 128);   // the last channel group may read past a row
  static constexpr int NW = Q8_NW;
  static constexpr int RED_BYTES_1 = G * CW * 4;              // per warp
  static constexpr int MERGE_BYTES = (G * RAP_MAX_SPLIT + 8) * 4;
  static constexpr int OFF_RED = 512;
  static constexpr int RED_BYTES = NW * RED_BYTES_1 > MERGE_BYTES ? NW * RED_BYTES_1 : MERGE_BYTES;
  static constexpr int OFF_STAGE = cround(OFF_RED + RED_BYTES, 128);
  static constexpr int fits(int nstg) { return OFF_STAGE + NW * nstg * STAGE_BYTES; }
  static constexpr int NSTG = fits(Q8_NSTG) <= SMEM_BUDGET ? Q8_NSTG : fits(3) <= SMEM_BUDGET ? 3 : 2;   // stages per warp
  static constexpr int SMEM = fits(NSTG);
  static constexpr int THREADS = NW * 32;
  static constexpr int ST = NW * Q8_BR;                       // positions per CTA tile
  static constexpr bool TMA = false;
  static_assert(SMEM <= SMEM_BUDGET, "ring does not fit");
  static_assert(NW * NSTG * 8 + NW * 64 <= OFF_RED - 16, "barriers and merge scalars sit below the reduction buffer");
  static_assert((K_BYTES % 16) == 0 && (V_BYTES % 16) == 0, "blocks are whole 16-byte units");
  // row of column n of n-tile t inside the warp's block: 4 n + t (rows 0, 4, .., 28 of a row of an odd number of
  // words start on banks 0, 28, 24, .., 4)
  static __device__ __forceinline__ constexpr int row(int t, int n) { return 4 * n + t; }
  // dims where the last k-step starts when 2P is not a multiple of 16: moved back so that it ends at (or, for a row
  // of 4 m + 2 code bytes, two bytes past) the end of the codes and starts on a word; what it covers twice, and the
  // two bytes past the codes, meet zeroed q
  static constexpr int LAST_BASE = ((2 * WK) % 4 == 2) ? 2 * WK - 14 : 2 * WK - 16;
  static constexpr bool LAST_SHIFTED = (2 * WK) % 16 != 0;
};

__device__ __forceinline__ void q8_mma_f16(float (&c)[4], uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1) {
  // rows 8..15 of A (registers a1, a3) are the padding of the head axis: zero
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %5}, {%7, %8}, {%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(0u), "r"(a2), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float q8_ex2(float x) {      // 2^x, one instruction; 2^(-inf) = 0
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t q8_pack_f16(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
__device__ __forceinline__ uint32_t q8_prmt(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t r;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
  return r;
}
__device__ __forceinline__ uint32_t q8_hsub2(uint32_t a, uint32_t b) {
  uint32_t r;
  asm("sub.rn.f16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
  return r;
}
__device__ __forceinline__ float q8_bf16_bits(uint32_t h) { return __uint_as_float(h << 16); }
constexpr uint32_t Q8_EXP = 0x64646464u;        // high byte of the fp16 numbers 1024 .. 1279
constexpr uint32_t Q8_1152 = 0x64806480u;       // fp16 pair (1152, 1152)

template <int G, int WK, int DV>
__global__ void __launch_bounds__(Q8Cfg<G, WK, DV>::THREADS, 2) attn_q8_kernel(const ScanParams p) {
  using C = Q8Cfg<G, WK, DV>;
  constexpr int ST = C::ST, NW = C::NW, NSTG = C::NSTG, NKS = C::NKS, NCG = C::NCG, CW = C::CW;
  constexpr int KSW = C::KS / 4, VSW = C::VS / 4;          // words per quantised row
  constexpr int MMA_BR = Q8_BR;
  constexpr int THREADS = C::THREADS;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  unsigned char* smem = smem_raw;
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
  if (p.balanced) {
    // the plan (reads the lengths only): computed by the first warp into the reduction buffer, which is free until
    // the first merge; batches too large for that buffer are planned by every thread on its own
    int* pref = reinterpret_cast<int*>(red);
    const bool shared_plan = sk_plan_shared(p.seq_len, p.B, p.Hkv, p.len_add, p.S_cap, ST, (int)gridDim.x, pref,
                                            C::RED_BYTES / 4, &plan);
    if (!shared_plan) plan = sk_plan(p.seq_len, p.B, p.Hkv, p.len_add, p.S_cap, ST, (int)gridDim.x);
    // Everything below reads q~ and the cache rows the previous kernel in the stream wrote, and writes what the next
    // one may depend on: wait for the predecessor first, and only then let the successor start (it may begin to
    // stream its weights while this scan runs, and waits for this kernel before it writes anything this one reads).
    pdl_wait();
    pdl_launch_dependents();
    if (blockIdx.x == 0) {   // sequences without any row are scanned by nobody: their output is zero
      for (int i = tid; i < p.B * p.Hkv; i += THREADS) p.unit_cnt_other[i] = 0;   // counters a launch that gave up left behind
      if (tid == 0) *p.dyn_next_other = 0;          // and the piece counter a bf16 tensor-core launch before this one used
      for (int bb = 0; bb < p.B; ++bb) {
        const bool empty = shared_plan ? pref[bb] == (bb > 0 ? pref[bb - 1] : 0)
                                       : sk_tiles_of(p.seq_len, bb, p.len_add, p.S_cap, ST) == 0;
        if (empty)
          for (int i = tid; i < p.Hq * DV; i += THREADS) p.out[(size_t)bb * p.Hq * DV + i] = 0.f;
      }
    }
    if ((int)blockIdx.x >= plan.nc) return;
    cur = (int)((long long)blockIdx.x * plan.T / plan.nc);
    hi = (int)((long long)(blockIdx.x + 1) * plan.T / plan.nc);
    if (cur >= hi) return;
    int pb = 0;
    if (shared_plan) {       // the unit that holds tile `cur`
      b = sk_seq_of(pref, p.B, cur);
      pb = b > 0 ? pref[b - 1] : 0;
    } else {
      for (b = 0; b < p.B; ++b) {
        const int nb = sk_tiles_of(p.seq_len, b, p.len_add, p.S_cap, ST) * p.Hkv;
        if (cur < pb + nb) break;
        pb += nb;
      }
    }
    const int ntb = sk_tiles_of(p.seq_len, b, p.len_add, p.S_cap, ST);
    h = (cur - pb) / ntb;
    unit_start = pb + h * ntb;
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

  // fragment addressing inside a block.  K: this thread supplies column gid of every n-tile (block row 4 gid + t)
  // and, of a k-step that starts at byte `base` of the row, the word base / 4 + tq: its bytes 0, 1 are the k-slots
  // 2 tq, 2 tq + 1, its bytes 2, 3 the k-slots 2 tq + 8, 2 tq + 9.
  const int krow = 4 * gid * KSW + tq;                      // + t KSW for n-tile t, + base / 4 for the step
  // V: the k-slots 2 tq, 2 tq + 1 of n-tile t are block rows 8 tq + t and 8 tq + 4 + t; word gid of a 32-channel group
  const int vrow = 8 * tq * VSW + gid;
  int st = 0;                  // ring position and phase of this warp, running on across units
  uint32_t parity = 0;
  bool timed_out = false;
  const float cs = p.qscale;   // log2(e) / sqrt(D)

  for (;;) {   // one pass per segment (a single one unless the mode is balanced)
    int seg_tiles;
    {
      len = min(max(p.seq_len[b] + p.len_add, 0), p.S_cap);
      seg_tiles = (len + ST - 1) / ST;
      if (p.balanced) {
        t_begin = cur - unit_start;
        n_my = min(seg_tiles - t_begin, hi - cur);
        const int seg = (int)blockIdx.x - sk_cta_of(unit_start, plan);
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
    const unsigned char* kg = p.k + unit * (size_t)p.S_cap * (size_t)C::KS;
    const unsigned char* vg = p.v + unit * (size_t)p.S_cap * (size_t)C::VS;
    const int len8 = (len + 7) & ~7;                  // rows a copy may touch: S_cap is a multiple of 8
    // this warp's blocks: rows [(t_begin + i) ST + 32 warp, + 32) for i < n_blk, those that hold a valid row
    const int row_w = t_begin * ST + MMA_BR * warp;
    const int n_blk = len > row_w ? min(n_my, (len - row_w + ST - 1) / ST) : 0;

    auto issue_block = [&](int i, int stg) {          // all lanes converged; lane 0 issues
      const int j0 = row_w + i * ST;
      const int rows = min(MMA_BR, len8 - j0);
      const uint32_t bar = bar0 + 8 * stg, dst = wstage_u + stg * C::STAGE_BYTES;
      const uint32_t kb = (uint32_t)rows * C::KS, vb = (uint32_t)rows * C::VS;     // multiples of 16: rows is a multiple of 8
      if (lane == 0 && RAP_BOUNDS(j0 + rows - 1, p.S_cap, p.status, 0x202) && RAP_BOUNDS(stg, NSTG, p.status, 0x203) &&
          RAP_BOUNDS(rows - 1, MMA_BR, p.status, 0x204)) {
        mbar_expect_tx(bar, kb + vb);
        bulk_g2s(dst, kg + (size_t)j0 * C::KS, kb, bar);
        bulk_g2s(dst + C::K_BYTES, vg + (size_t)j0 * C::VS, vb, bar);
      }
    };
    {
      const int pre = min(n_blk, NSTG - 1);
      for (int i = 0; i < pre; ++i) issue_block(i, (st + i) % NSTG);
    }

    // ---- q as the A operand (fp16): head gid; of the step that starts at dim `base` the dims base + 4 tq, + 1 (k-slots
    // 2 tq, 2 tq + 1) and base + 4 tq + 2, + 3 (k-slots 2 tq + 8, 2 tq + 9); zero for the padding heads, for dims an
    // earlier step covered and for dims past the row.  off_q = 1152 * (sum of the head's q): what the constant in
    // the K operand adds to every raw logit of this head.
    uint32_t qa[NKS][2];
    float off_q = 0.f;
    {
      const uint32_t* qrow = p.q + ((size_t)b * p.Hq + (size_t)h * G + (gid < G ? gid : 0)) * WK;
#pragma unroll
      for (int ks = 0; ks < NKS; ++ks) {
        const bool shifted = C::LAST_SHIFTED && ks == NKS - 1;
        const int wb = (shifted ? C::LAST_BASE : 16 * ks) / 2;     // first bf16 pair (word of q) of the step
#pragma unroll
        for (int hlf = 0; hlf < 2; ++hlf) {
          const int w = wb + 2 * tq + hlf;
          const bool fresh = w >= 8 * ks && w < WK;             // not covered by an earlier step, inside the row
          const uint32_t bits = (gid < G && fresh && RAP_BOUNDS(w, WK, p.status, 0x201)) ? qrow[w] : 0u;
          qa[ks][hlf] = q8_pack_f16(__uint_as_float(bits << 16), __uint_as_float(bits & 0xffff0000u));
          const __half2 hq = *reinterpret_cast<const __half2*>(&qa[ks][hlf]);
          off_q += __low2float(hq) + __high2float(hq);
        }
      }
      off_q += __shfl_xor_sync(0xffffffffu, off_q, 1);
      off_q += __shfl_xor_sync(0xffffffffu, off_q, 2);
      off_q *= 1152.f;
    }
    float o[NCG][4][4];           // [channel group][tile i: channels 4 g + i][accumulator registers]
#pragma unroll
    for (int cg = 0; cg < NCG; ++cg)
#pragma unroll
      for (int i4 = 0; i4 < 4; ++i4)
#pragma unroll
        for (int r = 0; r < 4; ++r) o[cg][i4][r] = 0.f;
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

      // ---- S^T = q K^T: four n-tiles (8 rows each), NKS steps of 16 dims; K operand = 1152 + code ----
      float s[4][4];
#pragma unroll
      for (int t = 0; t < 4; ++t) s[t][0] = s[t][1] = s[t][2] = s[t][3] = 0.f;
#pragma unroll
      for (int ks = 0; ks < NKS; ++ks) {
        const int w0 = ((C::LAST_SHIFTED && ks == NKS - 1) ? C::LAST_BASE : 16 * ks) / 4;
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          const uint32_t x = RAP_BOUNDS(krow + t * KSW + w0, C::K_BYTES / 4, p.status, 0x205) ? kw[krow + t * KSW + w0] : 0u;
          q8_mma_f16(s[t], qa[ks][0], qa[ks][1], q8_prmt(x, Q8_EXP, 0x4140u), q8_prmt(x, Q8_EXP, 0x4342u));
        }
      }

      // ---- scales of this thread's rows 4 (2 tq + e) + t (bf16 in the last two bytes of a row) ----
      float ksc[4][2], vsc[4][2];
#pragma unroll
      for (int t = 0; t < 4; ++t)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int r = C::row(t, 2 * tq + e);
          const bool valid = r < nrows;
          const bool sc_ok = RAP_BOUNDS(r, MMA_BR, p.status, 0x206);
          const uint32_t kb16 = sc_ok ? *reinterpret_cast<const uint16_t*>(stage + r * C::KS + C::KS - 2) : 0u;
          const uint32_t vb16 = sc_ok ? *reinterpret_cast<const uint16_t*>(stage + C::K_BYTES + r * C::VS + C::VS - 2) : 0u;
          ksc[t][e] = valid ? q8_bf16_bits(kb16) * cs : 0.f;
          vsc[t][e] = valid ? q8_bf16_bits(vb16) : 0.f;
        }

      // ---- softmax on the accumulators: x = (s - 1152 sum q) s_K log2(e)/sqrt(D) - m_ref ----
      float x[4][2];
      bool raise = false;
#pragma unroll
      for (int t = 0; t < 4; ++t)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          s[t][e] = (s[t][e] - off_q) * ksc[t][e];                     // the logit in base-2 units
          x[t][e] = s[t][e] - m_ref;
          if (nrows < MMA_BR && C::row(t, 2 * tq + e) >= nrows) x[t][e] = -INFINITY;
          raise |= x[t][e] > Q8_LAZY_SLACK;
        }
      if (__any_sync(0xffffffffu, raise)) {
        float mx = -INFINITY;
#pragma unroll
        for (int t = 0; t < 4; ++t)
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const bool masked = nrows < MMA_BR && C::row(t, 2 * tq + e) >= nrows;
            x[t][e] = masked ? -INFINITY : s[t][e];
            mx = fmaxf(mx, x[t][e]);
          }
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        const float m_new = fmaxf(m_ref, mx);                  // finite: every block holds a valid row
        const float alpha = q8_ex2(m_ref - m_new);             // first block: 2^(-inf) = 0
        m_ref = m_new;
        l_thr *= alpha;
#pragma unroll
        for (int cg = 0; cg < NCG; ++cg)
#pragma unroll
          for (int i4 = 0; i4 < 4; ++i4) {
            o[cg][i4][0] *= alpha;
            o[cg][i4][1] *= alpha;
          }
#pragma unroll
        for (int t = 0; t < 4; ++t)
#pragma unroll
          for (int e = 0; e < 2; ++e) x[t][e] -= m_ref;
      }
      uint32_t pa[4];          // p s_V as fp16 pairs: the A operand of the second contraction
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        const float p0 = q8_ex2(x[t][0]), p1 = q8_ex2(x[t][1]);
        l_thr += p0 + p1;
        pa[t] = q8_pack_f16(p0 * vsc[t][0], p1 * vsc[t][1]);
      }

      // ---- O += P V: two steps of 16 rows (n-tiles 2 kb, 2 kb + 1), NCG groups of 32 channels ----
      // (bounds-checking build: the word offsets do not depend on the data; the largest one is checked once per block
      // against the words this stage holds behind the K block)
      const bool v_ok = RAP_BOUNDS(vrow + (2 + 5) * VSW + 8 * (NCG - 1), (C::STAGE_BYTES - C::K_BYTES) / 4, p.status, 0x207);
#pragma unroll
      for (int kb = 0; kb < 2 && v_ok; ++kb) {
        // rows of this thread's k-slots: n-tile 2 kb -> 8 tq + 2 kb and 8 tq + 4 + 2 kb, n-tile 2 kb + 1 -> one row further
        const uint32_t* v0 = vw + vrow + 2 * kb * VSW;
#pragma unroll
        for (int cg = 0; cg < NCG; ++cg) {
          const uint32_t xa = v0[8 * cg], xb = v0[8 * cg + 4 * VSW];
          const uint32_t xc = v0[8 * cg + VSW], xd = v0[8 * cg + 5 * VSW];
          // channel pairs (0, 1) and (2, 3) of the word, each as (first row, second row) of the k-slot pair
          const uint32_t g01 = q8_prmt(xa, xb, 0x5140u), g23 = q8_prmt(xa, xb, 0x7362u);
          const uint32_t h01 = q8_prmt(xc, xd, 0x5140u), h23 = q8_prmt(xc, xd, 0x7362u);
#pragma unroll
          for (int i4 = 0; i4 < 4; ++i4) {
            const uint32_t gsrc = i4 < 2 ? g01 : g23, hsrc = i4 < 2 ? h01 : h23;
            const uint32_t sel = (i4 & 1) ? 0x4342u : 0x4140u;
            const uint32_t b0 = q8_hsub2(q8_prmt(gsrc, Q8_EXP, sel), Q8_1152);
            const uint32_t b1 = q8_hsub2(q8_prmt(hsrc, Q8_EXP, sel), Q8_1152);
            q8_mma_f16(o[cg][i4], pa[2 * kb], pa[2 * kb + 1], b0, b1);
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
    const float f = m_ref == -INFINITY ? 0.f : q8_ex2(m_ref - m_all);   // a warp without a block contributes nothing
    if (tq == 0) l_s[warp * 8 + gid] = l_thr * f;
    if (gid < G && RAP_BOUNDS(((size_t)warp * G + gid) * CW + CW - 1, C::RED_BYTES / 4, p.status, 0x208)) {
      float* rr = red + ((size_t)warp * G + gid) * CW;
#pragma unroll
      for (int cg = 0; cg < NCG; ++cg)
#pragma unroll
        for (int i4 = 0; i4 < 4; ++i4) {
          // accumulator columns 2 tq, 2 tq + 1 of tile i are the channels 4 (2 tq) + i and 4 (2 tq + 1) + i of the group
          rr[32 * cg + 8 * tq + i4] = o[cg][i4][0] * f;
          rr[32 * cg + 8 * tq + 4 + i4] = o[cg][i4][1] * f;
        }
    }
    __syncthreads();
    const bool ws_ok = RAP_BOUNDS((ws_base - p.ws) + (long long)(G - 1) * ws_head + DV + 1, p.ws_floats, p.status, 0x209);
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
      const int first = sk_cta_of(unit_start, plan);
      const int nseg = sk_cta_of(unit_start + seg_tiles - 1, plan) - first + 1;
      const int u = b * p.Hkv + h;
      if (tid == 0) *s_last = RAP_BOUNDS(u, p.B * p.Hkv, p.status, 0x20a) && atomicAdd(&p.unit_cnt[u], 1) == nseg - 1;
      __syncthreads();
      if (*s_last) {
        __threadfence();
        const float* ub = p.ws + ((size_t)b * p.Hq + (size_t)h * G) * RAP_MAX_SPLIT * (size_t)(DV + 2);
        const bool m_ok = RAP_BOUNDS((ub - p.ws) + (long long)(G - 1) * ws_head + (long long)(nseg - 1) * (DV + 2) + DV + 1,
                                     p.ws_floats, p.status, 0x20b) &&
                          RAP_BOUNDS(((size_t)b * p.Hq + (size_t)h * G + G - 1) * DV + DV - 1, (size_t)p.B * p.Hq * DV, p.status, 0x20c);
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
    if (cur >= hi) break;
    unit_start += seg_tiles;
    if (++h == p.Hkv) {
      h = 0;
      do { ++b; } while (b < p.B && sk_tiles_of(p.seq_len, b, p.len_add, p.S_cap, ST) == 0);
      if (b >= p.B) break;
    }
    __syncthreads();   // the reduction buffer and the merge scalars are reused by the next segment
  }   // segment loop
}

}  // namespace
