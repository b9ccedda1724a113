// Shape-specialised bf16 split-KV scan for rap_decode_attn on the plain FP32 pipes (Eq. 2 on the retained dims,
// Eq. 7, scale 1/sqrt(D)): the tier behind the tensor-core form of the scan (rap_attn_mma_kernel.cuh), kept for
// cross-checks and for the low-rank comparator's full-width K.
//
// The scan reads every cache byte once and does G flops per byte, so HBM bandwidth bounds it;
// what decides whether it gets there is the number of issue slots spent per cache word on the
// plain FP32 pipes (tensor cores are not used for this scan).  Everything that depends on the
// head shape -- K words per row (WK = P), V channels (DV = d_v'), group size G -- is a template
// parameter, so the inner loops are fully unrolled with immediate shared-memory offsets and
// no run-time predicates.
//
// One CTA (256 threads) scans tiles (64 to 192 positions) of one (sequence, KV head) unit at a time for
// all G query heads of that KV head.
//   * staging: K and V tiles are contiguous byte ranges of the dense-packed cache; warp 0
//     moves them with bulk async copies (mbarrier complete_tx) into a two-stage ring of large tiles.
//   * logits: warp c owns dim-chunk c (chunks are equal; the last one is shifted back into
//     the row and its overlapped words meet zeroed q), lane l owns positions l and l + 32.
//     q lives in registers pre-scaled by log2(e)/sqrt(D) as (even, odd) float pairs; each
//     32-bit cache word is unpacked by shift / mask and fed to packed fma.rn.f32x2.
//   * softmax: warp g < G adds the 8 chunk partials of head g.  The reference maximum is
//     lazy: it is raised (with a warp max and a rescale factor for the accumulators) only when
//     a logit exceeds it by more than 8, so p = 2^(s - m_ref) <= 256 and most tiles need neither
//     shuffles nor a rescale; the row sum stays per lane until the end of the scan.
//   * PV: thread (row group, channel pair) accumulates its rows two at a time per packed FMA.
//   * partials (acc[d_v'], m, l) of the split go to the workspace; in balanced mode the CTA that delivers a unit's
//     last partial merges them, with an explicit n_split a combine kernel does.
// Every mbarrier wait is bounded: on timeout the CTA records RAP_ETIMEOUT and leaves.
#pragma once
#include "rap_attn_common.cuh"

namespace {

constexpr int STHREADS = 256;
constexpr int SCHUNKS = 8;       // dim chunks of the logits phase (= warps)
constexpr float LAZY_MAX_SLACK = 8.f;

// positions per tile: the largest multiple of 32 (up to 192) whose two-stage ring fits beside the
// partial-logit and p buffers of a CTA (two CTAs per SM).  Large tiles spread the per-tile costs
// (barriers, waits, softmax bookkeeping) over more bytes and keep a whole tile in flight.
constexpr int scan_smem_bound(int G, int WK, int DV, int st) {
  const int k_row = WK * 4;
  const int wvp = (DV + 1) / 2, ng = (STHREADS / wvp) > st ? st : (STHREADS / wvp);
  const int ip = ((st + ng - 1) / ng + 1) / 2, gp = (G + 1) & ~1;
  const int pp = ng * (cround(ip * gp * 2, 32) + 8) * 4;                         // p buffer
  return 128 + SCHUNKS * (G * st + 4) * 4 + pp + 512 + 2 * (st * (k_row + DV * 2) + 256);
}
constexpr int scan_tile_rows(int G, int WK, int DV) {
  for (int st = 192; st > 64; st -= 32)
    if (scan_smem_bound(G, WK, DV, st) <= SMEM_BUDGET) return st;
  return 64;
}

template <int G, int WK, int DV>
struct ScanCfg {
  static constexpr int ST = scan_tile_rows(G, WK, DV);   // positions per tile
  static constexpr int RL = ST / 32;                           // rows per lane in the logits / softmax phases
  static constexpr int KV = (WK % 2) ? 1 : (WK % 4) ? 2 : 4;   // 32-bit words per K read
  // Rows of 128 / 256 bytes put every row on the same banks.  For those the logits mapping is
  // rotated: the 8 lanes of a quarter warp read 8 consecutive 16-byte units of ONE row (a contiguous
  // 128 bytes), lane j of the quarter owns units j, j + 8, ..., and the chunk index of the partial
  // logits is j instead of the warp.  Other multiples of 32 bytes fall back to padded row copies.
  static constexpr bool KROT = (WK % 8) == 0;
  static constexpr int KS = WK;                                // K row stride in shared memory (words)
  static constexpr int UNITS = WK / KV;
  static constexpr int CLU = (UNITS + SCHUNKS - 1) / SCHUNKS;  // reads per lane and row
  static constexpr int SPS = KROT ? G * ST + 4 : G * ST;       // partial-logit floats per chunk (bank-shifted when rotated)
  static constexpr int CL = CLU * KV;                          // words per chunk
  static constexpr bool VODD = (DV & 1) != 0;
  static constexpr int WVP = (DV + 1) / 2;                     // channel pairs per V row
  static constexpr int NG = (STHREADS / WVP) > ST ? ST : (STHREADS / WVP);   // PV row groups
  // Odd d_v': rows are 2-byte aligned, but with an even number of row groups every thread only meets rows
  // of one parity, and the aligned 32-bit word w of such a row holds channels (2w, 2w+1) for even rows and
  // (2w-1, 2w) for odd rows -- same word loads as for even d_v', the channel shift is applied once, when
  // the row groups are reduced.  (The half word that belongs to a neighbouring row is finite and dropped.)
  static constexpr bool VWORD = !VODD || (NG % 2) == 0;
  static constexpr int RPG = (ST + NG - 1) / NG;               // rows per group (largest)
  static constexpr int LASTN = ST - (RPG - 1) * NG;            // groups that own a row in the last slot
  static constexpr int IP = (RPG + 1) / 2;                     // row pairs per group
  static constexpr int Gp = (G + 1) & ~1;
  static constexpr int GS = cround(IP * Gp * 2, 32) + 8;       // p floats per group (bank-shifted)
  static constexpr int OFF_SPART = 128;
  static constexpr int OFF_PP = OFF_SPART + SCHUNKS * SPS * 4;
  static constexpr int OFF_ALPHA = OFF_PP + cround(NG * GS * 4, 16);
  static constexpr int OFF_STAGE = cround(OFF_ALPHA + 32, 128);
  static constexpr int V_OFF = cround(ST * KS * 4, 128);
  static constexpr int STAGE_BYTES = cround(V_OFF + ST * DV * 2, 128);
  static constexpr int NS_RAW = (SMEM_BUDGET - OFF_STAGE) / STAGE_BYTES;
  static constexpr int NS = NS_RAW > 4 ? 4 : NS_RAW;
  static constexpr int SMEM = OFF_STAGE + NS * STAGE_BYTES;
  static_assert(NS >= 2, "tile ring needs two stages");
  static_assert(NG * 2 * WVP * G <= SCHUNKS * SPS, "row-group reduction reuses the partial-logit buffer");
};

__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ uint64_t pack2u(uint32_t lo, uint32_t hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
// d = a * b + c on two packed fp32 lanes
__device__ __forceinline__ uint64_t ffma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t fmul2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}

template <int KV>
__device__ __forceinline__ void ld_words(const uint32_t* p, uint32_t (&x)[KV]) {
  if constexpr (KV == 1) {
    x[0] = *p;
  } else if constexpr (KV == 2) {
    const uint2 v = *reinterpret_cast<const uint2*>(p);
    x[0] = v.x; x[1] = v.y;
  } else {
    const uint4 v = *reinterpret_cast<const uint4*>(p);
    x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
  }
}

template <int G, int WK, int DV>
__global__ void __launch_bounds__(STHREADS, 2) attn_scan_kernel(const ScanParams p) {
  using C = ScanCfg<G, WK, DV>;
  constexpr int Gp = C::Gp;
  constexpr int ST = C::ST, RL = C::RL;
  extern __shared__ __align__(128) unsigned char smem[];
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem);
  float* s_part = reinterpret_cast<float*>(smem + C::OFF_SPART);   // [SCHUNKS][G][ST]; reused for the group reduction
  float* pp = reinterpret_cast<float*>(smem + C::OFF_PP);
  float* alpha_s = reinterpret_cast<float*>(smem + C::OFF_ALPHA);
  unsigned char* stages = smem + C::OFF_STAGE;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // what the current segment scans: tiles [t_begin, t_begin + n_my) of unit (b, h), partials to ws_base
  int b = 0, h = 0, len = 0, len8 = 0, t_begin = 0, n_my = 0;
  float* ws_base = nullptr;
  size_t ws_head = 0;
  const unsigned char* kg = nullptr;
  const unsigned char* vg = nullptr;
  // balanced mode: this CTA's range [cur, hi) of global tiles and the plan it comes from
  SkPlan plan;
  plan.T = 0; plan.nc = 0;
  int cur = 0, hi = 0, unit_start = 0;
  if (p.balanced) {
    plan = sk_plan(p.seq_len, p.B, p.Hkv, p.len_add, p.S_cap, ST, (int)gridDim.x);   // reads the lengths only
    // Everything below reads q~ and the cache rows the previous kernel in the stream wrote, and writes what the next
    // one may depend on: wait for the predecessor first, and only then let the successor start (it may begin to
    // stream its weights while this scan runs, and waits for this kernel before it writes anything this one reads).
    pdl_wait();
    pdl_launch_dependents();
    if (blockIdx.x == 0) {   // sequences without any row are scanned by nobody: their output is zero
      for (int i = tid; i < p.B * p.Hkv; i += STHREADS) p.unit_cnt_other[i] = 0;   // counters a launch that gave up left behind
      if (tid == 0) *p.dyn_next_other = 0;          // and the piece counter a tensor-core launch before this one used
      for (int bb = 0; bb < p.B; ++bb)
        if (sk_tiles_of(p.seq_len, bb, p.len_add, p.S_cap, ST) == 0)
          for (int i = tid; i < p.Hq * DV; i += STHREADS) p.out[(size_t)bb * p.Hq * DV + i] = 0.f;
    }
    if ((int)blockIdx.x >= plan.nc) return;
    cur = (int)((long long)blockIdx.x * plan.T / plan.nc);
    hi = (int)((long long)(blockIdx.x + 1) * plan.T / plan.nc);
    if (cur >= hi) return;
    // the unit that holds tile `cur`
    int pb = 0;
    for (b = 0; b < p.B; ++b) {
      const int nb = sk_tiles_of(p.seq_len, b, p.len_add, p.S_cap, ST) * p.Hkv;
      if (cur < pb + nb) break;
      pb += nb;
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
  const uint32_t bar0 = smem_u32(bars);
  const uint32_t stage0 = smem_u32(stages);

  if (tid == 0) {
#pragma unroll
    for (int s = 0; s < C::NS; ++s) mbar_init(bar0 + 8 * s, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  for (int i = tid; i < C::NG * C::GS; i += STHREADS) pp[i] = 0.f;   // slots of rows that never exist stay zero
  __syncthreads();

  // issued by warp 0 (all lanes converged): tile tl of this CTA into stage st
  auto issue_tile = [&](int tl, int st) {
    const int j0 = (t_begin + tl) * ST;
    const int rows = min(ST, len8 - j0);
    const uint32_t bar = bar0 + 8 * st;
    const uint32_t dst = stage0 + st * C::STAGE_BYTES;
    const uint32_t kb = (uint32_t)rows * WK * 4, vb = (uint32_t)rows * DV * 2;
    if (lane == 0) mbar_expect_tx(bar, kb + vb);
    __syncwarp();
    if (lane == 0) bulk_g2s(dst, kg + (size_t)j0 * (WK * 4), kb, bar);
    if (lane == 0) bulk_g2s(dst + C::V_OFF, vg + (size_t)j0 * (DV * 2), vb, bar);
  };
  // ---- this warp's dim chunk and its pre-scaled q registers ---------------------------------
  const int u_nom = warp * C::CLU;                         // first unit this chunk is responsible for
  const int u0 = min(u_nom, C::UNITS - C::CLU);            // first unit it reads (shifted back into the row)
  const int w0 = C::KROT ? (lane & 7) * 4 : u0 * C::KV;    // first word this thread reads in a row
  const int ustep = C::KROT ? 32 : C::KV;                  // words between its consecutive reads
  const int krow = C::KROT ? warp * 4 + (lane >> 3) : lane;   // its rows: krow and krow + 32
  const int kchunk = C::KROT ? (lane & 7) : warp;          // which of the 8 partial sums it produces
  // rotated mapping with a unit count that is not a multiple of 8: lanes past the row's last unit
  // re-read that last unit (their q is zero), never the next row
  int krot_off[C::KROT ? C::CLU : 1];
#pragma unroll
  for (int u = 0; u < (C::KROT ? C::CLU : 1); ++u) krot_off[u] = min((lane & 7) + 8 * u, C::UNITS - 1) * 4 - w0;
  uint64_t qr[G][C::CL];

  // ---- PV role ------------------------------------------------------------------------------
  const int grp = tid / C::WVP, wch = tid - grp * C::WVP;
  const bool pv_active = grp < C::NG;
  const bool last_slot_ok = grp < C::LASTN;    // does this group own a row in slot RPG - 1 ?
  const bool has_hi = 2 * wch + 1 < DV;        // odd DV: the last channel pair has one channel
  uint64_t accLo[G], accHi[G];     // (even-slot rows, odd-slot rows) partial sums of channels 2*wch and 2*wch+1
  const float* ppg = pp + (pv_active ? grp : 0) * C::GS;

  // softmax role: warp g < G, lanes own positions lane and lane + 32
  float m_ref, l_lane;
  int pidx[RL];
#pragma unroll
  for (int k = 0; k < RL; ++k) {
    const int j = lane + 32 * k, gj = j % C::NG, ij = j / C::NG;
    pidx[k] = gj * C::GS + (ij >> 1) * Gp * 2 + (ij & 1) + 2 * warp;
  }
  bool timed_out = false;
  int st = 0;                  // ring position and phase run on across segments
  uint32_t parity = 0;

  for (;;) {   // one pass per segment (a single one unless the mode is balanced)
  int seg_tiles;               // tiles of the current unit
  {
    len = min(max(p.seq_len[b] + p.len_add, 0), p.S_cap);
    len8 = (len + 7) & ~7;     // rows a copy may touch: S_cap is a multiple of 8
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
        for (int i = tid; i < G * (DV + 2); i += STHREADS) {
          const int g = i / (DV + 2), c = i - g * (DV + 2);
          ws_base[g * ws_head + c] = (c == DV) ? -INFINITY : 0.f;
        }
        return;
      }
    }
    const size_t unit = (size_t)b * p.Hkv + h;
    kg = p.k + unit * (size_t)p.S_cap * (size_t)(WK * 4);
    vg = p.v + unit * (size_t)p.S_cap * (size_t)(DV * 2);
  }
  if (warp == 0) {
    const int pre = min(n_my, C::NS - 1);
    for (int tl = 0; tl < pre; ++tl) issue_tile(tl, (st + tl) % C::NS);
  }
#pragma unroll
  for (int g = 0; g < G; ++g) {
    const uint32_t* qrow = p.q + ((size_t)b * p.Hq + (size_t)h * G + g) * WK;
#pragma unroll
    for (int i = 0; i < C::CL; ++i) {
      const bool mine = C::KROT ? ((lane & 7) + 8 * (i / C::KV)) < C::UNITS : (u0 + i / C::KV) >= u_nom;
      const uint32_t x = mine ? qrow[w0 + (i / C::KV) * ustep + i % C::KV] : 0u;   // (not read when not mine)
      qr[g][i] = pack2(__uint_as_float(x << 16) * p.qscale, __uint_as_float(x & 0xffff0000u) * p.qscale);
    }
    accLo[g] = accHi[g] = 0ull;
  }
  m_ref = -INFINITY;
  l_lane = 0.f;

  for (int tl = 0; tl < n_my; ++tl) {
    const bool ok = mbar_wait_bounded(bar0 + 8 * st, parity);
    unsigned char* stage = stages + st * C::STAGE_BYTES;
    const int j0 = (t_begin + tl) * ST;
    const int nj = min(ST, len - j0);
    if (nj < ST && ok) {
      // last tile of the sequence: rows >= nj were not written by this sequence; zero their V so
      // that the fixed-length PV loop meets 0 * 0 there
      uint16_t* vz = reinterpret_cast<uint16_t*>(stage + C::V_OFF);
      for (int i = nj * DV + tid; i < ST * DV; i += STHREADS) vz[i] = 0;
    }

    // ---- logits partials: rows lane, lane + 32; words [w0, w0 + CL) ------------------------
    {
      const uint32_t* rbase = reinterpret_cast<const uint32_t*>(stage) + krow * C::KS + w0;
#pragma unroll
      for (int rr = 0; rr < RL; rr += 2) {       // two rows (krow + 32 rr, krow + 32 rr + 32) per pass
        const bool two = rr + 1 < RL;
        const uint32_t* r0 = rbase + rr * 32 * C::KS;
        const uint32_t* r1 = r0 + (two ? 32 * C::KS : 0);
        uint64_t a0[G], a1[G];
#pragma unroll
        for (int g = 0; g < G; ++g) a0[g] = a1[g] = 0ull;
#pragma unroll
        for (int u = 0; u < C::CLU; ++u) {
          uint32_t x0[C::KV], x1[C::KV];
          const int uo = C::KROT ? krot_off[C::KROT ? u : 0] : u * ustep;
          ld_words<C::KV>(r0 + uo, x0);
          if (two) ld_words<C::KV>(r1 + uo, x1);
#pragma unroll
          for (int j = 0; j < C::KV; ++j) {
            const uint64_t k0 = pack2u(x0[j] << 16, x0[j] & 0xffff0000u);
#pragma unroll
            for (int g = 0; g < G; ++g) a0[g] = ffma2(k0, qr[g][u * C::KV + j], a0[g]);
            if (two) {
              const uint64_t k1 = pack2u(x1[j] << 16, x1[j] & 0xffff0000u);
#pragma unroll
              for (int g = 0; g < G; ++g) a1[g] = ffma2(k1, qr[g][u * C::KV + j], a1[g]);
            }
          }
        }
#pragma unroll
        for (int g = 0; g < G; ++g) {
          float e, o;
          unpack2(a0[g], e, o);
          s_part[kchunk * C::SPS + g * ST + krow + rr * 32] = e + o;
          if (two) {
            unpack2(a1[g], e, o);
            s_part[kchunk * C::SPS + g * ST + krow + rr * 32 + 32] = e + o;
          }
        }
      }
    }
    if (__syncthreads_or(!ok)) {   // sync #1: partial logits visible; the previous tile's stage is free
      timed_out = true;
      break;
    }
    if (warp == 0 && tl + C::NS - 1 < n_my) issue_tile(tl + C::NS - 1, st == 0 ? C::NS - 1 : st - 1);

    // ---- online softmax: warp g owns head g --------------------------------------------------
    if (warp < G) {
      const int g = warp;
      float sv[RL];
#pragma unroll
      for (int k = 0; k < RL; ++k) sv[k] = 0.f;
#pragma unroll
      for (int c = 0; c < SCHUNKS; ++c) {
#pragma unroll
        for (int k = 0; k < RL; ++k) sv[k] += s_part[c * C::SPS + g * ST + lane + 32 * k];
      }
      float mx = -INFINITY;
#pragma unroll
      for (int k = 0; k < RL; ++k) {
        if (lane + 32 * k >= nj) sv[k] = -INFINITY;
        mx = fmaxf(mx, sv[k]);
      }
      float alpha = 1.f;
      if (__any_sync(0xffffffffu, mx > m_ref + LAZY_MAX_SLACK)) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        const float m_new = fmaxf(m_ref, mx);
        alpha = exp2f(m_ref - m_new);     // first tile: 2^(-inf) = 0
        l_lane *= alpha;
        m_ref = m_new;
      }
#pragma unroll
      for (int k = 0; k < RL; ++k) {
        const float pk = exp2f(sv[k] - m_ref);
        l_lane += pk;
        pp[pidx[k]] = pk;
      }
      if (lane == 0) alpha_s[g] = alpha;
    }
    __syncthreads();   // sync #2: p and alpha visible

    // ---- PV: slots 0 .. RPG-1 of this thread's row group, two slots per packed FMA -----------
    if (pv_active) {
      {
        bool resc = false;
        float al[G];
#pragma unroll
        for (int g = 0; g < G; ++g) {
          al[g] = alpha_s[g];
          resc |= al[g] != 1.f;
        }
        if (resc) {
#pragma unroll
          for (int g = 0; g < G; ++g) {
            const uint64_t aa = pack2(al[g], al[g]);
            accLo[g] = fmul2(accLo[g], aa);
            accHi[g] = fmul2(accHi[g], aa);
          }
        }
      }
      const unsigned char* vt = stage + C::V_OFF;
#pragma unroll
      for (int ip = 0; ip < C::IP; ++ip) {
        const int iA = 2 * ip, iB = 2 * ip + 1;
        const bool okA = (iA < C::RPG - 1) || (iA == C::RPG - 1 && last_slot_ok);
        const bool okB = (iB < C::RPG - 1) || (iB == C::RPG - 1 && last_slot_ok);
        uint64_t lo, hi;
        if constexpr (C::VWORD) {
          constexpr int SLOT_WORDS = C::NG * DV / 2;      // words between a group's consecutive rows (NG * DV is even)
          const uint32_t* pa = reinterpret_cast<const uint32_t*>(vt) + ((grp * DV) >> 1) + wch;
          const uint32_t xa = okA ? pa[iA * SLOT_WORDS] : 0u;
          const uint32_t xb = okB ? pa[iB * SLOT_WORDS] : 0u;
          lo = pack2u(xa << 16, xb << 16);
          hi = pack2u(xa & 0xffff0000u, xb & 0xffff0000u);
        } else {
          const uint16_t* pa = reinterpret_cast<const uint16_t*>(vt) + grp * DV + 2 * wch;
          const uint32_t la = okA ? pa[iA * C::NG * DV] : 0u, lb = okB ? pa[iB * C::NG * DV] : 0u;
          const uint32_t ha = (okA && has_hi) ? pa[iA * C::NG * DV + 1] : 0u;
          const uint32_t hb = (okB && has_hi) ? pa[iB * C::NG * DV + 1] : 0u;
          lo = pack2u(la << 16, lb << 16);
          hi = pack2u(ha << 16, hb << 16);
        }
        const float* pr = ppg + ip * Gp * 2;
#pragma unroll
        for (int g2 = 0; g2 < Gp / 2; ++g2) {
          const float4 t = *reinterpret_cast<const float4*>(pr + 4 * g2);
          const uint64_t pg0 = pack2(t.x, t.y);
          accLo[2 * g2] = ffma2(lo, pg0, accLo[2 * g2]);
          accHi[2 * g2] = ffma2(hi, pg0, accHi[2 * g2]);
          if (2 * g2 + 1 < G) {
            const uint64_t pg1 = pack2(t.z, t.w);
            accLo[2 * g2 + 1] = ffma2(lo, pg1, accLo[2 * g2 + 1]);
            accHi[2 * g2 + 1] = ffma2(hi, pg1, accHi[2 * g2 + 1]);
          }
        }
      }
    }
    if (++st == C::NS) { st = 0; parity ^= 1u; }
  }

  if (timed_out) {
    if (tid == 0) {
      atomicCAS(&p.status[0], 0, (int)RAP_ETIMEOUT);
      p.status[1] = (b * p.Hkv + h) * RAP_MAX_SPLIT + (int)(blockIdx.x % RAP_MAX_SPLIT);
      // give copies still in flight a bounded chance to land before the shared memory is released
      for (int s = 0; s < C::NS; ++s) {
        mbar_wait_bounded(bar0 + 8 * s, 0);
        mbar_wait_bounded(bar0 + 8 * s, 1);
      }
    }
    __syncthreads();
    return;
  }

  // ---- reduce the PV row groups and write this split's partials --------------------------------
  __syncthreads();
  float* red = s_part;              // [NG][G][2 * WVP]
  constexpr int DVP = 2 * C::WVP;
  if (pv_active) {
#pragma unroll
    for (int g = 0; g < G; ++g) {
      const int ch = 2 * wch - ((C::VODD && C::VWORD) ? (grp & 1) : 0);   // odd rows of an odd d_v': shifted pairs
      float a, c;
      unpack2(accLo[g], a, c);
      if (ch >= 0) red[(grp * G + g) * DVP + ch] = a + c;
      unpack2(accHi[g], a, c);
      red[(grp * G + g) * DVP + ch + 1] = a + c;
    }
  }
  __syncthreads();
  for (int i = tid; i < G * DV; i += STHREADS) {
    const int g = i / DV, c = i - g * DV;
    float s = 0.f;
#pragma unroll
    for (int r = 0; r < C::NG; ++r) s += red[(r * G + g) * DVP + c];
    ws_base[g * ws_head + c] = s;
  }
  if (warp < G) {
    float l = l_lane;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
    if (lane == 0) {
      ws_base[warp * ws_head + DV] = m_ref;
      ws_base[warp * ws_head + DV + 1] = l;
    }
  }
  if (p.balanced) {
    // ---- the CTA that delivers a unit's last partial merges them (no separate combine launch) ------
    __shared__ int s_last;
    __threadfence();           // this CTA's partials are visible before its arrival is counted
    __syncthreads();
    const int first = sk_cta_of(unit_start, plan);
    const int nseg = sk_cta_of(unit_start + seg_tiles - 1, plan) - first + 1;
    const int u = b * p.Hkv + h;
    if (tid == 0) s_last = atomicAdd(&p.unit_cnt[u], 1) == nseg - 1;
    __syncthreads();
    if (s_last) {
      __threadfence();
      float* wgt = s_part;     // [G][64] segment weights, then G reciprocals of the denominators
      const float* ub = p.ws + ((size_t)b * p.Hq + (size_t)h * G) * RAP_MAX_SPLIT * (size_t)(DV + 2);
      if (warp < G) {
        const float* gb = ub + (size_t)warp * ws_head;
        float mv[2], lv[2];
#pragma unroll
        for (int k = 0; k < 2; ++k) {
          const int sg = lane + 32 * k;
          lv[k] = sg < nseg ? __ldcg(gb + (size_t)sg * (DV + 2) + DV + 1) : 0.f;
          mv[k] = (sg < nseg && lv[k] > 0.f) ? __ldcg(gb + (size_t)sg * (DV + 2) + DV) : -INFINITY;
        }
        float M = fmaxf(mv[0], mv[1]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
        float den = 0.f;
#pragma unroll
        for (int k = 0; k < 2; ++k) {
          const float wk = lv[k] > 0.f ? exp2f(mv[k] - M) : 0.f;
          wgt[warp * RAP_MAX_SPLIT + lane + 32 * k] = wk;
          den += wk * lv[k];
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) den += __shfl_xor_sync(0xffffffffu, den, o);
        if (lane == 0) wgt[G * RAP_MAX_SPLIT + warp] = den > 0.f ? 1.f / den : 0.f;
      }
      __syncthreads();
      for (int i = tid; i < G * DV; i += STHREADS) {
        const int g = i / DV, c = i - g * DV;
        const float* gb = ub + (size_t)g * ws_head + c;
        float num = 0.f;
        for (int sg = 0; sg < nseg; ++sg) num += wgt[g * RAP_MAX_SPLIT + sg] * __ldcg(gb + (size_t)sg * (DV + 2));
        p.out[((size_t)b * p.Hq + (size_t)h * G + g) * DV + c] = num * wgt[G * RAP_MAX_SPLIT + g];
      }
      if (tid == 0) p.unit_cnt[u] = 0;   // ready for the next call on this context
    }
  }
  // ---- next segment: the following unit, from its first tile ---------------------------------------
  if (!p.balanced) break;
  cur += n_my;
  if (cur >= hi) break;
  unit_start += seg_tiles;
  if (++h == p.Hkv) {
    h = 0;
    do { ++b; } while (b < p.B && sk_tiles_of(p.seq_len, b, p.len_add, p.S_cap, ST) == 0);
    if (b >= p.B) break;
  }
  __syncthreads();   // the row-group reduction buffer is the next segment's partial-logit buffer
  }   // segment loop
}

}  // namespace
