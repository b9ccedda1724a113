// Bandwidth-tuned bf16 split-KV scan for rap_decode_attn (Eq. 2 on the retained dims, Eq. 7,
// scale 1/sqrt(D)).  The scan is HBM-bound (G flops per cache byte), so the design goal is to
// keep ~100 KB of K/V tiles in flight per SM and to spend as few issue slots per cache word
// as the plain FP32 pipes allow; tensor cores are not used here.
//
// One CTA (256 threads) owns a contiguous range of 64-position tiles of one (sequence, KV
// head) unit and all G query heads of that KV head, so every cache byte is read from HBM once.
//   * staging: K and V tiles are contiguous byte ranges of the dense-packed cache; one elected
//     thread moves them with bulk async copies (cp.async.bulk, mbarrier complete_tx) into a
//     3-4 stage ring.  When a K row is a multiple of 32 bytes the rows are copied one by one
//     to a padded stride so that lane-per-position reads stay bank-conflict free.
//   * logits: warp c owns dim-chunk c of the K row, lane l owns positions l and l+32.  The
//     pre-scaled q chunk (log2(e)/sqrt(D) folded in) lives in registers as (even, odd) float
//     pairs; each 32-bit cache word is unpacked by shift/mask and fed to packed fma.rn.f32x2.
//   * online softmax: warp g < G sums the 8 chunk partials of head g, takes the tile max and
//     sum with warp shuffles, and writes p = 2^(s - m) in the order the PV phase reads it.
//   * PV: thread (group, channel pair) accumulates rows group, group+NG, ... two rows per
//     packed FMA; the V tile is read as consecutive 32-bit words (16-bit reads for odd d_v').
//   * partials (acc[d_v'], m, l) go to the context workspace; the combine kernel merges them.
// Every mbarrier wait is bounded: on timeout the CTA records RAP_ETIMEOUT and leaves.
#include <math.h>

#include "rap_internal.h"

namespace {

constexpr int FT = 64;          // positions per tile
constexpr int FTHREADS = 256;
constexpr int FCHUNKS = 8;      // dim chunks of the logits phase (= warps)
constexpr uint32_t WAIT_LIMIT = 1u << 21;
constexpr int SMEM_BUDGET = 115712;   // two CTAs per SM

struct FastParams {
  const uint32_t* q;          // [B][Hq][WK] bf16 pairs
  const unsigned char* k;     // [B][Hkv][S_cap][WK*4 bytes]
  const unsigned char* v;     // [B][Hkv][S_cap][dv*2 bytes]
  const int32_t* seq_len;
  float* ws;
  int32_t* status;
  int len_add, Hq, Hkv, WK, dv, S_cap, n_split;
  float qscale;
  int NS, kclass, kpad, ks;   // stages; K read width class (0/1/2 = 4/8/16 bytes); padded row copies; smem K row stride (words)
  int stage_bytes, v_off;
  int NG, WVP, IP, GS;        // PV row groups, channel pairs per row, pair iterations per group, pp group stride (floats)
  int off_pp, off_alpha, off_stage;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

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

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
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
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity) {
  for (uint32_t i = 0; i < WAIT_LIMIT; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}
// global -> this CTA's shared memory, completion counted in bytes on the mbarrier (no multicast)
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}

template <int G, int CLT>
__global__ void __launch_bounds__(FTHREADS, 2) attn_fast_kernel(const FastParams p) {
  constexpr int Gp = (G + 1) & ~1;
  extern __shared__ __align__(128) unsigned char smem[];
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem);
  float* s_part = reinterpret_cast<float*>(smem + 128);   // [FCHUNKS][G][FT]; reused for the group reduction
  float* pp = reinterpret_cast<float*>(smem + p.off_pp);
  float* alpha_s = reinterpret_cast<float*>(smem + p.off_alpha);
  unsigned char* stages = smem + p.off_stage;

  const int split = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int WK = p.WK, dv = p.dv;
  int len = p.seq_len[b] + p.len_add;
  len = min(max(len, 0), p.S_cap);
  const int n_tiles = (len + FT - 1) / FT;
  const int tps = (n_tiles + p.n_split - 1) / p.n_split;
  const int t_begin = min(n_tiles, split * tps), t_end = min(n_tiles, t_begin + tps);
  const int n_my = t_end - t_begin;
  const int len8 = (len + 7) & ~7;      // rows a copy may touch: S_cap is a multiple of 8
  float* ws_base = p.ws + (((size_t)b * p.Hq + (size_t)h * G) * p.n_split + split) * (size_t)(dv + 2);
  const size_t ws_head = (size_t)p.n_split * (dv + 2);

  if (n_my <= 0) {   // nothing to scan: neutral partials
    for (int i = tid; i < G * (dv + 2); i += FTHREADS) {
      const int g = i / (dv + 2), c = i - g * (dv + 2);
      ws_base[g * ws_head + c] = (c == dv) ? -INFINITY : 0.f;
    }
    return;
  }

  const size_t unit = (size_t)b * p.Hkv + h;
  const unsigned char* kg = p.k + unit * (size_t)p.S_cap * (size_t)(WK * 4);
  const unsigned char* vg = p.v + unit * (size_t)p.S_cap * (size_t)(dv * 2);
  const uint32_t bar0 = smem_u32(bars);
  const uint32_t stage0 = smem_u32(stages);

  if (tid == 0) {
    for (int s = 0; s < p.NS; ++s) mbar_init(bar0 + 8 * s, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  // issued by warp 0 (all lanes converged); tl = tile index local to this CTA
  auto issue_tile = [&](int tl) {
    const int st = tl % p.NS;
    const int j0 = (t_begin + tl) * FT;
    const int rows = min(FT, len8 - j0);
    const uint32_t bar = bar0 + 8 * st;
    const uint32_t dst = stage0 + st * p.stage_bytes;
    const uint32_t kb = (uint32_t)rows * WK * 4, vb = (uint32_t)rows * dv * 2;
    if (lane == 0) mbar_expect_tx(bar, kb + vb);
    __syncwarp();
    if (p.kpad) {
      for (int r = lane; r < rows; r += 32)
        bulk_g2s(dst + r * p.ks * 4, kg + (size_t)(j0 + r) * (WK * 4), WK * 4, bar);
    } else if (lane == 0) {
      bulk_g2s(dst, kg + (size_t)j0 * (WK * 4), kb, bar);
    }
    if (lane == 0) bulk_g2s(dst + p.v_off, vg + (size_t)j0 * (dv * 2), vb, bar);
  };
  if (warp == 0) {
    const int pre = min(n_my, p.NS - 1);
    for (int tl = 0; tl < pre; ++tl) issue_tile(tl);
  }

  // ---- this warp's dim chunk and its pre-scaled q registers ---------------------------------
  const int vw = 1 << p.kclass;                 // words per K read
  const int units = WK / vw;
  const int ubase = units / FCHUNKS, urem = units % FCHUNKS;
  const int w0 = (warp * ubase + min(warp, urem)) * vw;
  const int cl = (ubase + (warp < urem ? 1 : 0)) * vw;
  uint64_t qr[G][CLT];
#pragma unroll
  for (int g = 0; g < G; ++g) {
    const uint32_t* qrow = p.q + ((size_t)b * p.Hq + (size_t)h * G + g) * WK;
#pragma unroll
    for (int i = 0; i < CLT; ++i) {
      uint32_t x = (i < cl) ? qrow[w0 + i] : 0u;
      qr[g][i] = pack2(__uint_as_float(x << 16) * p.qscale, __uint_as_float(x & 0xffff0000u) * p.qscale);
    }
  }

  // ---- PV role ------------------------------------------------------------------------------
  const int NG = p.NG, WVP = p.WVP;
  const int grp = tid / WVP, wch = tid - grp * WVP;
  const bool pv_active = grp < NG;
  const bool vodd = dv & 1;
  uint64_t accLo[G], accHi[G];     // (row-pair partial a, partial b) of channels 2*wch and 2*wch+1
#pragma unroll
  for (int g = 0; g < G; ++g) accLo[g] = accHi[g] = 0ull;
  // softmax role: warp g < G, lanes own positions lane and lane+32
  float m_run = -INFINITY, l_run = 0.f;
  int pidx0, pidx1;
  {
    const int g0 = lane % NG, i0 = lane / NG, g1 = (lane + 32) % NG, i1 = (lane + 32) / NG;
    pidx0 = g0 * p.GS + (i0 >> 1) * Gp * 2 + (i0 & 1);
    pidx1 = g1 * p.GS + (i1 >> 1) * Gp * 2 + (i1 & 1);
  }
  bool timed_out = false;

  for (int tl = 0; tl < n_my; ++tl) {
    const int st = tl % p.NS;
    const uint32_t parity = (uint32_t)(tl / p.NS) & 1u;
    const bool ok = mbar_wait_bounded(bar0 + 8 * st, parity);
    const unsigned char* stage = stages + (size_t)st * p.stage_bytes;
    const int j0 = (t_begin + tl) * FT;
    const int nj = min(FT, len - j0);

    // ---- logits partials: rows lane, lane + 32; words [w0, w0 + cl) ------------------------
    {
      const uint32_t* kt = reinterpret_cast<const uint32_t*>(stage);
      const uint32_t* r0 = kt + lane * p.ks + w0;
      const uint32_t* r1 = r0 + 32 * p.ks;
      uint64_t a0[G], a1[G];
#pragma unroll
      for (int g = 0; g < G; ++g) a0[g] = a1[g] = 0ull;
      if (p.kclass == 0) {
#pragma unroll
        for (int i = 0; i < CLT; ++i) {
          if (i < cl) {
            const uint32_t x0 = r0[i], x1 = r1[i];
            const uint64_t k0 = pack2u(x0 << 16, x0 & 0xffff0000u), k1 = pack2u(x1 << 16, x1 & 0xffff0000u);
#pragma unroll
            for (int g = 0; g < G; ++g) {
              a0[g] = ffma2(k0, qr[g][i], a0[g]);
              a1[g] = ffma2(k1, qr[g][i], a1[g]);
            }
          }
        }
      } else if (p.kclass == 1) {
#pragma unroll
        for (int i = 0; i + 1 < CLT + 1 && i < CLT; i += 2) {
          if (i < cl) {
            const uint2 x0 = *reinterpret_cast<const uint2*>(r0 + i), x1 = *reinterpret_cast<const uint2*>(r1 + i);
            const uint32_t xs0[2] = {x0.x, x0.y}, xs1[2] = {x1.x, x1.y};
#pragma unroll
            for (int u = 0; u < 2; ++u) {
              if (i + u < CLT) {
                const uint64_t k0 = pack2u(xs0[u] << 16, xs0[u] & 0xffff0000u);
                const uint64_t k1 = pack2u(xs1[u] << 16, xs1[u] & 0xffff0000u);
#pragma unroll
                for (int g = 0; g < G; ++g) {
                  a0[g] = ffma2(k0, qr[g][i + u], a0[g]);
                  a1[g] = ffma2(k1, qr[g][i + u], a1[g]);
                }
              }
            }
          }
        }
      } else {
#pragma unroll
        for (int i = 0; i < CLT; i += 4) {
          if (i < cl) {
            const uint4 x0 = *reinterpret_cast<const uint4*>(r0 + i), x1 = *reinterpret_cast<const uint4*>(r1 + i);
            const uint32_t xs0[4] = {x0.x, x0.y, x0.z, x0.w}, xs1[4] = {x1.x, x1.y, x1.z, x1.w};
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              if (i + u < CLT) {
                const uint64_t k0 = pack2u(xs0[u] << 16, xs0[u] & 0xffff0000u);
                const uint64_t k1 = pack2u(xs1[u] << 16, xs1[u] & 0xffff0000u);
#pragma unroll
                for (int g = 0; g < G; ++g) {
                  a0[g] = ffma2(k0, qr[g][i + u], a0[g]);
                  a1[g] = ffma2(k1, qr[g][i + u], a1[g]);
                }
              }
            }
          }
        }
      }
#pragma unroll
      for (int g = 0; g < G; ++g) {
        float e, o;
        unpack2(a0[g], e, o);
        s_part[(warp * G + g) * FT + lane] = e + o;
        unpack2(a1[g], e, o);
        s_part[(warp * G + g) * FT + lane + 32] = e + o;
      }
    }
    if (__syncthreads_or(!ok)) {   // sync #1: partial logits visible; the previous tile's stage is free
      timed_out = true;
      break;
    }
    if (warp == 0 && tl + p.NS - 1 < n_my) issue_tile(tl + p.NS - 1);

    // ---- online softmax: warp g owns head g --------------------------------------------------
    if (warp < G) {
      const int g = warp;
      float s0 = 0.f, s1 = 0.f;
#pragma unroll
      for (int c = 0; c < FCHUNKS; ++c) {
        s0 += s_part[(c * G + g) * FT + lane];
        s1 += s_part[(c * G + g) * FT + lane + 32];
      }
      if (lane >= nj) s0 = -INFINITY;
      if (lane + 32 >= nj) s1 = -INFINITY;
      float mx = fmaxf(s0, s1);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      const float m_new = fmaxf(m_run, mx);
      const float p0 = exp2f(s0 - m_new), p1 = exp2f(s1 - m_new);
      float sum = p0 + p1;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
      const float alpha = exp2f(m_run - m_new);
      l_run = l_run * alpha + sum;
      m_run = m_new;
      pp[pidx0 + 2 * g] = p0;
      pp[pidx1 + 2 * g] = p1;
      if (lane == 0) alpha_s[g] = alpha;
    }
    __syncthreads();   // sync #2: p and alpha visible

    // ---- PV: rows grp, grp + NG, ... of this tile, two rows per packed FMA ------------------
    if (pv_active) {
#pragma unroll
      for (int g = 0; g < G; ++g) {
        const float a = alpha_s[g];
        if (a != 1.f) {
          const uint64_t aa = pack2(a, a);
          accLo[g] = ffma2(accLo[g], aa, 0ull);
          accHi[g] = ffma2(accHi[g], aa, 0ull);
        }
      }
      const int count = nj > grp ? (nj - grp + NG - 1) / NG : 0;
      const int npair = count >> 1;
      const float* ppg = pp + grp * p.GS;
      const unsigned char* vt = stage + p.v_off;
      if (!vodd) {
        const int WV = dv >> 1;
        const uint32_t* pa = reinterpret_cast<const uint32_t*>(vt) + grp * WV + wch;
        const int rstep = NG * WV;
#pragma unroll 2
        for (int ip = 0; ip < npair; ++ip) {
          const uint32_t xa = pa[0], xb = pa[rstep];
          pa += 2 * rstep;
          const uint64_t lo = pack2u(xa << 16, xb << 16), hi = pack2u(xa & 0xffff0000u, xb & 0xffff0000u);
          const float* pr = ppg + ip * Gp * 2;
#pragma unroll
          for (int g = 0; g + 1 < G; g += 2) {
            const float4 t = *reinterpret_cast<const float4*>(pr + 2 * g);
            const uint64_t pg0 = pack2(t.x, t.y), pg1 = pack2(t.z, t.w);
            accLo[g] = ffma2(lo, pg0, accLo[g]);
            accHi[g] = ffma2(hi, pg0, accHi[g]);
            accLo[g + 1] = ffma2(lo, pg1, accLo[g + 1]);
            accHi[g + 1] = ffma2(hi, pg1, accHi[g + 1]);
          }
          if (G & 1) {
            const float2 t = *reinterpret_cast<const float2*>(pr + 2 * (G - 1));
            const uint64_t pg0 = pack2(t.x, t.y);
            accLo[G - 1] = ffma2(lo, pg0, accLo[G - 1]);
            accHi[G - 1] = ffma2(hi, pg0, accHi[G - 1]);
          }
        }
        if (count & 1) {
          const uint32_t xa = pa[0];
          const uint64_t lo = pack2u(xa << 16, 0u), hi = pack2u(xa & 0xffff0000u, 0u);
          const float* pr = ppg + npair * Gp * 2;
#pragma unroll
          for (int g = 0; g < G; ++g) {
            const uint64_t pg = pack2(pr[2 * g], 0.f);
            accLo[g] = ffma2(lo, pg, accLo[g]);
            accHi[g] = ffma2(hi, pg, accHi[g]);
          }
        }
      } else {
        const uint16_t* pa = reinterpret_cast<const uint16_t*>(vt) + grp * dv + 2 * wch;
        const bool has_hi = 2 * wch + 1 < dv;
        const int rstep = NG * dv;
#pragma unroll 2
        for (int ip = 0; ip < npair; ++ip) {
          const uint32_t la = pa[0], lb = pa[rstep];
          const uint32_t ha = has_hi ? pa[1] : 0u, hb = has_hi ? pa[rstep + 1] : 0u;
          pa += 2 * rstep;
          const uint64_t lo = pack2u(la << 16, lb << 16), hi = pack2u(ha << 16, hb << 16);
          const float* pr = ppg + ip * Gp * 2;
#pragma unroll
          for (int g = 0; g + 1 < G; g += 2) {
            const float4 t = *reinterpret_cast<const float4*>(pr + 2 * g);
            const uint64_t pg0 = pack2(t.x, t.y), pg1 = pack2(t.z, t.w);
            accLo[g] = ffma2(lo, pg0, accLo[g]);
            accHi[g] = ffma2(hi, pg0, accHi[g]);
            accLo[g + 1] = ffma2(lo, pg1, accLo[g + 1]);
            accHi[g + 1] = ffma2(hi, pg1, accHi[g + 1]);
          }
          if (G & 1) {
            const float2 t = *reinterpret_cast<const float2*>(pr + 2 * (G - 1));
            const uint64_t pg0 = pack2(t.x, t.y);
            accLo[G - 1] = ffma2(lo, pg0, accLo[G - 1]);
            accHi[G - 1] = ffma2(hi, pg0, accHi[G - 1]);
          }
        }
        if (count & 1) {
          const uint32_t la = pa[0], ha = has_hi ? pa[1] : 0u;
          const uint64_t lo = pack2u(la << 16, 0u), hi = pack2u(ha << 16, 0u);
          const float* pr = ppg + npair * Gp * 2;
#pragma unroll
          for (int g = 0; g < G; ++g) {
            const uint64_t pg = pack2(pr[2 * g], 0.f);
            accLo[g] = ffma2(lo, pg, accLo[g]);
            accHi[g] = ffma2(hi, pg, accHi[g]);
          }
        }
      }
    }
  }

  if (timed_out) {
    if (tid == 0) {
      atomicCAS(&p.status[0], 0, (int)RAP_ETIMEOUT);
      p.status[1] = (b * p.Hkv + h) * p.n_split + split;
    }
    // give copies still in flight a bounded chance to land before the shared memory is released
    if (tid == 0) {
      for (int s = 0; s < p.NS; ++s) {
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
  const int DVP = 2 * WVP;
  if (pv_active) {
#pragma unroll
    for (int g = 0; g < G; ++g) {
      float a, c;
      unpack2(accLo[g], a, c);
      red[(grp * G + g) * DVP + 2 * wch] = a + c;
      unpack2(accHi[g], a, c);
      red[(grp * G + g) * DVP + 2 * wch + 1] = a + c;
    }
  }
  __syncthreads();
  for (int i = tid; i < G * dv; i += FTHREADS) {
    const int g = i / dv, c = i - g * dv;
    float s = 0.f;
    for (int r = 0; r < NG; ++r) s += red[(r * G + g) * DVP + c];
    ws_base[g * ws_head + c] = s;
  }
  if (warp < G && lane == 0) {
    ws_base[warp * ws_head + dv] = m_run;
    ws_base[warp * ws_head + dv + 1] = l_run;
  }
}

typedef void (*fast_kernel_t)(const FastParams);

template <int G>
fast_kernel_t pick_clt(int clt) {
  switch (clt) {
    case 4: return attn_fast_kernel<G, 4>;
    case 6: return attn_fast_kernel<G, 6>;
    case 8: return attn_fast_kernel<G, 8>;
  }
  return nullptr;
}

fast_kernel_t pick_kernel(int G, int clt) {
  switch (G) {
    case 1: return pick_clt<1>(clt);
    case 2: return pick_clt<2>(clt);
    case 3: return pick_clt<3>(clt);
    case 4: return clt == 7 ? attn_fast_kernel<4, 7> : pick_clt<4>(clt);
    case 5: return pick_clt<5>(clt);
  }
  return nullptr;
}

__global__ void attn_combine_fast_kernel(const float* __restrict__ ws, int n_split, int dv, float* __restrict__ out) {
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
  const float inv = den > 0.f ? 1.f / den : 0.f;
  for (int c = threadIdx.x; c < dv; c += blockDim.x) {
    float num = 0.f;
    for (int s = 0; s < n_split; ++s) {
      const float l = base[(size_t)s * (dv + 2) + dv + 1];
      if (l > 0.f) num += exp2f(base[(size_t)s * (dv + 2) + dv] - M) * base[(size_t)s * (dv + 2) + c];
    }
    out[bg * dv + c] = num * inv;
  }
}

inline int round_up(int x, int m) { return (x + m - 1) / m * m; }

}  // namespace

rap_status rap_launch_attn_fast(rap_ctx* ctx, const rap_attn_args& a, int n_split_req, cudaStream_t st) {
  const int G = a.Hq / a.Hkv;
  const int WK = a.P2 / 2, dv = a.dv;
  if (a.dtype != RAP_BF16 || G > 5 || WK < 1 || WK > 64 || dv < 16 || dv > 256) return RAP_EUNSUPPORTED;
  FastParams p;
  p.kclass = (WK % 4 == 0) ? 2 : (WK % 2 == 0) ? 1 : 0;
  p.kpad = (WK % 8 == 0) ? 1 : 0;
  p.ks = p.kpad ? WK + 4 : WK;
  const int vw = 1 << p.kclass;
  const int units = WK / vw;
  int clt_need = ((units + FCHUNKS - 1) / FCHUNKS) * vw;
  int clt = clt_need <= 4 ? 4 : clt_need <= 6 ? 6 : (clt_need == 7 && G == 4) ? 7 : 8;
  fast_kernel_t kern = pick_kernel(G, clt);
  if (!kern) return RAP_EUNSUPPORTED;
  p.WVP = (dv + 1) / 2;
  p.NG = FTHREADS / p.WVP;
  if (p.NG > FT) p.NG = FT;
  const int Gp = (G + 1) & ~1;
  p.IP = ((FT + p.NG - 1) / p.NG + 1) / 2;
  p.GS = round_up(p.IP * Gp * 2, 32) + 8;
  p.off_pp = 128 + FCHUNKS * G * FT * 4;
  p.off_alpha = p.off_pp + round_up(p.NG * p.GS * 4, 16);
  p.off_stage = round_up(p.off_alpha + 32, 128);
  p.v_off = round_up(FT * p.ks * 4, 128);
  p.stage_bytes = round_up(p.v_off + FT * dv * 2, 128);
  p.NS = (SMEM_BUDGET - p.off_stage) / p.stage_bytes;
  if (p.NS > 4) p.NS = 4;
  if (p.NS < 2) return RAP_EUNSUPPORTED;
  const size_t smem = (size_t)p.off_stage + (size_t)p.NS * p.stage_bytes;

  // split count: fill two CTAs per SM a whole number of times, splits of at least 8 tiles
  int n_split = n_split_req;
  if (n_split <= 0) {
    const long units_total = (long)a.B * a.Hkv;
    const int n_tiles = (a.h_len_max + FT - 1) / FT;
    const long slots = 2L * ctx->sm_count;
    double best = 1e30;
    n_split = 1;
    for (int ns = 1; ns <= RAP_MAX_SPLIT; ++ns) {
      const int tiles_per = (n_tiles + ns - 1) / ns;
      if (ns > 1 && tiles_per < 8) break;
      const long waves = (units_total * ns + slots - 1) / slots;
      const double cost = (double)waves * (tiles_per + 3);
      if (cost < best - 1e-9) { best = cost; n_split = ns; }
    }
  }
  p.q = (const uint32_t*)a.q; p.k = (const unsigned char*)a.k; p.v = (const unsigned char*)a.v;
  p.seq_len = a.seq_len; p.ws = ctx->d_attn_ws; p.status = ctx->d_status;
  p.len_add = a.len_add; p.Hq = a.Hq; p.Hkv = a.Hkv; p.WK = WK; p.dv = dv; p.S_cap = a.S_cap; p.n_split = n_split;
  p.qscale = (float)(1.4426950408889634 / sqrt((double)a.head_dim));
  RAP_CUDA_TRY(ctx, rap_raise_smem(ctx, kern, SMEM_BUDGET));
  dim3 grid(n_split, a.Hkv, a.B);
  kern<<<grid, FTHREADS, smem, st>>>(p);
  ctx->launches++;
  RAP_CUDA_TRY(ctx, cudaGetLastError());
  attn_combine_fast_kernel<<<a.B * a.Hq, 128, 0, st>>>(ctx->d_attn_ws, n_split, dv, a.out);
  ctx->launches++;
  RAP_CUDA_TRY(ctx, cudaGetLastError());
  return RAP_OK;
}
