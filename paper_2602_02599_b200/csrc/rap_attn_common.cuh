// Pieces shared by the split-KV decode kernels: the balanced work plan (which CTA scans which tiles of
// which (sequence, KV head) unit), bounded mbarrier waits and the bulk global -> shared copy.
#pragma once
#include <math.h>

#include "rap_internal.h"

namespace {

constexpr uint32_t WAIT_LIMIT = 1u << 21;
constexpr int SMEM_BUDGET = 115712;   // dynamic shared memory per CTA with two CTAs per SM

constexpr int cround(int x, int m) { return (x + m - 1) / m * m; }

using ScanParams = rap_scan_params;

// Balanced mode.  All tiles of all (sequence, KV head) units form one sequence, unit-major, of T
// tiles; CTA c of NC scans the tiles [c T / NC, (c + 1) T / NC), whatever units they belong to, so
// every CTA does the same amount of work for any batch, length mix and SM count.  A unit touched by
// several CTAs gets one partial per CTA ("segment"); segment index = CTA - first CTA of the unit.
// NC is capped so that no unit has more than RAP_MAX_SPLIT segments.  The scan and the combine
// kernel derive the same plan from seq_len with the helpers below.
struct SkPlan {
  int T;           // total tiles (the host side keeps B * H_kv * S_cap / 64 below 2^31)
  int nc;          // CTAs that take part (<= gridDim.x)
};
__device__ __forceinline__ int sk_tiles_of(const int32_t* seq_len, int b, int len_add, int S_cap, int tile_rows) {
  const int len = min(max(seq_len[b] + len_add, 0), S_cap);
  return (len + tile_rows - 1) / tile_rows;
}
__device__ __forceinline__ SkPlan sk_plan(const int32_t* seq_len, int B, int Hkv, int len_add, int S_cap, int tile_rows,
                                          int grid) {
  long long T = 0;
  int n_max = 0;
  for (int b = 0; b < B; ++b) {
    const int n = sk_tiles_of(seq_len, b, len_add, S_cap, tile_rows);
    T += (long long)n * Hkv;
    n_max = max(n_max, n);
  }
  SkPlan pl;
  pl.T = (int)T;
  pl.nc = 0;
  if (T > 0) {
    const long long cap = (long long)(RAP_MAX_SPLIT - 2) * T / n_max;     // segments per unit <= n_max NC / T + 2
    pl.nc = (int)max(1LL, min(min((long long)grid, cap), T));             // and every CTA owns at least one tile
  }
  return pl;
}
// The same plan, computed once per CTA by its first warp instead of by every thread: the inclusive prefix of the
// tiles of sequences 0..b (all KV heads) goes to `pref` (shared memory, room for `cap` ints, B <= cap - 2 or the
// function returns false and leaves everything to sk_plan), the total and the longest sequence to its last two
// slots.  Every thread of the CTA must call it; pref[0..B) stays valid until the caller reuses the memory.
__device__ __forceinline__ bool sk_plan_shared(const int32_t* seq_len, int B, int Hkv, int len_add, int S_cap, int tile_rows,
                                               int grid, int* pref, int cap, SkPlan* out) {
  if (B > cap - 2) return false;
  const int tid = threadIdx.x, lane = tid & 31;
  if (tid < 32) {
    int carry = 0, n_max = 0;
    for (int base = 0; base < B; base += 32) {
      const int bb = base + lane;
      const int n = bb < B ? sk_tiles_of(seq_len, bb, len_add, S_cap, tile_rows) : 0;
      n_max = max(n_max, n);
      int x = n * Hkv;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int y = __shfl_up_sync(0xffffffffu, x, o);
        if (lane >= o) x += y;
      }
      if (bb < B) pref[bb] = carry + x;
      carry += __shfl_sync(0xffffffffu, x, 31);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) n_max = max(n_max, __shfl_xor_sync(0xffffffffu, n_max, o));
    if (lane == 0) {
      pref[cap - 2] = carry;
      pref[cap - 1] = n_max;
    }
  }
  __syncthreads();
  const long long T = pref[cap - 2];
  const int n_max = pref[cap - 1];
  out->T = (int)T;
  out->nc = 0;
  if (T > 0) {
    const long long lim = (long long)(RAP_MAX_SPLIT - 2) * T / n_max;
    out->nc = (int)max(1LL, min(min((long long)grid, lim), T));
  }
  return true;
}
// sequence that holds global tile `cur` (< total), given the inclusive prefix: smallest b with pref[b] > cur
__device__ __forceinline__ int sk_seq_of(const int* pref, int B, int cur) {
  int lo = 0, hi = B - 1;
  while (lo < hi) {
    const int mid = (lo + hi) >> 1;
    if (pref[mid] > cur) hi = mid; else lo = mid + 1;
  }
  return lo;
}
// first CTA whose range holds global tile s:  max c with floor(c T / NC) <= s
__device__ __forceinline__ int sk_cta_of(int s, const SkPlan& pl) { return (int)((((long long)s + 1) * pl.nc - 1) / pl.T); }

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

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
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, uint32_t limit) {
  for (uint32_t i = 0; i < limit; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}
// one probe that never parks the thread (try_wait may, and then costs a few hundred cycles even when the phase is over)
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// the copy is normally ahead of the math: one probe, and the bounded polling loop out of line
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, uint32_t limit = WAIT_LIMIT) {
  if (mbar_test_wait(bar, parity)) return true;
  return mbar_wait_slow(bar, parity, limit);
}
// Programmatic dependent launch (no-ops in a kernel launched without the attribute): wait until the previous kernel
// in the stream has completed and its writes are visible; let the next kernel in the stream start its prologue.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// global -> this CTA's shared memory, completion counted in bytes on the mbarrier (no multicast)
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}

}  // namespace
