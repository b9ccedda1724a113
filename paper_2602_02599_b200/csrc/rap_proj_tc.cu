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
// A reduction split (grid.z) lets a decode-sized call use every SM; the RoPE / append epilogue
// kernel sums the splits.  Every mbarrier wait is bounded; a wait that gives up records
// RAP_ETIMEOUT in the device status word and the CTA winds down.
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
};

__device__ __forceinline__ void tc_mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

// Persistent: CTA c takes work items c, c + gridDim.x, ...  The stage ring runs on across items, and the
// accumulator is double buffered in tensor memory (2 x TN columns) so that the epilogue of one item
// overlaps the MMAs of the next.
template <int TN>
__global__ void __launch_bounds__(TC_THREADS, 1)
proj_tc_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_x, const TcParams p) {
  using C = TcCfg<TN>;
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
      for (int w = blockIdx.x; w < p.n_work && !timed_out; w += gridDim.x) {
        int n0, t0, ks, kb0, nkb;
        decode(w, n0, t0, ks, kb0, nkb);
        for (int kb = 0; kb < nkb; ++kb, ++kbg) {
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
        uint32_t r[32];
        if (nkb > 0 && ready) {
          tc_ld32(tmem_d + buf * TN + ((uint32_t)(quarter * 32) << 16) + (uint32_t)c0, r);
          asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        } else {
#pragma unroll
          for (int j = 0; j < 32; ++j) r[j] = 0u;
        }
        if (n < p.n_out) {
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const int t = t0 + c0 + j;
            if (t < p.T) ybase[(size_t)t * p.n_out + n] = __uint_as_float(r[j]);
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

template <int TN>
rap_status launch_tc(rap_ctx* ctx, const CUtensorMap& mw, const CUtensorMap& mx, const TcParams& p, dim3 grid,
                     cudaStream_t st) {
  RAP_CUDA_TRY(ctx, rap_raise_smem(ctx, proj_tc_kernel<TN>, TcCfg<TN>::SMEM));
  proj_tc_kernel<TN><<<grid, TC_THREADS, TcCfg<TN>::SMEM, st>>>(mw, mx, p);
  ctx->launches++;
  RAP_CUDA_TRY(ctx, cudaGetLastError());
  return RAP_OK;
}

}  // namespace

bool rap_tensor_map_bf16(rap_ctx* ctx, void* map128, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  return make_map(ctx, reinterpret_cast<CUtensorMap*>(map128), base, rows, cols, box_rows);
}

// Y[ks][T][N] (fp32, context workspace) = X[T][K] * W[N][K]^T, bf16 operands, K split over grid.z.
rap_status rap_launch_gemm_tc(rap_ctx* ctx, const void* x, const void* w, int T, int K, int N, int* ksplit_out,
                              cudaStream_t st) {
  if (T < 1 || (K % 8) != 0) return RAP_EUNSUPPORTED;     // tensor-map rows must be multiples of 16 bytes
  const int tn = T <= 32 ? 32 : T <= 64 ? 64 : T <= 128 ? 128 : 256;
  CUtensorMap mw, mx;
  if (!make_map(ctx, &mw, w, (uint64_t)N, (uint64_t)K, TC_BM)) return RAP_EUNSUPPORTED;
  if (!make_map(ctx, &mx, x, (uint64_t)T, (uint64_t)K, (uint32_t)tn)) return RAP_EUNSUPPORTED;
  const int row_tiles = (N + TC_BM - 1) / TC_BM, tok_tiles = (T + tn - 1) / tn;
  const int nkb = (K + TC_BK - 1) / TC_BK;
  // reduction split: enough CTAs for every SM on decode-sized calls, within the workspace
  int ksplit = ctx->sm_count / (row_tiles * tok_tiles);
  if (ksplit > RAP_MAX_KSPLIT) ksplit = RAP_MAX_KSPLIT;
  if (ksplit > nkb / 4) ksplit = nkb / 4;
  while (ksplit > 1 && (size_t)ksplit * T * N * sizeof(float) > ctx->proj_ws_bytes) --ksplit;
  if (ksplit < 1) ksplit = 1;
  int per = (nkb + ksplit - 1) / ksplit;
  ksplit = (nkb + per - 1) / per;          // no empty split
  if ((size_t)ksplit * T * N * sizeof(float) > ctx->proj_ws_bytes) return RAP_EUNSUPPORTED;
  TcParams p;
  p.y = ctx->d_proj_ws; p.status = ctx->d_status; p.T = T; p.n_out = N; p.nkb_total = nkb; p.nkb_per_split = per;
  p.row_tiles = row_tiles; p.tok_tiles = tok_tiles; p.n_work = row_tiles * tok_tiles * ksplit;
  dim3 grid(p.n_work < ctx->sm_count ? p.n_work : ctx->sm_count, 1, 1);
  *ksplit_out = ksplit;
  switch (tn) {
    case 32: return launch_tc<32>(ctx, mw, mx, p, grid, st);
    case 64: return launch_tc<64>(ctx, mw, mx, p, grid, st);
    case 128: return launch_tc<128>(ctx, mw, mx, p, grid, st);
    default: return launch_tc<256>(ctx, mw, mx, p, grid, st);
  }
}

rap_status rap_launch_proj_tc(rap_ctx* ctx, const rap_proj_args& a, int* ksplit_out, cudaStream_t st) {
  if (a.dtype != RAP_BF16) return RAP_EUNSUPPORTED;
  const int n_out = (a.Hq + a.Hkv) * a.P2 + a.Hkv * a.dv;
  return rap_launch_gemm_tc(ctx, a.x, a.w, a.T, a.hidden, n_out, ksplit_out, st);
}
