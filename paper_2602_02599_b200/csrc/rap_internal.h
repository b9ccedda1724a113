// Internal declarations shared by the translation units of the RAP decode library.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include <set>
#include <string>
#include <vector>

#include "rap.h"
#include "rap_debug.h"

#define RAP_MAX_SPLIT 64     // upper bound on sequence splits of the attention scan
#define RAP_MAX_GROUP 8      // largest G = H_q / H_kv
#define RAP_MAX_KSPLIT 8     // upper bound on reduction splits of the projection

struct rap_ctx {
  rap_model_desc desc;
  int device = 0;
  int sm_count = 0;
  bool tables_built = false;
  std::vector<int32_t> n_pairs;   // P_l
  std::vector<int32_t> n_vch;     // d_v'_l
  // library-owned device memory
  int32_t* d_status = nullptr;    // [2] = {code, detail}
  float* d_attn_ws = nullptr;     // split-KV partials
  size_t attn_ws_bytes = 0;
  int32_t* d_unit_cnt = nullptr;  // [2][max_batch][H_kv] partial-arrival counters of the balanced scan (zero between calls)
  uint32_t scan_epoch = 0;        // balanced scans launched so far: picks the counter set
  float* d_proj_ws = nullptr;     // fp32 projection results / split-K partials
  size_t proj_ws_bytes = 0;
  int32_t* d_proj_cnt = nullptr;  // fused projection: two sets of [row tiles][4] split-arrival counters (zero between calls)
  int proj_cnt_n = 0;             // counters per set
  uint32_t proj_epoch = 0;        // launches of the fused projection so far: picks the set
  void* d_stage_x = nullptr;      // staging for rap_decode_step_host
  float* d_stage_out = nullptr;
  void* d_stage_q = nullptr;
  void* d_oproj_x = nullptr;      // rap_out_proj: attention output rounded to the storage dtype
  void* d_pf_v = nullptr;         // prefill attention, odd d_v': V rows copied to an even row length (grown on demand)
  size_t pf_v_bytes = 0;
  void* d_lr_k = nullptr;         // low-rank comparator: rebuilt, rotated full-width K (grown on demand)
  size_t lr_k_bytes = 0;
  void* d_lr_cs = nullptr;        // low-rank comparator: (cos, sin) table [positions][D/2]
  size_t lr_cs_bytes = 0;
  int lr_cs_len = 0;              // positions the table currently covers
  size_t stage_x_bytes = 0, stage_out_bytes = 0;
  void* copy_in = nullptr;        // rap_decode_step_host: stream of the input copies behind layer 0's (cudaStream_t)
  void* copy_out = nullptr;       // rap_decode_step_host: stream of the early output copies
  void* ev_in = nullptr;          // the inputs of layers >= 1 have arrived (cudaEvent_t)
  void* ev_mid = nullptr;         // the layers before a cut have run
  // pinned host staging for rap_build_tables
  void* h_tables = nullptr;
  size_t h_tables_bytes = 0;
  void* tables_stream = nullptr;
  bool tables_inflight = false;
  // optional timing of the attention launches of rap_decode_step (event pairs on the caller's stream)
  std::vector<cudaEvent_t> prof_ev;   // 2 * capacity events
  int prof_pairs = 0;                 // pairs recorded since the last read
  std::set<const void*> attr_done;    // kernels whose dynamic shared-memory limit has been raised on this device
  struct MapSlot { const void* base; uint64_t rows, cols; uint32_t box; unsigned char map[128]; };
  std::vector<MapSlot> tmaps;         // encoded tensor maps, reused while (pointer, shape, box) repeat
  size_t tmap_next = 0;
  int32_t attn_variant = 0;
  long long dbg_ws_floats = 0;    // > 0: the next scan launch is told its workspace holds only this many floats (rap_debug.h)
  int32_t dbg_dyn_piece = -1, dbg_dyn_frac = 0;   // test hook: pieces claimed at run time, forced (-1: the launcher decides; rap_debug.h)
  int32_t dbg_arm_timeout = 0;    // the next tensor-core scan launch runs into a bounded wait on purpose (rap_debug.h)
  int32_t proj_variant = 0;       // 1: rap_qkv_rope_append always takes the two-stage path (GEMM, then the epilogue kernel)
  int64_t launches = 0;
  std::string cuda_error;
  // lazily created tensor maps / per-device attributes live in the .cu files
  bool smem_attr_set = false;
};

// cudaFuncSetAttribute(MaxDynamicSharedMemorySize) once per kernel and context
template <typename F>
static inline cudaError_t rap_raise_smem(rap_ctx* ctx, F fn, int bytes) {
  if (!ctx->attr_done.insert((const void*)fn).second) return cudaSuccess;
  return cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
}

// Index checks of the bounds-checking build (-DRAP_DEBUG_BOUNDS, a second library next to the normal one): RAP_BOUNDS(i,
// n, status, tag) is true when 0 <= i < n; otherwise it records RAP_EBOUNDS with `tag` in the device status word (the
// first failure wins) and the caller skips the access.  In the normal build it is the constant true and costs nothing.
#ifdef RAP_DEBUG_BOUNDS
#ifdef __CUDACC__
__device__ __forceinline__ bool rap_in_bounds(long long i, long long n, int32_t* status, int tag) {
  if (i >= 0 && i < n) return true;
  if (atomicCAS(&status[0], 0, (int)RAP_EBOUNDS) == 0) status[1] = tag;
  return false;
}
#endif
#define RAP_BOUNDS(i, n, status, tag) rap_in_bounds((long long)(i), (long long)(n), (status), (tag))
#else
#define RAP_BOUNDS(i, n, status, tag) true
#endif

static inline int rap_elem_bytes(int32_t dtype) { return dtype == RAP_F32 ? 4 : 2; }
static inline bool rap_aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

#define RAP_CUDA_TRY(ctx, expr)                                         \
  do {                                                                  \
    cudaError_t _e = (expr);                                            \
    if (_e != cudaSuccess) {                                            \
      (ctx)->cuda_error = std::string(#expr) + ": " + cudaGetErrorString(_e); \
      return RAP_ECUDA;                                                 \
    }                                                                   \
  } while (0)

// Parameters and lookup entry of the shape-specialised split-KV scan (rap_attn_scan_kernel.cuh).
struct rap_scan_params {
  const uint32_t* q;          // [B][Hq][WK] bf16 pairs
  const unsigned char* k;     // [B][Hkv][S_cap][WK * 4 bytes]
  const unsigned char* v;     // [B][Hkv][S_cap][DV * 2 bytes]
  const int32_t* seq_len;
  float* ws;
  long long ws_floats; // size of ws (used by the index checks of the bounds-checking build)
  int32_t* status;
  int len_add, Hq, Hkv, S_cap, n_split;
  float qscale;
  int32_t* unit_cnt;   // balanced mode: arrivals per (sequence, KV head) unit, zero between calls
  int32_t* unit_cnt_other;   // the set the previous launch used; cleared by this launch (two sets take turns)
  float* out;          // balanced mode: [B][Hq][DV], written by the CTA that completes a unit
  uint32_t wait_limit; // probes of a stage barrier before a warp gives up (RAP_ETIMEOUT)
  int dbg_skip_copy;   // test hook: the first warp of the first CTA arms its first stage and issues no copy for it
  int B;               // sequences (used by the balanced mode)
  int balanced;        // 0: grid (n_split, H_kv, B), equal tile ranges per split; 1: grid (CTAs), see SkPlan
  // Balanced mode, tensor-core form: the last tiles of the tile sequence are not assigned up front but cut into pieces
  // of dyn_piece tiles that the CTAs claim from a counter as they finish (0: everything is assigned up front)
  int dyn_piece;       // tiles per piece
  int dyn_frac_x256;   // share of all tiles handed out that way, in 256ths
  int dyn_guard;       // 1: the kernel drops the pieces when they turn out large against a CTA's own part (automatic mode)
  int32_t* dyn_next;   // next unclaimed piece of this launch (zero on entry)
  int32_t* dyn_next_other;   // the counter the previous launch used; cleared by this launch
};
struct rap_scan_entry {
  int G, WK, DV;       // query heads per KV head, K words per row (= P), V channels (= d_v')
  int smem, tile;      // dynamic shared memory, positions per tile
  int threads;         // CTA size
  int tma;             // 1: the kernel takes tensor maps of the K and V caches (boxes of 32 rows x 64 elements)
  const void* fn;      // the kernel, launched with cudaLaunchKernel
  const void* fn_dyn;  // tensor-core scan only: the instantiation that can hand tiles out at run time, or nullptr
};
// the instantiation built for this head shape, or nullptr (generated at build time):
// the FP32-pipe scan (rap_attn_scan_kernel.cuh) and the mma.sync scan (rap_attn_mma_kernel.cuh)
const rap_scan_entry* rap_scan_find(int G, int WK, int DV);
const rap_scan_entry* rap_mma_find(int G, int WK, int DV);
const rap_scan_entry* rap_q8_find(int G, int WK, int DV);      // the scan over an 8-bit quantised cache (rap_attn_q8_kernel.cuh)
// Tensor map over a row-major [rows][cols] bf16 matrix, boxes of box_rows x 64 elements, 128-byte swizzle,
// zero fill outside; cached in the context by (pointer, shape, box).  map128 receives the 128-byte CUtensorMap.
bool rap_tensor_map_bf16(rap_ctx* ctx, void* map128, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows);

// Launchers implemented in the kernel files.  All return RAP_OK or RAP_ECUDA.
struct rap_attn_args {
  const void* q; const void* k; const void* v;
  const int32_t* seq_len; int32_t len_add;      // effective length = seq_len[b] + len_add
  int32_t B, Hq, Hkv, P2, dv, S_cap, head_dim, dtype;
  int32_t n_split, h_len_max;
  float* out;
  int32_t pdl = 0;          // launch the scan with programmatic stream serialization (inside rap_decode_step)
};
rap_status rap_launch_attn(rap_ctx* ctx, const rap_attn_args& a, cudaStream_t st);

struct rap_proj_args {
  const void* x; const void* w; const void* bias;
  const int32_t* seq_id; const int32_t* pos; const int32_t* slot;   // seq_id/slot NULL => decode mode
  const double* inv_freq;   // this layer's [H_kv][D/2]
  void* q_out; void* k_cache; void* v_cache;
  int32_t T, hidden, Hq, Hkv, P2, dv, half_dim, B_cache, S_cap, dtype;
  int32_t pdl = 0;          // launch with programmatic stream serialization (inside rap_decode_step, after an attention launch)
};
rap_status rap_launch_qkv_rope_append(rap_ctx* ctx, const rap_proj_args& a, cudaStream_t st);

struct rap_lowrank_args {
  const void* q_full; const void* k_latent; const void* bk; const void* v;
  const int32_t* seq_len; int32_t B, Hq, Hkv, r, dv, S_cap, head_dim, dtype, pairing;
  double rope_theta; int32_t n_split, h_len_max; float* out;
};
rap_status rap_launch_lowrank_attn(rap_ctx* ctx, const rap_lowrank_args& a, cudaStream_t st);

rap_status rap_launch_pack(rap_ctx* ctx, int32_t layer, const void* wq, const void* wk, const void* wv,
                           const int32_t* k_dim_idx, const int32_t* v_idx, void* w_qkv,
                           const void* bq, const void* bk, const void* bv, void* bias, cudaStream_t st);
rap_status rap_launch_advance(rap_ctx* ctx, int32_t* seq_len, int32_t B, cudaStream_t st);
rap_status rap_launch_prefill_attn(rap_ctx* ctx, int B, int T, const void* q, const void* k, const void* v, int P2,
                                   int dv, int S_cap, const int32_t* start, float* out, cudaStream_t st);
rap_status rap_launch_pack_wo(rap_ctx* ctx, int32_t layer, const void* wo, const int32_t* v_idx, void* dst, cudaStream_t st);
rap_status rap_launch_out_proj(rap_ctx* ctx, int32_t layer, int32_t T, const float* attn_out, const void* wo_tilde,
                               void* y, cudaStream_t st);

// 8-bit cache quantisation (rap_q8.cu, rap_attn_q8.cu)
rap_status rap_launch_quantize_rows(rap_ctx* ctx, int32_t dtype_in, long long n_rows, int W, const void* src, void* dst,
                                    cudaStream_t st);
rap_status rap_launch_qkv_rope_append_q8(rap_ctx* ctx, const rap_proj_args& a, cudaStream_t st);
rap_status rap_launch_attn_q8(rap_ctx* ctx, const rap_attn_args& a, cudaStream_t st);
