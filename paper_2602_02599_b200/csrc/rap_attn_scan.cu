// Launch side of the shape-specialised split-KV scans: kernel lookup by head shape, the balanced /
// equal-split launch and the combine kernel of the equal-split mode.  The kernel templates live in
// rap_attn_scan_kernel.cuh (FP32 pipes) and rap_attn_mma_kernel.cuh (mma.sync); their instantiations (one
// per supported (G, P, d_v')) are generated into several translation units at build time (build.py) and
// found through rap_scan_find / rap_mma_find.
#include "rap_attn_common.cuh"

namespace {

// out[b][g][c] = sum_s 2^(m_s - M) acc_s[c] / sum_s 2^(m_s - M) l_s ; empty splits have l = 0.
// Balanced mode (seq_len != nullptr): the unit's segment count follows from the same plan the scan used.
__global__ void __launch_bounds__(128) attn_scan_combine_kernel(const float* __restrict__ ws, int n_split, int dv,
                                                                float* __restrict__ out,
                                                                const int32_t* __restrict__ seq_len, int B, int Hq,
                                                                int Hkv, int len_add, int S_cap, int tile_rows,
                                                                int scan_grid) {
  const size_t bg = blockIdx.x;
  int stride = n_split;
  if (seq_len != nullptr) {
    const int b = (int)(bg / Hq), h = (int)(bg % Hq) / (Hq / Hkv);
    const SkPlan pl = sk_plan(seq_len, B, Hkv, len_add, S_cap, tile_rows, scan_grid);
    int pb = 0;
    for (int bb = 0; bb < b; ++bb) pb += sk_tiles_of(seq_len, bb, len_add, S_cap, tile_rows) * Hkv;
    const int n = sk_tiles_of(seq_len, b, len_add, S_cap, tile_rows);
    const int start = pb + h * n;
    n_split = n > 0 ? sk_cta_of(start + n - 1, pl) - sk_cta_of(start, pl) + 1 : 0;
    stride = RAP_MAX_SPLIT;
  }
  const float* base = ws + bg * stride * (size_t)(dv + 2);
  __shared__ float wgt[RAP_MAX_SPLIT];
  __shared__ float inv_s;
  if (threadIdx.x < 32) {
    float M = -INFINITY;
    for (int s = threadIdx.x; s < n_split; s += 32)
      if (base[(size_t)s * (dv + 2) + dv + 1] > 0.f) M = fmaxf(M, base[(size_t)s * (dv + 2) + dv]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
    float den = 0.f;
    for (int s = threadIdx.x; s < n_split; s += 32) {
      const float l = base[(size_t)s * (dv + 2) + dv + 1];
      const float w = l > 0.f ? exp2f(base[(size_t)s * (dv + 2) + dv] - M) : 0.f;
      wgt[s] = w;
      den += w * l;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) den += __shfl_xor_sync(0xffffffffu, den, o);
    if (threadIdx.x == 0) inv_s = den > 0.f ? 1.f / den : 0.f;
  }
  __syncthreads();
  const float inv = inv_s;
  for (int c = threadIdx.x; c < dv; c += blockDim.x) {
    float num = 0.f;
    for (int s = 0; s < n_split; ++s) {
      const float w = wgt[s];
      if (w > 0.f) num += w * base[(size_t)s * (dv + 2) + c];
    }
    out[bg * dv + c] = num * inv;
  }
}

}  // namespace

static rap_status launch_split_kv(rap_ctx* ctx, const rap_attn_args& a, int n_split_req, cudaStream_t st,
                                  const rap_scan_entry* e, bool is_mma) {
  // n_split = 0: balanced mode, one CTA per resident slot; an explicit n_split keeps equal ranges per split
  const bool balanced = n_split_req <= 0 && (long long)a.B * a.Hkv * ((a.S_cap + 63) / 64) < (1LL << 31);
  int n_split = balanced ? RAP_MAX_SPLIT : n_split_req;
  if (n_split <= 0) {   // (only for tile counts beyond 2^31) equal ranges, a few waves of CTAs
    n_split = (8 * ctx->sm_count + a.B * a.Hkv - 1) / (a.B * a.Hkv);
    n_split = n_split > RAP_MAX_SPLIT ? RAP_MAX_SPLIT : n_split < 1 ? 1 : n_split;
  }
  ScanParams p;
  p.q = (const uint32_t*)a.q; p.k = (const unsigned char*)a.k; p.v = (const unsigned char*)a.v;
  p.seq_len = a.seq_len; p.ws = ctx->d_attn_ws; p.status = ctx->d_status;
  p.ws_floats = (long long)(ctx->attn_ws_bytes / sizeof(float));
  if (ctx->dbg_ws_floats > 0) {      // test hook: understate the workspace (it is as large as ever), see rap_debug.h
    p.ws_floats = ctx->dbg_ws_floats;
    ctx->dbg_ws_floats = 0;
  }
  p.len_add = a.len_add; p.Hq = a.Hq; p.Hkv = a.Hkv; p.S_cap = a.S_cap; p.n_split = n_split;
  p.qscale = (float)(1.4426950408889634 / sqrt((double)a.head_dim));
  p.B = a.B; p.balanced = balanced ? 1 : 0;
  {   // two counter sets take turns; each launch clears the one its predecessor used
    const size_t n_units = (size_t)ctx->desc.max_batch * ctx->desc.n_kv_heads;
    const uint32_t set = balanced ? (ctx->scan_epoch++ & 1u) : 0u;
    p.unit_cnt = ctx->d_unit_cnt + set * n_units;
    p.unit_cnt_other = ctx->d_unit_cnt + (set ^ 1u) * n_units;
    p.dyn_next = ctx->d_unit_cnt + 2 * n_units + set;
    p.dyn_next_other = ctx->d_unit_cnt + 2 * n_units + (set ^ 1u);
  }
  // Long launches of the tensor-core form: the CTAs do not stream at the same pace (the memory system shares its
  // bandwidth unevenly), so the last tenth of the tiles is not assigned up front but claimed piece by piece by
  // whoever is done.  A piece costs a pipeline refill and a partial, so short launches (under ~100 tiles per CTA)
  // keep the fixed split -- and the kernel without that logic, which starts and ends a microsecond or two sooner; a
  // piece is long enough that no unit gets more than ~24 of them.  (Measured on the quantised cache: no gain, a
  // piece's overhead weighs twice as much there.)
  p.dyn_piece = 0;
  p.dyn_frac_x256 = 0;
  p.dyn_guard = 0;
  const void* fn = e->fn;
  if (balanced && is_mma && e->fn_dyn) {
    const long long unit_tiles = (a.h_len_max + e->tile - 1) / e->tile;
    const long long per_cta = (long long)a.B * a.Hkv * unit_tiles / (2 * ctx->sm_count);
    if (ctx->dbg_dyn_piece >= 0) {
      p.dyn_piece = ctx->dbg_dyn_piece;
      p.dyn_frac_x256 = ctx->dbg_dyn_frac;
    } else if (per_cta >= 96) {
      p.dyn_piece = (int)(unit_tiles / 24 > 16 ? unit_tiles / 24 : 16);
      p.dyn_frac_x256 = 26;
      p.dyn_guard = 1;
    }
    if (p.dyn_piece > 0 && p.dyn_frac_x256 > 0) fn = e->fn_dyn;
  }
  p.out = a.out;
  p.wait_limit = WAIT_LIMIT;
  p.dbg_skip_copy = 0;
  if (ctx->dbg_arm_timeout && !e->tma && is_mma) {
    // test hook (rap_debug_arm_wait_timeout): one stage of this launch is armed without a copy and polled a few
    // thousand times only, so the launch reports RAP_ETIMEOUT and leaves its units unfinished
    p.wait_limit = 4096;
    p.dbg_skip_copy = 1;
    ctx->dbg_arm_timeout = 0;
  }
  RAP_CUDA_TRY(ctx, rap_raise_smem(ctx, fn, e->smem));
  const int scan_grid = 2 * ctx->sm_count;
  dim3 grid(n_split, a.Hkv, a.B);
  if (balanced) grid = dim3(scan_grid, 1, 1);
  alignas(64) unsigned char map_k[128] = {0}, map_v[128] = {0};   // CUtensorMap images (kernels without maps ignore them)
  if (e->tma) {
    const uint64_t rows = (uint64_t)a.B * a.Hkv * a.S_cap;
    if (!rap_tensor_map_bf16(ctx, map_k, a.k, rows, (uint64_t)a.P2, 32) ||
        !rap_tensor_map_bf16(ctx, map_v, a.v, rows, (uint64_t)a.dv, 32))
      return RAP_EUNSUPPORTED;
  }
  void* args[] = {&p, map_k, map_v};
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(e->threads);
  cfg.dynamicSmemBytes = (size_t)e->smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = a.pdl ? 1 : 0;      // the kernel waits for its predecessor before it reads q~ or a cache row
  RAP_CUDA_TRY(ctx, cudaLaunchKernelExC(&cfg, fn, args));
  ctx->launches++;
  RAP_CUDA_TRY(ctx, cudaGetLastError());
  if (balanced) {
    return RAP_OK;   // merged inside the scan kernel
  }
  attn_scan_combine_kernel<<<a.B * a.Hq, 128, 0, st>>>(ctx->d_attn_ws, n_split, a.dv, a.out, nullptr, a.B, a.Hq, a.Hkv,
                                                       a.len_add, a.S_cap, e->tile, scan_grid);
  ctx->launches++;
  RAP_CUDA_TRY(ctx, cudaGetLastError());
  return RAP_OK;
}

rap_status rap_launch_attn_scan(rap_ctx* ctx, const rap_attn_args& a, int n_split_req, cudaStream_t st) {
  if (a.dtype != RAP_BF16 || (a.P2 & 1)) return RAP_EUNSUPPORTED;
  const rap_scan_entry* e = rap_scan_find(a.Hq / a.Hkv, a.P2 / 2, a.dv);
  return e ? launch_split_kv(ctx, a, n_split_req, st, e, false) : RAP_EUNSUPPORTED;
}

rap_status rap_launch_attn_mma(rap_ctx* ctx, const rap_attn_args& a, int n_split_req, cudaStream_t st) {
  if (a.dtype != RAP_BF16 || (a.P2 & 1)) return RAP_EUNSUPPORTED;
  const rap_scan_entry* e = rap_mma_find(a.Hq / a.Hkv, a.P2 / 2, a.dv);
  return e ? launch_split_kv(ctx, a, n_split_req, st, e, true) : RAP_EUNSUPPORTED;
}

// a.k / a.v are quantised caches (rap_q8.cu); same plan, workspace and merge as the other two scans
rap_status rap_launch_attn_q8_mma(rap_ctx* ctx, const rap_attn_args& a, int n_split_req, cudaStream_t st) {
  if (a.dtype != RAP_BF16 || (a.P2 & 1)) return RAP_EUNSUPPORTED;
  const rap_scan_entry* e = rap_q8_find(a.Hq / a.Hkv, a.P2 / 2, a.dv);
  return e ? launch_split_kv(ctx, a, n_split_req, st, e, false) : RAP_EUNSUPPORTED;
}
