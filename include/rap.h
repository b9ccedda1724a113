/*
 * rap.h -- C ABI of the B200-native RAP (RoPE-Aligned Pruning) decode path.
 *
 * The library implements the online consequence of RAP: attention over a KV cache whose
 * K rows keep only whole retained RoPE pairs (2P dims) and whose V rows keep only
 * retained channels (d_v' dims); the pair selection E_k is fused offline into a shrunken
 * W~_q = W_q E_k^T, so no decode step ever rebuilds a full-width K (Section 4, Step 3;
 * Eq. 6, Eq. 7; Algorithm 1).
 *
 * Conventions
 *   - plain C; every entry point returns rap_status (0 = OK) and never throws, aborts or
 *     traps.  Arguments are validated on the host BEFORE anything is launched.
 *   - pointers named d_* are DEVICE pointers, h_* are HOST pointers; all are owned by the
 *     caller.  The library owns only what rap_create allocates (a device status word, the
 *     split-KV / projection workspace and the staging buffers of rap_decode_step_host),
 *     released by rap_destroy.
 *   - all GPU work is enqueued on the caller's stream (`stream` is a cudaStream_t passed as
 *     void*, NULL = the legacy default stream) and is asynchronous unless stated otherwise.
 *   - device buffers must be 16-byte aligned (RAP_EALIGN otherwise).
 *   - weights are stored [out][in] row-major, so y = W x.
 *   - notation: L layers, hidden = model width, H_q / H_kv query / KV heads, G = H_q/H_kv,
 *     D = original head_dim, P_l retained pairs and d_v'_l retained V channels of layer l,
 *     B batch, S_cap cache capacity in rows.
 *   - layouts are dense-packed, no padding:
 *       q~      [T][H_q][2P]                       (storage dtype)
 *       K cache [B][H_kv][S_cap][2P]   per layer   (storage dtype)
 *       V cache [B][H_kv][S_cap][d_v'] per layer   (storage dtype)
 *       out     [B][H_q][d_v']                     (fp32, reduced V coordinates)
 *     Reduced K/q dims are pair-interleaved: reduced dims (2c, 2c+1) are the two members of
 *     the c-th retained pair, pairs in ascending original index.
 */
#ifndef RAP_H_
#define RAP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  RAP_OK = 0,
  RAP_EINVAL = 1,       /* NULL required pointer, bad enum, value out of range          */
  RAP_ESHAPE = 2,       /* shape outside what the context was created for               */
  RAP_ECAPACITY = 3,    /* a cache slot / sequence length exceeds S_cap                 */
  RAP_EALIGN = 4,       /* device pointer not 16-byte aligned, or S_cap not multiple of 8 */
  RAP_EUNSUPPORTED = 5, /* valid request this build does not implement                  */
  RAP_ECUDA = 6,        /* a CUDA runtime call failed (see rap_last_cuda_error)          */
  RAP_ETIMEOUT = 7,     /* a bounded device-side wait gave up (device status word)      */
  RAP_ESTATE = 8,       /* call order: tables not built yet for this context            */
  RAP_EBOUNDS = 9       /* only from a library built with RAP_DEBUG_BOUNDS: a kernel's index check failed
                           (device status word; detail = which check); the access was skipped  */
} rap_status;

typedef enum { RAP_F32 = 0, RAP_BF16 = 1 } rap_dtype;

/* RoPE pairing of the model (Section 3): pair i = dims (i, i + D/2), or (2i, 2i + 1). */
typedef enum { RAP_PAIR_HALF = 0, RAP_PAIR_ADJACENT = 1 } rap_pairing;

typedef struct {
  int32_t n_layers, hidden, n_q_heads, n_kv_heads, head_dim; /* D even, H_q % H_kv == 0, G <= 8 */
  double rope_theta;                                         /* theta_base of Eq. 3           */
  int32_t pairing;                                           /* rap_pairing                   */
  int32_t dtype;                                             /* rap_dtype of X, W~, q~, caches */
  int32_t max_batch;                                         /* largest B of a decode call    */
  int32_t max_rows;                                          /* largest T of an append call   */
} rap_model_desc;

typedef struct rap_ctx rap_ctx;

/* Create / destroy a context.  rap_create validates the description, selects the current
 * device and allocates the library-owned device buffers (cudaMalloc).  RAP_EINVAL on a bad
 * description, RAP_ECUDA when no sm_100 device or an allocation fails. */
rap_status rap_create(const rap_model_desc* desc, rap_ctx** out);
rap_status rap_destroy(rap_ctx* ctx);

const char* rap_status_string(rap_status s);
/* Text of the last CUDA error seen by this context ("" if none). Host memory owned by ctx. */
const char* rap_last_cuda_error(const rap_ctx* ctx);

/* Per-head budget at retain ratio rho (Section 4.2 "Balanced K/V"; Table 13): whole pairs
 * P = floor(rho*D/2 + 1/2) and V channels d_v' = floor(rho*D + 1/2), rounded independently.
 * RAP_EINVAL unless 0 < rho <= 1 and D even. */
rap_status rap_retained_counts(double rho, int32_t head_dim, int32_t* n_pairs, int32_t* n_vch);

/* Budget-Alloc (Algorithm 2): layer-adaptive pair budgets m_l proportional to the layer score
 * sigma_l = mean over heads and pairs of h_k_pair_scores [L][H_kv][D/2] (HOST fp64, finite, non-negative), with
 * mean retain ratio rho; head-uniform inside a layer; V keeps 2 m_l channels (Balanced K/V).  The paper
 * does not fix the rounding: the integer total is round(rho * D/2 * L), layers whose proportional share
 * leaves [1, D/2] are pinned to the bound and the rest re-shared, shares are floored and the missing
 * units go to the largest fractional parts (ties: lower layer).  Host-only, no GPU work.  The results
 * feed rap_build_tables. */
rap_status rap_budget_alloc(int32_t n_layers, int32_t n_kv_heads, int32_t head_dim, const double* h_k_pair_scores,
                            double rho, int32_t* h_n_pairs, int32_t* h_n_vch);

/* Element offset of (b, h, pos, c) in a cache of row width W: ((b*H_kv + h)*S_cap + pos)*W + c. */
size_t rap_cache_elem_offset(int32_t n_kv_heads, int32_t S_cap, int32_t W, int32_t b, int32_t h,
                             int32_t pos, int32_t c);

/* ---- tables (Algorithm 2, selection step; Eq. 6 RAPIndex; Eq. 3 frequencies) --------
 * For every (layer l, KV head h): keep the n_pairs[l] RoPE pairs with the largest score and
 * the n_vch[l] V channels with the largest score (ties: lower index), each list ascending.
 *   h_k_pair_scores [L][H_kv][D/2], h_v_chan_scores [L][H_kv][D]  HOST fp64
 *   h_n_pairs[L] in [1, D/2], h_n_vch[L] in [1, D]                HOST
 * Outputs are DEVICE buffers with fixed strides (unused tail = -1 / 0.0):
 *   d_k_pair_idx int32 [L][H_kv][D/2]   retained original pair indices i_c
 *   d_k_dim_idx  int32 [L][H_kv][D]     RAPIndex: original in-head dim of reduced dim r
 *   d_v_idx      int32 [L][H_kv][D]     retained original V channels
 *   d_inv_freq   fp64  [L][H_kv][D/2]   theta^(-2 i_c / D): the ORIGINAL pair's frequency
 * The per-layer counts are recorded in the context and used by every later call.
 * Deterministic.  Work: host selection, then async copies on `stream` from context-owned
 * pinned memory (a later rap_build_tables on the same context first synchronizes `stream`). */
rap_status rap_build_tables(rap_ctx* ctx, const double* h_k_pair_scores, const double* h_v_chan_scores,
                            const int32_t* h_n_pairs, const int32_t* h_n_vch,
                            int32_t* d_k_pair_idx, int32_t* d_k_dim_idx, int32_t* d_v_idx,
                            double* d_inv_freq, void* stream);

/* Tables of a model whose RoPE does not use theta^(-2i/D): frequency-scaled variants (Section 4, "Practical
 * Considerations", "RoPE variants": they change the frequencies or their scaling but keep the 2x2 rotation
 * blocks, so the pair selection applies unchanged).  h_pair_freq [L][D/2] HOST fp64 (finite) is the model's own
 * frequency, in radians per position, of ORIGINAL pair i of layer l; retained pair c of (l, h) gets
 * d_inv_freq[l][h][c] = h_pair_freq[l][i_c] -- index-aware, as in rap_build_tables -- and the online path is the
 * same.  A variant that also rescales the rotated vectors by a constant (an attention temperature) folds that
 * constant into the rows of W~_q offline; it needs no table.  Everything else as rap_build_tables. */
rap_status rap_build_tables_freq(rap_ctx* ctx, const double* h_k_pair_scores, const double* h_v_chan_scores,
                                 const double* h_pair_freq, const int32_t* h_n_pairs, const int32_t* h_n_vch,
                                 int32_t* d_k_pair_idx, int32_t* d_k_dim_idx, int32_t* d_v_idx, double* d_inv_freq,
                                 void* stream);

/* Tables of a hybrid model (Section 4, "Hybrid compression"): RAP on the layers that use RoPE, plain
 * channel pruning of K on the layers that do not (h_rope_layer[l] == 0).  For such a layer K keeps the
 * 2 * h_n_pairs[l] channels with the largest h_k_chan_scores [L][H_kv][D] (ascending, no pair structure:
 * its d_k_pair_idx row stays -1) and its frequency row is zero, so the shared online path rotates by the
 * identity there.  Everything else as rap_build_tables. */
rap_status rap_build_tables_hybrid(rap_ctx* ctx, const double* h_k_pair_scores, const double* h_k_chan_scores,
                                   const double* h_v_chan_scores, const int32_t* h_rope_layer,
                                   const int32_t* h_n_pairs, const int32_t* h_n_vch, int32_t* d_k_pair_idx,
                                   int32_t* d_k_dim_idx, int32_t* d_v_idx, double* d_inv_freq, void* stream);

/* Tables of a model that rotates only the first h_rot_dims[l] dims of every head (appendix "RoPE in Recent Open
 * LLMs", partial rotary; Section 4, "Hybrid compression": RAP on the rotated dims, channel pruning on the rest).
 * Layer l with R = h_rot_dims[l] (even, 0..D): rotated pairs i = 0..R/2-1 have members (i, i + R/2) (or
 * (2i, 2i+1) with adjacent pairing) and frequency theta^(-2i/R); the h_n_rot_pairs[l] (0..R/2) best of them by
 * h_k_pair_scores[l][h][0..R/2) are kept.  Of the unrotated dims R..D-1 the 2 * (h_n_pairs[l] -
 * h_n_rot_pairs[l]) (at most D - R) best by h_k_chan_scores[l][h][R..D) are kept.  The reduced K row is
 * [kept pairs, members adjacent | kept channels ascending]; a slot that holds unrotated channels has
 * d_k_pair_idx = -1 and frequency zero, so the shared online path rotates it by the identity.  R = D gives
 * rap_build_tables, R = 0 a layer of rap_build_tables_hybrid without RoPE.  Everything else as rap_build_tables;
 * RAP_EINVAL for counts outside those ranges. */
rap_status rap_build_tables_partial(rap_ctx* ctx, const double* h_k_pair_scores, const double* h_k_chan_scores,
                                    const double* h_v_chan_scores, const int32_t* h_rot_dims,
                                    const int32_t* h_n_rot_pairs, const int32_t* h_n_pairs, const int32_t* h_n_vch,
                                    int32_t* d_k_pair_idx, int32_t* d_k_dim_idx, int32_t* d_v_idx,
                                    double* d_inv_freq, void* stream);

/* ---- offline weight gather (Algorithm 1: W~_k, W~_q = W_q E_k^T, W~_v) ----------------
 * Index selection, no arithmetic.  d_wq [H_q*D][hidden], d_wk / d_wv [H_kv*D][hidden] are the
 * dense weights of `layer`; d_w_qkv [N_out][hidden] receives the rows
 *   q head g: RAPIndex of KV head g/G (2P rows) | k head h: RAPIndex of h | v head h: v_idx of h,
 * N_out = (H_q + H_kv)*2P + H_kv*d_v'.  Optional bias vectors are gathered the same way
 * (d_bq/d_bk/d_bv -> d_bias [N_out]; pass NULL for all four when there is no bias). */
rap_status rap_pack_weights(rap_ctx* ctx, int32_t layer, const void* d_wq, const void* d_wk,
                            const void* d_wv, const int32_t* d_k_dim_idx, const int32_t* d_v_idx,
                            void* d_w_qkv, const void* d_bq, const void* d_bk, const void* d_bv,
                            void* d_bias, void* stream);

/* ---- pruned QKV projection + index-aware RoPE + append (Eq. 1, Eq. 3, Section 4) ---
 * T rows of hidden states.  Row r belongs to sequence d_seq_id[r] (0..B-1), sits at position
 * d_pos[r] and is written to cache row d_slot[r].  For every row:
 *   y = W~_qkv x (+ bias), fp32 accumulate;
 *   q~ and k~ pairs c rotate by the angle pos * inv_freq[l][h][c] (q head g uses KV head g/G);
 *   q~, k~, v~ are rounded once to the storage dtype; q~ -> d_q_out [T][H_q][2P],
 *   k~ -> K cache row (seq, h, slot), v~ -> V cache row (seq, h, slot).
 * d_bias may be NULL.  d_k_cache / d_v_cache are THIS layer's buffers with B_cache sequences.
 * h_slot_max: the caller's upper bound on every d_slot value (RAP_ECAPACITY if >= S_cap);
 * the kernel also skips, and records in the device status word, any row whose slot or
 * sequence id is out of range.  T <= max_rows. */
rap_status rap_qkv_rope_append(rap_ctx* ctx, int32_t layer, int32_t T, const void* d_x,
                               const void* d_w_qkv, const void* d_bias, const int32_t* d_seq_id,
                               const int32_t* d_pos, const int32_t* d_slot, int32_t h_slot_max,
                               const double* d_inv_freq, void* d_q_out, void* d_k_cache,
                               void* d_v_cache, int32_t B_cache, int32_t S_cap, void* stream);

/* ---- split-KV decode attention on the reduced dims (Eq. 2, Eq. 7, scale 1/sqrt(D)) ----
 * For each sequence b and query head g (KV head h = g/G):
 *   s_j = q~_g . K[b,h,j] / sqrt(D),  j in [0, d_seq_len[b]);  p = softmax(s);
 *   out[b,g,:] = sum_j p_j V[b,h,j,:].
 * d_seq_len[b] counts valid cache rows INCLUDING the row just appended (>= 1; a sequence
 * with length 0 produces zeros).  h_seq_len_max: caller's bound on d_seq_len (<= S_cap).
 * The scale uses the ORIGINAL head_dim.  n_split = 0 lets the library choose the number of
 * sequence splits; partial (max, sum, accumulator) triples live in the context workspace,
 * so two calls on the same context must not overlap on the GPU.  B <= max_batch. */
rap_status rap_decode_attn(rap_ctx* ctx, int32_t layer, int32_t B, const void* d_q,
                           const void* d_k_cache, const void* d_v_cache, int32_t S_cap,
                           const int32_t* d_seq_len, int32_t h_seq_len_max, int32_t n_split,
                           float* d_out, void* stream);

/* ---- composition with 8-bit cache quantisation (Introduction and Related Work: pruning the width of the cache and
 * lowering the bit-width of what is cached are orthogonal; the appendix on composing RAP with quantisation uses a
 * plain symmetric round-to-nearest quantiser).  The paper fixes no cache format; the reading taken here: every
 * compact cache row x of width W (W = 2P for K, d_v' for V) keeps int8 codes c_i in [-127, 127] and one scale
 *     s = bf16(max_i |x_i| / 127),   c_i = clip(rint(x_i / s), -127, 127),   x_i ~ c_i s
 * (an all-zero row has s = 0), decided in fp32 with round-half-even.  A quantised row occupies
 * rap_q8_row_bytes(W) = (W + 2) rounded up to a multiple of 4 bytes: the codes, each stored as the unsigned byte
 * c_i + 128, then zero padding, and the bf16 scale in the last two bytes.  Quantised caches are
 * [B][H_kv][S_cap][row bytes], dense; q~ is not quantised.
 *   rap_quantize_rows       d_rows [n_rows][W] (dtype_in = RAP_F32 or RAP_BF16) -> d_q8 [n_rows][row bytes]; also the
 *                           way to convert an existing cache of a layer (n_rows = B * H_kv * S_cap).
 *   rap_qkv_rope_append_q8  rap_qkv_rope_append with the new K and V rows quantised straight from their fp32 values
 *                           (no rounding to the storage dtype in between); q~ as in rap_qkv_rope_append.
 *   rap_decode_attn_q8      rap_decode_attn over quantised caches: Eq. 2 on K_j = c^K_j s^K_j, V_j = c^V_j s^V_j.
 *   rap_decode_step_q8      rap_decode_step over quantised caches (h_k8 / h_v8: HOST arrays of L device pointers):
 *                           per layer the quantising append, then the attention over the quantised cache.
 * Arguments, errors and stream behaviour as for the unquantised calls; head_dim <= 256. */
size_t rap_q8_row_bytes(int32_t W);
rap_status rap_quantize_rows(rap_ctx* ctx, int32_t dtype_in, int64_t n_rows, int32_t W, const void* d_rows, void* d_q8,
                             void* stream);
rap_status rap_qkv_rope_append_q8(rap_ctx* ctx, int32_t layer, int32_t T, const void* d_x, const void* d_w_qkv,
                                  const void* d_bias, const int32_t* d_seq_id, const int32_t* d_pos,
                                  const int32_t* d_slot, int32_t h_slot_max, const double* d_inv_freq, void* d_q_out,
                                  void* d_k8, void* d_v8, int32_t B_cache, int32_t S_cap, void* stream);
rap_status rap_decode_attn_q8(rap_ctx* ctx, int32_t layer, int32_t B, const void* d_q, const void* d_k8, const void* d_v8,
                              int32_t S_cap, const int32_t* d_seq_len, int32_t h_seq_len_max, int32_t n_split,
                              float* d_out, void* stream);

rap_status rap_decode_step_q8(rap_ctx* ctx, int32_t B, const void* d_x, const void* const* h_w_qkv,
                              const void* const* h_bias, const double* d_inv_freq, void* const* h_k8,
                              void* const* h_v8, int32_t S_cap, int32_t* d_seq_len, int32_t h_seq_len_max,
                              int32_t n_split, void* d_q_scratch, float* d_out, size_t out_layer_stride,
                              int32_t advance, void* stream);

/* ---- decode attention without any allocation (the paper has no counterpart) --------------
 * Same result as rap_decode_attn, for callers that cannot allocate device memory: code running
 * inside someone else's memory budget (a serving engine that hands out every byte of HBM up
 * front), inside a region where cudaMalloc is forbidden or would synchronize the device, or
 * before/without a rap_ctx (rap_create allocates).  It takes the shape directly instead of a
 * context and calls no cudaMalloc / cudaFree or any other allocating routine.
 *   dtype: rap_dtype of d_q and the caches; n_pairs = P, n_vch = d_v' of this layer;
 *   d_q [B][H_q][2P], d_k_cache [B][H_kv][S_cap][2P], d_v_cache [B][H_kv][S_cap][d_v'],
 *   d_seq_len[b] valid rows (as in rap_decode_attn), d_out [B][H_q][d_v'] fp32.
 * Scratch: the split-KV partials go to a 4 MiB array that is part of the library image
 * (RAP_NOALLOC_WS_FLOATS floats, defined below); every GPU that loads the library holds those 4 MiB
 * until the process exits.  A call needs B * H_q * n_split * (d_v' + 2) floats: with
 * n_split = 0 the library picks a split count that fits; RAP_ESHAPE if the requested n_split
 * does not fit, if even one split does not (B * H_q * (d_v' + 2) > RAP_NOALLOC_WS_FLOATS), or if B or H_kv
 * exceeds 65535 (they index the launch grid).
 * The first call on each device looks up the array's device address (with that device
 * current); make that first call outside any stream capture.
 * All calls on a device share the one array and it keeps the previous call's contents.  The
 * kernels write every partial they later read, so nothing needs clearing, but two calls whose
 * kernels overlap on the GPU (different streams, or a graph with parallel branches) race on
 * it: serialize them.  Always uses the shape-generic kernel (any 2P, d_v' <= 256, G <= 8). */
#define RAP_NOALLOC_WS_FLOATS (1u << 20)
rap_status rap_decode_attn_noalloc(int32_t dtype, int32_t B, int32_t n_q_heads, int32_t n_kv_heads,
                                   int32_t head_dim, int32_t n_pairs, int32_t n_vch, const void* d_q,
                                   const void* d_k_cache, const void* d_v_cache, int32_t S_cap,
                                   const int32_t* d_seq_len, int32_t h_seq_len_max, int32_t n_split,
                                   float* d_out, void* stream);

/* ---- causal attention of a block of new tokens on the reduced dims (Eq. 2 for every t of the block) --
 * Prefill-side counterpart of rap_decode_attn: each of the B sequences has T new tokens whose q~ rows are
 * d_q [B][T][H_q][2P] and whose K / V rows are already in the caches (written by rap_qkv_rope_append) at
 * rows d_start[b] .. d_start[b] + T - 1; token i attends rows 0 .. d_start[b] + i.
 * d_out [B][T][H_q][d_v'] fp32.  h_start_max: caller's bound on d_start (RAP_ECAPACITY if
 * h_start_max + T > S_cap).  Tensor-core kernel, bf16 storage only (RAP_EUNSUPPORTED for fp32 stacks).
 * For a layer with an odd d_v' the call first copies the visible V rows to an even row length in a
 * context-owned workspace of B * H_kv * S_cap * (d_v' + 1) elements; the workspace is allocated (and the
 * stream synchronized) the first time a call needs that much, so make that call outside a stream capture.
 * Calls on one context must not overlap on the GPU (the workspace is shared, and growing it frees the old one
 * after synchronizing only the calling stream). */
rap_status rap_prefill_attn(rap_ctx* ctx, int32_t layer, int32_t B, int32_t T, const void* d_q, const void* d_k_cache,
                            const void* d_v_cache, int32_t S_cap, const int32_t* d_start, int32_t h_start_max,
                            float* d_out, void* stream);

/* ---- output projection on the retained V channels (Algorithm 1: W~_o = E_v W_o) ------------
 * rap_pack_wo: offline column gather.  d_wo [hidden][H_q*D] is the dense W_o of `layer` (stored
 * [out][in]); d_wo_tilde [hidden][H_q*d_v'] receives, for query head g and retained channel c, the
 * column g*D + v_idx[g/G][c] -- the only columns a reduced attention output can reach.
 * rap_out_proj: y[t] = W~_o o[t] for T <= max_batch rows; d_attn_out [T][H_q][d_v'] is the fp32 output
 * of rap_decode_attn, d_y [T][hidden] is written in the storage dtype (fp32 accumulate, one rounding;
 * for bf16 the attention output is first rounded to bf16, as a bf16 model would hand it to W_o).
 * RAP_EUNSUPPORTED unless H_q*d_v' is a multiple of 8 (bf16) / 4 (fp32). */
rap_status rap_pack_wo(rap_ctx* ctx, int32_t layer, const void* d_wo, const int32_t* d_v_idx, void* d_wo_tilde,
                       void* stream);
rap_status rap_out_proj(rap_ctx* ctx, int32_t layer, int32_t T, const float* d_attn_out, const void* d_wo_tilde,
                        void* d_y, void* stream);

/* ---- one decode step over all layers (projection + RoPE + append, then attention, per layer) -------------------------------------
 * Layer l consumes d_x + l*B*hidden (one hidden-state row per sequence) and produces
 * d_out + l*out_layer_stride ([B][H_q][d_v'_l] fp32).  d_seq_len[b] = rows cached BEFORE the
 * step: the new token takes position = slot = d_seq_len[b] and attends over d_seq_len[b]+1
 * rows (Eq. 2 runs over the prefix including t).  h_seq_len_max bounds d_seq_len (< S_cap).
 * h_w_qkv / h_bias / h_k_cache / h_v_cache are HOST arrays of L device pointers (h_bias may be
 * NULL).  d_q_scratch: caller's [B][H_q][D] storage-dtype scratch for q~.  If advance != 0 a
 * final kernel adds 1 to every d_seq_len[b]. */
rap_status rap_decode_step(rap_ctx* ctx, int32_t B, const void* d_x, const void* const* h_w_qkv,
                           const void* const* h_bias, const double* d_inv_freq,
                           void* const* h_k_cache, void* const* h_v_cache, int32_t S_cap,
                           int32_t* d_seq_len, int32_t h_seq_len_max, int32_t n_split,
                           void* d_q_scratch, float* d_out, size_t out_layer_stride,
                           int32_t advance, void* stream);

/* Same step with HOST input and output: h_x [L][B][hidden] (storage dtype) is copied to the
 * device, the step runs, out is copied back to h_out [L][out_layer_stride] and the stream is
 * synchronized before returning.  With pinned host memory the copies are asynchronous and overlap the
 * layers: the inputs of layers >= 1 arrive on a context-owned stream while layer 0 runs, and the outputs
 * of all but the last layer leave on another while later layers run.  h_x must stay unchanged and h_out
 * unread until the call returns. */
rap_status rap_decode_step_host(rap_ctx* ctx, int32_t B, const void* h_x, const void* const* h_w_qkv,
                                const void* const* h_bias, const double* d_inv_freq,
                                void* const* h_k_cache, void* const* h_v_cache, int32_t S_cap,
                                int32_t* d_seq_len, int32_t h_seq_len_max, int32_t n_split,
                                float* h_out, size_t out_layer_stride, int32_t advance, void* stream);

/* ---- comparator: low-rank cache with per-step reconstruction (Section 3) ------------------
 * Measurement-only counterpart of a weight-side low-rank method at equal cached dims: the K
 * cache holds UNROTATED latents [B][H_kv][S_cap][r]; every call rebuilds K_j = latent_j B_k[h]
 * (d_bk [H_kv][r][D], storage dtype), applies full-width RoPE at position j, and attends with
 * the full-width, already rotated d_q_full [B][H_q][D].  V side as in rap_decode_attn with
 * row width d_v.  Output [B][H_q][d_v] fp32. */
rap_status rap_lowrank_decode_attn(rap_ctx* ctx, int32_t B, int32_t r, int32_t d_v, const void* d_q_full,
                                   const void* d_k_latent, const void* d_bk, const void* d_v_cache,
                                   int32_t S_cap, const int32_t* d_seq_len, int32_t h_seq_len_max,
                                   int32_t n_split, float* d_out, void* stream);

/* Reads (and clears) the device status word after synchronizing `stream`.  code is a
 * rap_status (RAP_OK, RAP_ECAPACITY for a skipped out-of-range row, RAP_ETIMEOUT for a bounded
 * wait that gave up); detail identifies the row / stage. */
rap_status rap_get_last_device_status(rap_ctx* ctx, int32_t* code, int32_t* detail, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* RAP_H_ */
