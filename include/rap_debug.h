/*
 * rap_debug.h -- test, accounting and profiling hooks of the RAP decode library.
 *
 * These entry points are exported by the same shared library as rap.h but are not part of the
 * product interface: they count launches, time the attention launches of a decode step and force
 * a kernel tier so that tests and profiles can reach every one of them.  Same conventions as rap.h.
 */
#ifndef RAP_DEBUG_H_
#define RAP_DEBUG_H_

#include "rap.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Number of kernels this context has launched since creation (for launch accounting). */
int64_t rap_kernel_launch_count(const rap_ctx* ctx);

/* Timing of the attention launches inside rap_decode_step / rap_decode_step_host, for roofline
 * reports: after rap_profile_attn(ctx, capacity) the next `capacity` attention launches (one per layer
 * and step) are bracketed by CUDA events on the caller's stream; rap_profile_attn_read waits for them,
 * returns the summed device time in milliseconds and the number of launches covered, and rearms the
 * same events.  capacity = 0 switches the timing off.  Event creation happens in rap_profile_attn. */
rap_status rap_profile_attn(rap_ctx* ctx, int32_t capacity);
rap_status rap_profile_attn_read(rap_ctx* ctx, float* ms_sum, int32_t* n_calls);

/* Forces a kernel variant for rap_decode_attn: 0 = automatic (the shape-specialised scans when the
 * head shape has one, the tensor-core form first; the low-rank comparator's fast path), 1 = fully generic
 * kernels only, 2 = skip the shape-specialised scans, 3 = skip only the tensor-core form of the
 * shape-specialised scan, 4 = the tensor-core form or nothing (bf16 calls return RAP_EUNSUPPORTED when the
 * head shape has no instantiation of it).  Meant for tests and profiling. */
rap_status rap_set_attn_variant(rap_ctx* ctx, int32_t variant);

/* Forces the form of rap_qkv_rope_append: 0 = automatic (decode-sized bf16 calls, T <= 32, run as one kernel with
 * the RoPE / append epilogue fused into the tcgen05 GEMM), 1 = always two stages (GEMM into the fp32 workspace, then
 * the epilogue kernel).  Meant for tests, which check the two forms against each other and against the oracle. */
rap_status rap_set_proj_variant(rap_ctx* ctx, int32_t variant);

/* Makes one bounded device-side wait run out, without faulting or hanging anything: the next launch of the
 * tensor-core scan of rap_decode_attn (head shapes staged by plain bulk copies) has the first warp of its first CTA
 * arm one stage barrier without issuing the copy for it, and polls stage barriers a few thousand times instead of
 * millions.  That warp gives up, its CTA records RAP_ETIMEOUT in the device status word, waits (bounded) for its
 * other copies and returns; every other CTA finishes normally.  The units that CTA touched stay unfinished (their
 * outputs are not written).  Later launches run normally: each launch clears the arrival counters its predecessor
 * used, so nothing has to be reset by hand.  The hook disarms itself when it is used. */
rap_status rap_debug_arm_wait_timeout(rap_ctx* ctx);

/* The tensor-core scan of rap_decode_attn (head shapes of the shaped workloads: the five retain ratios at D = 128,
 * 3 to 5 query heads per KV head) normally decides by the size of a launch whether its last tiles are handed
 * out at run time (pieces of some tiles, claimed from a counter by the CTAs as they finish) or assigned up front like
 * the rest.  This forces the choice for every later launch on the context, so that small test cases take the run-time
 * path: piece_tiles > 0 tiles per piece and frac_x256 / 256 of all tiles handed out that way; piece_tiles = 0: nothing
 * is handed out at run time; piece_tiles = -1: back to the automatic choice.  The result of a launch does not depend on
 * which CTA ends up with which piece (a piece is a fixed range of tiles, and partials are merged in tile order). */
rap_status rap_debug_set_scan_pieces(rap_ctx* ctx, int32_t piece_tiles, int32_t frac_x256);

/* Shows that the index checks of the bounds-checking build (librap_b200_dbg.so, compiled with -DRAP_DEBUG_BOUNDS) are
 * live, without any access leaving a buffer: the next shape-specialised scan launch is told that the split-KV
 * workspace holds only n_floats floats (it is as large as ever).  In the bounds-checking build the writes of partials
 * beyond that claim are skipped and the device status word reports RAP_EBOUNDS; in the normal build, which has no
 * checks, the call changes nothing.  The hook disarms itself when it is used; 0 switches it off. */
rap_status rap_debug_claim_scan_workspace(rap_ctx* ctx, int64_t n_floats);

#ifdef __cplusplus
}
#endif
#endif /* RAP_DEBUG_H_ */
