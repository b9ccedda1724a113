"""ctypes binding of the RAP decode C ABI (include/rap.h): argument marshalling only.

Every function has the name of the C entry point it calls.  Tensors are torch CUDA tensors
used as device buffers (data_ptr()), the stream is torch's current stream.  Nothing is
computed in Python and there is no CPU fallback: a missing library raises at first use.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, byref, c_char_p, c_double, c_int32, c_int64, c_size_t, c_void_p

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# RAP_LIBRARY selects another build of the same library (the bounds-checking one, librap_b200_dbg.so, in tests)
LIB_PATH = os.environ.get("RAP_LIBRARY") or os.path.join(_HERE, "librap_b200.so")

RAP_OK, RAP_EINVAL, RAP_ESHAPE, RAP_ECAPACITY, RAP_EALIGN, RAP_EUNSUPPORTED, RAP_ECUDA, RAP_ETIMEOUT, RAP_ESTATE, RAP_EBOUNDS = range(10)
RAP_F32, RAP_BF16 = 0, 1
RAP_PAIR_HALF, RAP_PAIR_ADJACENT = 0, 1

EXPORTS = [
    "rap_create", "rap_destroy", "rap_status_string", "rap_last_cuda_error", "rap_retained_counts",
    "rap_cache_elem_offset", "rap_build_tables", "rap_pack_weights", "rap_qkv_rope_append",
    "rap_decode_attn", "rap_decode_step", "rap_decode_step_host", "rap_lowrank_decode_attn",
    "rap_get_last_device_status", "rap_kernel_launch_count", "rap_set_attn_variant",
    "rap_decode_attn_noalloc", "rap_profile_attn", "rap_profile_attn_read",
    "rap_pack_wo", "rap_out_proj", "rap_budget_alloc", "rap_prefill_attn", "rap_build_tables_hybrid",
    "rap_build_tables_partial", "rap_build_tables_freq", "rap_set_proj_variant", "rap_debug_arm_wait_timeout", "rap_debug_claim_scan_workspace", "rap_debug_set_scan_pieces",
    "rap_q8_row_bytes", "rap_quantize_rows", "rap_qkv_rope_append_q8", "rap_decode_attn_q8", "rap_decode_step_q8",
]


class rap_model_desc(ctypes.Structure):
    _fields_ = [("n_layers", c_int32), ("hidden", c_int32), ("n_q_heads", c_int32), ("n_kv_heads", c_int32),
                ("head_dim", c_int32), ("rope_theta", c_double), ("pairing", c_int32), ("dtype", c_int32),
                ("max_batch", c_int32), ("max_rows", c_int32)]


class RapError(RuntimeError):
    def __init__(self, status, where, detail=""):
        self.status = status
        msg = f"{where}: {_lib().rap_status_string(status).decode()}"
        if detail:
            msg += f" ({detail})"
        super().__init__(msg)


_LIB = None


def _lib():
    """Load librap_b200.so (built in-tree by build.py); raises if it is not there."""
    global _LIB
    if _LIB is not None:
        return _LIB
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2602_02599_b200.build` "
                           "(there is no fallback path)")
    lib = ctypes.CDLL(LIB_PATH)
    P = c_void_p
    lib.rap_create.argtypes = [POINTER(rap_model_desc), POINTER(P)]
    lib.rap_destroy.argtypes = [P]
    lib.rap_status_string.argtypes = [c_int32]
    lib.rap_status_string.restype = c_char_p
    lib.rap_last_cuda_error.argtypes = [P]
    lib.rap_last_cuda_error.restype = c_char_p
    lib.rap_retained_counts.argtypes = [c_double, c_int32, POINTER(c_int32), POINTER(c_int32)]
    lib.rap_cache_elem_offset.argtypes = [c_int32] * 7
    lib.rap_cache_elem_offset.restype = c_size_t
    lib.rap_build_tables.argtypes = [P] * 10
    lib.rap_build_tables_freq.argtypes = [P] * 11
    lib.rap_build_tables_hybrid.argtypes = [P] * 12
    lib.rap_build_tables_partial.argtypes = [P] * 13
    lib.rap_pack_weights.argtypes = [P, c_int32] + [P] * 11
    lib.rap_qkv_rope_append.argtypes = [P, c_int32, c_int32, P, P, P, P, P, P, c_int32, P, P, P, P, c_int32, c_int32, P]
    lib.rap_decode_attn.argtypes = [P, c_int32, c_int32, P, P, P, c_int32, P, c_int32, c_int32, P, P]
    lib.rap_decode_step.argtypes = [P, c_int32, P, P, P, P, P, P, c_int32, P, c_int32, c_int32, P, P, c_size_t, c_int32, P]
    lib.rap_decode_step_host.argtypes = [P, c_int32, P, P, P, P, P, P, c_int32, P, c_int32, c_int32, P, c_size_t, c_int32, P]
    lib.rap_lowrank_decode_attn.argtypes = [P, c_int32, c_int32, c_int32, P, P, P, P, c_int32, P, c_int32, c_int32, P, P]
    lib.rap_get_last_device_status.argtypes = [P, POINTER(c_int32), POINTER(c_int32), P]
    lib.rap_kernel_launch_count.argtypes = [P]
    lib.rap_kernel_launch_count.restype = c_int64
    lib.rap_set_attn_variant.argtypes = [P, c_int32]
    lib.rap_set_proj_variant.argtypes = [P, c_int32]
    lib.rap_debug_arm_wait_timeout.argtypes = [P]
    lib.rap_debug_set_scan_pieces.argtypes = [P, c_int32, c_int32]
    lib.rap_debug_claim_scan_workspace.argtypes = [P, c_int64]
    lib.rap_q8_row_bytes.argtypes = [c_int32]
    lib.rap_q8_row_bytes.restype = c_size_t
    lib.rap_quantize_rows.argtypes = [P, c_int32, c_int64, c_int32, P, P, P]
    lib.rap_qkv_rope_append_q8.argtypes = lib.rap_qkv_rope_append.argtypes
    lib.rap_decode_attn_q8.argtypes = lib.rap_decode_attn.argtypes
    lib.rap_decode_step_q8.argtypes = lib.rap_decode_step.argtypes
    lib.rap_budget_alloc.argtypes = [c_int32, c_int32, c_int32, P, c_double, P, P]
    lib.rap_prefill_attn.argtypes = [P, c_int32, c_int32, c_int32, P, P, P, c_int32, P, c_int32, P, P]
    lib.rap_pack_wo.argtypes = [P, c_int32, P, P, P, P]
    lib.rap_out_proj.argtypes = [P, c_int32, c_int32, P, P, P, P]
    lib.rap_profile_attn.argtypes = [P, c_int32]
    lib.rap_profile_attn_read.argtypes = [P, POINTER(ctypes.c_float), POINTER(c_int32)]
    lib.rap_decode_attn_noalloc.argtypes = [c_int32] * 7 + [P, P, P, c_int32, P, c_int32, c_int32, P, P]
    for name in EXPORTS:
        fn = getattr(lib, name)
        if fn.restype is ctypes.c_int:       # default: every other entry point returns rap_status
            fn.restype = c_int32
    _LIB = lib
    return lib


def _ptr(t):
    """Device (or host) address of a torch tensor / numpy array / raw int; None -> NULL."""
    if t is None:
        return None
    if isinstance(t, int):
        return c_void_p(t)
    if isinstance(t, np.ndarray):
        return c_void_p(t.ctypes.data)
    return c_void_p(t.data_ptr())


def _stream():
    import torch
    return c_void_p(torch.cuda.current_stream().cuda_stream)


def _ptr_array(tensors):
    arr = (c_void_p * len(tensors))()
    for i, t in enumerate(tensors):
        arr[i] = None if t is None else (t if isinstance(t, int) else t.data_ptr())
    return arr


def rap_retained_counts(rho, head_dim):
    P, dv = c_int32(), c_int32()
    s = _lib().rap_retained_counts(rho, head_dim, byref(P), byref(dv))
    if s:
        raise RapError(s, "rap_retained_counts")
    return P.value, dv.value


def rap_budget_alloc(k_pair_scores, rho, head_dim):
    """(n_pairs [L], n_vch [L]) int32 arrays of Algorithm 2 for host scores [L][H_kv][D/2]."""
    ks = np.ascontiguousarray(k_pair_scores, dtype=np.float64)
    L, H = ks.shape[0], ks.shape[1]
    n_pairs, n_vch = np.zeros(L, dtype=np.int32), np.zeros(L, dtype=np.int32)
    s = _lib().rap_budget_alloc(L, H, head_dim, _ptr(ks), float(rho), _ptr(n_pairs), _ptr(n_vch))
    if s:
        raise RapError(s, "rap_budget_alloc")
    return n_pairs, n_vch


def rap_q8_row_bytes(W):
    return int(_lib().rap_q8_row_bytes(W))


def rap_cache_elem_offset(n_kv_heads, S_cap, W, b, h, pos, c):
    return _lib().rap_cache_elem_offset(n_kv_heads, S_cap, W, b, h, pos, c)


def _noalloc_ws_floats():
    """RAP_NOALLOC_WS_FLOATS as include/rap.h defines it (the one place the limit is written down)."""
    import re
    text = open(os.path.join(os.path.dirname(_HERE), "include", "rap.h")).read()
    m = re.search(r"#define\s+RAP_NOALLOC_WS_FLOATS\s+\(1u\s*<<\s*(\d+)\)", text)
    if not m:
        raise RuntimeError("include/rap.h does not define RAP_NOALLOC_WS_FLOATS as (1u << n)")
    return 1 << int(m.group(1))


NOALLOC_WS_FLOATS = _noalloc_ws_floats()


def rap_decode_attn_noalloc(dtype, B, n_q_heads, n_kv_heads, head_dim, n_pairs, n_vch, d_q, d_k_cache, d_v_cache,
                            S_cap, d_seq_len, h_seq_len_max, n_split, d_out):
    """Decode attention for callers that must not allocate: no context, scratch in the library's
    own 4 MiB static device array (shared by all calls on a device; overlapping calls race)."""
    s = _lib().rap_decode_attn_noalloc(dtype, B, n_q_heads, n_kv_heads, head_dim, n_pairs, n_vch, _ptr(d_q),
                                       _ptr(d_k_cache), _ptr(d_v_cache), S_cap, _ptr(d_seq_len), h_seq_len_max,
                                       n_split, _ptr(d_out), _stream())
    if s:
        need = B * n_q_heads * max(n_split, 1) * (n_vch + 2)
        raise RapError(s, "rap_decode_attn_noalloc",
                       f"needs {need} scratch floats, the static array holds {NOALLOC_WS_FLOATS}" if s == RAP_ESHAPE else "")


class RapContext:
    """Owns one rap_ctx.  Methods are the C entry points with the ctx argument bound."""

    def __init__(self, n_layers, hidden, n_q_heads, n_kv_heads, head_dim, rope_theta, pairing, dtype,
                 max_batch, max_rows=None):
        self.desc = rap_model_desc(n_layers, hidden, n_q_heads, n_kv_heads, head_dim, float(rope_theta),
                                   int(pairing), int(dtype), max_batch, max_rows or max_batch)
        self._ctx = c_void_p()
        s = _lib().rap_create(byref(self.desc), byref(self._ctx))
        if s:
            detail = _lib().rap_last_cuda_error(self._ctx).decode() if self._ctx else ""
            if self._ctx:
                _lib().rap_destroy(self._ctx)
                self._ctx = c_void_p()
            raise RapError(s, "rap_create", detail)

    def _check(self, s, where):
        if s:
            raise RapError(s, where, _lib().rap_last_cuda_error(self._ctx).decode())

    def close(self):
        if self._ctx:
            _lib().rap_destroy(self._ctx)
            self._ctx = c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- entry points --------------------------------------------------------------------
    def rap_build_tables(self, k_pair_scores, v_chan_scores, n_pairs, n_vch, d_k_pair_idx, d_k_dim_idx,
                         d_v_idx, d_inv_freq):
        ks = np.ascontiguousarray(k_pair_scores, dtype=np.float64)
        vs = np.ascontiguousarray(v_chan_scores, dtype=np.float64)
        npairs = np.ascontiguousarray(n_pairs, dtype=np.int32)
        nvch = np.ascontiguousarray(n_vch, dtype=np.int32)
        self._check(_lib().rap_build_tables(self._ctx, _ptr(ks), _ptr(vs), _ptr(npairs), _ptr(nvch),
                                            _ptr(d_k_pair_idx), _ptr(d_k_dim_idx), _ptr(d_v_idx),
                                            _ptr(d_inv_freq), _stream()), "rap_build_tables")

    def rap_build_tables_freq(self, k_pair_scores, v_chan_scores, pair_freq, n_pairs, n_vch, d_k_pair_idx, d_k_dim_idx,
                              d_v_idx, d_inv_freq):
        arrs = [np.ascontiguousarray(a, dtype=np.float64) for a in (k_pair_scores, v_chan_scores, pair_freq)]
        ints = [np.ascontiguousarray(a, dtype=np.int32) for a in (n_pairs, n_vch)]
        self._check(_lib().rap_build_tables_freq(self._ctx, _ptr(arrs[0]), _ptr(arrs[1]), _ptr(arrs[2]), _ptr(ints[0]),
                                                 _ptr(ints[1]), _ptr(d_k_pair_idx), _ptr(d_k_dim_idx), _ptr(d_v_idx),
                                                 _ptr(d_inv_freq), _stream()), "rap_build_tables_freq")

    def rap_build_tables_hybrid(self, k_pair_scores, k_chan_scores, v_chan_scores, rope_layer, n_pairs, n_vch,
                                d_k_pair_idx, d_k_dim_idx, d_v_idx, d_inv_freq):
        arrs = [np.ascontiguousarray(a, dtype=np.float64) for a in (k_pair_scores, k_chan_scores, v_chan_scores)]
        ints = [np.ascontiguousarray(a, dtype=np.int32) for a in (rope_layer, n_pairs, n_vch)]
        self._check(_lib().rap_build_tables_hybrid(self._ctx, _ptr(arrs[0]), _ptr(arrs[1]), _ptr(arrs[2]), _ptr(ints[0]),
                                                   _ptr(ints[1]), _ptr(ints[2]), _ptr(d_k_pair_idx), _ptr(d_k_dim_idx),
                                                   _ptr(d_v_idx), _ptr(d_inv_freq), _stream()), "rap_build_tables_hybrid")

    def rap_build_tables_partial(self, k_pair_scores, k_chan_scores, v_chan_scores, rot_dims, n_rot_pairs, n_pairs, n_vch,
                                 d_k_pair_idx, d_k_dim_idx, d_v_idx, d_inv_freq):
        arrs = [np.ascontiguousarray(a, dtype=np.float64) for a in (k_pair_scores, k_chan_scores, v_chan_scores)]
        ints = [np.ascontiguousarray(a, dtype=np.int32) for a in (rot_dims, n_rot_pairs, n_pairs, n_vch)]
        self._check(_lib().rap_build_tables_partial(self._ctx, _ptr(arrs[0]), _ptr(arrs[1]), _ptr(arrs[2]), _ptr(ints[0]),
                                                    _ptr(ints[1]), _ptr(ints[2]), _ptr(ints[3]), _ptr(d_k_pair_idx),
                                                    _ptr(d_k_dim_idx), _ptr(d_v_idx), _ptr(d_inv_freq), _stream()),
                    "rap_build_tables_partial")

    def rap_pack_weights(self, layer, d_wq, d_wk, d_wv, d_k_dim_idx, d_v_idx, d_w_qkv,
                         d_bq=None, d_bk=None, d_bv=None, d_bias=None):
        self._check(_lib().rap_pack_weights(self._ctx, layer, _ptr(d_wq), _ptr(d_wk), _ptr(d_wv),
                                            _ptr(d_k_dim_idx), _ptr(d_v_idx), _ptr(d_w_qkv), _ptr(d_bq),
                                            _ptr(d_bk), _ptr(d_bv), _ptr(d_bias), _stream()), "rap_pack_weights")

    def rap_qkv_rope_append(self, layer, T, d_x, d_w_qkv, d_bias, d_seq_id, d_pos, d_slot, h_slot_max,
                            d_inv_freq, d_q_out, d_k_cache, d_v_cache, B_cache, S_cap):
        self._check(_lib().rap_qkv_rope_append(self._ctx, layer, T, _ptr(d_x), _ptr(d_w_qkv), _ptr(d_bias),
                                               _ptr(d_seq_id), _ptr(d_pos), _ptr(d_slot), h_slot_max,
                                               _ptr(d_inv_freq), _ptr(d_q_out), _ptr(d_k_cache), _ptr(d_v_cache),
                                               B_cache, S_cap, _stream()), "rap_qkv_rope_append")

    def rap_decode_attn(self, layer, B, d_q, d_k_cache, d_v_cache, S_cap, d_seq_len, h_seq_len_max, n_split, d_out):
        self._check(_lib().rap_decode_attn(self._ctx, layer, B, _ptr(d_q), _ptr(d_k_cache), _ptr(d_v_cache), S_cap,
                                           _ptr(d_seq_len), h_seq_len_max, n_split, _ptr(d_out), _stream()),
                    "rap_decode_attn")

    def rap_quantize_rows(self, dtype_in, n_rows, W, d_rows, d_q8):
        self._check(_lib().rap_quantize_rows(self._ctx, dtype_in, n_rows, W, _ptr(d_rows), _ptr(d_q8), _stream()),
                    "rap_quantize_rows")

    def rap_qkv_rope_append_q8(self, layer, T, d_x, d_w_qkv, d_bias, d_seq_id, d_pos, d_slot, h_slot_max, d_inv_freq,
                               d_q_out, d_k8, d_v8, B_cache, S_cap):
        self._check(_lib().rap_qkv_rope_append_q8(self._ctx, layer, T, _ptr(d_x), _ptr(d_w_qkv), _ptr(d_bias),
                                                  _ptr(d_seq_id), _ptr(d_pos), _ptr(d_slot), h_slot_max,
                                                  _ptr(d_inv_freq), _ptr(d_q_out), _ptr(d_k8), _ptr(d_v8), B_cache,
                                                  S_cap, _stream()), "rap_qkv_rope_append_q8")

    def rap_decode_attn_q8(self, layer, B, d_q, d_k8, d_v8, S_cap, d_seq_len, h_seq_len_max, n_split, d_out):
        self._check(_lib().rap_decode_attn_q8(self._ctx, layer, B, _ptr(d_q), _ptr(d_k8), _ptr(d_v8), S_cap,
                                              _ptr(d_seq_len), h_seq_len_max, n_split, _ptr(d_out), _stream()),
                    "rap_decode_attn_q8")

    def rap_decode_step(self, B, d_x, w_qkv, bias, d_inv_freq, k_cache, v_cache, S_cap, d_seq_len,
                        h_seq_len_max, n_split, d_q_scratch, d_out, out_layer_stride, advance):
        """w_qkv / bias / k_cache / v_cache: per-layer lists of tensors, or prebuilt pointer arrays."""
        args = [a if isinstance(a, ctypes.Array) or a is None else _ptr_array(a) for a in (w_qkv, bias, k_cache, v_cache)]
        self._check(_lib().rap_decode_step(self._ctx, B, _ptr(d_x), args[0], args[1], _ptr(d_inv_freq), args[2],
                                           args[3], S_cap, _ptr(d_seq_len), h_seq_len_max, n_split,
                                           _ptr(d_q_scratch), _ptr(d_out), out_layer_stride, advance, _stream()),
                    "rap_decode_step")

    def rap_decode_step_q8(self, B, d_x, w_qkv, bias, d_inv_freq, k8, v8, S_cap, d_seq_len, h_seq_len_max, n_split,
                           d_q_scratch, d_out, out_layer_stride, advance):
        args = [a if isinstance(a, ctypes.Array) or a is None else _ptr_array(a) for a in (w_qkv, bias, k8, v8)]
        self._check(_lib().rap_decode_step_q8(self._ctx, B, _ptr(d_x), args[0], args[1], _ptr(d_inv_freq), args[2], args[3],
                                              S_cap, _ptr(d_seq_len), h_seq_len_max, n_split, _ptr(d_q_scratch),
                                              _ptr(d_out), out_layer_stride, advance, _stream()), "rap_decode_step_q8")

    def rap_decode_step_host(self, B, h_x, w_qkv, bias, d_inv_freq, k_cache, v_cache, S_cap, d_seq_len,
                             h_seq_len_max, n_split, h_out, out_layer_stride, advance):
        args = [a if isinstance(a, ctypes.Array) or a is None else _ptr_array(a) for a in (w_qkv, bias, k_cache, v_cache)]
        self._check(_lib().rap_decode_step_host(self._ctx, B, _ptr(h_x), args[0], args[1], _ptr(d_inv_freq), args[2],
                                                args[3], S_cap, _ptr(d_seq_len), h_seq_len_max, n_split,
                                                _ptr(h_out), out_layer_stride, advance, _stream()),
                    "rap_decode_step_host")

    def rap_lowrank_decode_attn(self, B, r, d_v, d_q_full, d_k_latent, d_bk, d_v_cache, S_cap, d_seq_len,
                                h_seq_len_max, n_split, d_out):
        self._check(_lib().rap_lowrank_decode_attn(self._ctx, B, r, d_v, _ptr(d_q_full), _ptr(d_k_latent), _ptr(d_bk),
                                                   _ptr(d_v_cache), S_cap, _ptr(d_seq_len), h_seq_len_max, n_split,
                                                   _ptr(d_out), _stream()), "rap_lowrank_decode_attn")

    def rap_get_last_device_status(self):
        code, detail = c_int32(), c_int32()
        self._check(_lib().rap_get_last_device_status(self._ctx, byref(code), byref(detail), _stream()),
                    "rap_get_last_device_status")
        return code.value, detail.value

    def rap_kernel_launch_count(self):
        return int(_lib().rap_kernel_launch_count(self._ctx))

    def rap_prefill_attn(self, layer, B, T, d_q, d_k_cache, d_v_cache, S_cap, d_start, h_start_max, d_out):
        self._check(_lib().rap_prefill_attn(self._ctx, layer, B, T, _ptr(d_q), _ptr(d_k_cache), _ptr(d_v_cache), S_cap,
                                            _ptr(d_start), h_start_max, _ptr(d_out), _stream()), "rap_prefill_attn")

    def rap_pack_wo(self, layer, d_wo, d_v_idx, d_wo_tilde):
        self._check(_lib().rap_pack_wo(self._ctx, layer, _ptr(d_wo), _ptr(d_v_idx), _ptr(d_wo_tilde), _stream()),
                    "rap_pack_wo")

    def rap_out_proj(self, layer, T, d_attn_out, d_wo_tilde, d_y):
        self._check(_lib().rap_out_proj(self._ctx, layer, T, _ptr(d_attn_out), _ptr(d_wo_tilde), _ptr(d_y), _stream()),
                    "rap_out_proj")

    def rap_profile_attn(self, capacity):
        self._check(_lib().rap_profile_attn(self._ctx, capacity), "rap_profile_attn")

    def rap_profile_attn_read(self):
        ms, n = ctypes.c_float(), c_int32()
        self._check(_lib().rap_profile_attn_read(self._ctx, byref(ms), byref(n)), "rap_profile_attn_read")
        return ms.value, n.value

    def rap_debug_claim_scan_workspace(self, n_floats):
        self._check(_lib().rap_debug_claim_scan_workspace(self._ctx, n_floats), "rap_debug_claim_scan_workspace")

    def rap_debug_arm_wait_timeout(self):
        self._check(_lib().rap_debug_arm_wait_timeout(self._ctx), "rap_debug_arm_wait_timeout")

    def rap_debug_set_scan_pieces(self, piece_tiles, frac_x256):
        self._check(_lib().rap_debug_set_scan_pieces(self._ctx, piece_tiles, frac_x256), "rap_debug_set_scan_pieces")

    def rap_set_proj_variant(self, variant):
        self._check(_lib().rap_set_proj_variant(self._ctx, variant), "rap_set_proj_variant")

    def rap_set_attn_variant(self, variant):
        self._check(_lib().rap_set_attn_variant(self._ctx, variant), "rap_set_attn_variant")


def ptr_array(tensors):
    """Host array of device pointers for the per-layer arguments of rap_decode_step."""
    return _ptr_array(tensors)
