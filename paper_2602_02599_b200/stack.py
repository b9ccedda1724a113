"""Device-buffer holder for one attention stack: allocation and pointer bookkeeping only.

torch allocates the device memory and provides the stream; every computation is a call
into the C ABI through binding.RapContext.
"""
from __future__ import annotations

import numpy as np
import torch

from . import binding
from .binding import RapContext


def torch_dtype(name):
    return torch.float32 if name == "f32" else torch.bfloat16


class DecodeStack:
    """Tables, shrunken weights and compact caches of `w` (a synth.Workload) on one GPU."""

    def __init__(self, w, n_pairs=None, n_vch=None, batch=None, s_cap=None, max_rows=None, device="cuda:0",
                 alloc_cache=True):
        self.w = w
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        self.B = w.batch if batch is None else batch
        self.L = w.n_layers
        self.n_pairs = [w.n_pairs] * self.L if n_pairs is None else list(n_pairs)
        self.n_vch = [w.n_vch] * self.L if n_vch is None else list(n_vch)
        self.s_cap = s_cap if s_cap is not None else ((w.seq + 64 + 7) // 8) * 8
        self.dt = torch_dtype(w.dtype)
        self.ctx = RapContext(w.n_layers, w.hidden, w.n_q_heads, w.n_kv_heads, w.head_dim, w.rope_theta,
                              w.pairing, binding.RAP_F32 if w.dtype == "f32" else binding.RAP_BF16,
                              self.B, max_rows or self.B)
        D, H = w.head_dim, w.n_kv_heads
        dev = self.device
        self.k_pair_idx = torch.empty((self.L, H, D // 2), dtype=torch.int32, device=dev)
        self.k_dim_idx = torch.empty((self.L, H, D), dtype=torch.int32, device=dev)
        self.v_idx = torch.empty((self.L, H, D), dtype=torch.int32, device=dev)
        self.inv_freq = torch.empty((self.L, H, D // 2), dtype=torch.float64, device=dev)
        self.w_qkv = [None] * self.L
        self.bias = None
        self.k_cache = [None] * self.L
        self.v_cache = [None] * self.L
        if alloc_cache:
            for l in range(self.L):
                self.alloc_layer_cache(l)
        self.seq_len = torch.zeros((self.B,), dtype=torch.int32, device=dev)
        self.q_scratch = torch.empty((max(self.B, max_rows or 0), w.n_q_heads, D), dtype=self.dt, device=dev)
        self.out_stride = self.B * w.n_q_heads * max(self.n_vch)
        self.out = torch.empty((self.L, self.out_stride), dtype=torch.float32, device=dev)
        self._ptrs = None

    def n_out(self, l):
        w = self.w
        return (w.n_q_heads + w.n_kv_heads) * 2 * self.n_pairs[l] + w.n_kv_heads * self.n_vch[l]

    def alloc_layer_cache(self, l):
        w = self.w
        self.k_cache[l] = torch.empty((self.B, w.n_kv_heads, self.s_cap, 2 * self.n_pairs[l]), dtype=self.dt,
                                      device=self.device)
        self.v_cache[l] = torch.empty((self.B, w.n_kv_heads, self.s_cap, self.n_vch[l]), dtype=self.dt,
                                      device=self.device)
        self._ptrs = None

    def build_tables(self, k_pair_scores, v_chan_scores):
        self.ctx.rap_build_tables(k_pair_scores, v_chan_scores, self.n_pairs, self.n_vch, self.k_pair_idx,
                                  self.k_dim_idx, self.v_idx, self.inv_freq)

    def set_packed_weights(self, l, w_np):
        """Upload an already shrunken W~_qkv [N_out][hidden] (host fp32 array), stored in the stack dtype."""
        self.w_qkv[l] = torch.from_numpy(np.ascontiguousarray(w_np)).to(self.device).to(self.dt).contiguous()
        self._ptrs = None

    def pack_from_full(self, l, Wq, Wk, Wv):
        """Upload dense weights and gather the retained rows on the device (rap_pack_weights)."""
        up = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(self.device).to(self.dt).contiguous()
        dq, dk, dv = up(Wq), up(Wk), up(Wv)
        self.w_qkv[l] = torch.empty((self.n_out(l), self.w.hidden), dtype=self.dt, device=self.device)
        self.ctx.rap_pack_weights(l, dq, dk, dv, self.k_dim_idx, self.v_idx, self.w_qkv[l])
        torch.cuda.current_stream().synchronize()
        self._ptrs = None

    def pointer_arrays(self):
        if self._ptrs is None:
            self._ptrs = (binding.ptr_array(self.w_qkv), None if self.bias is None else binding.ptr_array(self.bias),
                          binding.ptr_array(self.k_cache), binding.ptr_array(self.v_cache))
        return self._ptrs

    def qkv_rope_append(self, l, x, seq_id, pos, slot, slot_max, q_out=None):
        T = x.shape[0]
        q_out = self.q_scratch if q_out is None else q_out
        self.ctx.rap_qkv_rope_append(l, T, x, self.w_qkv[l], None if self.bias is None else self.bias[l], seq_id,
                                     pos, slot, slot_max, self.inv_freq, q_out, self.k_cache[l], self.v_cache[l],
                                     self.B, self.s_cap)
        return q_out

    def decode_attn(self, l, q, seq_len, len_max, n_split=0, out=None):
        out = self.out[l] if out is None else out
        self.ctx.rap_decode_attn(l, self.B, q, self.k_cache[l], self.v_cache[l], self.s_cap, seq_len, len_max,
                                 n_split, out)
        return out

    def decode_step(self, x, len_max, n_split=0, advance=0):
        wq, bs, kc, vc = self.pointer_arrays()
        self.ctx.rap_decode_step(self.B, x, wq, bs, self.inv_freq, kc, vc, self.s_cap, self.seq_len, len_max,
                                 n_split, self.q_scratch, self.out, self.out_stride, advance)
        return self.out

    def decode_step_host(self, h_x, h_out, len_max, n_split=0, advance=0):
        wq, bs, kc, vc = self.pointer_arrays()
        self.ctx.rap_decode_step_host(self.B, h_x, wq, bs, self.inv_freq, kc, vc, self.s_cap, self.seq_len, len_max,
                                      n_split, h_out, self.out_stride, advance)
        return h_out

    def fill_synthetic(self, seed, tail=256, chunk=2048):
        """Seeded synthetic state for the large workloads: packed weights N(0, 0.02^2) from synth, cache
        positions [0, seq) filled on the device with iid N(0, hidden * 0.02^2) (the law of projected
        hidden states), then the last `tail` positions of every sequence rewritten through
        rap_qkv_rope_append in `chunk`-row calls so the real append path is exercised at scale."""
        from . import synth
        w = self.w
        for l in range(self.L):
            self.set_packed_weights(l, synth.draw_packed_weights(w, l))
        g = torch.Generator(device=self.device).manual_seed(seed)
        sigma = float(np.sqrt(w.hidden) * 0.02)
        for l in range(self.L):
            self.k_cache[l].normal_(0.0, sigma, generator=g)
            self.v_cache[l].normal_(0.0, sigma, generator=g)
        tail = min(tail, w.seq)
        rows_b = np.repeat(np.arange(self.B, dtype=np.int32), tail)
        rows_p = np.tile(np.arange(w.seq - tail, w.seq, dtype=np.int32), self.B)
        for l in range(self.L):
            xg = torch.Generator(device=self.device).manual_seed(seed + 7919 * (l + 1))
            for c0 in range(0, len(rows_b), chunk):
                c1 = min(len(rows_b), c0 + chunk)
                x = torch.empty((c1 - c0, w.hidden), dtype=self.dt, device=self.device).normal_(0.0, 1.0, generator=xg)
                sid = torch.from_numpy(rows_b[c0:c1]).to(self.device)
                pos = torch.from_numpy(rows_p[c0:c1]).to(self.device)
                qo = torch.empty((c1 - c0, w.n_q_heads, 2 * self.n_pairs[l]), dtype=self.dt, device=self.device)
                self.qkv_rope_append(l, x, sid, pos, pos, int(rows_p[c0:c1].max()), q_out=qo)
        torch.cuda.synchronize()

    def close(self):
        self.ctx.close()
