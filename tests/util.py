"""Helpers shared by the GPU parity tests: run the oracle chain and the device chain on the
same seeded inputs.  The oracle and the CUDA path only meet here, in the tests."""
import numpy as np
import torch

from oracle import rap_oracle as O
from paper_2602_02599_b200 import synth
from paper_2602_02599_b200.stack import DecodeStack

BF16_MAX_ABS, BF16_REL_L2 = 1.5e-2, 5e-3     # attention output vs fp64 on the same bf16 inputs
F32_MAX_ABS = 1e-5


def to_np64(t):
    return t.detach().to(torch.float64).cpu().numpy()


def oracle_tables(w, ks, vs, n_pairs=None, n_vch=None):
    n_pairs = [w.n_pairs] * w.n_layers if n_pairs is None else n_pairs
    n_vch = [w.n_vch] * w.n_layers if n_vch is None else n_vch
    return O.build_tables(ks, vs, n_pairs, n_vch, w.head_dim, w.rope_theta, w.pairing)


def rel_l2(got, want):
    return float(np.linalg.norm(got - want) / max(np.linalg.norm(want), 1e-30))


def check_attn(got, want, dtype):
    err = float(np.abs(got - want).max())
    if dtype == "f32":
        assert err <= F32_MAX_ABS, f"max-abs {err:.3e} > {F32_MAX_ABS}"
    else:
        r = rel_l2(got, want)
        assert err <= BF16_MAX_ABS and r <= BF16_REL_L2, f"max-abs {err:.3e}, rel-L2 {r:.3e}"
    return err


def check_projection(got, want, dtype, what):
    """q~/k~/v~ after the single storage rounding: one storage ulp of the value plus the fp32
    accumulation error of the dot product (1e-3 of the row's largest entry for bf16)."""
    got, want = np.asarray(got, np.float64), np.asarray(want, np.float64)
    if dtype == "f32":
        tol = 1e-5 * np.ones_like(want)
    else:
        ulp = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(want), 1e-30))) - 7)
        tol = ulp + 1e-3 * np.abs(want).max(axis=-1, keepdims=True)
    bad = np.abs(got - want) > tol
    assert not bad.any(), f"{what}: {bad.sum()} entries off, worst {np.abs(got - want).max():.3e}"


def build_small_stack(w, ks, vs, full_weights=True, s_cap=None, max_rows=None, n_pairs=None, n_vch=None):
    """DecodeStack with tables built and weights uploaded; returns (stack, oracle tables, host W~ list)."""
    st = DecodeStack(w, n_pairs=n_pairs, n_vch=n_vch, s_cap=s_cap, max_rows=max_rows)
    st.build_tables(ks, vs)
    tabs = oracle_tables(w, ks, vs, n_pairs, n_vch)
    w_host = []
    for l in range(w.n_layers):
        P, dv = st.n_pairs[l], st.n_vch[l]
        if full_weights:
            Wq, Wk, Wv = synth.draw_full_weights(w, l)
            st.pack_from_full(l, Wq, Wk, Wv)
            wr = [O.round_storage(a, w.dtype) for a in (Wq, Wk, Wv)]
            w_host.append(O.gather_weights(wr[0], wr[1], wr[2], tabs, l, P, dv, w.head_dim))
        else:
            wp = synth.draw_packed_weights(w, l)
            st.set_packed_weights(l, wp)
            w_host.append(O.round_storage(wp, w.dtype))
    return st, tabs, w_host


def prefill_both(st, tabs, w_host, w, lens, step_tag=0, chunk=None):
    """Fill the caches the real way on both sides: every sequence b gets lens[b] tokens at positions
    0..lens[b]-1 through rap_qkv_rope_append (device) and the projection, RoPE and append steps of the oracle.  Returns oracle caches
    (list per layer of (K, V) fp64 arrays [B][H_kv][S_cap][W])."""
    B = st.B
    rows = [(b, p) for b in range(B) for p in range(int(lens[b]))]
    seq_id = np.array([r[0] for r in rows], dtype=np.int32)
    pos = np.array([r[1] for r in rows], dtype=np.int32)
    T = len(rows)
    chunk = chunk or T
    caches = []
    for l in range(w.n_layers):
        P, dv = st.n_pairs[l], st.n_vch[l]
        X = synth.draw_hidden(w, l, step_tag, T)
        Xr = O.round_storage(X, w.dtype)
        K = np.zeros((B, w.n_kv_heads, st.s_cap, 2 * P))
        V = np.zeros((B, w.n_kv_heads, st.s_cap, dv))
        q, k, v = O.qkv_rope(Xr, w_host[l], None, pos, tabs["inv_freq"][l], w.n_q_heads, w.n_kv_heads, P, dv)
        O.append(K, V, k, v, seq_id, pos, w.dtype)
        caches.append((K, V))
        st.k_cache[l].zero_()
        st.v_cache[l].zero_()
        for c0 in range(0, T, chunk):
            c1 = min(T, c0 + chunk)
            dx = torch.from_numpy(X[c0:c1]).to(st.device).to(st.dt).contiguous()
            dsid = torch.from_numpy(seq_id[c0:c1]).to(st.device)
            dpos = torch.from_numpy(pos[c0:c1]).to(st.device)
            qo = torch.empty((c1 - c0, w.n_q_heads, 2 * P), dtype=st.dt, device=st.device)
            st.qkv_rope_append(l, dx, dsid, dpos, dpos, int(pos[c0:c1].max()), q_out=qo)
    torch.cuda.synchronize()
    return caches


def unpack_q8(t, W):
    """A quantised cache tensor (uint8 [..., row bytes]) -> (codes int8 [..., W], scales fp64 [...]): the codes come
    first, each stored as code + 128; the bf16 scale sits in the last two bytes of the row."""
    a = t.detach().cpu().numpy()
    codes = (a[..., :W].astype(np.int16) - 128).astype(np.int8)
    bits = a[..., -2].astype(np.uint32) | (a[..., -1].astype(np.uint32) << 8)
    scales = (bits << 16).astype(np.uint32).view(np.float32).astype(np.float64)
    return codes, scales


def pack_q8(codes, scales, row_bytes):
    """Oracle-side codes and (bf16-valued) scales -> the byte layout of a quantised cache, as a uint8 array."""
    codes = np.asarray(codes, dtype=np.int8)
    out = np.zeros(codes.shape[:-1] + (row_bytes,), dtype=np.uint8)
    out[..., : codes.shape[-1]] = (codes.astype(np.int16) + 128).astype(np.uint8)
    bits = (np.asarray(scales, dtype=np.float32).view(np.uint32) >> 16).astype(np.uint16)
    out[..., -2] = (bits & 0xFF).astype(np.uint8)
    out[..., -1] = (bits >> 8).astype(np.uint8)
    return out
