"""CPU oracle for the RAP (RoPE-Aligned Pruning) decode path -- TEST INFRASTRUCTURE ONLY.

A plain, slow NumPy fp64 statement of what the decode path computes, written from the
paper's definitions.  It shares no code, table, constant or helper with the CUDA
library and never imports it.  Only the tests, the smoke check and the CPU-baseline
leg of the benchmark may call into this module; the product path never does.

Two definitions of the same result live here:

  (R) the *reduced* path  -- tables -> gathered weights -> projection -> index-aware
      RoPE on the retained pairs -> append -> attention over 2P / d_v' dims.  This is
      the result the CUDA kernels are compared with.
  (F) the *full-dimensional masked* path -- textbook RoPE attention at the original
      head_dim with the removed K pairs zeroed and V restricted to retained channels.
      The paper proves (R) == (F) (Appendix "Full-dimensional representation",
      masked-logit equivalence); (F) exists only to pin (R).

Output projection (gather_wo / out_proj): pinned by the identity W~_o o_reduced = W_o E_v^T o_reduced
(expanding the reduced output back to D channels with zeros and using the dense W_o) and by a
loop-written column gather.

Pins (in tests/test_oracle_pins.py): rho=1 equals an independent textbook RoPE GQA
attention; (R)==(F) for rho<1 in both pairings; the per-pair relative-rotation
identity R_m^T R_n = R_(n-m); position-shift invariance; E_k E_k^T = I and
E_k R_t = R_(t,S) E_k (also for a frequency table that is not theta^(-2i/D)); the retained-fraction column of Table 13; the bytes/token row
of Table 15; brute-force loops on tiny inputs; closed-form softmax cases.

Cache quantisation (quantize_rows and the functions on top of it): a reading of a composition the paper only
names; pinned by exact rational arithmetic on hand-made rows, the half-step round-trip bound, exact
power-of-two scale equivariance and closed forms.

Parity unpinned: the paper prints no worked numeric example of an attention output, so
absolute outputs are pinned only through the identities and closed forms above.
The low-rank comparator (lowrank_decode_attn) is pinned only against the textbook
attention it reduces to when the latent factor is a selection matrix.

Notation follows the paper: D = original head_dim, P = retained RoPE pairs per KV
head (m_l in the paper), d_v' = retained V channels, G = H_q / H_kv, theta = RoPE base.
"""
from __future__ import annotations

import math

import numpy as np

PAIR_HALF = 0       # pair i = dims (i, i + D/2)      ("half apart", Section 3)
PAIR_ADJACENT = 1   # pair i = dims (2i, 2i + 1)      ("next to each other", Section 3)


# --------------------------------------------------------------------------------------
# storage rounding
# --------------------------------------------------------------------------------------
def round_bf16(x):
    """Round to bfloat16 (round-to-nearest-even on the fp32 bit pattern), return fp64.

    bf16 is the top 16 bits of an IEEE fp32; values are first rounded to fp32.
    """
    a = np.asarray(x, dtype=np.float32)
    bits = a.view(np.uint32).astype(np.uint64)
    lsb = (bits >> np.uint64(16)) & np.uint64(1)
    rounded = (bits + np.uint64(0x7FFF) + lsb) & np.uint64(0xFFFF0000)
    out = rounded.astype(np.uint32).view(np.float32)
    # NaN payloads are not produced by the synthetic inputs; keep inf/nan as they are.
    out = np.where(np.isfinite(a), out, a)
    return out.astype(np.float64)


def round_storage(x, dtype):
    """Round to the storage dtype of a config ('f32' or 'bf16'), return fp64."""
    if dtype == "bf16":
        return round_bf16(x)
    if dtype == "f32":
        return np.asarray(x, dtype=np.float32).astype(np.float64)
    raise ValueError(f"unknown storage dtype {dtype!r}")


def bf16_bits(x):
    """The 16-bit patterns of values that are already exactly representable in bf16."""
    a = np.asarray(x, dtype=np.float32)
    return (a.view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def build_tables_hybrid(k_pair_scores, k_chan_scores, v_chan_scores, rope_layer, n_pairs, n_vch, head_dim,
                        rope_theta, pairing):
    """Tables of a model whose layers are not all rotary (Section 4, "Hybrid compression": RAP where
    RoPE is used, plain channel pruning of K elsewhere).

    rope_layer[l] != 0: as build_tables.  rope_layer[l] == 0 (no positional rotation in that layer):
    K keeps the 2 * n_pairs[l] channels with the largest k_chan_scores [L][H_kv][D], ascending, no pair
    structure (k_pair_idx stays -1), and the frequency row is zero, i.e. the rotation of the shared
    online path is the identity for that layer."""
    tabs = build_tables(k_pair_scores, v_chan_scores, n_pairs, n_vch, head_dim, rope_theta, pairing)
    kc = np.asarray(k_chan_scores, dtype=np.float64)
    L, H, D = kc.shape
    for l in range(L):
        if rope_layer[l]:
            continue
        n = 2 * int(n_pairs[l])
        for h in range(H):
            tabs["k_pair_idx"][l, h, :] = -1
            tabs["k_dim_idx"][l, h, :] = -1
            tabs["k_dim_idx"][l, h, :n] = top_k_ascending(kc[l, h], n)
            tabs["inv_freq"][l, h, :] = 0.0
    return tabs


def build_tables_partial(k_pair_scores, k_chan_scores, v_chan_scores, rot_dims, n_rot_pairs, n_pairs, n_vch,
                         head_dim, rope_theta, pairing):
    """Tables of a model that rotates only the first rot_dims[l] dims of every head (Appendix "RoPE in Recent
    Open LLMs": partial rotary; Section 4, "Hybrid compression": RAP on the rotated part, channel pruning
    on the rest).

    Layer l, KV head h.  Rotated part: pairs i = 0 .. R/2 - 1 with R = rot_dims[l], members (i, i + R/2)
    (HALF pairing inside the rotated block) or (2i, 2i + 1) (ADJACENT), frequency theta ** (-2 i / R); the
    n_rot_pairs[l] pairs with the largest k_pair_scores[l, h, :R/2] are kept, ascending.  Unrotated part:
    channels R .. D - 1; the 2 * (n_pairs[l] - n_rot_pairs[l]) channels with the largest
    k_chan_scores[l, h, R:] are kept, ascending.  The reduced K row is [kept pairs, members adjacent |
    kept channels]; the frequency of a slot that holds unrotated channels is zero (identity rotation), so the
    online path is the same as for a fully rotary layer.  V as in build_tables.
    R = D reproduces build_tables, R = 0 a layer without positional rotation."""
    kp = np.asarray(k_pair_scores, dtype=np.float64)
    kc = np.asarray(k_chan_scores, dtype=np.float64)
    vs = np.asarray(v_chan_scores, dtype=np.float64)
    L, H, D = vs.shape
    assert D == head_dim
    tabs = {"k_pair_idx": np.full((L, H, D // 2), -1, dtype=np.int32),
            "k_dim_idx": np.full((L, H, D), -1, dtype=np.int32),
            "v_idx": np.full((L, H, D), -1, dtype=np.int32),
            "inv_freq": np.zeros((L, H, D // 2), dtype=np.float64)}
    for l in range(L):
        R, Pr, P = int(rot_dims[l]), int(n_rot_pairs[l]), int(n_pairs[l])
        C = 2 * (P - Pr)
        assert R % 2 == 0 and 0 <= R <= D and 0 <= Pr <= R // 2 and 0 <= C <= D - R
        for h in range(H):
            pairs = top_k_ascending(kp[l, h, : R // 2], Pr) if Pr else np.zeros(0, dtype=np.int64)
            for c, i in enumerate(pairs):
                i = int(i)
                tabs["k_pair_idx"][l, h, c] = i
                a, b = (i, i + R // 2) if pairing == PAIR_HALF else (2 * i, 2 * i + 1)
                tabs["k_dim_idx"][l, h, 2 * c] = a
                tabs["k_dim_idx"][l, h, 2 * c + 1] = b
                tabs["inv_freq"][l, h, c] = float(rope_theta) ** (-(2.0 * i) / R)
            if C:
                tabs["k_dim_idx"][l, h, 2 * Pr: 2 * P] = R + top_k_ascending(kc[l, h, R:], C)
            tabs["v_idx"][l, h, : int(n_vch[l])] = top_k_ascending(vs[l, h], int(n_vch[l]))
    return tabs


# --------------------------------------------------------------------------------------
# Tables  (Algorithm 2, selection step; Eq. 6 RAPIndex; Eq. 3 frequencies)
# --------------------------------------------------------------------------------------
def retained_counts(rho, head_dim):
    """Per-head budget at retain ratio rho: P whole pairs for K, d_v' channels for V.

    Reading: both are rounded half-up independently, P = floor(rho*D/2 + 1/2) and
    d_v' = floor(rho*D + 1/2).  This reproduces the retained fractions of Table 13.
    """
    P = int(math.floor(rho * (head_dim // 2) + 0.5))
    dv = int(math.floor(rho * head_dim + 0.5))
    return P, dv


def top_k_ascending(scores, k):
    """Indices of the k largest scores (ties: lower index wins), returned ascending."""
    scores = np.asarray(scores, dtype=np.float64)
    order = sorted(range(scores.shape[0]), key=lambda i: (-scores[i], i))
    return np.array(sorted(order[:k]), dtype=np.int32)


def rap_index(pair_idx, head_dim, pairing):
    """RAPIndex of Eq. 6: original in-head dimension of every reduced dimension.

    Reading: reduced dims are pair-interleaved -- reduced (2c, 2c+1) are the two
    members of the c-th retained pair, pairs in ascending original order.
    """
    out = np.empty(2 * len(pair_idx), dtype=np.int32)
    for c, i in enumerate(pair_idx):
        if pairing == PAIR_HALF:
            out[2 * c], out[2 * c + 1] = i, i + head_dim // 2
        elif pairing == PAIR_ADJACENT:
            out[2 * c], out[2 * c + 1] = 2 * i, 2 * i + 1
        else:
            raise ValueError("pairing")
    return out


def build_tables(k_pair_scores, v_chan_scores, n_pairs, n_vch, head_dim, rope_theta, pairing):
    """Tables for every (layer, KV head).

    k_pair_scores [L][H_kv][D/2], v_chan_scores [L][H_kv][D] (fp64), n_pairs[L], n_vch[L].
    Returns dict of fixed-stride arrays (unused tail = -1 / 0.0):
      k_pair_idx int32 [L][H_kv][D/2], k_dim_idx int32 [L][H_kv][D] (RAPIndex),
      v_idx int32 [L][H_kv][D], inv_freq fp64 [L][H_kv][D/2].
    inv_freq[c] = theta ** (-2 i_c / D) with i_c the ORIGINAL 0-based pair index
    (index-aware rotation, Section 4; Eq. 3).
    """
    ks = np.asarray(k_pair_scores, dtype=np.float64)
    vs = np.asarray(v_chan_scores, dtype=np.float64)
    L, H, half = ks.shape
    D = head_dim
    assert half == D // 2 and vs.shape == (L, H, D)
    k_pair_idx = np.full((L, H, half), -1, dtype=np.int32)
    k_dim_idx = np.full((L, H, D), -1, dtype=np.int32)
    v_idx = np.full((L, H, D), -1, dtype=np.int32)
    inv_freq = np.zeros((L, H, half), dtype=np.float64)
    for l in range(L):
        P, dv = int(n_pairs[l]), int(n_vch[l])
        for h in range(H):
            pairs = top_k_ascending(ks[l, h], P)
            k_pair_idx[l, h, :P] = pairs
            k_dim_idx[l, h, : 2 * P] = rap_index(pairs, D, pairing)
            v_idx[l, h, :dv] = top_k_ascending(vs[l, h], dv)
            for c in range(P):
                inv_freq[l, h, c] = float(rope_theta) ** (-2.0 * float(pairs[c]) / float(D))
    return dict(k_pair_idx=k_pair_idx, k_dim_idx=k_dim_idx, v_idx=v_idx, inv_freq=inv_freq)


def build_tables_freq(k_pair_scores, v_chan_scores, pair_freq, n_pairs, n_vch, head_dim, pairing):
    """Tables of a model whose RoPE has its own per-pair frequencies (Section 4, "Practical Considerations":
    frequency-scaled variants keep the 2x2 rotation blocks, so the pair selection applies unchanged).

    pair_freq [L][D/2] is the frequency (radians per position) of ORIGINAL pair i in layer l.  Reading: the
    selection is build_tables's; the retained pair c of (l, h) rotates at the frequency of its original pair,
    inv_freq[l, h, c] = pair_freq[l, i_c]  (index-aware, exactly as for the standard table).  A constant
    rescaling of the rotated vectors, which some variants add, is linear and belongs to W~_q; it is not part
    of the tables."""
    pf = np.asarray(pair_freq, dtype=np.float64)
    tabs = build_tables(k_pair_scores, v_chan_scores, n_pairs, n_vch, head_dim, 2.0, pairing)
    L, H, half = tabs["k_pair_idx"].shape
    assert pf.shape == (L, half)
    tabs["inv_freq"][:] = 0.0
    for l in range(L):
        for h in range(H):
            for c in range(int(n_pairs[l])):
                tabs["inv_freq"][l, h, c] = pf[l, int(tabs["k_pair_idx"][l, h, c])]
    return tabs


def selection_matrix(index, width):
    """Binary E of Eq. 6: E[r, index[r]] = 1 (rows = reduced dims, cols = original dims)."""
    E = np.zeros((len(index), width), dtype=np.float64)
    for r, j in enumerate(index):
        E[r, j] = 1.0
    return E


# --------------------------------------------------------------------------------------
# Weight gather  (Algorithm 1, construction step: W~_k, W~_q = W_q E_k^T, W~_v)
# --------------------------------------------------------------------------------------
def gather_weights(Wq, Wk, Wv, tables, layer, n_pairs_l, n_vch_l, head_dim):
    """Build W~_qkv [N_out][hidden] for one layer from full [out][in] weights.

    Row order: q heads 0..H_q-1 (2P rows each, using the RAPIndex of KV head g // G),
    then k heads (2P rows each), then v heads (d_v' rows each).
    """
    D = head_dim
    Hq, Hkv = Wq.shape[0] // D, Wk.shape[0] // D
    G = Hq // Hkv
    P2, dv = 2 * n_pairs_l, n_vch_l
    rows = []
    for g in range(Hq):
        idx = tables["k_dim_idx"][layer, g // G, :P2]
        rows.append(Wq[g * D + idx, :])
    for h in range(Hkv):
        idx = tables["k_dim_idx"][layer, h, :P2]
        rows.append(Wk[h * D + idx, :])
    for h in range(Hkv):
        idx = tables["v_idx"][layer, h, :dv]
        rows.append(Wv[h * D + idx, :])
    return np.concatenate(rows, axis=0)


# --------------------------------------------------------------------------------------
# Projection (Eq. 1 on the reduced widths), then index-aware RoPE (Eq. 3)
# --------------------------------------------------------------------------------------
def project(x, w_qkv, bias=None):
    """y[t] = W~_qkv x[t] (+ bias): x [T][hidden], w_qkv [N_out][hidden] -> [T][N_out], fp64."""
    y = np.asarray(x, dtype=np.float64) @ np.asarray(w_qkv, dtype=np.float64).T
    if bias is not None:
        y = y + np.asarray(bias, dtype=np.float64)[None, :]
    return y


def rope_reduced(vec, pos, inv_freq):
    """Rotate the P retained pairs of one reduced vector (length 2P) at position pos.

    Pair c occupies reduced dims (2c, 2c+1) and turns by the angle pos * inv_freq[c],
    with the 2x2 block [[cos, -sin], [sin, cos]] of Eq. 3.
    """
    v = np.array(vec, dtype=np.float64)
    out = np.empty_like(v)
    for c in range(len(v) // 2):
        phi = float(pos) * float(inv_freq[c])
        a, b = v[2 * c], v[2 * c + 1]
        out[2 * c] = a * math.cos(phi) - b * math.sin(phi)
        out[2 * c + 1] = a * math.sin(phi) + b * math.cos(phi)
    return out


def qkv_rope(x, w_qkv, bias, pos, inv_freq_l, Hq, Hkv, P, dv):
    """Projection and index-aware RoPE for T rows: returns unrounded fp64 (q [T][Hq][2P], k [T][Hkv][2P], v [T][Hkv][dv]).

    inv_freq_l: [H_kv][>=P] table of this layer; q head g uses KV head g // G's entries.
    """
    y = project(x, w_qkv, bias)
    T = y.shape[0]
    G = Hq // Hkv
    P2 = 2 * P
    q = np.empty((T, Hq, P2))
    k = np.empty((T, Hkv, P2))
    v = np.empty((T, Hkv, dv))
    for t in range(T):
        for g in range(Hq):
            q[t, g] = rope_reduced(y[t, g * P2:(g + 1) * P2], pos[t], inv_freq_l[g // G])
        off = Hq * P2
        for h in range(Hkv):
            k[t, h] = rope_reduced(y[t, off + h * P2: off + (h + 1) * P2], pos[t], inv_freq_l[h])
        off += Hkv * P2
        for h in range(Hkv):
            v[t, h] = y[t, off + h * dv: off + (h + 1) * dv]
    return q, k, v


# --------------------------------------------------------------------------------------
# Append, then attention (Eq. 2 on the reduced dims, Eq. 7, scale 1/sqrt(D))
# --------------------------------------------------------------------------------------
def append(k_cache, v_cache, k_new, v_new, seq_id, slot, dtype):
    """Write rounded k/v rows into caches [B][H_kv][S_cap][W]; returns nothing.

    Row r goes to sequence seq_id[r], cache row slot[r].  One rounding to the storage
    dtype happens here (and on q in the caller).
    """
    for r in range(k_new.shape[0]):
        k_cache[seq_id[r], :, slot[r], :] = round_storage(k_new[r], dtype)
        v_cache[seq_id[r], :, slot[r], :] = round_storage(v_new[r], dtype)


def decode_attn(q, k_cache, v_cache, seq_len, head_dim):
    """softmax(q K^T / sqrt(D)) V over rows [0, len_b) of each sequence.

    q [B][H_q][2P]; k_cache [B][H_kv][S_cap][2P]; v_cache [B][H_kv][S_cap][d_v'];
    seq_len[b] counts valid rows including the newest one.  Output [B][H_q][d_v'] in
    reduced V coordinates.  The scale uses the ORIGINAL head_dim D (Section 4, Step 3).
    """
    q = np.asarray(q, dtype=np.float64)
    B, Hq, _ = q.shape
    Hkv = k_cache.shape[1]
    G = Hq // Hkv
    dv = v_cache.shape[3]
    out = np.zeros((B, Hq, dv), dtype=np.float64)
    for b in range(B):
        n = int(seq_len[b])
        for g in range(Hq):
            h = g // G
            K = np.asarray(k_cache[b, h, :n], dtype=np.float64)
            V = np.asarray(v_cache[b, h, :n], dtype=np.float64)
            s = (K @ q[b, g]) / math.sqrt(float(head_dim))
            p = np.exp(s - s.max())
            p = p / p.sum()
            out[b, g] = p @ V
    return out


def prefill_attn(q, k_cache, v_cache, start, head_dim):
    """Causal attention of T new tokens per sequence over the reduced dims (Eq. 2 for every t of
    the block: token i of sequence b sits at cache row start[b] + i and attends rows 0 .. start[b] + i).

    q [B][T][H_q][2P]; caches as in decode_attn, already holding the T new rows; output
    [B][T][H_q][d_v'].  Written in the masked-matrix form softmax(Q K^T / sqrt(D) + mask) V, on purpose
    unlike decode_attn's per-query loop: the two are pinned against each other.
    """
    q = np.asarray(q, dtype=np.float64)
    B, T, Hq, _ = q.shape
    Hkv = k_cache.shape[1]
    G = Hq // Hkv
    dv = v_cache.shape[3]
    out = np.zeros((B, T, Hq, dv), dtype=np.float64)
    for b in range(B):
        n = int(start[b]) + T
        rows = np.arange(n)[None, :]
        allowed = rows <= (int(start[b]) + np.arange(T))[:, None]           # [T][n] causal mask
        for g in range(Hq):
            h = g // G
            K = np.asarray(k_cache[b, h, :n], dtype=np.float64)
            V = np.asarray(v_cache[b, h, :n], dtype=np.float64)
            S = (q[b, :, g, :] @ K.T) / math.sqrt(float(head_dim))
            S = np.where(allowed, S, -np.inf)
            Pm = np.exp(S - S.max(axis=1, keepdims=True))
            Pm = Pm / Pm.sum(axis=1, keepdims=True)
            out[b, :, g, :] = Pm @ V
    return out


def attn_partial(q_g, K, V, head_dim):
    """(m, l, acc) of one split: m = max logit, l = sum exp(s-m), acc = sum exp(s-m) V."""
    if K.shape[0] == 0:
        return -np.inf, 0.0, np.zeros(V.shape[1])
    s = (np.asarray(K, dtype=np.float64) @ q_g) / math.sqrt(float(head_dim))
    m = s.max()
    e = np.exp(s - m)
    return m, e.sum(), e @ np.asarray(V, dtype=np.float64)


def combine_partials(parts):
    """Log-sum-exp merge of (m, l, acc) partials; empty splits (m = -inf, l = 0) drop out."""
    M = max(m for m, _, _ in parts)
    num = sum(math.exp(m - M) * acc for m, l, acc in parts if l > 0.0)
    den = sum(math.exp(m - M) * l for m, l, acc in parts if l > 0.0)
    return num / den


# --------------------------------------------------------------------------------------
# (F) full-dimensional masked path and the textbook reference -- pins only
# --------------------------------------------------------------------------------------
def textbook_inv_freq(head_dim, rope_theta):
    """Standard RoPE table: theta ** (-2 i / D), i = 0 .. D/2 - 1 (Eq. 3)."""
    return np.array([float(rope_theta) ** (-(2.0 * i) / head_dim) for i in range(head_dim // 2)])


def textbook_rope(x, pos, head_dim, rope_theta, pairing):
    """Full-width RoPE of one head vector in the usual framework formulation.

    HALF pairing: x * cos + rotate_half(x) * sin with cos/sin = table repeated twice and
    rotate_half(x) = concat(-x[D/2:], x[:D/2]).  ADJACENT pairing: the interleaved form.
    Written independently of rope_reduced on purpose.
    """
    x = np.asarray(x, dtype=np.float64)
    D = head_dim
    ang = float(pos) * textbook_inv_freq(D, rope_theta)
    if pairing == PAIR_HALF:
        cos = np.concatenate([np.cos(ang), np.cos(ang)])
        sin = np.concatenate([np.sin(ang), np.sin(ang)])
        rot = np.concatenate([-x[D // 2:], x[: D // 2]])
        return x * cos + rot * sin
    cos = np.repeat(np.cos(ang), 2)
    sin = np.repeat(np.sin(ang), 2)
    rot = np.empty_like(x)
    rot[0::2] = -x[1::2]
    rot[1::2] = x[0::2]
    return x * cos + rot * sin


def full_masked_attention(X_hist, Wq, Wk, Wv, k_pair_idx, v_idx, head_dim, rope_theta, pairing,
                          Hq, Hkv, n_pairs_l, n_vch_l, scale_dim=None):
    """(F): one sequence, tokens X_hist [n][hidden] at positions 0..n-1, query = last token.

    Full W_q, W_k, W_v ([heads*D][hidden]); textbook RoPE over all D/2 pairs; K dims of
    removed pairs zeroed (W_k M_S); V restricted to the retained channels; scale
    1/sqrt(D).  Returns [H_q][d_v'].
    """
    D = head_dim
    n = X_hist.shape[0]
    G = Hq // Hkv
    X = np.asarray(X_hist, dtype=np.float64)
    qfull = (np.asarray(Wq, dtype=np.float64) @ X[-1]).reshape(Hq, D)
    kfull = (X @ np.asarray(Wk, dtype=np.float64).T).reshape(n, Hkv, D)
    vfull = (X @ np.asarray(Wv, dtype=np.float64).T).reshape(n, Hkv, D)
    out = np.zeros((Hq, n_vch_l))
    sd = float(D if scale_dim is None else scale_dim)
    for g in range(Hq):
        h = g // G
        mask = np.zeros(D)
        for i in k_pair_idx[h, :n_pairs_l]:
            if pairing == PAIR_HALF:
                mask[i] = mask[i + D // 2] = 1.0
            else:
                mask[2 * i] = mask[2 * i + 1] = 1.0
        qr = textbook_rope(qfull[g], n - 1, D, rope_theta, pairing)
        s = np.empty(n)
        for j in range(n):
            kr = textbook_rope(kfull[j, h], j, D, rope_theta, pairing) * mask
            s[j] = float(qr @ kr) / math.sqrt(sd)
        p = np.exp(s - s.max())
        p /= p.sum()
        out[g] = p @ vfull[:, h, :][:, v_idx[h, :n_vch_l]]
    return out


def reduced_attention_from_hidden(X_hist, w_qkv, inv_freq_l, Hq, Hkv, P, dv, head_dim,
                                  dtype=None, bias=None):
    """(R) end to end for one sequence: tokens X_hist at positions 0..n-1, query = last.

    Builds the cache the real way (projection, RoPE and append for every token) and runs the attention.  dtype=None keeps
    everything in fp64 (used by the identity pins); 'bf16'/'f32' rounds q, k, v once.
    Returns (out [H_q][d_v'], q [H_q][2P], K [H_kv][n][2P], V [H_kv][n][d_v']).
    """
    n = X_hist.shape[0]
    q, k, v = qkv_rope(X_hist, w_qkv, bias, np.arange(n), inv_freq_l, Hq, Hkv, P, dv)
    if dtype is not None:
        q, k, v = round_storage(q, dtype), round_storage(k, dtype), round_storage(v, dtype)
    K = np.transpose(k, (1, 0, 2))[None]
    V = np.transpose(v, (1, 0, 2))[None]
    out = decode_attn(q[-1][None], K, V, [n], head_dim)
    return out[0], q[-1], K[0], V[0]


# --------------------------------------------------------------------------------------
# low-rank comparator (Section 3: cache X A_k, rebuild K = latent B_k, full RoPE each step)
# --------------------------------------------------------------------------------------
def lowrank_decode_attn(q_full, k_latent, B_k, v_cache, seq_len, head_dim, rope_theta, pairing):
    """Decode attention of a weight-side low-rank method at equal cached dims.

    q_full [B][H_q][D] is already rotated at its own position.  k_latent
    [B][H_kv][S_cap][r] is unrotated; every step rebuilds K_j = latent_j B_k[h] ([r][D]),
    applies full-width RoPE at position j, and attends with scale 1/sqrt(D).  V side is a
    d_v'-wide cache as in RAP (the V factor is absorbed into W_o).
    """
    q_full = np.asarray(q_full, dtype=np.float64)
    B, Hq, D = q_full.shape
    Hkv = k_latent.shape[1]
    G = Hq // Hkv
    out = np.zeros((B, Hq, v_cache.shape[3]))
    for b in range(B):
        n = int(seq_len[b])
        for h in range(Hkv):
            Kfull = np.asarray(k_latent[b, h, :n], dtype=np.float64) @ np.asarray(B_k[h], dtype=np.float64)
            Krot = np.stack([textbook_rope(Kfull[j], j, D, rope_theta, pairing) for j in range(n)])
            V = np.asarray(v_cache[b, h, :n], dtype=np.float64)
            for g in range(h * G, (h + 1) * G):
                s = (Krot @ q_full[b, g]) / math.sqrt(float(D))
                p = np.exp(s - s.max())
                p /= p.sum()
                out[b, g] = p @ V
    return out


# --------------------------------------------------------------------------------------
# Budget-Alloc (Algorithm 2, layer-adaptive budgets with mean retain ratio rho)
# --------------------------------------------------------------------------------------
def budget_alloc(k_pair_scores, rho, head_dim):
    """Per-layer pair budgets m_l proportional to the layer score with mean retain ratio rho.

    sigma_l = mean over heads and pairs of the pair scores (Algorithm 2, layer score).
    The paper fixes m_l ~ sigma_l and (1/L) sum m_l / (D/2) = rho but not the rounding; the
    reading taken here: the integer total is round(rho * D/2 * L); real-valued targets are
    proportional to sigma_l, layers whose target leaves [1, D/2] are pinned to the bound and the
    rest re-shared (water-filling); targets are floored and the missing units go to the largest
    fractional parts (ties: lower layer).  V keeps 2 m_l channels (Balanced K/V).
    Returns (n_pairs [L], n_vch [L]) as int arrays."""
    sc = np.asarray(k_pair_scores, dtype=np.float64)
    L, P = sc.shape[0], head_dim // 2
    sigma = sc.reshape(L, -1).mean(axis=1)
    total = int(math.floor(rho * P * L + 0.5))
    total = min(max(total, L), P * L)
    fixed = {}
    while True:
        free = [l for l in range(L) if l not in fixed]
        rest = total - sum(fixed.values())
        ssum = sum(sigma[l] for l in free)
        target = {l: (rest * sigma[l] / ssum if ssum > 0 else rest / len(free)) for l in free}
        over = [l for l in free if target[l] > P]
        under = [l for l in free if target[l] < 1]
        if over:                       # pin the layers that want more than everything first
            for l in over:
                fixed[l] = P
        elif under:
            for l in under:
                fixed[l] = 1
        else:
            break
        if len(fixed) == L:
            target = {}
            break
    m = np.zeros(L, dtype=np.int64)
    for l, v in fixed.items():
        m[l] = v
    free = sorted(target)
    for l in free:
        m[l] = int(math.floor(target[l]))
    missing = total - int(m.sum())
    order = sorted(free, key=lambda l: (-(target[l] - math.floor(target[l])), l))
    i = 0
    while missing > 0 and order:
        l = order[i % len(order)]
        if m[l] < P:
            m[l] += 1
            missing -= 1
        i += 1
        if i > 4 * len(order) + missing:
            break
    return m.astype(np.int32), (2 * m).astype(np.int32)


# --------------------------------------------------------------------------------------
# output projection on the retained V channels (Algorithm 1: W~_o = E_v W_o absorbs the V selection)
# --------------------------------------------------------------------------------------
def gather_wo(Wo, tables, layer, n_vch_l, head_dim, Hq, Hkv):
    """W~_o [hidden][H_q * d_v'] from the dense W_o [hidden][H_q * D] (weights stored [out][in]).

    Input column g * D + u of W_o multiplies channel u of query head g's attention output; only
    the retained channels u in S_v of KV head g // G ever carry a value, so W~_o keeps exactly
    those columns, in the order of the reduced output (head-major, channels ascending)."""
    D, G, dv = head_dim, Hq // Hkv, n_vch_l
    cols = []
    for g in range(Hq):
        cols.append(g * D + np.asarray(tables["v_idx"][layer, g // G, :dv]))
    return np.asarray(Wo)[:, np.concatenate(cols)]


def out_proj(attn_out, wo_tilde):
    """y[t] = W~_o o[t]: attn_out [T][H_q][d_v'] (reduced V coordinates) -> [T][hidden], fp64."""
    o = np.asarray(attn_out, dtype=np.float64)
    return o.reshape(o.shape[0], -1) @ np.asarray(wo_tilde, dtype=np.float64).T


# --------------------------------------------------------------------------------------
# composition with KV-cache quantisation (Introduction and Related Work: pruning the cache width and lowering
# the bit-width of what is cached are orthogonal; the paper's own composition study uses a plain symmetric
# round-to-nearest quantiser)
# --------------------------------------------------------------------------------------
def quantize_rows(x):
    """8-bit symmetric round-to-nearest quantisation of cache rows, one scale per row.

    Reading (the paper names the quantiser family, not a cache format): every compact cache row x [W] keeps
    codes c_i in [-127, 127] and one scale s with x_i ~ c_i * s:
        s  = bf16( max_i |x_i| / 127 )          the scale is stored in the cache's 16-bit float type
        c_i = clip( rint( x_i / s ), -127, 127 )  round half to even; an all-zero row has s = 0 and c = 0.
    The decision is taken in fp32 (x as fp32, both divisions in fp32), the precision the kernels take it in.
    x [..., W] -> (codes int8 [..., W], scales fp64 [...], holding bf16 values)."""
    x32 = np.asarray(x, dtype=np.float32)
    amax = np.max(np.abs(x32), axis=-1)
    s32 = (amax / np.float32(127.0)).astype(np.float32)
    s = round_bf16(s32).astype(np.float32)
    safe = np.where(s > 0, s, np.float32(1.0)).astype(np.float32)
    c = np.rint((x32 / safe[..., None]).astype(np.float32))
    c = np.clip(c, -127.0, 127.0)
    c = np.where((s > 0)[..., None], c, 0.0)
    return c.astype(np.int8), s.astype(np.float64)


def dequantize_rows(codes, scales):
    """x_i = c_i * s, fp64."""
    return np.asarray(codes, dtype=np.float64) * np.asarray(scales, dtype=np.float64)[..., None]


def append_q8(k_codes, k_scales, v_codes, v_scales, k_new, v_new, seq_id, slot):
    """Quantised append: rows k_new [T][H_kv][2P], v_new [T][H_kv][d_v'] (after RoPE, before any rounding)
    are quantised row by row and written to codes [B][H_kv][S_cap][W] / scales [B][H_kv][S_cap]."""
    for r in range(k_new.shape[0]):
        c, s = quantize_rows(k_new[r])
        k_codes[seq_id[r], :, slot[r], :] = c
        k_scales[seq_id[r], :, slot[r]] = s
        c, s = quantize_rows(v_new[r])
        v_codes[seq_id[r], :, slot[r], :] = c
        v_scales[seq_id[r], :, slot[r]] = s


def decode_attn_q8(q, k_codes, k_scales, v_codes, v_scales, seq_len, head_dim):
    """Eq. 2 on the reduced dims over a quantised cache: the attention of decode_attn on the dequantised rows
    K_j = c^K_j s^K_j, V_j = c^V_j s^V_j (q is not quantised)."""
    return decode_attn(q, dequantize_rows(k_codes, k_scales), dequantize_rows(v_codes, v_scales), seq_len, head_dim)


def kv_bytes_per_token_q8(n_layers, n_kv_heads, k_width, v_width):
    """Resident bytes per token of the quantised cache as the library lays it out: per row the codes, then a
    16-bit scale in the last two bytes of a row padded to a multiple of four bytes."""
    row = lambda w: (w + 2 + 3) // 4 * 4
    return n_layers * n_kv_heads * (row(k_width) + row(v_width))


# --------------------------------------------------------------------------------------
# closed-form accounting (Table 3 cost model; Table 15 bytes per token)
# --------------------------------------------------------------------------------------
def kv_bytes_per_token(n_layers, n_kv_heads, k_width, v_width, elem_bytes):
    """Resident KV state per token: L * H_kv * (K width + V width) * bytes."""
    return n_layers * n_kv_heads * (k_width + v_width) * elem_bytes


def attn_read_bytes(B, n_kv_heads, length, k_width, v_width, elem_bytes):
    """Bytes of pruned cache one decode step of one layer must read."""
    return B * n_kv_heads * length * (k_width + v_width) * elem_bytes
