"""Pins for the CPU oracle: what the paper and the mathematics fix, checked on the CPU.

Every check here compares the oracle with something other than itself: a textbook
formulation written separately, an identity the paper proves, a number the paper prints,
a closed form, or brute-force loops on tiny inputs.
"""
import math
import os

import numpy as np
import pytest
import torch

from oracle import rap_oracle as O
from paper_2602_02599_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _small(pairing=O.PAIR_HALF, rho=0.75, D=16, Hq=4, Hkv=2, hidden=24, n=7, seed=3, L=1):
    """Tiny full-weight model: everything needed for both (R) and (F)."""
    rng = np.random.default_rng(seed)
    P, dv = O.retained_counts(rho, D)
    ks = rng.lognormal(0, 1, (L, Hkv, D // 2))
    vs = rng.lognormal(0, 1, (L, Hkv, D))
    tabs = O.build_tables(ks, vs, [P] * L, [dv] * L, D, 10000.0, pairing)
    Wq = rng.normal(0, 0.3, (Hq * D, hidden))
    Wk = rng.normal(0, 0.3, (Hkv * D, hidden))
    Wv = rng.normal(0, 0.3, (Hkv * D, hidden))
    X = rng.normal(0, 1, (n, hidden))
    return dict(P=P, dv=dv, tabs=tabs, Wq=Wq, Wk=Wk, Wv=Wv, X=X, D=D, Hq=Hq, Hkv=Hkv,
                pairing=pairing, theta=10000.0, ks=ks, vs=vs)


def _reduced(m, layer=0, **kw):
    w = O.gather_weights(m["Wq"], m["Wk"], m["Wv"], m["tabs"], layer, m["P"], m["dv"], m["D"])
    return O.reduced_attention_from_hidden(m["X"], w, m["tabs"]["inv_freq"][layer], m["Hq"], m["Hkv"],
                                           m["P"], m["dv"], m["D"], **kw)


def _full(m, layer=0, **kw):
    return O.full_masked_attention(m["X"], m["Wq"], m["Wk"], m["Wv"], m["tabs"]["k_pair_idx"][layer],
                                   m["tabs"]["v_idx"][layer], m["D"], m["theta"], m["pairing"],
                                   m["Hq"], m["Hkv"], m["P"], m["dv"], **kw)


# ---- storage rounding ------------------------------------------------------------------
def test_round_bf16_matches_library_rounding():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.normal(0, 1, 5000), rng.normal(0, 1e-3, 2000), rng.normal(0, 1e4, 2000),
                        [0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895314e38, 1e-40]]).astype(np.float32)
    want = torch.from_numpy(x).to(torch.bfloat16).to(torch.float64).numpy()
    got = O.round_bf16(x)
    assert np.array_equal(got, want)
    # ties go to even: 1 + 2^-8 is halfway between 1 and 1 + 2^-7
    assert O.round_bf16(np.float32(1.00390625)) == 1.0
    assert O.round_bf16(np.float32(1.01171875)) == 1.015625


# ---- tables ----------------------------------------------------------------------------
def test_counts_match_table13():
    rows = [l.split() for l in open(os.path.join(GOLD, "table13_retained_fraction.txt"))
            if l.strip() and not l.startswith("#")]
    assert len(rows) == 5
    for rho, frac in rows:
        P, dv = O.retained_counts(float(rho), 128)
        assert f"{P / 64:.3f}" == frac or abs(P / 64 - float(frac)) < 5.1e-4
    # the budgets the workloads name
    assert O.retained_counts(0.75, 64) == (24, 48)
    assert O.retained_counts(0.9, 128) == (58, 115)
    assert O.retained_counts(0.7, 128) == (45, 90)
    assert O.retained_counts(1.0, 128) == (64, 128)
    for rho, (P, dv) in synth.SWEEP_COUNTS.items():
        assert O.retained_counts(rho, 128) == (P, dv)


def test_bytes_per_token_table15():
    rows = dict(l.split() for l in open(os.path.join(GOLD, "table15_bytes_per_token.txt"))
                if l.strip() and not l.startswith("#"))
    dense = O.kv_bytes_per_token(32, 8, 128, 128, 2)
    assert dense == int(rows["dense"]) * 1024
    P, dv = O.retained_counts(0.7, 128)
    rap = O.kv_bytes_per_token(32, 8, 2 * P, dv, 2)
    assert rap == 92160
    assert abs(rap / 1024 - float(rows["rap0.7"])) < 1.0 and rap / dense < 0.705


def test_cost_model_table3():
    rows = dict((l.split()[0], l.split()[1:]) for l in open(os.path.join(GOLD, "table3_cost_model.txt"))
                if l.strip() and not l.startswith("#"))
    # RAP: cache, params and FLOPs of the K/V side all scale with the retained fraction.
    S, H, D = 1000, 32, 128
    for rho in (0.9, 0.7, 0.5):
        P, dv = O.retained_counts(rho, D)
        assert O.attn_read_bytes(1, 1, S, 2 * P, dv, 1) / (2 * S * D) == pytest.approx(rho, abs=0.007)
        assert (H * D) * (2 * P + dv) / (2 * H * D * D) == pytest.approx(rho, abs=0.007)
    assert 0.7 / (2 * 32) == pytest.approx(float(rows["palu_leftover_rho0.7_H32"][0]), abs=5e-4)
    assert 4096 * 4096 / 1e6 == pytest.approx(float(rows["wq_millions"][0]), abs=5e-3)
    assert 4096 * 1024 / 1e6 == pytest.approx(float(rows["wk_millions"][0]), abs=5e-3)


def test_topk_brute_force_and_ties():
    rng = np.random.default_rng(1)
    for _ in range(50):
        n = int(rng.integers(1, 12))
        k = int(rng.integers(1, n + 1))
        s = rng.integers(0, 4, n).astype(np.float64)          # many ties
        got = O.top_k_ascending(s, k)
        # brute force: repeatedly take the largest remaining, lowest index on ties
        left, pick = list(range(n)), []
        for _ in range(k):
            best = left[0]
            for i in left:
                if s[i] > s[best]:
                    best = i
            pick.append(best)
            left.remove(best)
        assert list(got) == sorted(pick)
    s = rng.lognormal(0, 1, 64)
    assert list(O.top_k_ascending(s, 20)) == sorted(np.argsort(-s, kind="stable")[:20].tolist())
    assert list(O.top_k_ascending([1.0, 5.0, 5.0, 5.0, 0.0], 2)) == [1, 2]


@pytest.mark.parametrize("pairing", [O.PAIR_HALF, O.PAIR_ADJACENT])
def test_selection_matrix_properties(pairing):
    m = _small(pairing=pairing, D=16, rho=0.6)
    D, P = m["D"], m["P"]
    for h in range(m["Hkv"]):
        pairs = m["tabs"]["k_pair_idx"][0, h, :P]
        idx = m["tabs"]["k_dim_idx"][0, h, :2 * P]
        assert np.all(np.diff(pairs) > 0) and pairs.min() >= 0 and pairs.max() < D // 2
        assert np.all(m["tabs"]["k_pair_idx"][0, h, P:] == -1)
        assert np.all(m["tabs"]["k_dim_idx"][0, h, 2 * P:] == -1)
        E = O.selection_matrix(idx, D)
        assert np.array_equal(E @ E.T, np.eye(2 * P))                 # E_k E_k^T = I
        M = E.T @ E
        assert np.array_equal(M, np.diag(np.diag(M))) and set(np.diag(M)) <= {0.0, 1.0}
        # whole pairs only: both members kept or both dropped
        for i in range(D // 2):
            a, b = (i, i + D // 2) if pairing == O.PAIR_HALF else (2 * i, 2 * i + 1)
            assert M[a, a] == M[b, b] == (1.0 if i in pairs else 0.0)
        # E_k R_t = R_(t,S) E_k : selecting after the full rotation == index-aware rotation
        x = np.random.default_rng(h).normal(size=D)
        for t in (0, 1, 17, 4097):
            lhs = E @ O.textbook_rope(x, t, D, m["theta"], pairing)
            rhs = O.rope_reduced(E @ x, t, m["tabs"]["inv_freq"][0, h])
            assert np.allclose(lhs, rhs, rtol=0, atol=1e-12)
        # frequencies are those of the ORIGINAL pair indices
        want = np.array([m["theta"] ** (-2.0 * i / D) for i in pairs])
        assert np.allclose(m["tabs"]["inv_freq"][0, h, :P], want, rtol=1e-15, atol=0)
        v = m["tabs"]["v_idx"][0, h, :m["dv"]]
        assert np.all(np.diff(v) > 0) and v.min() >= 0 and v.max() < D


# ---- rho = 1: nothing removed -> textbook RoPE GQA attention ----------------------------
def _textbook_gqa(X, Wq, Wk, Wv, D, Hq, Hkv, theta):
    """Plain rotate-half RoPE attention written with array ops, no RAP objects at all."""
    n = X.shape[0]
    inv = 1.0 / (theta ** (np.arange(0, D, 2) / D))
    ang = np.arange(n)[:, None] * inv[None, :]
    cos = np.concatenate([np.cos(ang), np.cos(ang)], axis=1)
    sin = np.concatenate([np.sin(ang), np.sin(ang)], axis=1)

    def rot(x):   # x [n][heads][D]
        x1, x2 = x[..., : D // 2], x[..., D // 2:]
        return x * cos[:, None, :] + np.concatenate([-x2, x1], axis=-1) * sin[:, None, :]

    q = rot((X @ Wq.T).reshape(n, Hq, D))[-1]
    k = rot((X @ Wk.T).reshape(n, Hkv, D))
    v = (X @ Wv.T).reshape(n, Hkv, D)
    out = np.zeros((Hq, D))
    for g in range(Hq):
        h = g // (Hq // Hkv)
        s = k[:, h, :] @ q[g] / np.sqrt(D)
        p = np.exp(s - s.max())
        out[g] = (p / p.sum()) @ v[:, h, :]
    return out


def test_rho1_equals_textbook_attention():
    m = _small(rho=1.0, D=16, Hq=6, Hkv=2, n=9)
    out, _, _, _ = _reduced(m)
    ref = _textbook_gqa(m["X"], m["Wq"], m["Wk"], m["Wv"], m["D"], m["Hq"], m["Hkv"], m["theta"])
    # reduced V coordinates at rho=1 are all channels in ascending order
    assert np.allclose(out, ref, rtol=0, atol=1e-12)


# ---- rho < 1: reduced path == full-dimensional masked path ------------------------------
@pytest.mark.parametrize("pairing", [O.PAIR_HALF, O.PAIR_ADJACENT])
@pytest.mark.parametrize("rho", [0.75, 0.4])
def test_reduced_equals_full_masked(pairing, rho):
    m = _small(pairing=pairing, rho=rho, D=16, Hq=4, Hkv=2, n=8, seed=11)
    out, _, _, _ = _reduced(m)
    ref = _full(m)
    assert np.allclose(out, ref, rtol=0, atol=1e-12)


def test_negative_controls_break_the_identity():
    m = _small(rho=0.5, D=16, n=8, seed=5)
    out, _, _, _ = _reduced(m)
    # a 1/sqrt(2P) scale is NOT what the method computes
    wrong_scale = _full(m, scale_dim=2 * m["P"])
    assert np.abs(out - wrong_scale).max() > 1e-4
    # re-indexed frequencies theta^(-2c/D) (c = reduced index) are not index-aware
    w = O.gather_weights(m["Wq"], m["Wk"], m["Wv"], m["tabs"], 0, m["P"], m["dv"], m["D"])
    reidx = np.tile(O.textbook_inv_freq(m["D"], m["theta"])[None, :], (m["Hkv"], 1))
    bad, _, _, _ = O.reduced_attention_from_hidden(m["X"], w, reidx, m["Hq"], m["Hkv"], m["P"], m["dv"], m["D"])
    assert np.abs(bad - _full(m)).max() > 1e-4
    # gathering W_q with another KV head's indices breaks it as well
    tabs2 = {k: v.copy() for k, v in m["tabs"].items()}
    tabs2["k_dim_idx"][0, 0], tabs2["k_dim_idx"][0, 1] = m["tabs"]["k_dim_idx"][0, 1], m["tabs"]["k_dim_idx"][0, 0]
    assert not np.array_equal(tabs2["k_dim_idx"], m["tabs"]["k_dim_idx"])
    w_bad = O.gather_weights(m["Wq"], m["Wk"], m["Wv"], m["tabs"], 0, m["P"], m["dv"], m["D"])
    w_swapped = O.gather_weights(m["Wq"], m["Wk"], m["Wv"], tabs2, 0, m["P"], m["dv"], m["D"])
    nq = m["Hq"] * 2 * m["P"]
    w_bad[:nq] = w_swapped[:nq]          # q rows follow the wrong head, k rows the right one
    bad, _, _, _ = O.reduced_attention_from_hidden(m["X"], w_bad, m["tabs"]["inv_freq"][0], m["Hq"], m["Hkv"],
                                                   m["P"], m["dv"], m["D"])
    assert np.abs(bad - _full(m)).max() > 1e-4


# ---- R_m^T R_n = R_(n-m): per-pair relative formula, shift invariance ---------------------
def test_per_pair_relative_rotation_identity():
    rng = np.random.default_rng(7)
    P = 5
    inv = 10000.0 ** (-2.0 * np.array([0, 3, 4, 9, 15]) / 32)
    q, k = rng.normal(size=2 * P), rng.normal(size=2 * P)
    for m_pos, n_pos in [(0, 0), (5, 2), (100, 131), (4096, 17)]:
        lhs = O.rope_reduced(q, m_pos, inv) @ O.rope_reduced(k, n_pos, inv)
        rhs = 0.0
        for c in range(P):
            aq, bq, ak, bk = q[2 * c], q[2 * c + 1], k[2 * c], k[2 * c + 1]
            d = (n_pos - m_pos) * inv[c]
            rhs += (aq * ak + bq * bk) * math.cos(d) + (bq * ak - aq * bk) * math.sin(d)
        assert lhs == pytest.approx(rhs, abs=1e-11)
    # rotation by 0 is the identity; rotation preserves the norm of every pair
    assert np.array_equal(O.rope_reduced(q, 0, inv), q)
    r = O.rope_reduced(q, 77, inv)
    assert np.allclose(r[0::2] ** 2 + r[1::2] ** 2, q[0::2] ** 2 + q[1::2] ** 2, atol=1e-12)
    # quarter turn: (a, b) -> (-b, a) when pos * inv_freq = pi / 2
    r = O.rope_reduced([2.0, 3.0], 1, [math.pi / 2])
    assert r == pytest.approx([-3.0, 2.0], abs=1e-15)


def test_position_shift_invariance():
    m = _small(rho=0.75, D=16, n=6, seed=2)
    w = O.gather_weights(m["Wq"], m["Wk"], m["Wv"], m["tabs"], 0, m["P"], m["dv"], m["D"])
    n = m["X"].shape[0]

    def logits(offset):
        q, k, _ = O.qkv_rope(m["X"], w, None, np.arange(n) + offset, m["tabs"]["inv_freq"][0],
                             m["Hq"], m["Hkv"], m["P"], m["dv"])
        return np.array([[q[-1, g] @ k[j, g // 2] for j in range(n)] for g in range(m["Hq"])])

    base = logits(0)
    for off in (1, 1000, 100000):
        assert np.allclose(logits(off), base, rtol=0, atol=1e-9)


# ---- attention: brute force and closed forms ---------------------------------------------
def test_attention_brute_force_tiny():
    rng = np.random.default_rng(4)
    B, Hq, Hkv, P2, dv, cap, D = 2, 4, 2, 4, 3, 5, 8
    q = rng.normal(size=(B, Hq, P2))
    K = rng.normal(size=(B, Hkv, cap, P2))
    V = rng.normal(size=(B, Hkv, cap, dv))
    lens = [3, 5]
    got = O.decode_attn(q, K, V, lens, D)
    for b in range(B):
        for g in range(Hq):
            h = g // 2
            s = []
            for j in range(lens[b]):
                acc = 0.0
                for d in range(P2):
                    acc += q[b, g, d] * K[b, h, j, d]
                s.append(acc / math.sqrt(D))
            mx = max(s)
            e = [math.exp(x - mx) for x in s]
            z = sum(e)
            for c in range(dv):
                want = sum(e[j] / z * V[b, h, j, c] for j in range(lens[b]))
                assert got[b, g, c] == pytest.approx(want, abs=1e-14)


def test_attention_closed_forms():
    V = np.array([[[[1.0, 2.0], [5.0, -2.0], [9.0, 9.0]]]])
    K = np.array([[[[0.3, 0.1], [0.3, 0.1], [7.0, 7.0]]]])
    q = np.array([[[1.0, -2.0]]])
    # one cached token: the output is that token's V row
    assert np.array_equal(O.decode_attn(q, K, V, [1], 4)[0, 0], [1.0, 2.0])
    # two tokens with equal logits: the mean of the two V rows; the third row is not read
    assert O.decode_attn(q, K, V, [2], 4)[0, 0] == pytest.approx([3.0, 0.0], abs=1e-15)
    # scale 1/sqrt(D): logits (ln 3) * sqrt(D) / sqrt(D) -> weights 3:1
    D = 16
    K2 = np.array([[[[math.log(3.0) * math.sqrt(D)], [0.0]]]])
    V2 = np.array([[[[1.0], [0.0]]]])
    assert O.decode_attn(np.array([[[1.0]]]), K2, V2, [2], D)[0, 0, 0] == pytest.approx(0.75, abs=1e-15)


def test_split_combine_invariance():
    rng = np.random.default_rng(9)
    n, P2, dv, D = 53, 6, 5, 16
    q, K, V = rng.normal(size=P2) * 3, rng.normal(size=(n, P2)), rng.normal(size=(n, dv))
    ref = O.decode_attn(q[None, None], K[None, None], V[None, None], [n], D)[0, 0]
    for cuts in ([0, 53], [0, 1, 53], [0, 10, 10, 31, 53], [0, 0, 20, 53, 53]):
        parts = [O.attn_partial(q, K[a:b], V[a:b], D) for a, b in zip(cuts[:-1], cuts[1:])]
        assert np.allclose(O.combine_partials(parts), ref, rtol=0, atol=1e-13)


def test_append_layout():
    K = np.full((2, 2, 4, 2), -7.0)
    V = np.full((2, 2, 4, 3), -7.0)
    k_new = np.arange(8, dtype=np.float64).reshape(2, 2, 2) + 1.00390625
    v_new = np.arange(12, dtype=np.float64).reshape(2, 2, 3)
    O.append(K, V, k_new, v_new, seq_id=[1, 0], slot=[3, 0], dtype="bf16")
    assert np.array_equal(K[1, :, 3, :], O.round_bf16(k_new[0])) and np.array_equal(V[0, :, 0, :], v_new[1])
    touched = np.zeros((2, 2, 4), bool)
    touched[1, :, 3] = touched[0, :, 0] = True
    assert np.all(K[~touched] == -7.0) and np.all(V[~touched] == -7.0)


# ---- low-rank comparator ------------------------------------------------------------------
def test_lowrank_comparator_reduces_to_textbook():
    """With B_k = E_k (a selection) and latent = unrotated reduced K, rebuilding + full RoPE
    equals the masked full-dim attention, i.e. the RAP result."""
    m = _small(rho=0.5, D=16, Hq=4, Hkv=2, n=6, seed=21)
    D, P, Hkv, Hq = m["D"], m["P"], m["Hkv"], m["Hq"]
    n = m["X"].shape[0]
    w = O.gather_weights(m["Wq"], m["Wk"], m["Wv"], m["tabs"], 0, P, m["dv"], D)
    y = O.project(m["X"], w)
    off = Hq * 2 * P
    latent = np.stack([y[:, off + h * 2 * P: off + (h + 1) * 2 * P] for h in range(Hkv)])[None]
    off += Hkv * 2 * P
    V = np.stack([y[:, off + h * m["dv"]: off + (h + 1) * m["dv"]] for h in range(Hkv)])[None]
    Bk = np.stack([O.selection_matrix(m["tabs"]["k_dim_idx"][0, h, :2 * P], D) for h in range(Hkv)])
    qfull = (m["Wq"] @ m["X"][-1]).reshape(Hq, D)
    qrot = np.stack([O.textbook_rope(qfull[g], n - 1, D, m["theta"], m["pairing"]) for g in range(Hq)])[None]
    got = O.lowrank_decode_attn(qrot, latent, Bk, V, [n], D, m["theta"], m["pairing"])[0]
    assert np.allclose(got, _full(m), rtol=0, atol=1e-12)


# ---- output projection on the retained V channels --------------------------------------------
def test_out_proj_equals_dense_wo_on_zero_expanded_output():
    """W~_o o_reduced == W_o (E_v^T o_reduced): expanding the reduced attention output back to D
    channels (zeros where V was pruned) and applying the dense W_o gives the same hidden vector."""
    m = _small(rho=0.5, D=16, Hq=4, Hkv=2, n=5, seed=31)
    D, Hq, Hkv, dv, hidden = m["D"], m["Hq"], m["Hkv"], m["dv"], m["X"].shape[1]
    rng = np.random.default_rng(8)
    Wo = rng.normal(0, 0.05, (hidden, Hq * D))
    o = rng.normal(0, 1.0, (3, Hq, dv))
    wt = O.gather_wo(Wo, m["tabs"], 0, dv, D, Hq, Hkv)
    assert wt.shape == (hidden, Hq * dv)
    got = O.out_proj(o, wt)
    G = Hq // Hkv
    full = np.zeros((3, Hq, D))
    for g in range(Hq):
        for c in range(dv):
            full[:, g, m["tabs"]["v_idx"][0, g // G, c]] = o[:, g, c]
    want = full.reshape(3, Hq * D) @ Wo.T
    assert np.allclose(got, want, rtol=0, atol=1e-13)
    # the gather itself, column by column
    for g in range(Hq):
        for c in range(dv):
            assert np.array_equal(wt[:, g * dv + c], Wo[:, g * D + m["tabs"]["v_idx"][0, g // G, c]])
    # negative control: using another head's V selection breaks the identity
    bad = O.gather_wo(Wo, m["tabs"], 0, dv, D, Hq, Hkv)[:, ::-1]
    assert np.abs(O.out_proj(o, bad) - want).max() > 1e-3


# ---- Budget-Alloc (Algorithm 2) ----------------------------------------------------------------
def test_budget_alloc_properties():
    rng = np.random.default_rng(4)
    D, L, H = 128, 32, 8
    for rho in (0.5, 0.7, 0.9):
        sc = rng.lognormal(0, 1, (L, H, D // 2)) * np.linspace(0.6, 1.6, L)[:, None, None]
        m, nv = O.budget_alloc(sc, rho, D)
        sigma = sc.reshape(L, -1).mean(axis=1)
        assert m.sum() == round(rho * 64 * L)                      # mean retain ratio = rho (Algorithm 2)
        assert m.min() >= 1 and m.max() <= 64 and np.array_equal(nv, 2 * m)   # whole pairs; V keeps 2 m_l
        order = np.argsort(sigma)
        assert np.all(np.diff(m[order]) >= 0)                     # more sensitive layers never get less
        if m.max() < 64 and m.min() > 1:                          # no clipping: proportional up to rounding
            t = rho * 64 * L * sigma / sigma.sum()
            assert np.abs(m - t).max() < 1.0
    # equal layer scores: the uniform budget (rho * D/2 whole pairs everywhere when that is an integer;
    # otherwise the layers differ by at most one pair and the mean is kept)
    m, _ = O.budget_alloc(np.ones((8, 2, 64)), 0.75, 128)
    assert np.array_equal(m, np.full(8, 48))
    m, _ = O.budget_alloc(np.ones((8, 2, 64)), 0.7, 128)
    assert m.sum() == 358 and set(m.tolist()) == {44, 45}
    # the tie rule, worked by hand: total = round(0.7 * 64 * 8) = 358, every share is 358 / 8 = 44.75, the floors
    # give 8 * 44 = 352, and the six missing pairs go to equal fractional parts in layer order: layers 0..5
    assert m.tolist() == [45, 45, 45, 45, 45, 45, 44, 44]
    # two layers with a larger fraction come first, then the tie among the others is broken by layer index:
    # scores (1, 1, 1.1, 1, 1.1, 1), rho = 0.5, D = 16: total 24, shares 3.871 (x4) and 4.258 (x2), floors 3 / 4
    # sum to 20, the four missing pairs go to fraction 0.871 in layer order -> layers 0, 1, 3, 5
    sc = np.ones((6, 1, 8)) * np.array([1, 1, 1.1, 1, 1.1, 1])[:, None, None]
    m, nv = O.budget_alloc(sc, 0.5, 16)
    assert m.tolist() == [4, 4, 4, 4, 4, 4] and nv.tolist() == [8] * 6
    sc = np.ones((6, 1, 8)) * np.array([1, 1, 1.3, 1, 1.3, 1])[:, None, None]
    # shares 24 / 6.6 = 3.636 (x4) and 4.727 (x2): floors 3, 3, 4, 3, 4, 3 = 20; fractions 0.727 (layers 2, 4) beat
    # 0.636, so they take two of the four missing pairs and the tie among the rest gives the other two to layers 0, 1
    m, _ = O.budget_alloc(sc, 0.5, 16)
    assert m.tolist() == [4, 4, 5, 3, 5, 3]
    # one dominant layer is capped at all pairs and the rest share what is left
    sc = np.ones((4, 1, 32)); sc[0] *= 100
    m, _ = O.budget_alloc(sc, 0.5, 64)
    assert m[0] == 32 and m.sum() == 64 and np.all(m[1:] >= 10)


# ---- prefill (causal block) attention on the reduced dims --------------------------------------
def test_prefill_attn_equals_per_token_decode_attention():
    """The masked-matrix form equals running the decode definition token by token with the prefix length
    of each token (Eq. 2 holds for every t), and the first token of an empty cache returns V_0."""
    rng = np.random.default_rng(17)
    B, T, Hq, Hkv, P2, dv, D, cap = 2, 5, 4, 2, 6, 5, 8, 16
    K = rng.normal(0, 1, (B, Hkv, cap, P2))
    V = rng.normal(0, 1, (B, Hkv, cap, dv))
    q = rng.normal(0, 1, (B, T, Hq, P2))
    start = [3, 0]
    got = O.prefill_attn(q, K, V, start, D)
    for i in range(T):
        want = O.decode_attn(q[:, i], K, V, [start[0] + i + 1, start[1] + i + 1], D)
        assert np.allclose(got[:, i], want, rtol=0, atol=1e-13)
    assert np.allclose(got[1, 0], np.repeat(V[1, :, 0, :], Hq // Hkv, axis=0), rtol=0, atol=1e-15)
    # a future row must not leak: changing rows after a token's position leaves its output unchanged
    K2, V2 = K.copy(), V.copy()
    K2[:, :, 6:, :] += 5.0
    V2[:, :, 6:, :] -= 3.0
    got2 = O.prefill_attn(q, K2, V2, start, D)
    assert np.array_equal(got2[0, :3], got[0, :3]) and not np.allclose(got2[0, 3:], got[0, 3:])


# ---- hybrid models: layers without RoPE are channel-pruned -------------------------------------------
def test_nope_layer_tables_give_plain_channel_pruned_attention():
    """In a layer without positional rotation the reduced path (zero frequencies, per-channel K selection)
    equals full-width dot-product attention with the dropped K channels zeroed -- written out with loops."""
    m = _small(rho=0.5, D=16, Hq=4, Hkv=2, n=6, seed=41)
    D, Hq, Hkv, P, dv = m["D"], m["Hq"], m["Hkv"], m["P"], m["dv"]
    rng = np.random.default_rng(3)
    kc = rng.lognormal(0, 1, (1, Hkv, D))
    tabs = O.build_tables_hybrid(m["ks"], kc, m["vs"], [0], [P], [dv], D, m["theta"], m["pairing"])
    assert np.all(tabs["inv_freq"] == 0.0) and np.all(tabs["k_pair_idx"] == -1)
    for h in range(Hkv):
        want = np.sort(np.argsort(-kc[0, h], kind="stable")[: 2 * P])
        assert np.array_equal(tabs["k_dim_idx"][0, h, : 2 * P], want)
    w = O.gather_weights(m["Wq"], m["Wk"], m["Wv"], tabs, 0, P, dv, D)
    got, _, _, _ = O.reduced_attention_from_hidden(m["X"], w, tabs["inv_freq"][0], Hq, Hkv, P, dv, D)
    # full-width reference without any rotation
    X, n, G = m["X"], m["X"].shape[0], Hq // Hkv
    want = np.zeros((Hq, dv))
    for g in range(Hq):
        h = g // G
        keep = set(int(i) for i in tabs["k_dim_idx"][0, h, : 2 * P])
        q = m["Wq"][g * D:(g + 1) * D] @ X[-1]
        s = np.empty(n)
        for j in range(n):
            k = m["Wk"][h * D:(h + 1) * D] @ X[j]
            s[j] = sum(q[d] * k[d] for d in range(D) if d in keep) / math.sqrt(D)
        pr = np.exp(s - s.max()); pr /= pr.sum()
        for c in range(dv):
            u = tabs["v_idx"][0, h, c]
            want[g, c] = sum(pr[j] * float(m["Wv"][h * D + u] @ X[j]) for j in range(n))
    assert np.allclose(got, want, rtol=0, atol=1e-12)
    # a rotary layer of the same call is unchanged
    t2 = O.build_tables_hybrid(np.concatenate([m["ks"], m["ks"]]), np.concatenate([kc, kc]), np.concatenate([m["vs"], m["vs"]]),
                               [1, 0], [P, P], [dv, dv], D, m["theta"], m["pairing"])
    assert np.array_equal(t2["k_dim_idx"][0], m["tabs"]["k_dim_idx"][0]) and np.array_equal(t2["inv_freq"][0], m["tabs"]["inv_freq"][0])


# ---- partial rotary: RAP on the rotated dims of a head, channel pruning on the rest -----------------
def test_partial_rotary_tables_reduce_to_the_full_and_the_unrotated_case():
    m = _small(rho=0.75, D=16, Hq=4, Hkv=2, n=5, seed=17)
    D, Hkv, P, dv = m["D"], m["Hkv"], m["P"], m["dv"]
    kc = np.random.default_rng(4).lognormal(0, 1, (1, Hkv, D))
    full = O.build_tables_partial(m["ks"], kc, m["vs"], [D], [P], [P], [dv], D, m["theta"], m["pairing"])
    for key in ("k_pair_idx", "k_dim_idx", "v_idx", "inv_freq"):
        assert np.array_equal(full[key], m["tabs"][key]), key
    none = O.build_tables_partial(m["ks"], kc, m["vs"], [0], [0], [P], [dv], D, m["theta"], m["pairing"])
    want = O.build_tables_hybrid(m["ks"], kc, m["vs"], [0], [P], [dv], D, m["theta"], m["pairing"])
    for key in ("k_pair_idx", "k_dim_idx", "v_idx", "inv_freq"):
        assert np.array_equal(none[key], want[key]), key


@pytest.mark.parametrize("pairing", [O.PAIR_HALF, O.PAIR_ADJACENT])
def test_partial_rotary_reduced_path_equals_full_width_attention(pairing):
    """Rotate only the first R dims of each head (the usual formulation, applied to that block with its own
    table theta^(-2i/R)), zero the dropped K dims, keep the retained V channels: the reduced path built from
    build_tables_partial gives the same output."""
    m = _small(pairing=pairing, rho=0.75, D=16, Hq=4, Hkv=2, n=6, seed=29)
    D, Hq, Hkv, dv, X = m["D"], m["Hq"], m["Hkv"], m["dv"], m["X"]
    R, Pr, P = 8, 3, 5                          # 3 of 4 rotated pairs, 4 of 8 unrotated channels
    kc = np.random.default_rng(8).lognormal(0, 1, (1, Hkv, D))
    tabs = O.build_tables_partial(m["ks"], kc, m["vs"], [R], [Pr], [P], [dv], D, m["theta"], pairing)
    # structure: pairs inside the rotated block, channels outside, zero frequency on the channel slots
    for h in range(Hkv):
        dims = tabs["k_dim_idx"][0, h, : 2 * P]
        assert len(set(dims.tolist())) == 2 * P and np.all(dims[: 2 * Pr] < R) and np.all(dims[2 * Pr:] >= R)
        assert np.all(np.diff(dims[2 * Pr:]) > 0) and np.all(tabs["inv_freq"][0, h, Pr:] == 0.0)
        for c in range(Pr):
            i = int(tabs["k_pair_idx"][0, h, c])
            assert tabs["inv_freq"][0, h, c] == m["theta"] ** (-2.0 * i / R)
        want_ch = R + np.sort(np.argsort(-kc[0, h, R:], kind="stable")[: 2 * (P - Pr)])
        assert np.array_equal(dims[2 * Pr:], want_ch)
    w = O.gather_weights(m["Wq"], m["Wk"], m["Wv"], tabs, 0, P, dv, D)
    got, _, _, _ = O.reduced_attention_from_hidden(X, w, tabs["inv_freq"][0], Hq, Hkv, P, dv, D)
    n, G = X.shape[0], Hq // Hkv

    def rot(x, pos):
        return np.concatenate([O.textbook_rope(x[:R], pos, R, m["theta"], pairing), x[R:]])

    want = np.zeros((Hq, dv))
    for g in range(Hq):
        h = g // G
        keep = [int(d) for d in tabs["k_dim_idx"][0, h, : 2 * P]]
        q = rot(m["Wq"][g * D:(g + 1) * D] @ X[-1], n - 1)
        s = np.empty(n)
        for j in range(n):
            k = rot(m["Wk"][h * D:(h + 1) * D] @ X[j], j)
            s[j] = sum(q[d] * k[d] for d in keep) / math.sqrt(D)
        pr = np.exp(s - s.max()); pr /= pr.sum()
        for c in range(dv):
            u = tabs["v_idx"][0, h, c]
            want[g, c] = sum(pr[j] * float(m["Wv"][h * D + u] @ X[j]) for j in range(n))
    assert np.allclose(got, want, rtol=0, atol=1e-12)
    # the pin bites: a table that forgets the block-local frequency (theta^(-2i/D) instead of /R) fails it
    bad = {k: v.copy() for k, v in tabs.items()}
    for h in range(Hkv):
        for c in range(Pr):
            bad["inv_freq"][0, h, c] = m["theta"] ** (-2.0 * int(tabs["k_pair_idx"][0, h, c]) / D)
    got_bad, _, _, _ = O.reduced_attention_from_hidden(X, w, bad["inv_freq"][0], Hq, Hkv, P, dv, D)
    assert not np.allclose(got_bad, want, rtol=0, atol=1e-6)


# ---- frequency-scaled RoPE variants (Section 4, "Practical Considerations") -----------------------
def _full_width_rope_with_table(x, pos, freq, pairing):
    """Full-width RoPE of one head vector with an arbitrary per-pair frequency table, written as D/2 explicit
    2x2 rotations (no RAP object, no oracle call)."""
    D = len(x)
    y = np.array(x, dtype=np.float64)
    for i in range(D // 2):
        a, b = (i, i + D // 2) if pairing == O.PAIR_HALF else (2 * i, 2 * i + 1)
        c, s = math.cos(pos * freq[i]), math.sin(pos * freq[i])
        y[a], y[b] = x[a] * c - x[b] * s, x[a] * s + x[b] * c
    return y


@pytest.mark.parametrize("pairing", [O.PAIR_HALF, O.PAIR_ADJACENT])
def test_scaled_frequency_tables_keep_the_pair_identities(pairing):
    """A model table that is not theta^(-2i/D) (every pair slowed down by its own factor, as a context-extension
    variant does): the selection is unchanged, E_k R_t = R_(t,S) E_k holds with the scaled full table, the reduced
    attention equals full-width attention under that table with the removed pairs zeroed, and taking the table
    by reduced position c instead of original pair i_c breaks it."""
    m = _small(pairing=pairing, D=16, rho=0.6, n=9, seed=21, L=2)
    D, P, dv, Hq, Hkv = m["D"], m["P"], m["dv"], m["Hq"], m["Hkv"]
    rng = np.random.default_rng(8)
    base = np.array([m["theta"] ** (-2.0 * i / D) for i in range(D // 2)])
    freq = np.stack([base * rng.uniform(0.1, 1.0, D // 2), base / np.linspace(1.0, 8.0, D // 2)])   # [L][D/2]
    tabs = O.build_tables_freq(m["ks"], m["vs"], freq, [P] * 2, [dv] * 2, D, pairing)
    for key in ("k_pair_idx", "k_dim_idx", "v_idx"):
        assert np.array_equal(tabs[key], m["tabs"][key])
    # the standard table through the same call reproduces build_tables
    std = O.build_tables_freq(m["ks"], m["vs"], np.stack([base, base]), [P] * 2, [dv] * 2, D, pairing)
    assert np.allclose(std["inv_freq"], m["tabs"]["inv_freq"], rtol=1e-15, atol=0)
    G = Hq // Hkv
    for l in range(2):
        for h in range(Hkv):
            pairs = tabs["k_pair_idx"][l, h, :P]
            assert np.array_equal(tabs["inv_freq"][l, h, :P], freq[l][pairs])
            assert np.all(tabs["inv_freq"][l, h, P:] == 0.0)
            E = O.selection_matrix(tabs["k_dim_idx"][l, h, :2 * P], D)
            x = np.random.default_rng(10 * l + h).normal(size=D)
            for t in (0, 3, 250, 4097):
                lhs = E @ _full_width_rope_with_table(x, t, freq[l], pairing)
                assert np.allclose(lhs, O.rope_reduced(E @ x, t, tabs["inv_freq"][l, h]), rtol=0, atol=1e-12)
        # attention: reduced path with the gathered table == full width with the scaled table, removed pairs zeroed
        w = O.gather_weights(m["Wq"], m["Wk"], m["Wv"], tabs, l, P, dv, D)
        out, _, _, _ = O.reduced_attention_from_hidden(m["X"], w, tabs["inv_freq"][l], Hq, Hkv, P, dv, D)
        n = m["X"].shape[0]
        qf = (m["Wq"] @ m["X"][-1]).reshape(Hq, D)
        kf = (m["X"] @ m["Wk"].T).reshape(n, Hkv, D)
        vf = (m["X"] @ m["Wv"].T).reshape(n, Hkv, D)
        ref = np.zeros((Hq, dv))
        for g in range(Hq):
            h = g // G
            keep = np.zeros(D)
            keep[tabs["k_dim_idx"][l, h, :2 * P]] = 1.0
            qr = _full_width_rope_with_table(qf[g], n - 1, freq[l], pairing)
            s = np.array([qr @ (_full_width_rope_with_table(kf[j, h], j, freq[l], pairing) * keep) for j in range(n)])
            p = np.exp(s / math.sqrt(D) - (s / math.sqrt(D)).max())
            ref[g] = (p / p.sum()) @ vf[:, h, :][:, tabs["v_idx"][l, h, :dv]]
        assert np.allclose(out, ref, rtol=0, atol=1e-12)
        # negative control: frequencies taken by reduced position instead of by original pair
        wrong = np.zeros_like(tabs["inv_freq"][l])
        wrong[:, :P] = freq[l][:P]
        bad, _, _, _ = O.reduced_attention_from_hidden(m["X"], w, wrong, Hq, Hkv, P, dv, D)
        assert np.abs(bad - ref).max() > 1e-4


# ---- composition with KV-cache quantisation -----------------------------------------------------------
def _bf16_exact(fr):
    """Nearest bf16 (8 significant bits, ties to even) of a positive Fraction, as a Fraction -- exact arithmetic."""
    from fractions import Fraction
    e = 0
    while fr >= 2 ** (e + 1):
        e += 1
    while fr < 2 ** e:
        e -= 1
    ulp = Fraction(2) ** (e - 7)
    n = fr / ulp
    lo = n.numerator // n.denominator
    rem = n - lo
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and lo % 2 == 1):
        lo += 1
    return lo * ulp


def test_quantize_rows_against_exact_rational_arithmetic():
    """Codes and scale of hand-made rows recomputed with Fractions (no floating point): s = bf16(fp32(amax / 127)),
    c = round-half-even(x / s) clipped to +-127.  The rows are fp32 numbers, so the Fractions are their exact values;
    the fp32 divisions of the oracle are checked to land on the same codes, ties and clipping included."""
    from fractions import Fraction
    rng = np.random.default_rng(2)
    rows = [np.array([1.27, -0.635, 0.01, 0.0], dtype=np.float32),
            np.array([3.0, -3.0, 1.5, 0.75, 0.011811024], dtype=np.float32),
            np.array([1e-3, -2e-3, 5e-4], dtype=np.float32),
            rng.normal(0, 1.3, 90).astype(np.float32), rng.normal(0, 40.0, 115).astype(np.float32),
            np.zeros(7, dtype=np.float32)]
    for x in rows:
        codes, s = O.quantize_rows(x)
        amax = max(abs(Fraction(float(v))) for v in x)
        if amax == 0:
            assert s == 0.0 and not codes.any()
            continue
        s32 = Fraction(float(np.float32(float(amax)) / np.float32(127.0)))      # one fp32 division: the stated precision
        s_exact = _bf16_exact(s32)
        assert Fraction(float(s)) == s_exact
        for v, c in zip(x, codes):
            ratio = Fraction(float(v)) / s_exact
            # the fp32 quotient is the rounding of this exact ratio; away from .5 boundaries the code is fixed by it
            lo = ratio.numerator // ratio.denominator
            frac = ratio - lo
            want = lo + (1 if frac > Fraction(1, 2) else 0)
            if abs(frac - Fraction(1, 2)) < Fraction(1, 2 ** 12):
                assert int(c) in (max(-127, min(127, lo)), max(-127, min(127, lo + 1)))
            else:
                assert int(c) == max(-127, min(127, want)), (float(v), float(s), int(c), want)
    # the worked row: amax 1.27 -> s = bf16(0.01) = 0.010009765625 -> 126.88, -63.44, 0.999, 0
    codes, s = O.quantize_rows(np.array([1.27, -0.635, 0.01, 0.0], dtype=np.float32))
    assert s == 0.010009765625 and codes.tolist() == [127, -63, 1, 0]


def test_quantize_rows_round_trip_scale_equivariance_and_layout():
    rng = np.random.default_rng(5)
    x = (rng.normal(0, 1, (4, 3, 50, 90)) * rng.lognormal(0, 2, (4, 3, 50, 1))).astype(np.float32)
    codes, s = O.quantize_rows(x)
    assert codes.dtype == np.int8 and codes.shape == x.shape and s.shape == x.shape[:-1]
    assert np.abs(codes.astype(int)).max() <= 127
    back = O.dequantize_rows(codes, s)
    # round to nearest: half a step per element (the largest element may also lose what clipping to 127 takes:
    # the bf16 scale can sit up to 2^-9 below amax / 127)
    step = s[..., None]
    assert np.all(np.abs(back - x) <= 0.5 * step + np.abs(x) * 2.0 ** -8 + 1e-30)
    assert np.all(np.abs(back - x)[np.abs(codes) < 127] <= (0.5 * step * np.ones_like(x))[np.abs(codes) < 127] * (1 + 1e-6))
    # every row uses its range: the largest element maps to +-127 or +-126
    assert np.all(np.abs(codes).max(axis=-1) >= 126)
    # scaling a row by a power of two scales s by it and leaves the codes alone (all operations are exact then)
    c2, s2 = O.quantize_rows(x * np.float32(8.0))
    assert np.array_equal(c2, codes) and np.array_equal(s2, 8.0 * s)
    # rows are independent: a per-tensor scale would wipe out the small rows
    small = np.abs(x).max(axis=-1) < 0.05 * np.abs(x).max()
    assert small.any() and np.all(np.abs(codes[small]).max(axis=-1) >= 126)
    # the scale is a bf16 number
    assert np.array_equal(O.round_bf16(s), s)
    # all elements equal: one code value, +-127 or +-126, and the row comes back within half a step
    c, sc = O.quantize_rows(np.full((1, 16), -0.3, dtype=np.float32))
    assert len(set(c.ravel().tolist())) == 1 and c[0, 0] in (-127, -126) and abs(c[0, 0] * sc[0] + 0.3) <= 0.5 * sc[0]


def test_quantised_append_and_attention_closed_forms():
    """append_q8 writes exactly the named rows; decode_attn_q8 is Eq. 2 on c * s: a single cached row returns that
    row's dequantised V, equal K rows average the dequantised V rows, and the output moves by no more than the
    quantisation step of V when the cache is quantised (a bound, not a tolerance)."""
    rng = np.random.default_rng(9)
    B, Hkv, G, cap, P2, dv, D = 2, 2, 2, 8, 6, 5, 8
    k8 = np.zeros((B, Hkv, cap, P2), np.int8); ks = np.zeros((B, Hkv, cap))
    v8 = np.zeros((B, Hkv, cap, dv), np.int8); vs = np.zeros((B, Hkv, cap))
    k_new = rng.normal(0, 1, (3, Hkv, P2)); v_new = rng.normal(0, 2, (3, Hkv, dv))
    O.append_q8(k8, ks, v8, vs, k_new, v_new, [0, 1, 0], [0, 0, 1])
    touched = np.zeros((B, Hkv, cap), bool); touched[0, :, 0] = touched[1, :, 0] = touched[0, :, 1] = True
    assert not k8[~touched].any() and not vs[~touched].any() and np.all(ks[touched] > 0)
    assert np.array_equal(k8[0, :, 1], O.quantize_rows(k_new[2])[0]) and np.array_equal(vs[1, :, 0], O.quantize_rows(v_new[1])[1])
    q = rng.normal(0, 1, (B, Hkv * G, P2))
    out = O.decode_attn_q8(q, k8, ks, v8, vs, [2, 1], D)
    Vd = O.dequantize_rows(v8, vs)
    assert np.allclose(out[1], np.repeat(Vd[1, :, 0], G, axis=0), rtol=0, atol=1e-15)          # one row: its V
    k8[0, :, 1] = k8[0, :, 0]; ks[0, :, 1] = ks[0, :, 0]                                       # equal K rows: the mean
    out = O.decode_attn_q8(q, k8, ks, v8, vs, [2, 1], D)
    assert np.allclose(out[0], np.repeat(0.5 * (Vd[0, :, 0] + Vd[0, :, 1]), G, axis=0), rtol=0, atol=1e-15)
    # against the unquantised cache with the same K: a convex combination of V rows moves by at most half a V step
    Kd = O.dequantize_rows(k8, ks)
    Vfull = np.zeros((B, Hkv, cap, dv)); Vfull[0, :, 0] = v_new[0]; Vfull[0, :, 1] = v_new[2]; Vfull[1, :, 0] = v_new[1]
    ref = O.decode_attn(q, Kd, Vfull.astype(np.float32), [2, 1], D)
    assert np.abs(out - ref).max() <= 0.5 * vs.max() * (1 + 2.0 ** -7)
    # bytes per token of the layout: codes + 16-bit scale, rows padded to four bytes (8B shape, rho = 0.7: 184 B / head)
    assert O.kv_bytes_per_token_q8(32, 8, 90, 90) == 32 * 8 * (92 + 92)
    assert O.kv_bytes_per_token_q8(1, 1, 116, 115) == 120 + 120 and O.kv_bytes_per_token_q8(1, 1, 128, 128) == 264
