"""Parity at the workloads' full batch, context and head shapes, in the launch configuration the
benchmark times (same B, S, split heuristic; two layers instead of all, since the grid does not
depend on the layer count).  The oracle cannot afford whole outputs at these sizes, so it checks
sampled (layer, sequence, KV head) units one by one: it downloads that unit's cache slice and the
device's own q~ rows and recomputes the attention in fp64; the new token's q~ / k~ / v~ are checked
for every head against the fp64 projection + RoPE of the same bf16 inputs."""
from dataclasses import replace

import numpy as np
import pytest
import torch

from oracle import rap_oracle as O
from paper_2602_02599_b200 import synth
from paper_2602_02599_b200.stack import DecodeStack

import util

pytestmark = pytest.mark.gpu


def _sampled_units(L, B, H, n, rng):
    units = {(0, 0, 0), (L - 1, B - 1, H - 1), (0, B - 1, 0), (L - 1, 0, H - 1), (0, 0, H - 1), (L - 1, B - 1, 0)}
    while len(units) < n:
        units.add((int(rng.integers(L)), int(rng.integers(B)), int(rng.integers(H))))
    return sorted(units)


def _run(name, ragged):
    w = replace(synth.CONFIGS[name], n_layers=2)
    st = DecodeStack(w, max_rows=max(w.batch, 2048))
    st.build_tables(*synth.draw_scores(w))
    util_tabs = util.oracle_tables(w, *synth.draw_scores(w))
    st.fill_synthetic(w.seed)
    L, B, Hq, Hkv, G, D = w.n_layers, w.batch, w.n_q_heads, w.n_kv_heads, w.group, w.head_dim
    P, dv = w.n_pairs, w.n_vch
    lens = synth.ragged_lengths(w) if ragged else np.full(B, w.seq, dtype=np.int32)
    st.seq_len.copy_(torch.from_numpy(lens))
    X = np.stack([synth.draw_hidden(w, l, 3, B) for l in range(L)])
    dx = torch.from_numpy(X).to(st.device).to(st.dt).contiguous()
    q_dev = []
    # the step the benchmark times, layer by layer so that each layer's q~ can be kept
    seq_id = torch.arange(B, dtype=torch.int32, device=st.device)
    pos = st.seq_len.clone()
    for l in range(L):
        st.qkv_rope_append(l, dx[l], seq_id, pos, pos, int(lens.max()))
        q_dev.append(st.q_scratch.reshape(-1)[: B * Hq * 2 * P].reshape(B, Hq, 2 * P).clone())
        st.decode_attn(l, st.q_scratch, pos + 1, int(lens.max()) + 1)
    torch.cuda.synchronize()
    assert st.ctx.rap_get_last_device_status() == (0, 0)
    # a2-a4: every head of the new token in both layers
    for l in range(L):
        w_host = O.round_storage(synth.draw_packed_weights(w, l), w.dtype)
        q, k, v = O.qkv_rope(O.round_storage(X[l], w.dtype), w_host, None, lens, util_tabs["inv_freq"][l], Hq, Hkv, P, dv)
        util.check_projection(util.to_np64(q_dev[l]), O.round_storage(q, w.dtype), w.dtype, f"{name} q layer {l}")
        idx = torch.from_numpy(lens.astype(np.int64)).to(st.device)
        bsel = torch.arange(B, device=st.device)
        k_dev = st.k_cache[l][bsel, :, idx, :]
        v_dev = st.v_cache[l][bsel, :, idx, :]
        util.check_projection(util.to_np64(k_dev), O.round_storage(k, w.dtype), w.dtype, f"{name} k layer {l}")
        util.check_projection(util.to_np64(v_dev), O.round_storage(v, w.dtype), w.dtype, f"{name} v layer {l}")
    # a5: sampled units, full-length fp64 recomputation
    rng = np.random.default_rng(11)
    worst = 0.0
    for (l, b, h) in _sampled_units(L, B, Hkv, 16, rng):
        n = int(lens[b]) + 1
        K = util.to_np64(st.k_cache[l][b, h, :n])[None, None]
        V = util.to_np64(st.v_cache[l][b, h, :n])[None, None]
        q = util.to_np64(q_dev[l][b, h * G:(h + 1) * G])[None]
        want = O.decode_attn(q, K, V, [n], D)[0]
        got = util.to_np64(st.out[l][: B * Hq * dv]).reshape(B, Hq, dv)[b, h * G:(h + 1) * G]
        worst = max(worst, util.check_attn(got, want, w.dtype))
    st.close()
    return worst


@pytest.mark.parametrize("name", ["3b", "8b", "14b", "sweep1.0", "sweep0.9", "sweep0.8", "sweep0.7", "sweep0.5"])
def test_full_size_uniform_lengths(name):
    _run(name, ragged=False)


@pytest.mark.parametrize("name", ["3b", "8b", "14b"])
def test_full_size_ragged_lengths(name):
    _run(name, ragged=True)
