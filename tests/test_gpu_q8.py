"""Composition with 8-bit cache quantisation: the CUDA quantiser, the quantising append and the attention over a
quantised cache against the CPU oracle (quantize_rows / append_q8 / decode_attn_q8), through the C ABI."""
from dataclasses import replace

import numpy as np
import pytest
import torch

from oracle import rap_oracle as O
from paper_2602_02599_b200 import binding, synth
from paper_2602_02599_b200.stack import DecodeStack

import util

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("W", [90, 115, 128, 64, 116, 1, 33])
@pytest.mark.parametrize("dtype_in", ["f32", "bf16"])
def test_quantize_rows_bit_exact(W, dtype_in):
    """Codes, scales and padding of rap_quantize_rows equal the oracle's bit for bit on the same inputs: rows of very
    different magnitudes, an all-zero row, a row of equal elements, values on rounding ties."""
    w = synth.scaled_down(synth.LLAMA_8B, n_layers=1, batch=1, seq=8, hidden=256)
    st = DecodeStack(w, s_cap=8, alloc_cache=False)
    rng = np.random.default_rng(W)
    n = 1000
    x = (rng.normal(0, 1, (n, W)) * rng.lognormal(0, 3, (n, 1))).astype(np.float32)
    x[0] = 0.0
    x[1] = -0.3
    x[2, : min(W, 5)] = np.array([127.0, 63.5, -62.5, 0.5, -1.5], dtype=np.float32)[: min(W, 5)]     # s = 1: ties to even
    if dtype_in == "bf16":
        x = O.round_bf16(x).astype(np.float32)
    dx = torch.from_numpy(x).to(st.device)
    if dtype_in == "bf16":
        dx = dx.to(torch.bfloat16)
    rb = binding.rap_q8_row_bytes(W)
    assert rb == (W + 2 + 3) // 4 * 4
    out = torch.full((n, rb), 0xAB, dtype=torch.uint8, device=st.device)
    st.ctx.rap_quantize_rows(binding.RAP_F32 if dtype_in == "f32" else binding.RAP_BF16, n, W, dx, out)
    torch.cuda.synchronize()
    codes, scales = O.quantize_rows(x)
    assert np.array_equal(out.cpu().numpy(), util.pack_q8(codes, scales, rb))
    got_c, got_s = util.unpack_q8(out, W)
    assert np.array_equal(got_c, codes) and np.array_equal(got_s, scales)
    if W >= 5:
        assert got_c[2, :5].tolist() == [127, 64, -62, 0, -2] and got_s[2] == 1.0
    st.close()


def _q8_caches(st, l):
    w = st.w
    kb, vb = binding.rap_q8_row_bytes(2 * st.n_pairs[l]), binding.rap_q8_row_bytes(st.n_vch[l])
    k8 = torch.zeros((st.B, w.n_kv_heads, st.s_cap, kb), dtype=torch.uint8, device=st.device)
    v8 = torch.zeros((st.B, w.n_kv_heads, st.s_cap, vb), dtype=torch.uint8, device=st.device)
    return k8, v8


@pytest.mark.parametrize("name", ["tiny", "8b", "3b", "sweep1.0"])
def test_q8_append_and_attention_end_to_end(name):
    """Caches filled through rap_qkv_rope_append_q8 (every row quantised from its fp32 value), then one more token and
    rap_decode_attn_q8.  The codes are compared with the oracle's quantisation of its own fp64 projection: the two
    sides round different fp32 numbers (fp32 against fp64 accumulation), so a code may differ by one where a value
    sits next to a rounding boundary, never by more, and only rarely; the scale agrees to a bf16 step.  The attention is
    judged on the device's own codes, scales and q~."""
    base = synth.CONFIGS[name]
    w = base if name == "tiny" else synth.scaled_down(base, n_layers=2, batch=2, seq=300, hidden=512)
    lens = [w.seq] if w.batch == 1 else [300, 211]
    ks, vs = synth.draw_scores(w)
    st, tabs, w_host = util.build_small_stack(w, ks, vs, full_weights=True, max_rows=256)
    B, Hq, Hkv, D = w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim
    rows = [(b, p) for b in range(B) for p in range(lens[b] + 1)]          # the last row of each sequence is the new token
    seq_id = np.array([r[0] for r in rows], dtype=np.int32)
    pos = np.array([r[1] for r in rows], dtype=np.int32)
    T = len(rows)
    for l in range(w.n_layers):
        P, dv = st.n_pairs[l], st.n_vch[l]
        k8, v8 = _q8_caches(st, l)
        X = synth.draw_hidden(w, l, 0, T)
        q_dev = torch.empty((T, Hq, 2 * P), dtype=st.dt, device=st.device)
        for c0 in range(0, T, 256):
            c1 = min(T, c0 + 256)
            dx = torch.from_numpy(X[c0:c1]).to(st.device).to(st.dt).contiguous()
            sid, ps = torch.from_numpy(seq_id[c0:c1]).to(st.device), torch.from_numpy(pos[c0:c1]).to(st.device)
            st.ctx.rap_qkv_rope_append_q8(l, c1 - c0, dx, st.w_qkv[l], None, sid, ps, ps, int(pos[c0:c1].max()), st.inv_freq,
                                          q_dev[c0:c1], k8, v8, B, st.s_cap)
        torch.cuda.synchronize()
        assert st.ctx.rap_get_last_device_status() == (0, 0)
        q, k, v = O.qkv_rope(O.round_storage(X, w.dtype), w_host[l], None, pos, tabs["inv_freq"][l], Hq, Hkv, P, dv)
        util.check_projection(util.to_np64(q_dev), O.round_storage(q, w.dtype), w.dtype, f"q layer {l}")
        kc_o = np.zeros((B, Hkv, st.s_cap, 2 * P), np.int8); ks_o = np.zeros((B, Hkv, st.s_cap))
        vc_o = np.zeros((B, Hkv, st.s_cap, dv), np.int8); vs_o = np.zeros((B, Hkv, st.s_cap))
        O.append_q8(kc_o, ks_o, vc_o, vs_o, k, v, seq_id, pos)
        for dev, W, c_o, s_o, what in ((k8, 2 * P, kc_o, ks_o, "K"), (v8, dv, vc_o, vs_o, "V")):
            c_d, s_d = util.unpack_q8(dev, W)
            written = np.zeros(c_d.shape[:3], bool)
            written[seq_id, :, pos] = True
            assert not dev.cpu().numpy()[~written].any()                        # nothing but the named rows was touched
            diff = np.abs(c_d.astype(int) - c_o.astype(int))[written]
            assert diff.max() <= 1, what
            assert (diff != 0).mean() < 0.02, (what, (diff != 0).mean())
            assert np.all(np.abs(s_d - s_o)[written] <= 2.0 ** -7 * s_o[written] + 1e-30), what
            raw = dev.cpu().numpy()
            assert not raw[..., W:-2].any()                                    # padding bytes are zero
        # attention of the new token of every sequence over its whole prefix, on the device's own cache
        last = np.array([i for i, (b, p) in enumerate(rows) if p == lens[b]])
        dq = q_dev[torch.from_numpy(last).to(st.device)].contiguous()
        dl = torch.tensor([n + 1 for n in lens], dtype=torch.int32, device=st.device)
        kc_d, ks_d = util.unpack_q8(k8, 2 * P)
        vc_d, vs_d = util.unpack_q8(v8, dv)
        want = O.decode_attn_q8(util.to_np64(dq), kc_d, ks_d, vc_d, vs_d, [n + 1 for n in lens], D)
        for n_split in (0, 3):
            out = torch.full((B, Hq, dv), float("nan"), dtype=torch.float32, device=st.device)
            st.ctx.rap_decode_attn_q8(l, B, dq, k8, v8, st.s_cap, dl, max(lens) + 1, n_split, out)
            torch.cuda.synchronize()
            util.check_attn(util.to_np64(out), want, w.dtype)
        # the quantised cache stays close to the unquantised one: not a parity statement, a sanity bound on the reading
        Kf = np.zeros((B, Hkv, st.s_cap, 2 * P)); Vf = np.zeros((B, Hkv, st.s_cap, dv))
        O.append(Kf, Vf, k, v, seq_id, pos, "f32")
        ref = O.decode_attn(util.to_np64(dq), Kf, Vf, [n + 1 for n in lens], D)
        assert np.abs(want - ref).max() < 0.05 * np.abs(Vf).max()
    st.close()


def _random_q8_case(w, lens, n_split, seed=0, variant=0, q_gain=1.0):
    """rap_decode_attn_q8 alone on caches quantised by rap_quantize_rows from random rows, every unit checked."""
    st = DecodeStack(w, s_cap=((max(lens) + 8 + 7) // 8) * 8)
    st.ctx.rap_set_attn_variant(variant)
    st.build_tables(*synth.draw_scores(w))
    g = torch.Generator(device=st.device).manual_seed(seed)
    P2, dv = 2 * w.n_pairs, w.n_vch
    sig = float(np.sqrt(w.hidden) * 0.02)
    st.k_cache[0].normal_(0, sig, generator=g)
    st.v_cache[0].normal_(0, sig, generator=g)
    # rows of different magnitudes, so that the per-row scales matter
    ramp = (1.0 + 0.01 * torch.arange(st.s_cap, device=st.device, dtype=torch.float32) % 3.0).view(1, 1, -1, 1)
    st.v_cache[0].copy_((st.v_cache[0].float() * ramp).to(st.dt))
    k8, v8 = _q8_caches(st, 0)
    n_rows = st.B * w.n_kv_heads * st.s_cap
    dt_in = binding.RAP_F32 if w.dtype == "f32" else binding.RAP_BF16
    st.ctx.rap_quantize_rows(dt_in, n_rows, P2, st.k_cache[0], k8)
    st.ctx.rap_quantize_rows(dt_in, n_rows, dv, st.v_cache[0], v8)
    q = torch.empty((w.batch, w.n_q_heads, P2), dtype=st.dt, device=st.device).normal_(0, sig * q_gain, generator=g)
    dl = torch.tensor(lens, dtype=torch.int32, device=st.device)
    out = torch.full((w.batch, w.n_q_heads, dv), float("nan"), dtype=torch.float32, device=st.device)
    st.ctx.rap_decode_attn_q8(0, w.batch, q, k8, v8, st.s_cap, dl, int(max(lens)), n_split, out)
    torch.cuda.synchronize()
    assert st.ctx.rap_get_last_device_status() == (0, 0)
    kc, ksc = util.unpack_q8(k8, P2)
    vc, vsc = util.unpack_q8(v8, dv)
    assert np.array_equal(kc, O.quantize_rows(util.to_np64(st.k_cache[0]))[0])
    want = O.decode_attn_q8(util.to_np64(q), kc, ksc, vc, vsc, [max(1, n) for n in lens], w.head_dim)
    for b, n in enumerate(lens):
        if n == 0:
            want[b] = 0.0
    util.check_attn(util.to_np64(out), want, w.dtype)
    st.close()


@pytest.mark.parametrize("name", ["3b", "8b", "14b", "sweep1.0", "sweep0.8", "sweep0.5"])
@pytest.mark.parametrize("n_split", [0, 5])
def test_q8_attention_longer_sequences(name, n_split):
    w = synth.scaled_down(synth.CONFIGS[name], n_layers=1, batch=4, seq=4096)
    _random_q8_case(w, [4096, 2500, 1, 33], n_split, seed=n_split)


@pytest.mark.parametrize("variant", [0, 1])
@pytest.mark.parametrize("lens", [[0, 5000, 0, 1, 129, 0], [1, 1, 1, 1, 1, 1, 1, 1], [63, 64, 65, 127, 128, 129]])
def test_q8_attention_mixed_lengths_and_generic_kernel(variant, lens):
    """Empty sequences, one-row sequences, block and tile boundaries; variant 1 forces the shape-generic kernel."""
    w = synth.scaled_down(synth.LLAMA_8B, n_layers=1, batch=len(lens), seq=max(lens))
    _random_q8_case(w, lens, 0, seed=len(lens), variant=variant)
    _random_q8_case(w, lens, 4, seed=len(lens) + 1, variant=variant)


@pytest.mark.parametrize("q_gain", [12.0, 0.05])
def test_q8_attention_peaked_and_flat_softmax(q_gain):
    w = synth.scaled_down(synth.LLAMA_8B, n_layers=1, batch=3, seq=2500)
    _random_q8_case(w, [2500, 1333, 40], 0, seed=7, q_gain=q_gain)


def test_q8_attention_head_shape_without_specialised_scan_and_fp32():
    w = replace(synth.scaled_down(synth.LLAMA_8B, n_layers=1, batch=2, seq=700), n_pairs=37, n_vch=70, n_q_heads=16)
    _random_q8_case(w, [700, 333], 0, seed=1)
    w = replace(synth.TINY, batch=2, seq=200)
    _random_q8_case(w, [200, 77], 0, seed=2)
    _random_q8_case(w, [200, 77], 3, seed=3)


@pytest.mark.parametrize("name", ["8b", "3b", "14b"])
def test_q8_full_size_sampled_units(name):
    """rap_decode_attn_q8 at the workloads' full batch and context, in the launch configuration the benchmark times
    (balanced split, one layer resident): sampled (sequence, KV head) units recomputed by the oracle from that unit's
    codes and scales, ragged lengths included."""
    w = replace(synth.CONFIGS[name], n_layers=1)
    st = DecodeStack(w)
    st.build_tables(*synth.draw_scores(w))
    g = torch.Generator(device=st.device).manual_seed(w.seed)
    sig = float(np.sqrt(w.hidden) * 0.02)
    st.k_cache[0].normal_(0, sig, generator=g)
    st.v_cache[0].normal_(0, sig, generator=g)
    B, Hq, Hkv, G, P2, dv = w.batch, w.n_q_heads, w.n_kv_heads, w.group, 2 * w.n_pairs, w.n_vch
    kb, vb = binding.rap_q8_row_bytes(P2), binding.rap_q8_row_bytes(dv)
    n_rows = B * Hkv * st.s_cap
    k8 = torch.empty((B, Hkv, st.s_cap, kb), dtype=torch.uint8, device=st.device)
    v8 = torch.empty((B, Hkv, st.s_cap, vb), dtype=torch.uint8, device=st.device)
    st.ctx.rap_quantize_rows(binding.RAP_BF16, n_rows, P2, st.k_cache[0], k8)
    st.ctx.rap_quantize_rows(binding.RAP_BF16, n_rows, dv, st.v_cache[0], v8)
    st.k_cache[0] = st.v_cache[0] = None          # the bf16 rows are no longer needed
    torch.cuda.empty_cache()
    q = torch.empty((B, Hq, P2), dtype=st.dt, device=st.device).normal_(0, sig, generator=g)
    out = torch.empty((B, Hq, dv), dtype=torch.float32, device=st.device)
    rng = np.random.default_rng(3)
    for lens in (np.full(B, w.seq + 1, dtype=np.int32), synth.ragged_lengths(w) + 1):
        dl = torch.from_numpy(lens.astype(np.int32)).to(st.device)
        out.fill_(float("nan"))
        st.ctx.rap_decode_attn_q8(0, B, q, k8, v8, st.s_cap, dl, int(lens.max()), 0, out)
        torch.cuda.synchronize()
        assert st.ctx.rap_get_last_device_status() == (0, 0)
        assert not torch.isnan(out).any()
        units = {(0, 0), (B - 1, Hkv - 1), (0, Hkv - 1), (B - 1, 0)}
        while len(units) < 8:
            units.add((int(rng.integers(B)), int(rng.integers(Hkv))))
        for b, h in sorted(units):
            n = int(lens[b])
            kc, ks = util.unpack_q8(k8[b, h, :n], P2)
            vc, vs = util.unpack_q8(v8[b, h, :n], dv)
            want = O.decode_attn_q8(util.to_np64(q[b, h * G:(h + 1) * G])[None], kc[None, None], ks[None, None], vc[None, None],
                                    vs[None, None], [n], w.head_dim)[0]
            util.check_attn(util.to_np64(out[b, h * G:(h + 1) * G]), want, w.dtype)
    st.close()


@pytest.mark.parametrize("name,T", [("8b", 32), ("8b", 5), ("3b", 17), ("sweep1.0", 1)])
def test_q8_decode_sized_append(name, T):
    """Decode-sized rap_qkv_rope_append_q8 calls (T <= 32: the token-tile width the step uses; scattered sequences and
    slots).  q~ equals, bit for bit, what the unquantised entry point writes for the same rows (every rotating kernel
    rounds the same way); against the oracle: codes within one step, scales within a bf16 step (fp32 against fp64
    accumulation); nothing but the named rows is touched."""
    w = synth.scaled_down(synth.CONFIGS[name], n_layers=2, batch=3, seq=64, hidden=512)
    ks, vs = synth.draw_scores(w)
    st, tabs, w_host = util.build_small_stack(w, ks, vs, full_weights=True, max_rows=64)
    B, Hq, Hkv = w.batch, w.n_q_heads, w.n_kv_heads
    rng = np.random.default_rng(5)
    seq_id = rng.integers(0, B, size=T).astype(np.int32)
    pos = np.zeros(T, np.int32)
    for b in range(B):                                   # distinct slots per sequence
        m = seq_id == b
        pos[m] = rng.permutation(60)[: m.sum()]
    sid, ps = torch.from_numpy(seq_id).to(st.device), torch.from_numpy(pos).to(st.device)
    for l in range(w.n_layers):
        P, dv = st.n_pairs[l], st.n_vch[l]
        X = synth.draw_hidden(w, l, 3, T)
        dx = torch.from_numpy(X).to(st.device).to(st.dt).contiguous()
        k8, v8 = _q8_caches(st, l)
        q_dev = torch.full((T, Hq, 2 * P), float("nan"), dtype=st.dt, device=st.device)
        st.ctx.rap_qkv_rope_append_q8(l, T, dx, st.w_qkv[l], None, sid, ps, ps, int(pos.max()), st.inv_freq, q_dev, k8, v8, B,
                                      st.s_cap)
        q_plain = torch.full((T, Hq, 2 * P), float("nan"), dtype=st.dt, device=st.device)
        st.qkv_rope_append(l, dx, sid, ps, ps, int(pos.max()), q_out=q_plain)
        torch.cuda.synchronize()
        assert st.ctx.rap_get_last_device_status() == (0, 0)
        assert torch.equal(q_dev, q_plain)
        q, k, v = O.qkv_rope(O.round_storage(X, w.dtype), w_host[l], None, pos, tabs["inv_freq"][l], Hq, Hkv, P, dv)
        util.check_projection(util.to_np64(q_dev), O.round_storage(q, w.dtype), w.dtype, f"q layer {l}")
        kc_o = np.zeros((B, Hkv, st.s_cap, 2 * P), np.int8); ks_o = np.zeros((B, Hkv, st.s_cap))
        vc_o = np.zeros((B, Hkv, st.s_cap, dv), np.int8); vs_o = np.zeros((B, Hkv, st.s_cap))
        O.append_q8(kc_o, ks_o, vc_o, vs_o, k, v, seq_id, pos)
        for dev, W, c_o, s_o, what in ((k8, 2 * P, kc_o, ks_o, "K"), (v8, dv, vc_o, vs_o, "V")):
            c_d, s_d = util.unpack_q8(dev, W)
            written = np.zeros(c_d.shape[:3], bool)
            written[seq_id, :, pos] = True
            assert not dev.cpu().numpy()[~written].any()
            diff = np.abs(c_d.astype(int) - c_o.astype(int))[written]
            assert diff.max() <= 1, what
            assert (diff != 0).mean() < 0.02, (what, (diff != 0).mean())
            assert np.all(np.abs(s_d - s_o)[written] <= 2.0 ** -7 * s_o[written] + 1e-30), what
            assert not dev.cpu().numpy()[..., W:-2].any()
    st.close()


@pytest.mark.parametrize("name", ["8b", "3b"])
def test_q8_decode_step_equals_the_separate_calls_and_the_oracle(name):
    """rap_decode_step_q8 (all layers: quantising append, then attention over the quantised cache; consecutive launches
    overlap) against the same step made of rap_qkv_rope_append_q8 + rap_decode_attn_q8 calls -- bit for bit, caches
    and outputs -- and its attention against the oracle on the device's own codes; the lengths advance."""
    w = synth.scaled_down(synth.CONFIGS[name], n_layers=3, batch=2, seq=300, hidden=512)
    lens = np.array([300, 211], dtype=np.int32)
    ks, vs = synth.draw_scores(w)
    st, tabs, w_host = util.build_small_stack(w, ks, vs, full_weights=False, max_rows=256)
    B, Hq, Hkv, D, L = w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.n_layers
    g = torch.Generator(device=st.device).manual_seed(11)
    sig = float(np.sqrt(w.hidden) * 0.02)
    k8, v8 = [], []
    n_rows = B * Hkv * st.s_cap
    for l in range(L):
        st.k_cache[l].normal_(0, sig, generator=g)
        st.v_cache[l].normal_(0, sig, generator=g)
        a, b = _q8_caches(st, l)
        st.ctx.rap_quantize_rows(binding.RAP_BF16, n_rows, 2 * st.n_pairs[l], st.k_cache[l], a)
        st.ctx.rap_quantize_rows(binding.RAP_BF16, n_rows, st.n_vch[l], st.v_cache[l], b)
        k8.append(a)
        v8.append(b)
    x = torch.empty((L, B, w.hidden), dtype=st.dt, device=st.device).normal_(0, 1, generator=g)
    # the step as separate calls, on copies
    k8_ref, v8_ref = [t.clone() for t in k8], [t.clone() for t in v8]
    dl = torch.from_numpy(lens).to(st.device)
    sid = torch.arange(B, dtype=torch.int32, device=st.device)
    out_ref, q_ref = [], []
    for l in range(L):
        q = torch.empty((B, Hq, 2 * st.n_pairs[l]), dtype=st.dt, device=st.device)
        st.ctx.rap_qkv_rope_append_q8(l, B, x[l], st.w_qkv[l], None, sid, dl, dl, int(lens.max()), st.inv_freq, q, k8_ref[l],
                                      v8_ref[l], B, st.s_cap)
        o = torch.empty((B, Hq, st.n_vch[l]), dtype=torch.float32, device=st.device)
        st.ctx.rap_decode_attn_q8(l, B, q, k8_ref[l], v8_ref[l], st.s_cap, dl + 1, int(lens.max()) + 1, 0, o)
        out_ref.append(o)
        q_ref.append(q)
    st.seq_len.copy_(dl)
    st.out.fill_(float("nan"))
    st.ctx.rap_decode_step_q8(B, x, st.w_qkv, None, st.inv_freq, k8, v8, st.s_cap, st.seq_len, int(lens.max()), 0, st.q_scratch,
                              st.out, st.out_stride, 1)
    torch.cuda.synchronize()
    assert st.ctx.rap_get_last_device_status() == (0, 0)
    assert st.seq_len.cpu().tolist() == (lens + 1).tolist()
    for l in range(L):
        P2, dv = 2 * st.n_pairs[l], st.n_vch[l]
        assert torch.equal(k8[l], k8_ref[l]) and torch.equal(v8[l], v8_ref[l])
        got = st.out[l][: B * Hq * dv].reshape(B, Hq, dv)
        assert torch.equal(got, out_ref[l])
        kc, ksc = util.unpack_q8(k8[l], P2)
        vc, vsc = util.unpack_q8(v8[l], dv)
        want = O.decode_attn_q8(util.to_np64(q_ref[l]), kc, ksc, vc, vsc, lens + 1, D)
        util.check_attn(util.to_np64(got), want, w.dtype)
    st.close()
