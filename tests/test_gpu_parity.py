"""Parity of the CUDA path (through the C ABI) against the CPU oracle, on the same seeded inputs."""
import numpy as np
import pytest
import torch

from oracle import rap_oracle as O
from paper_2602_02599_b200 import binding, synth
from paper_2602_02599_b200.stack import DecodeStack

import util

pytestmark = pytest.mark.gpu


def _tables_equal(st, tabs):
    torch.cuda.synchronize()
    assert np.array_equal(st.k_pair_idx.cpu().numpy(), tabs["k_pair_idx"])
    assert np.array_equal(st.k_dim_idx.cpu().numpy(), tabs["k_dim_idx"])
    assert np.array_equal(st.v_idx.cpu().numpy(), tabs["v_idx"])
    got, want = st.inv_freq.cpu().numpy(), tabs["inv_freq"]
    assert np.allclose(got, want, rtol=4e-16, atol=0)


@pytest.mark.parametrize("name", ["tiny", "3b", "8b", "14b", "sweep0.5", "sweep1.0"])
def test_tables_bit_exact_all_layers(name):
    w = synth.CONFIGS[name]
    ks, vs = synth.draw_scores(w)
    st = DecodeStack(w, batch=1, s_cap=8, alloc_cache=False)
    st.build_tables(ks, vs)
    _tables_equal(st, util.oracle_tables(w, ks, vs))
    st.close()


def test_tables_ties_adjacent_pairing_and_per_layer_budgets():
    from dataclasses import replace
    w = replace(synth.TINY, n_layers=3, pairing=1)
    rng = np.random.default_rng(5)
    ks = rng.integers(0, 3, (3, 2, 32)).astype(np.float64)        # heavy ties
    vs = rng.integers(0, 3, (3, 2, 64)).astype(np.float64)
    n_pairs, n_vch = [32, 1, 17], [1, 64, 33]
    st = DecodeStack(w, n_pairs=n_pairs, n_vch=n_vch, batch=1, s_cap=8, alloc_cache=False)
    st.build_tables(ks, vs)
    _tables_equal(st, util.oracle_tables(w, ks, vs, n_pairs, n_vch))
    st.close()


def test_pack_weights_bit_exact():
    w = synth.scaled_down(synth.LLAMA_8B, n_layers=2, batch=1, seq=8, hidden=256)
    ks, vs = synth.draw_scores(w)
    st, tabs, w_host = util.build_small_stack(w, ks, vs, full_weights=True)
    for l in range(w.n_layers):
        assert np.array_equal(util.to_np64(st.w_qkv[l]), w_host[l])
    st.close()


def _end_to_end(w, lens_before, n_split=0, with_bias=False, chunk=None, n_pairs=None, n_vch=None):
    """Prefill lens_before[b] tokens per sequence, then one decode step; compare every stage."""
    ks, vs = synth.draw_scores(w)
    T_pre = int(np.sum(lens_before))
    st, tabs, w_host = util.build_small_stack(w, ks, vs, full_weights=True, max_rows=max(chunk or T_pre, w.batch),
                                              n_pairs=n_pairs, n_vch=n_vch)
    B, Hq, Hkv, D = w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim
    bias_host = None
    if with_bias:
        bias_host, st.bias = [], []
        for l in range(w.n_layers):
            b = synth.draw_bias(w, l, st.n_out(l))
            st.bias.append(torch.from_numpy(b).to(st.device).to(st.dt))
            bias_host.append(O.round_storage(b, w.dtype))
    caches = util.prefill_both(st, tabs, w_host, w, lens_before, chunk=chunk) if not with_bias else None
    if with_bias:   # bias path: empty caches, first token only
        caches = [(np.zeros((B, Hkv, st.s_cap, 2 * st.n_pairs[l])), np.zeros((B, Hkv, st.s_cap, st.n_vch[l])))
                  for l in range(w.n_layers)]
        for l in range(w.n_layers):
            st.k_cache[l].zero_(); st.v_cache[l].zero_()
        lens_before = np.zeros(B, dtype=np.int32)
    lens_before = np.asarray(lens_before, dtype=np.int32)
    st.seq_len.copy_(torch.from_numpy(lens_before))
    X = np.stack([synth.draw_hidden(w, l, 1, B) for l in range(w.n_layers)])
    dx = torch.from_numpy(X).to(st.device).to(st.dt).contiguous()
    # canaries around what the step may write
    for l in range(w.n_layers):
        for b in range(B):
            st.k_cache[l][b, :, lens_before[b] + 1:, :] = -77.0
            st.v_cache[l][b, :, lens_before[b] + 1:, :] = -77.0
    before = [(st.k_cache[l].clone(), st.v_cache[l].clone()) for l in range(w.n_layers)]
    st.decode_step(dx, int(lens_before.max()), n_split=n_split, advance=1)
    torch.cuda.synchronize()
    assert st.ctx.rap_get_last_device_status() == (0, 0)
    assert np.array_equal(st.seq_len.cpu().numpy(), lens_before + 1)
    worst = 0.0
    for l in range(w.n_layers):
        P, dv = st.n_pairs[l], st.n_vch[l]
        Xr = O.round_storage(X[l], w.dtype)
        q, k, v = O.qkv_rope(Xr, w_host[l], None if bias_host is None else bias_host[l], lens_before,
                             tabs["inv_freq"][l], Hq, Hkv, P, dv)
        Kd, Vd = util.to_np64(st.k_cache[l]), util.to_np64(st.v_cache[l])
        Kb, Vb = util.to_np64(before[l][0]), util.to_np64(before[l][1])
        # slot layout: exactly the rows (b, :, len_b) changed
        changed_k = np.any(Kd != Kb, axis=-1)
        changed_v = np.any(Vd != Vb, axis=-1)
        expect = np.zeros_like(changed_k)
        for b in range(B):
            expect[b, :, lens_before[b]] = True
        assert np.array_equal(changed_k | expect, expect) and np.array_equal(changed_v | expect, expect)
        k_dev = np.stack([Kd[b, :, lens_before[b], :] for b in range(B)])
        v_dev = np.stack([Vd[b, :, lens_before[b], :] for b in range(B)])
        util.check_projection(k_dev, O.round_storage(k, w.dtype), w.dtype, f"k layer {l}")
        util.check_projection(v_dev, O.round_storage(v, w.dtype), w.dtype, f"v layer {l}")
        # attention judged on the device's own rounded q~ and cache rows (projection, RoPE and append are checked above)
        # -> recompute q~ on the device into a separate buffer
        dq = torch.empty((B, Hq, 2 * P), dtype=st.dt, device=st.device)
        tmp_k, tmp_v = st.k_cache[l].clone(), st.v_cache[l].clone()
        dpos = torch.from_numpy(lens_before).to(st.device)
        dsid = torch.arange(B, dtype=torch.int32, device=st.device)
        st.qkv_rope_append(l, dx[l], dsid, dpos, dpos, int(lens_before.max()), q_out=dq)
        torch.cuda.synchronize()
        assert torch.equal(tmp_k, st.k_cache[l]) and torch.equal(tmp_v, st.v_cache[l])   # idempotent rewrite
        util.check_projection(util.to_np64(dq), O.round_storage(q, w.dtype), w.dtype, f"q layer {l}")
        want = O.decode_attn(util.to_np64(dq), Kd, Vd, lens_before + 1, D)
        got = util.to_np64(st.out[l][: B * Hq * dv]).reshape(B, Hq, dv)
        worst = max(worst, util.check_attn(got, want, w.dtype))
        # and the whole chain against the oracle's own caches (looser: rounding of k/v may differ by an ulp)
        if w.dtype == "f32":
            Ko, Vo = caches[l]
            O.append(Ko, Vo, k, v, np.arange(B), lens_before, w.dtype)
            want2 = O.decode_attn(O.round_storage(q, w.dtype), Ko, Vo, lens_before + 1, D)
            assert np.abs(got - want2).max() <= util.F32_MAX_ABS
    st.close()
    return worst


def test_config1_tiny_fp32_end_to_end():
    w = synth.TINY
    err = _end_to_end(w, [w.seq])
    assert err <= 1e-5


@pytest.mark.parametrize("n_split", [1, 3, 64])
def test_config1_split_counts(n_split):
    _end_to_end(synth.TINY, [synth.TINY.seq], n_split=n_split)


def test_rope_at_large_positions_fp32():
    """Index-aware RoPE far out (positions up to 10^6 with the cache slot kept small): the device reduces the fp64
    angle before it takes the fp32 sine and cosine, so q~ and the appended K row stay within the fp32 tolerance."""
    w = synth.TINY
    ks, vs = synth.draw_scores(w)
    st, tabs, w_host = util.build_small_stack(w, ks, vs, full_weights=True, max_rows=8)
    pos = np.array([0, 1, 4097, 32768, 99999, 1000003], dtype=np.int32)
    T = len(pos)
    X = synth.draw_hidden(w, 0, 7, T)
    dx = torch.from_numpy(X).to(st.device).to(st.dt).contiguous()
    dq = torch.empty((T, w.n_q_heads, 2 * w.n_pairs), dtype=st.dt, device=st.device)
    sid = torch.zeros(T, dtype=torch.int32, device=st.device)
    slot = torch.arange(T, dtype=torch.int32, device=st.device)
    st.qkv_rope_append(0, dx, sid, torch.from_numpy(pos).to(st.device), slot, T - 1, q_out=dq)
    torch.cuda.synchronize()
    q, k, v = O.qkv_rope(O.round_storage(X, w.dtype), w_host[0], None, pos, tabs["inv_freq"][0], w.n_q_heads,
                         w.n_kv_heads, w.n_pairs, w.n_vch)
    util.check_projection(util.to_np64(dq), q, w.dtype, "q at large positions")
    Kd = util.to_np64(st.k_cache[0])
    k_dev = np.stack([Kd[0, :, t, :] for t in range(T)])
    util.check_projection(k_dev, k, w.dtype, "k at large positions")
    # the rotation is not the identity out there: an unrotated row would miss by far more than the tolerance
    assert np.abs(k_dev[-1] - O.qkv_rope(O.round_storage(X, w.dtype), w_host[0], None, np.zeros(T, np.int32),
                                         tabs["inv_freq"][0], w.n_q_heads, w.n_kv_heads, w.n_pairs, w.n_vch)[1][-1]).max() > 1e-2
    st.close()


def test_tiny_with_bias():
    _end_to_end(synth.TINY, [0], with_bias=True)


@pytest.mark.parametrize("name", ["3b", "8b", "14b", "sweep1.0", "sweep0.8", "sweep0.5"])
def test_scaled_down_bf16_twins(name):
    w = synth.scaled_down(synth.CONFIGS[name], n_layers=2, batch=2, seq=512, hidden=512)
    _end_to_end(w, [512, 475], chunk=256)


@pytest.mark.parametrize("lens", [[0, 1], [63, 64], [65, 127], [128, 129], [1, 300]])
def test_ragged_and_tile_boundaries(lens):
    w = synth.scaled_down(synth.LLAMA_8B, n_layers=1, batch=2, seq=320, hidden=256)
    _end_to_end(w, lens, chunk=256)
    _end_to_end(w, lens, n_split=7, chunk=256)


def test_adjacent_pairing_end_to_end():
    from dataclasses import replace
    w = replace(synth.TINY, pairing=1, seq=40)
    _end_to_end(w, [40])


def _random_attn_case(w, lens, n_split, seed=0, variant=0, q_gain=1.0, ramp=0.0, pieces=None):
    """rap_decode_attn alone on random caches (no projection), every unit checked.  q_gain scales q (peaked
    softmax); ramp > 0 makes the K rows grow with the position (the running maximum keeps moving); pieces =
    (tiles per piece, 256ths of all tiles) forces the tensor-core scan to hand that share out at run time."""
    st = DecodeStack(w, s_cap=((max(lens) + 8 + 7) // 8) * 8)
    st.ctx.rap_set_attn_variant(variant)
    if pieces is not None:
        st.ctx.rap_debug_set_scan_pieces(*pieces)
    ks, vs = synth.draw_scores(w)
    st.build_tables(ks, vs)
    g = torch.Generator(device=st.device).manual_seed(seed)
    P2, dv = 2 * w.n_pairs, w.n_vch
    sig = float(np.sqrt(w.hidden) * 0.02)
    for l in range(w.n_layers):
        st.k_cache[l].normal_(0, sig, generator=g)
        st.v_cache[l].normal_(0, sig, generator=g)
    q = torch.empty((w.batch, w.n_q_heads, P2), dtype=st.dt, device=st.device).normal_(0, sig * q_gain, generator=g)
    if ramp > 0:
        pos = torch.arange(st.s_cap, device=st.device, dtype=torch.float32).view(1, 1, -1, 1)
        for l in range(w.n_layers):
            st.k_cache[l].copy_((st.k_cache[l].float() * (1.0 + ramp * pos)).to(st.dt))
    dl = torch.tensor(lens, dtype=torch.int32, device=st.device)
    for l in range(w.n_layers):
        out = st.decode_attn(l, q, dl, int(max(lens)), n_split=n_split)
        torch.cuda.synchronize()
        # the definition needs at least one row; the library returns zeros for an empty sequence
        want = O.decode_attn(util.to_np64(q), util.to_np64(st.k_cache[l]), util.to_np64(st.v_cache[l]),
                             [max(1, n) for n in lens], w.head_dim)
        for b, n in enumerate(lens):
            if n == 0:
                want[b] = 0.0
        got = util.to_np64(out[: w.batch * w.n_q_heads * dv]).reshape(w.batch, w.n_q_heads, dv)
        util.check_attn(got, want, w.dtype)
    assert st.ctx.rap_get_last_device_status() == (0, 0)
    st.close()


@pytest.mark.parametrize("name", ["3b", "8b", "14b", "sweep1.0", "sweep0.9", "sweep0.8", "sweep0.5"])
@pytest.mark.parametrize("n_split", [0, 5])
def test_attention_only_longer_sequences(name, n_split):
    w = synth.scaled_down(synth.CONFIGS[name], n_layers=1, batch=3, seq=4096)
    _random_attn_case(w, [4096, 2500, 1], n_split)


@pytest.mark.parametrize("name", ["3b", "8b", "14b", "sweep1.0", "sweep0.5"])
@pytest.mark.parametrize("pieces", [(1, 128), (2, 64), (3, 200), (7, 38), (1, 256)])
def test_attention_pieces_claimed_at_run_time(name, pieces):
    """The tensor-core scan with a share of its tiles handed out at run time (long launches do that by themselves;
    here it is forced on small ones, down to pieces of one tile, up to every tile): pieces are fixed tile ranges and
    partials are merged in tile order, so the result is the one the oracle defines whoever scans what -- ragged
    lengths, an empty sequence, units cut by several pieces, twice in a row on the same context (the counters of the
    first launch are cleared by the second)."""
    w = synth.scaled_down(synth.CONFIGS[name], n_layers=2, batch=4, seq=4096)
    _random_attn_case(w, [4096, 2500, 1, 700], 0, seed=sum(pieces), variant=4, pieces=pieces)
    _random_attn_case(w, [300, 0, 3999, 129], 0, seed=pieces[0], variant=4, pieces=pieces)


def test_attention_pieces_and_tiers_take_turns():
    """Launches that hand pieces out at run time use a counter that the NEXT balanced launch on the context clears,
    whichever kernel that is: tensor-core scan with pieces, FP32-pipe scan, tensor-core scan again, explicit splits in
    between -- every result against the oracle."""
    w = synth.scaled_down(synth.CONFIGS["8b"], n_layers=1, batch=3, seq=4096)
    lens = [4096, 1500, 77]
    st = DecodeStack(w, s_cap=4104)
    st.build_tables(*synth.draw_scores(w))
    g = torch.Generator(device=st.device).manual_seed(4)
    sig = float(np.sqrt(w.hidden) * 0.02)
    st.k_cache[0].normal_(0, sig, generator=g)
    st.v_cache[0].normal_(0, sig, generator=g)
    q = torch.empty((w.batch, w.n_q_heads, 2 * w.n_pairs), dtype=st.dt, device=st.device).normal_(0, sig, generator=g)
    dl = torch.tensor(lens, dtype=torch.int32, device=st.device)
    want = O.decode_attn(util.to_np64(q), util.to_np64(st.k_cache[0]), util.to_np64(st.v_cache[0]), lens, w.head_dim)
    st.ctx.rap_debug_set_scan_pieces(2, 100)
    for variant, n_split in ((4, 0), (3, 0), (4, 0), (4, 3), (4, 0), (3, 0), (3, 0), (4, 0), (4, 0)):
        st.ctx.rap_set_attn_variant(variant)
        st.out.fill_(float("nan"))
        out = st.decode_attn(0, q, dl, max(lens), n_split=n_split)
        torch.cuda.synchronize()
        got = util.to_np64(out[: w.batch * w.n_q_heads * w.n_vch]).reshape(w.batch, w.n_q_heads, w.n_vch)
        util.check_attn(got, want, w.dtype)
    assert st.ctx.rap_get_last_device_status() == (0, 0)
    st.close()


@pytest.mark.parametrize("name", ["3b", "8b", "14b", "sweep1.0", "sweep0.5"])
@pytest.mark.parametrize("n_split", [0, 5])
def test_attention_fp32_pipe_scan(name, n_split):
    """The shape-specialised scan on the FP32 pipes (the tier behind the tensor-core form) against the oracle."""
    w = synth.scaled_down(synth.CONFIGS[name], n_layers=1, batch=3, seq=4096)
    _random_attn_case(w, [4096, 2500, 1], n_split, variant=3)


@pytest.mark.parametrize("G,P,dv", [(8, 45, 90), (1, 58, 115), (6, 51, 102), (2, 45, 90), (4, 22, 44), (4, 20, 40),
                                    (5, 41, 82), (3, 63, 126), (4, 64, 64), (7, 32, 64), (8, 64, 128),
                                    (4, 24, 48), (5, 16, 32), (3, 48, 96), (4, 56, 112)])
def test_attention_tensor_core_scan_head_shapes(G, P, dv):
    """The tensor-core form of the scan, forced (variant 4 fails instead of falling back): group sizes 1..8,
    odd and even d_v', the three row-spreading steps of the fragment loads (P odd, P = 2 mod 4, P = 0 mod 4),
    the shapes staged through swizzling tensor maps and other multiples of 8 (which keep some bank conflicts);
    ragged lengths, a block with one row, both split modes."""
    from dataclasses import replace
    base = synth.scaled_down(synth.LLAMA_8B, n_layers=1, batch=4, seq=3000)
    w = replace(base, n_pairs=P, n_vch=dv, n_q_heads=G * base.n_kv_heads)
    _random_attn_case(w, [3000, 1777, 1, 33], 0, seed=P + G, variant=4)
    _random_attn_case(w, [129, 0, 2999, 96], 3, seed=P, variant=4)
    # a cache capacity that is not a multiple of the 32-row block: the last block of every unit reaches into the
    # next unit's rows, and the last unit's past the end of the cache (where tensor-map boxes are zero-filled)
    _random_attn_case(w, [3010, 3010, 3010, 3010], 0, seed=G, variant=4)


@pytest.mark.parametrize("G,P,dv", [(2, 37, 70), (4, 45, 90), (3, 58, 115), (5, 64, 128), (1, 8, 16), (4, 30, 61),
                                    (5, 32, 64)])
@pytest.mark.parametrize("n_split", [0, 5])
def test_attention_run_time_shape_scan(G, P, dv, n_split):
    """The bf16 scan that takes the head shape at run time -- the tier a shape without any instantiation falls to
    (G = 2, P = 37, d_v' = 70 has none), forced here for instantiated shapes too (variant 2 skips both
    shape-specialised scans): odd, 2 mod 4 and 0 mod 4 pair counts, rows that are multiples of 32 bytes (padded
    in shared memory), odd and even d_v', ragged lengths, a one-row sequence and an empty one."""
    from dataclasses import replace
    base = synth.scaled_down(synth.LLAMA_8B, n_layers=1, batch=4, seq=3000)
    w = replace(base, n_pairs=P, n_vch=dv, n_q_heads=G * base.n_kv_heads)
    _random_attn_case(w, [3000, 1777, 1, 33], n_split, seed=P + G, variant=2)
    _random_attn_case(w, [129, 0, 2999, 96], n_split, seed=P, variant=2)


def test_attention_shape_without_instantiation_takes_the_default_path():
    """No forced tier: a head shape nobody instantiated still goes through rap_decode_attn and meets the oracle,
    and the tensor-core-or-nothing variant refuses it."""
    from dataclasses import replace
    base = synth.scaled_down(synth.LLAMA_8B, n_layers=1, batch=3, seq=2000)
    w = replace(base, n_pairs=37, n_vch=70, n_q_heads=2 * base.n_kv_heads)
    _random_attn_case(w, [2000, 1, 777], 0, seed=3)
    with pytest.raises(binding.RapError) as e:
        _random_attn_case(w, [2000, 1, 777], 0, seed=3, variant=4)
    assert e.value.status == binding.RAP_EUNSUPPORTED


@pytest.mark.parametrize("variant", [4, 3, 2])
@pytest.mark.parametrize("q_gain,ramp", [(12.0, 0.0), (3.0, 0.002), (0.05, 0.0)])
def test_attention_peaked_moving_and_flat_softmax(variant, q_gain, ramp):
    """Logit regimes that exercise the lazy reference maximum of both shape-specialised scans: nearly one-hot
    weights (large q), a maximum that keeps rising along the sequence (K grows with the position, so every
    few blocks rescale the accumulators) and nearly uniform weights."""
    w = synth.scaled_down(synth.LLAMA_8B, n_layers=1, batch=3, seq=2500)
    _random_attn_case(w, [2500, 1333, 40], 0, seed=7, variant=variant, q_gain=q_gain, ramp=ramp)
    _random_attn_case(w, [2500, 1333, 40], 4, seed=8, variant=variant, q_gain=q_gain, ramp=ramp)


def test_attention_generic_variant_matches():
    w = synth.scaled_down(synth.LLAMA_8B, n_layers=1, batch=2, seq=1500)
    st = DecodeStack(w, s_cap=1504)
    st.build_tables(*synth.draw_scores(w))
    g = torch.Generator(device=st.device).manual_seed(1)
    st.k_cache[0].normal_(0, 1.3, generator=g)
    st.v_cache[0].normal_(0, 1.3, generator=g)
    q = torch.empty((2, w.n_q_heads, 2 * w.n_pairs), dtype=st.dt, device=st.device).normal_(0, 1.3, generator=g)
    dl = torch.tensor([1500, 777], dtype=torch.int32, device=st.device)
    a = st.decode_attn(0, q, dl, 1500).clone()
    st.ctx.rap_set_attn_variant(1)
    b = st.decode_attn(0, q, dl, 1500).clone()
    torch.cuda.synchronize()
    assert (a - b).abs().max().item() < 2e-5
    st.close()


@pytest.mark.parametrize("n_layers", [2, 4, 7])      # below 4 layers the copies do not overlap the layers; 7: odd cut
def test_decode_step_host_matches_device_step(n_layers):
    w = synth.scaled_down(synth.LLAMA_8B, n_layers=n_layers, batch=2, seq=256, hidden=256)
    ks, vs = synth.draw_scores(w)
    st, tabs, w_host = util.build_small_stack(w, ks, vs, full_weights=False)
    g = torch.Generator(device=st.device).manual_seed(3)
    for l in range(w.n_layers):
        st.k_cache[l].normal_(0, 1.0, generator=g)
        st.v_cache[l].normal_(0, 1.0, generator=g)
    st.seq_len.fill_(256)
    X = np.stack([synth.draw_hidden(w, l, 9, w.batch) for l in range(w.n_layers)])
    hx = torch.from_numpy(X).to(st.dt).contiguous().pin_memory()
    dx = hx.to(st.device)
    ref = st.decode_step(dx, 256).clone()
    kref = [c.clone() for c in st.k_cache]
    for l in range(w.n_layers):                      # undo the append so the host step redoes the same work
        st.k_cache[l][:, :, 256, :] = 0
        st.v_cache[l][:, :, 256, :] = 0
    h_out = torch.empty((w.n_layers, st.out_stride), dtype=torch.float32).pin_memory()
    h_out.fill_(float("nan"))
    st.decode_step_host(hx, h_out, 256, advance=1)
    assert torch.equal(h_out, ref.cpu())
    assert all(torch.equal(a, b) for a, b in zip(kref, st.k_cache))
    assert st.seq_len.cpu().tolist() == [257, 257]
    assert st.ctx.rap_kernel_launch_count() > 0
    st.close()


def test_argument_validation_on_device_context():
    w = synth.scaled_down(synth.LLAMA_8B, n_layers=1, batch=2, seq=64, hidden=256)
    st = DecodeStack(w, s_cap=72)
    lib = binding._lib()
    ctx = st.ctx._ctx
    P = binding._ptr
    q = torch.zeros((2, w.n_q_heads, 90), dtype=st.dt, device=st.device)
    sl = torch.ones(2, dtype=torch.int32, device=st.device)
    # tables not built yet
    assert lib.rap_decode_attn(ctx, 0, 2, P(q), P(st.k_cache[0]), P(st.v_cache[0]), 72, P(sl), 1, 0, P(st.out), None) == binding.RAP_ESTATE
    st.build_tables(*synth.draw_scores(w))
    call = lambda **kw: lib.rap_decode_attn(ctx, kw.get("layer", 0), kw.get("B", 2), kw.get("q", P(q)), P(st.k_cache[0]),
                                            P(st.v_cache[0]), kw.get("cap", 72), P(sl), kw.get("lmax", 1),
                                            kw.get("ns", 0), P(st.out), None)
    assert call() == binding.RAP_OK
    assert call(layer=1) == binding.RAP_EINVAL
    assert call(B=3) == binding.RAP_ESHAPE
    assert call(q=None) == binding.RAP_EINVAL
    assert call(q=binding.c_void_p(q.data_ptr() + 2)) == binding.RAP_EALIGN
    assert call(cap=70) == binding.RAP_EALIGN
    assert call(lmax=73) == binding.RAP_ECAPACITY
    assert call(ns=65) == binding.RAP_ESHAPE
    x = torch.zeros((2, w.hidden), dtype=st.dt, device=st.device)
    st.set_packed_weights(0, synth.draw_packed_weights(w, 0))
    ids = torch.arange(2, dtype=torch.int32, device=st.device)
    app = lambda slot_max, T=2: lib.rap_qkv_rope_append(ctx, 0, T, P(x), P(st.w_qkv[0]), None, P(ids), P(ids), P(ids),
                                                        slot_max, P(st.inv_freq), P(st.q_scratch), P(st.k_cache[0]),
                                                        P(st.v_cache[0]), 2, 72, None)
    assert app(1) == binding.RAP_OK
    assert app(72) == binding.RAP_ECAPACITY
    assert app(1, T=3) == binding.RAP_ESHAPE
    # a slot the host bound did not catch is skipped on the device and reported
    bad = torch.tensor([0, 500], dtype=torch.int32, device=st.device)
    st.k_cache[0].fill_(5.0)
    assert lib.rap_qkv_rope_append(ctx, 0, 2, P(x), P(st.w_qkv[0]), None, P(ids), P(ids), P(bad), 1, P(st.inv_freq),
                                   P(st.q_scratch), P(st.k_cache[0]), P(st.v_cache[0]), 2, 72, None) == binding.RAP_OK
    code, detail = st.ctx.rap_get_last_device_status()
    assert (code, detail) == (binding.RAP_ECAPACITY, 1)
    assert torch.all(st.k_cache[0][1] == 5.0)
    assert st.ctx.rap_get_last_device_status() == (0, 0)
    st.close()


@pytest.mark.parametrize("dtype,pairing", [("f32", 0), ("f32", 1), ("bf16", 0)])
def test_lowrank_comparator_matches_oracle(dtype, pairing):
    """rap_lowrank_decode_attn (latent K rebuilt and rotated at full width every call) against the
    oracle's definition on the same storage-rounded inputs; ragged lengths, several splits."""
    from dataclasses import replace
    w = replace(synth.scaled_down(synth.LLAMA_8B, n_layers=1, batch=3, seq=300), dtype=dtype, pairing=pairing,
                head_dim=64 if dtype == "f32" else 128)
    D, Hq, Hkv, B = w.head_dim, w.n_q_heads, w.n_kv_heads, w.batch
    r, dv = (44, 45) if D == 64 else (90, 90)
    lens = [300, 129, 1]
    cap = 304
    dt = torch.float32 if dtype == "f32" else torch.bfloat16
    rng = np.random.default_rng(77)
    sig = float(np.sqrt(w.hidden) * 0.02)
    lat = O.round_storage(rng.standard_normal((B, Hkv, cap, r)) * sig, dtype)
    V = O.round_storage(rng.standard_normal((B, Hkv, cap, dv)) * sig, dtype)
    Bk = O.round_storage(synth.draw_lowrank_factor(w, 0, r), dtype)
    qf = O.round_storage(rng.standard_normal((B, Hq, D)) * sig, dtype)
    ctx = binding.RapContext(1, w.hidden, Hq, Hkv, D, w.rope_theta, pairing,
                             binding.RAP_F32 if dtype == "f32" else binding.RAP_BF16, B)
    dev = torch.device("cuda:0")
    up = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev).to(dt).contiguous()
    d_lat, d_V, d_Bk, d_q = up(lat), up(V), up(Bk), up(qf)
    dl = torch.tensor(lens, dtype=torch.int32, device=dev)
    want = O.lowrank_decode_attn(qf, lat, Bk, V, lens, D, w.rope_theta, pairing)
    for variant in (0, 1):      # 0: tensor-core rebuild + fast scan where the shape allows; 1: reference kernel
        ctx.rap_set_attn_variant(variant)
        for n_split in (0, 1, 3):
            out = torch.full((B, Hq, dv), float("nan"), dtype=torch.float32, device=dev)
            ctx.rap_lowrank_decode_attn(B, r, dv, d_q, d_lat, d_Bk, d_V, cap, dl, max(lens), n_split, out)
            torch.cuda.synchronize()
            util.check_attn(util.to_np64(out), want, dtype)
    assert ctx.rap_get_last_device_status() == (0, 0)
    ctx.close()


@pytest.mark.parametrize("lens", [[0, 5000, 0, 1, 129, 0], [7000], [1, 1, 1, 1, 1, 1, 1, 1], [0, 0, 3]])
def test_balanced_split_mixed_lengths(lens):
    """n_split = 0 lets every CTA scan an equal share of the global tile sequence: empty sequences,
    one long sequence (segment cap), many one-tile units and CTA ranges that cross unit boundaries."""
    w = synth.scaled_down(synth.LLAMA_8B, n_layers=1, batch=len(lens), seq=max(lens))
    _random_attn_case(w, lens, 0, seed=len(lens))


@pytest.mark.parametrize("name,hidden,T", [("tiny", None, 1), ("8b", 512, 2), ("3b", 512, 5), ("14b", 512, 4), ("8b", None, 32)])
def test_out_proj_matches_oracle(name, hidden, T):
    """rap_pack_wo (column gather, bit-exact) and rap_out_proj (W~_o times the reduced attention output)
    against the oracle on the same storage-rounded inputs; the last case is the 8B shape at batch 32."""
    w = synth.scaled_down(synth.CONFIGS[name], n_layers=2, batch=T, seq=8, hidden=hidden)
    ks, vs = synth.draw_scores(w)
    st = DecodeStack(w, s_cap=16, alloc_cache=False)
    st.build_tables(ks, vs)
    tabs = util.oracle_tables(w, ks, vs)
    rng = np.random.default_rng(12)
    for l in range(w.n_layers):
        Wo = synth.draw_wo(w, l)
        d_wo = torch.from_numpy(Wo).to(st.device).to(st.dt).contiguous()
        d_wt = torch.empty((w.hidden, w.n_q_heads * w.n_vch), dtype=st.dt, device=st.device)
        st.ctx.rap_pack_wo(l, d_wo, st.v_idx, d_wt)
        want_wt = O.gather_wo(O.round_storage(Wo, w.dtype), tabs, l, w.n_vch, w.head_dim, w.n_q_heads, w.n_kv_heads)
        torch.cuda.synchronize()
        assert np.array_equal(util.to_np64(d_wt), want_wt)
        o = rng.standard_normal((T, w.n_q_heads, w.n_vch)).astype(np.float32)
        d_o = torch.from_numpy(o).to(st.device)
        d_y = torch.full((T, w.hidden), float("nan"), dtype=st.dt, device=st.device)
        st.ctx.rap_out_proj(l, T, d_o, d_wt, d_y)
        torch.cuda.synchronize()
        want = O.out_proj(O.round_storage(o, w.dtype), want_wt)
        util.check_projection(util.to_np64(d_y), O.round_storage(want, w.dtype), w.dtype, f"{name} out_proj layer {l}")
    assert st.ctx.rap_get_last_device_status() == (0, 0)
    st.close()


def test_layer_adaptive_budgets_end_to_end():
    """Budgets from rap_budget_alloc (Algorithm 2: per-layer P_l, d_v' = 2 P_l) through tables, projection,
    append and attention: every layer has its own row widths."""
    w = synth.scaled_down(synth.LLAMA_8B, n_layers=4, batch=2, seq=300, hidden=256)
    ks, _ = synth.draw_scores(w)
    ks = ks * np.array([0.5, 1.0, 1.6, 0.9])[:, None, None]
    n_pairs, n_vch = binding.rap_budget_alloc(ks, 0.7, w.head_dim)
    assert len(set(n_pairs.tolist())) > 1 and n_pairs.sum() == round(0.7 * 64 * 4)
    _end_to_end(w, [300, 211], chunk=256, n_pairs=n_pairs.tolist(), n_vch=n_vch.tolist())


@pytest.mark.parametrize("P,dv", [(24, 48), (40, 80), (41, 82), (56, 112), (16, 32), (63, 126)])
def test_layer_adaptive_head_shapes_attention(P, dv):
    """Head shapes that layer-adaptive budgets produce (d_v' = 2P), through the default tier."""
    from dataclasses import replace
    w = replace(synth.scaled_down(synth.LLAMA_8B, n_layers=1, batch=3, seq=3000), n_pairs=P, n_vch=dv)
    _random_attn_case(w, [3000, 1777, 1], 0, seed=P)
    _random_attn_case(w, [3000, 1777, 1], 3, seed=P)


@pytest.mark.parametrize("n_layers,pieces", [(2, None), (3, (1, 128)), (2, (2, 256))])
def test_decode_step_replays_from_a_cuda_graph(n_layers, pieces):
    """rap_decode_step reads the sequence lengths on the device and its balanced scan has a fixed grid, so a
    step captured once can be replayed as the lengths advance: two replays equal two eager steps bit for bit.  Also
    with the scan handing tiles out at run time (forced on this small case): with an odd number of layers two
    consecutive launches of the replay use the same piece counter, which the launch before must have left at zero."""
    w = synth.scaled_down(synth.LLAMA_8B, n_layers=n_layers, batch=2, seq=300, hidden=256)
    ks, vs = synth.draw_scores(w)
    st, tabs, w_host = util.build_small_stack(w, ks, vs, full_weights=False)
    if pieces is not None:
        st.ctx.rap_debug_set_scan_pieces(*pieces)
    g = torch.Generator(device=st.device).manual_seed(5)
    for l in range(w.n_layers):
        st.k_cache[l].normal_(0, 1.0, generator=g)
        st.v_cache[l].normal_(0, 1.0, generator=g)
    k0 = [c.clone() for c in st.k_cache]
    v0 = [c.clone() for c in st.v_cache]
    x = torch.empty((w.n_layers, w.batch, w.hidden), dtype=st.dt, device=st.device).normal_(0, 1, generator=g)

    def reset():
        for l in range(w.n_layers):
            st.k_cache[l].copy_(k0[l])
            st.v_cache[l].copy_(v0[l])
        st.seq_len.copy_(torch.tensor([300, 123], dtype=torch.int32))

    reset()
    eager = []
    for i in range(2):
        st.decode_step(x, 300 + i, advance=1)
        eager.append(st.out.clone())
    torch.cuda.synchronize()
    reset()
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    with torch.cuda.graph(graph, stream=side):
        st.decode_step(x, 301, advance=1)      # the host bound covers both replays
    reset()                                    # capture does not run the work, but keep the state explicit
    for i in range(2):
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(st.out, eager[i])
    P2, dv = 2 * st.n_pairs[n_layers - 1], st.n_vch[n_layers - 1]
    q_last = st.q_scratch.flatten()[: w.batch * w.n_q_heads * P2].reshape(w.batch, w.n_q_heads, P2)
    want = O.decode_attn(util.to_np64(q_last), util.to_np64(st.k_cache[n_layers - 1]), util.to_np64(st.v_cache[n_layers - 1]),
                         [302, 125], w.head_dim)      # the last layer of the last replay against the definition
    util.check_attn(util.to_np64(st.out[n_layers - 1][: w.batch * w.n_q_heads * dv]).reshape(w.batch, w.n_q_heads, dv), want, w.dtype)
    assert st.seq_len.cpu().tolist() == [302, 125]
    assert st.ctx.rap_get_last_device_status() == (0, 0)
    st.close()


@pytest.mark.parametrize("name,T,starts", [("8b", 150, [0, 37]), ("3b", 100, [5, 0]), ("14b", 70, [64, 1]),
                                           ("sweep1.0", 130, [0, 200]), ("sweep0.8", 65, [63, 0]), ("sweep0.5", 128, [0, 128])])
def test_prefill_attn_matches_oracle(name, T, starts):
    _prefill_case(name, T, starts)


def _prefill_case(name, T, starts, q_gain=1.0, ramp=0.0):
    """rap_prefill_attn (tensor-core causal block attention on the reduced dims) against the oracle's masked
    matrix form on the same bf16 caches and q~: several query blocks, ragged starts, tile-boundary lengths."""
    w = synth.scaled_down(synth.CONFIGS[name], n_layers=1, batch=len(starts), seq=max(starts) + T)
    st = DecodeStack(w, s_cap=((max(starts) + T + 8 + 7) // 8) * 8)
    st.build_tables(*synth.draw_scores(w))
    g = torch.Generator(device=st.device).manual_seed(T)
    sig = float(np.sqrt(w.hidden) * 0.02)
    st.k_cache[0].normal_(0, sig, generator=g)
    st.v_cache[0].normal_(0, sig, generator=g)
    B, Hq, P2, dv = w.batch, w.n_q_heads, 2 * w.n_pairs, w.n_vch
    q = torch.empty((B, T, Hq, P2), dtype=st.dt, device=st.device).normal_(0, sig * q_gain, generator=g)
    if ramp > 0:      # K grows with the position: the running maximum keeps moving, the accumulators get rescaled
        pos = torch.arange(st.s_cap, device=st.device, dtype=torch.float32).view(1, 1, -1, 1)
        st.k_cache[0].copy_((st.k_cache[0].float() * (1.0 + ramp * pos)).to(st.dt))
    ds = torch.tensor(starts, dtype=torch.int32, device=st.device)
    want = O.prefill_attn(util.to_np64(q), util.to_np64(st.k_cache[0]), util.to_np64(st.v_cache[0]), starts, w.head_dim)
    for variant in (0, 1):       # 0: tcgen05 kernel, 1: warp-level mma.sync kernel
        st.ctx.rap_set_attn_variant(variant)
        out = torch.full((B, T, Hq, dv), float("nan"), dtype=torch.float32, device=st.device)
        st.ctx.rap_prefill_attn(0, B, T, q, st.k_cache[0], st.v_cache[0], st.s_cap, ds, max(starts), out)
        torch.cuda.synchronize()
        util.check_attn(util.to_np64(out).reshape(B * T, Hq, dv), want.reshape(B * T, Hq, dv), w.dtype)
    assert st.ctx.rap_get_last_device_status() == (0, 0)
    st.close()


@pytest.mark.parametrize("T,starts", [(1, [0, 300]), (257, [63, 0]), (129, [1, 64])])
def test_prefill_attn_block_edges(T, starts):
    """Blocks of one token, of one token more than two query tiles, and of one more than a tile; starts on and
    next to key-tile boundaries."""
    _prefill_case("8b", T, starts)


def test_prefill_attn_many_key_tiles_odd_value_width():
    """A block long enough for the key-tile pipeline to reach its steady state (18 key tiles per query tile), on the
    shape whose V rows have an odd width: their staging is the slowest producer, so the softmax groups run ahead
    of the MMA-issuing lanes as far as the barriers let them."""
    _prefill_case("3b", 1100, [0])


@pytest.mark.parametrize("q_gain,ramp", [(10.0, 0.0), (3.0, 0.004)])
def test_prefill_attn_peaked_and_moving_maximum(q_gain, ramp):
    """Nearly one-hot weights, and a maximum that rises along the keys so that the kernels keep rescaling their
    accumulators (in tensor memory for the tcgen05 kernel)."""
    _prefill_case("8b", 300, [0, 500], q_gain=q_gain, ramp=ramp)


def _decode_step_with_tables(st, tabs, w, lens):
    """Weights gathered with `tabs`, caches filled the real way, one decode step through the unchanged online
    path; appended K rows and the attention output against the oracle."""
    L = w.n_layers
    P, dv, Hq, Hkv, B = w.n_pairs, w.n_vch, w.n_q_heads, w.n_kv_heads, w.batch
    w_host = []
    for l in range(L):
        Wq, Wk, Wv = synth.draw_full_weights(w, l)
        st.pack_from_full(l, Wq, Wk, Wv)
        wr = [O.round_storage(a, w.dtype) for a in (Wq, Wk, Wv)]
        w_host.append(O.gather_weights(wr[0], wr[1], wr[2], tabs, l, P, dv, w.head_dim))
        assert np.array_equal(util.to_np64(st.w_qkv[l]), w_host[l])
    util.prefill_both(st, tabs, w_host, w, lens, chunk=256)
    st.seq_len.copy_(torch.tensor(lens, dtype=torch.int32))
    X = np.stack([synth.draw_hidden(w, l, 1, B) for l in range(L)])
    dx = torch.from_numpy(X).to(st.device).to(st.dt).contiguous()
    st.decode_step(dx, max(lens), advance=0)
    torch.cuda.synchronize()
    for l in range(L):
        q, k, v = O.qkv_rope(O.round_storage(X[l], w.dtype), w_host[l], None, np.array(lens), tabs["inv_freq"][l], Hq, Hkv, P, dv)
        Kd, Vd = util.to_np64(st.k_cache[l]), util.to_np64(st.v_cache[l])
        k_dev = np.stack([Kd[b, :, lens[b], :] for b in range(B)])
        util.check_projection(k_dev, O.round_storage(k, w.dtype), w.dtype, f"k layer {l}")
        want = O.decode_attn(O.round_storage(q, w.dtype), Kd, Vd, np.array(lens) + 1, w.head_dim)
        got = util.to_np64(st.out[l][: B * Hq * dv]).reshape(B, Hq, dv)
        util.check_attn(got, want, w.dtype)
    assert st.ctx.rap_get_last_device_status() == (0, 0)


def test_hybrid_tables_and_nope_layer_end_to_end():
    """rap_build_tables_hybrid: layer 0 rotary, layer 1 without RoPE (channel-pruned K, zero frequencies).
    Tables bit-exact against the oracle, then one decode step through the unchanged online path."""
    w = synth.scaled_down(synth.LLAMA_8B, n_layers=2, batch=2, seq=200, hidden=256)
    ks, vs = synth.draw_scores(w)
    kc = np.random.default_rng(6).lognormal(0, 1, (2, w.n_kv_heads, w.head_dim))
    rope_layer = [1, 0]
    st = DecodeStack(w, max_rows=256)
    st.ctx.rap_build_tables_hybrid(ks, kc, vs, rope_layer, st.n_pairs, st.n_vch, st.k_pair_idx, st.k_dim_idx, st.v_idx,
                                   st.inv_freq)
    tabs = O.build_tables_hybrid(ks, kc, vs, rope_layer, st.n_pairs, st.n_vch, w.head_dim, w.rope_theta, w.pairing)
    _tables_equal(st, tabs)
    _decode_step_with_tables(st, tabs, w, [200, 77])
    st.close()


def test_partial_rotary_tables_end_to_end():
    """rap_build_tables_partial: a fully rotary layer, a layer that rotates 64 of 128 dims (22 of its 45 pair
    slots hold rotated pairs, the rest unrotated channels), one that rotates 32 dims and one without RoPE.
    Tables bit-exact against the oracle, then one decode step through the unchanged online path; out-of-range
    counts are refused."""
    w = synth.scaled_down(synth.LLAMA_8B, n_layers=4, batch=2, seq=150, hidden=256)
    ks, vs = synth.draw_scores(w)
    kc = np.random.default_rng(9).lognormal(0, 1, (4, w.n_kv_heads, w.head_dim))
    D, P = w.head_dim, w.n_pairs
    rot_dims = [D, 64, 32, 0]
    n_rot = [P, 22, 16, 0]          # layer 1: 22 of 32 pairs + 46 of 64 channels; layer 2: all 16 pairs + 58 of 96
    st = DecodeStack(w, max_rows=256)
    args = (st.n_pairs, st.n_vch, st.k_pair_idx, st.k_dim_idx, st.v_idx, st.inv_freq)
    st.ctx.rap_build_tables_partial(ks, kc, vs, rot_dims, n_rot, *args)
    tabs = O.build_tables_partial(ks, kc, vs, rot_dims, n_rot, st.n_pairs, st.n_vch, D, w.rope_theta, w.pairing)
    _tables_equal(st, tabs)
    _decode_step_with_tables(st, tabs, w, [150, 61])
    for bad_rot, bad_n in (([D, 63, 32, 0], n_rot), ([D, 64, 32, 0], [P, 33, 16, 0]), ([D, 64, 32, 0], [P, 22, 16, 1]),
                           ([D, 64, 32, 0], [P, 10, 16, 0])):      # odd R; pairs > R/2; pairs without rotary dims; channels > D - R
        with pytest.raises(binding.RapError) as e:
            st.ctx.rap_build_tables_partial(ks, kc, vs, bad_rot, bad_n, *args)
        assert e.value.status == 1
    st.close()


def test_frequency_scaled_tables_end_to_end():
    """rap_build_tables_freq: the model's own per-pair frequency table (every pair of the standard table slowed
    down by its own factor, different per layer) instead of theta^(-2i/D).  Index tables and the gathered
    frequencies equal the oracle's exactly; one decode step through the unchanged online path (appended K rows and
    the attention output against the oracle); then a block of new tokens through rap_prefill_attn on the caches that
    the scaled rotation wrote.  The frequencies are far from the standard ones, so a path that ignored the table
    would miss the appended rows by much more than the tolerance."""
    w = synth.scaled_down(synth.LLAMA_8B, n_layers=2, batch=2, seq=200, hidden=256)
    ks, vs = synth.draw_scores(w)
    D, half, L = w.head_dim, w.head_dim // 2, w.n_layers
    base = w.rope_theta ** (-2.0 * np.arange(half) / D)
    rng = np.random.default_rng(31)
    freq = np.stack([base / np.linspace(1.0, 16.0, half), base * rng.uniform(0.2, 1.0, half)])
    st = DecodeStack(w, max_rows=256)
    st.ctx.rap_build_tables_freq(ks, vs, freq, st.n_pairs, st.n_vch, st.k_pair_idx, st.k_dim_idx, st.v_idx, st.inv_freq)
    tabs = O.build_tables_freq(ks, vs, freq, st.n_pairs, st.n_vch, D, w.pairing)
    torch.cuda.synchronize()
    for key, dev in (("k_pair_idx", st.k_pair_idx), ("k_dim_idx", st.k_dim_idx), ("v_idx", st.v_idx), ("inv_freq", st.inv_freq)):
        assert np.array_equal(dev.cpu().numpy(), tabs[key]), key
    std = util.oracle_tables(w, ks, vs)
    assert np.abs(tabs["inv_freq"] - std["inv_freq"]).max() > 0.1
    lens = [200, 77]
    _decode_step_with_tables(st, tabs, w, lens)
    # the standard table would have put the new K rows somewhere else entirely
    l, P, dv = 1, w.n_pairs, w.n_vch
    X = O.round_storage(synth.draw_hidden(w, l, 1, w.batch), w.dtype)
    w_host = util.to_np64(st.w_qkv[l])
    _, k_std, _ = O.qkv_rope(X, w_host, None, np.array(lens), std["inv_freq"][l], w.n_q_heads, w.n_kv_heads, P, dv)
    Kd = util.to_np64(st.k_cache[l])
    k_dev = np.stack([Kd[b, :, lens[b], :] for b in range(w.batch)])
    assert np.abs(k_dev - k_std).max() > 0.1
    # prefill-side attention over the same caches: 60 new tokens per sequence written through the scaled rotation
    T = 60
    rows = [(b, lens[b] + 1 + i) for b in range(w.batch) for i in range(T)]
    sid = torch.tensor([r[0] for r in rows], dtype=torch.int32, device=st.device)
    pos = torch.tensor([r[1] for r in rows], dtype=torch.int32, device=st.device)
    xb = torch.from_numpy(synth.draw_hidden(w, l, 2, len(rows))).to(st.device).to(st.dt).contiguous()
    q = torch.empty((len(rows), w.n_q_heads, 2 * P), dtype=st.dt, device=st.device)
    st.qkv_rope_append(l, xb, sid, pos, pos, int(pos.max()), q_out=q)
    start = torch.tensor([n + 1 for n in lens], dtype=torch.int32, device=st.device)
    out = torch.full((w.batch, T, w.n_q_heads, dv), float("nan"), dtype=torch.float32, device=st.device)
    st.ctx.rap_prefill_attn(l, w.batch, T, q, st.k_cache[l], st.v_cache[l], st.s_cap, start, max(lens) + 1, out)
    torch.cuda.synchronize()
    qo, ko, _ = O.qkv_rope(O.round_storage(util.to_np64(xb), w.dtype), w_host, None, pos.cpu().numpy(), tabs["inv_freq"][l],
                           w.n_q_heads, w.n_kv_heads, P, dv)
    util.check_projection(util.to_np64(q), O.round_storage(qo, w.dtype), w.dtype, "q of the block")
    want = O.prefill_attn(util.to_np64(q).reshape(w.batch, T, w.n_q_heads, 2 * P), util.to_np64(st.k_cache[l]),
                          util.to_np64(st.v_cache[l]), [n + 1 for n in lens], D)
    util.check_attn(util.to_np64(out).reshape(w.batch * T, w.n_q_heads, dv), want.reshape(w.batch * T, w.n_q_heads, dv), w.dtype)
    assert st.ctx.rap_get_last_device_status() == (0, 0)
    st.close()


@pytest.mark.parametrize("name,T,with_bias", [("8b", 32, False), ("3b", 16, True), ("14b", 4, False), ("sweep1.0", 1, True),
                                              ("sweep0.5", 7, False), ("8b", 31, True)])
def test_fused_projection_against_the_oracle_and_the_two_stage_form(name, T, with_bias):
    """Decode-sized rap_qkv_rope_append runs as one kernel (RoPE, rounding and append fused into the tcgen05 GEMM's
    epilogue, finished by whichever warp delivers a row block's last reduction split).  Rows of several sequences at
    scattered slots and far-apart positions, with and without a bias, on head shapes whose q / k / v sections start in
    the middle of a 32-row block (odd d_v' included): q~, the K rows and the V rows against the oracle, against the
    two-stage form of the same call, canaries around every written row, and twice in a row (the arrival counters
    must come back to zero)."""
    w = synth.scaled_down(synth.CONFIGS[name], n_layers=2, batch=3, seq=64, hidden=1024)
    ks, vs = synth.draw_scores(w)
    st, tabs, w_host = util.build_small_stack(w, ks, vs, full_weights=False, s_cap=4096, max_rows=32)
    Hq, Hkv, P, dv = w.n_q_heads, w.n_kv_heads, w.n_pairs, w.n_vch
    rng = np.random.default_rng(T)
    sid = rng.integers(0, w.batch, T).astype(np.int32)
    slot = rng.choice(4096, size=T, replace=False).astype(np.int32)        # distinct rows, so the result is unique
    pos = np.where(rng.random(T) < 0.5, slot, rng.integers(0, 120000, T)).astype(np.int32)
    d_sid, d_slot, d_pos = (torch.from_numpy(a).to(st.device) for a in (sid, slot, pos))
    bias_host = None
    if with_bias:
        st.bias, bias_host = [], []
        for l in range(w.n_layers):
            b = synth.draw_bias(w, l, st.n_out(l))
            st.bias.append(torch.from_numpy(b).to(st.device).to(st.dt))
            bias_host.append(O.round_storage(b, w.dtype))
    for l in range(w.n_layers):
        X = synth.draw_hidden(w, l, 5, T)
        dx = torch.from_numpy(X).to(st.device).to(st.dt).contiguous()
        q, k, v = O.qkv_rope(O.round_storage(X, w.dtype), w_host[l], None if bias_host is None else bias_host[l], pos,
                             tabs["inv_freq"][l], Hq, Hkv, P, dv)
        results = []
        for variant, rounds in ((0, 2), (1, 1)):        # fused (twice), then the two-stage form
            st.ctx.rap_set_proj_variant(variant)
            for _ in range(rounds):
                st.k_cache[l].fill_(-77.0)
                st.v_cache[l].fill_(-77.0)
                dq = torch.full((T, Hq, 2 * P), float("nan"), dtype=st.dt, device=st.device)
                n0 = st.ctx.rap_kernel_launch_count()
                st.qkv_rope_append(l, dx, d_sid, d_pos, d_slot, int(slot.max()), q_out=dq)
                torch.cuda.synchronize()
                assert st.ctx.rap_kernel_launch_count() - n0 == (1 if variant == 0 else 2)
                assert st.ctx.rap_get_last_device_status() == (0, 0)
                Kd, Vd = util.to_np64(st.k_cache[l]), util.to_np64(st.v_cache[l])
                written = np.zeros(Kd.shape[:3], dtype=bool)
                written[sid, :, slot] = True
                assert np.all(Kd[~written] == -77.0) and np.all(Vd[~written] == -77.0)
                k_dev, v_dev = Kd[sid, :, slot, :], Vd[sid, :, slot, :]
                util.check_projection(util.to_np64(dq), O.round_storage(q, w.dtype), w.dtype, f"q layer {l}")
                util.check_projection(k_dev, O.round_storage(k, w.dtype), w.dtype, f"k layer {l}")
                util.check_projection(v_dev, O.round_storage(v, w.dtype), w.dtype, f"v layer {l}")
                results.append((util.to_np64(dq), k_dev, v_dev))
        for a, b in zip(results[0], results[1]):
            assert np.array_equal(a, b)                  # the same call twice: bit-identical
        for a, b in zip(results[0], results[2]):         # the two forms differ by the rounding order of one product
            assert np.abs(a - b).max() <= 2.0 ** -7 * max(1e-30, np.abs(b).max())
        assert np.array_equal(results[0][2], results[2][2])          # V rows take no rotation: identical
    st.ctx.rap_set_proj_variant(0)
    st.close()


def test_fused_projection_skips_and_reports_an_out_of_range_row():
    w = synth.scaled_down(synth.LLAMA_8B, n_layers=1, batch=2, seq=64, hidden=256)
    st, tabs, w_host = util.build_small_stack(w, *synth.draw_scores(w), full_weights=False, s_cap=72, max_rows=8)
    x = torch.ones((3, w.hidden), dtype=st.dt, device=st.device)
    sid = torch.tensor([0, 1, 5], dtype=torch.int32, device=st.device)      # the third row names a sequence that is not there
    pos = torch.tensor([3, 4, 5], dtype=torch.int32, device=st.device)
    st.k_cache[0].fill_(5.0)
    st.v_cache[0].fill_(5.0)
    n0 = st.ctx.rap_kernel_launch_count()
    st.qkv_rope_append(0, x, sid, pos, pos, 5)
    torch.cuda.synchronize()
    assert st.ctx.rap_kernel_launch_count() - n0 == 1
    assert st.ctx.rap_get_last_device_status() == (binding.RAP_ECAPACITY, 2)
    changed = (st.k_cache[0] != 5.0).any(dim=-1).cpu().numpy()
    expect = np.zeros_like(changed)
    expect[0, :, 3] = expect[1, :, 4] = True
    assert np.array_equal(changed, expect)
    st.close()


def test_bounded_wait_gives_up_reports_and_the_next_launches_recover():
    """A device-side wait that cannot complete (a stage barrier armed by the test hook without a copy behind it, polled
    a few thousand times): the launch ends by itself, the status word says RAP_ETIMEOUT, the context stays usable,
    and the launches after it are right again without any reset from the host -- each launch clears the arrival
    counters its predecessor used, so the units the timed-out CTA left half counted do not poison later merges."""
    w = synth.scaled_down(synth.LLAMA_8B, n_layers=1, batch=3, seq=3000)
    lens = [3000, 1777, 640]
    st = DecodeStack(w, s_cap=3008)
    st.build_tables(*synth.draw_scores(w))
    g = torch.Generator(device=st.device).manual_seed(4)
    sig = float(np.sqrt(w.hidden) * 0.02)
    st.k_cache[0].normal_(0, sig, generator=g)
    st.v_cache[0].normal_(0, sig, generator=g)
    q = torch.empty((w.batch, w.n_q_heads, 2 * w.n_pairs), dtype=st.dt, device=st.device).normal_(0, sig, generator=g)
    dl = torch.tensor(lens, dtype=torch.int32, device=st.device)
    want = O.decode_attn(util.to_np64(q), util.to_np64(st.k_cache[0]), util.to_np64(st.v_cache[0]), lens, w.head_dim)
    shape = (w.batch, w.n_q_heads, w.n_vch)

    def run():
        out = st.decode_attn(0, q, dl, max(lens))
        torch.cuda.synchronize()
        return util.to_np64(out[: int(np.prod(shape))]).reshape(shape)

    util.check_attn(run(), want, w.dtype)
    assert st.ctx.rap_get_last_device_status() == (0, 0)
    st.out.fill_(float("nan"))
    st.ctx.rap_debug_arm_wait_timeout()
    got = run()                                   # returns: the wait is bounded
    assert np.isnan(got[0, : w.group]).all()      # the first unit (sequence 0, KV head 0) was never finished ...
    finished = ~np.isnan(got).any(axis=-1)
    assert finished.sum() >= finished.size - 2 * w.group          # ... the CTA touched two units at most
    util.check_attn(got[finished], want[finished], w.dtype)
    # no status read, no reset: two more launches (one per counter set) are complete and right
    for _ in range(2):
        st.out.fill_(float("nan"))
        util.check_attn(run(), want, w.dtype)
    code, detail = st.ctx.rap_get_last_device_status()
    assert code == binding.RAP_ETIMEOUT
    assert st.ctx.rap_get_last_device_status() == (0, 0)
    util.check_attn(run(), want, w.dtype)
    st.close()
