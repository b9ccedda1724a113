"""rap_decode_attn_noalloc: the entry point for callers that cannot allocate device memory
(engines that own the whole HBM budget, code that runs where cudaMalloc is off limits).  Its
split-KV scratch is a static array inside the library, so the checks here are: same result as
rap_decode_attn and as the CPU oracle (Eq. 2 on the device's own q~ and cache rows), also on a
second call that finds the first call's partials in the array; no device memory taken by a call;
and a clear refusal of a request the array cannot hold.  Collected last on purpose."""
import numpy as np
import pytest
import torch

from oracle import rap_oracle as O
from paper_2602_02599_b200 import binding, synth
from paper_2602_02599_b200.stack import DecodeStack

import util

pytestmark = pytest.mark.gpu


def _case(w, lens, n_split, seed):
    st = DecodeStack(w, s_cap=((max(lens) + 8 + 7) // 8) * 8)
    st.build_tables(*synth.draw_scores(w))
    g = torch.Generator(device=st.device).manual_seed(seed)
    sig = float(np.sqrt(w.hidden) * 0.02)
    st.k_cache[0].normal_(0, sig, generator=g)
    st.v_cache[0].normal_(0, sig, generator=g)
    q = torch.empty((w.batch, w.n_q_heads, 2 * w.n_pairs), dtype=st.dt, device=st.device).normal_(0, sig, generator=g)
    dl = torch.tensor(lens, dtype=torch.int32, device=st.device)
    want = st.decode_attn(0, q, dl, int(max(lens)))[: w.batch * w.n_q_heads * w.n_vch].clone()
    return st, q, dl, want


@pytest.mark.parametrize("name", ["tiny", "8b"])
def test_noalloc_matches_decode_attn_on_two_calls_in_a_row(name):
    base = synth.CONFIGS[name]
    w = synth.scaled_down(base, n_layers=1, batch=3, seq=1200)
    dtype = binding.RAP_F32 if w.dtype == "f32" else binding.RAP_BF16
    # two different problems back to back: the second call starts from the first call's partials
    for call, (lens, n_split) in enumerate([([1200, 700, 1], 0), ([90, 1200, 333], 5)]):
        st, q, dl, want = _case(w, lens, n_split, seed=call)
        got = torch.full_like(want, float("nan"))
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        binding.rap_decode_attn_noalloc(dtype, w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.n_pairs, w.n_vch,
                                        q, st.k_cache[0], st.v_cache[0], st.s_cap, dl, max(lens), n_split, got)
        torch.cuda.synchronize()
        if call == 1:      # the first call on a device may load the library's kernels; the second takes nothing
            assert torch.cuda.mem_get_info()[0] == free_before
        util.check_attn(util.to_np64(got), util.to_np64(want), w.dtype)
        # and against the definition itself, on the same stored q~ and cache rows
        oracle = O.decode_attn(util.to_np64(q), util.to_np64(st.k_cache[0]), util.to_np64(st.v_cache[0]), lens, w.head_dim)
        util.check_attn(util.to_np64(got).reshape(oracle.shape), oracle, w.dtype)
        st.close()


def test_noalloc_rejects_what_the_static_array_cannot_hold():
    w = synth.scaled_down(synth.LLAMA_8B, n_layers=1, batch=2, seq=64)
    st, q, dl, _ = _case(w, [64, 64], 0, seed=0)
    out = torch.zeros((2, w.n_q_heads, w.n_vch), dtype=torch.float32, device=st.device)
    lib = binding._lib()
    P = binding._ptr
    call = lambda B, ns: lib.rap_decode_attn_noalloc(binding.RAP_BF16, B, w.n_q_heads, w.n_kv_heads, w.head_dim,
                                                     w.n_pairs, w.n_vch, P(q), P(st.k_cache[0]), P(st.v_cache[0]),
                                                     st.s_cap, P(dl), 64, ns, P(out), None)
    assert call(2, 1) == binding.RAP_OK
    # B * H_q * (d_v' + 2) floats for ONE split already exceed 2^20: refused before any launch
    big_B = binding.NOALLOC_WS_FLOATS // (w.n_q_heads * (w.n_vch + 2)) + 1
    assert call(big_B, 0) == binding.RAP_ESHAPE
    # an explicit split count that does not fit is refused too (a fitting one is chosen when n_split = 0)
    B_mid = binding.NOALLOC_WS_FLOATS // (w.n_q_heads * (w.n_vch + 2) * 4)
    assert call(B_mid, 8) == binding.RAP_ESHAPE
    # more sequences than the launch grid can index: refused as a shape, not reported as a failed launch
    narrow = lambda B: lib.rap_decode_attn_noalloc(binding.RAP_BF16, B, 1, 1, 16, 1, 1, P(q), P(st.k_cache[0]),
                                                   P(st.v_cache[0]), st.s_cap, P(dl), 64, 1, P(out), None)
    assert narrow(65536) == binding.RAP_ESHAPE
    with pytest.raises(binding.RapError, match="static array holds"):
        binding.rap_decode_attn_noalloc(binding.RAP_BF16, big_B, w.n_q_heads, w.n_kv_heads, w.head_dim, w.n_pairs,
                                        w.n_vch, q, st.k_cache[0], st.v_cache[0], st.s_cap, dl, 64, 0, out)
    torch.cuda.synchronize()
    st.close()
