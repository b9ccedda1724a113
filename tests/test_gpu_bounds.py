"""The bounds-checking build of the library (librap_b200_dbg.so: the same sources with -DRAP_DEBUG_BOUNDS): every
hand-computed shared-memory and global index of the tensor-core scans (bf16 and quantised) and of the fused
projection epilogue is checked on the device; a failed check is recorded in the device status word and the access is
skipped.  The parity tests that reach those kernels at their edges (one-row sequences, tile and block boundaries,
more splits than tiles, odd d_v', ragged batches, rows that straddle the q / k / v sections) run again on that
library in a child process; all of them assert a clean status word.  One more case shows that the checks are live."""
import os
import subprocess
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
pytestmark = pytest.mark.gpu

EDGE_CASES = ("ragged_and_tile_boundaries or tensor_core_scan_head_shapes or balanced_split_mixed_lengths or "
              "fused_projection or q8_attention_mixed_lengths or q8_attention_longer or q8_append_and_attention or "
              "scaled_down_bf16_twins or layer_adaptive_head_shapes or peaked_moving_and_flat")


def _debug_library():
    from paper_2602_02599_b200 import build
    return build.build_debug()


def test_edge_cases_pass_with_every_index_checked():
    env = dict(os.environ, RAP_LIBRARY=_debug_library())
    r = subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", "test_gpu_parity.py"),
                        os.path.join(ROOT, "tests", "test_gpu_q8.py"), "-m", "gpu", "-x", "-q", "-k", EDGE_CASES],
                       cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]
    assert " passed" in r.stdout and "failed" not in r.stdout


_LIVE = r"""
import sys, numpy as np, torch
sys.path.insert(0, %r); sys.path.insert(0, %r)
from paper_2602_02599_b200 import binding, synth
from paper_2602_02599_b200.stack import DecodeStack
from oracle import rap_oracle as O
import util
w = synth.scaled_down(synth.LLAMA_8B, n_layers=1, batch=2, seq=900)
st = DecodeStack(w, s_cap=904)
st.build_tables(*synth.draw_scores(w))
g = torch.Generator(device=st.device).manual_seed(1)
st.k_cache[0].normal_(0, 1.0, generator=g); st.v_cache[0].normal_(0, 1.0, generator=g)
q = torch.empty((2, w.n_q_heads, 2 * w.n_pairs), dtype=st.dt, device=st.device).normal_(0, 1.0, generator=g)
dl = torch.tensor([900, 411], dtype=torch.int32, device=st.device)
want = O.decode_attn(util.to_np64(q), util.to_np64(st.k_cache[0]), util.to_np64(st.v_cache[0]), [900, 411], w.head_dim)
def run():
    out = st.decode_attn(0, q, dl, 900); torch.cuda.synchronize()
    return util.to_np64(out[: want.size]).reshape(want.shape)
util.check_attn(run(), want, w.dtype)
assert st.ctx.rap_get_last_device_status() == (0, 0)
st.ctx.rap_debug_claim_scan_workspace(16)          # the workspace is as large as ever; the kernel is told 16 floats
run()
code, detail = st.ctx.rap_get_last_device_status()
print("STATUS", code, hex(detail))
util.check_attn(run(), want, w.dtype)               # the hook disarmed itself; the next launch is right again
assert st.ctx.rap_get_last_device_status() == (0, 0)
st.close()
"""


def test_the_index_checks_are_live():
    """A scan launch that is told its workspace is 16 floats long: in the bounds-checking build the partial writes are
    skipped and RAP_EBOUNDS is reported (nothing leaves a buffer: the workspace has its real size); the same script
    on the normal library, which carries no checks, reports a clean status."""
    script = _LIVE % (ROOT, os.path.join(ROOT, "tests"))
    for lib, want in ((_debug_library(), "STATUS 9 0x109"), (None, "STATUS 0 0x0")):
        env = dict(os.environ)
        env.pop("RAP_LIBRARY", None)
        if lib:
            env["RAP_LIBRARY"] = lib
        r = subprocess.run([sys.executable, "-c", script], cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)
        assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-3000:]
        assert want in r.stdout, r.stdout
