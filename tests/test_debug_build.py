"""The bounds-checked build (SVIP_DEBUG_BOUNDS + SVIP_NVTX) compiles and exports the same ABI; on a GPU it runs
a small published configuration, aligned and unaligned, with no load outside the logits buffers."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_debug_build_compiles_and_exports_the_abi():
    import ctypes as C
    import re
    from paper_2411_18462_b200 import build
    path = build.build(debug=True)
    assert os.path.basename(path) == "libsvip_debug.so" and os.path.exists(path)
    lib = C.CDLL(path)
    text = open(os.path.join(ROOT, "include", "svip.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    for name in sorted(set(re.findall(r"\b(svip_[a-z_0-9]+)\s*\(", text))):
        assert hasattr(lib, name), name


CHILD = r'''
import numpy as np, torch, sys
sys.path.insert(0, %r); sys.path.insert(0, %r)
import svip_testlib as tl
from oracle import svip_oracle as O
from paper_2411_18462_b200 import Context, workloads as W, binding
assert binding.library_path().endswith("libsvip_debug.so")
ctx = Context(0, 4096)
w = W.make_workload("chat", B=4, K_max=6)
for S in (0, 1, 3):
    ctx.set_cluster_size(S)
    got = tl.gpu_draft_step(ctx, w.q_logits, w.T, w.h, w.draft_uniforms)
    tl.check_draft_against_oracle(O, w.q_logits, w.T, w.h, w.draft_uniforms, got, "debug build")
    tok = got[0].astype(np.int32)
    uv, _ = tl.guard_accept_uniforms(O, tok, w.q_logits, w.target_logits, w.cu_rows, w.T, w.verify_uniforms)
    res = tl.gpu_verify(ctx, tok, w.q_logits, w.target_logits, w.cu_rows, w.K_max, w.T, uv, fixed_K=True)
    tl.check_verify_against_oracle(O, tok, w.q_logits, w.target_logits, w.cu_rows, w.T, uv, res, "debug build")
    # unaligned rows: the vector loads reach into the 16-byte granules around a row, never beyond
    x = w.q_logits[:5, :4099].copy()
    got = tl.gpu_draft_step(ctx, x, 1.0, 0.3, w.draft_uniforms[:5], pad_elems=3, row_stride=4101)
    tl.check_draft_against_oracle(O, x, 1.0, 0.3, w.draft_uniforms[:5], got, "debug build, unaligned")
assert ctx.read_status() == 0, "a load outside the buffers was reported"
ctx.set_cluster_size(0)
print("debug build ok")
''' % (ROOT, os.path.join(ROOT, "tests"))


@pytest.mark.gpu
def test_debug_build_runs_clean_on_the_gpu():
    from paper_2411_18462_b200 import build
    path = build.build(debug=True)
    env = dict(os.environ, SVIP_LIBRARY=path)
    out = subprocess.run([sys.executable, "-c", CHILD], env=env, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0 and "debug build ok" in out.stdout, out.stdout[-2000:] + out.stderr[-4000:]
