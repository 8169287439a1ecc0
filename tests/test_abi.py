"""Host-only checks of the C ABI: the library loads without a GPU, exports every function the
header declares, and rejects bad arguments on the host before touching CUDA."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2411_18462_b200 import build, binding
    build.build()
    return binding.library()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "svip.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(svip_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert {"svip_draft_step", "svip_verify", "svip_pack_ragged", "svip_create", "svip_graph_launch"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_strerror_and_version(lib):
    assert lib.svip_version() >= 100
    assert lib.svip_strerror(0) == b"ok"
    for code in (-1, -2, -3, -4, -5):
        assert lib.svip_strerror(code) not in (b"ok", b"unknown status")
    assert lib.svip_strerror(-99) == b"unknown status"


def test_null_context_is_invalid_argument(lib):
    assert lib.svip_draft_step(None, 16, 0, 1, 8, 8, 1.0, 0.3, 16, 16, 16, 16, None, None) == -1
    assert lib.svip_pack_ragged(None, 16, 1, 1, 16, None, None, None) == -1
    assert lib.svip_verify(None, 16, 16, 8, None, -1, 0, 16, 8, 0, None, 1, 1, 2, 8, 1.0, 16, 16, 16, None) == -1
    assert lib.svip_create(None, 0, 16) == -1
    h = C.c_void_p()
    assert lib.svip_create(C.byref(h), 0, 0) == -1
    assert lib.svip_create(C.byref(h), -1, 16) == -1
    assert lib.svip_destroy(None) == -1
    assert lib.svip_graph_launch(None, None) == -1
    assert lib.svip_graph_destroy(None) == -1
    assert lib.svip_set_cluster_size(None, 1) == -1
    assert lib.svip_row_threshold(None, 16, 0, 1, 8, 8, 1.0, 2, 0.9, 16, None, None) == -1
    assert lib.svip_draft_step_at(None, 16, 0, 1, 8, 8, 8, 16, 1, 1.0, 0.3, 16, None, 16, 16, 16, None, None) == -1
    assert lib.svip_draft_step_filtered(None, 16, 0, 1, 8, 8, 1.0, 0.3, 16, None, 16, 16, 16, 16, None, None) == -1
    assert lib.svip_verify_filtered(None, 16, 16, 8, None, 16, -1, 0, 16, 8, 16, None, 0, None, 1, 1, 2, 8, 1.0, 16, 16,
                                    16, None) == -1
    assert lib.svip_draft_step_truncated(None, 16, 0, 1, 8, 8, 1.0, 0.3, 2, 0.9, 16, None, 16, 16, 16, 16, None, None) == -1
    assert lib.svip_graph_loop_end(None) == -1
    body = C.c_void_p()
    assert lib.svip_graph_loop_begin(None, None, 16, 4, C.byref(body)) == -1
    assert lib.svip_launch_count(None) == 0
    assert lib.svip_selftest_wait_timeout(None, 1000, None) == -1


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    from paper_2411_18462_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "_LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(binding.SvipError):
        binding.library()
