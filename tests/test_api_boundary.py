"""The C-ABI boundary without a GPU: the built library loads, exports every function the public header
declares, and rejects bad arguments on the host before any device work."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "hsd.h")


@pytest.fixture(scope="module")
def B():
    from paper_2602_12957_b200 import build
    build.build()
    from paper_2602_12957_b200 import binding
    return binding


def declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"HSD_API[^;(]*?\b(hsd_[a-z0-9_]+)\s*\(", text)))


def test_header_declares_the_three_named_calls():
    names = declared_functions()
    for n in ("hsd_verify_regions", "hsd_verify_page", "hsd_kv_commit", "hsd_create", "hsd_destroy"):
        assert n in names
    assert len(names) >= 15


def test_library_exports_every_declared_function_and_the_binding_lists_them(B):
    lib = C.CDLL(B.LIB_PATH)
    names = declared_functions()
    for n in names:
        assert getattr(lib, n) is not None
    assert sorted(B.EXPORTS) == names
    for n in names:
        assert hasattr(B, n), f"binding lacks {n}"


def test_status_strings(B):
    assert B.hsd_status_string(0) == "ok"
    seen = {B.hsd_status_string(s) for s in range(-8, 1)}
    assert len(seen) == 9 and "unknown status" not in seen
    assert B.hsd_status_string(-99) == "unknown status"


def test_constants_match_the_header(B):
    text = open(HEADER).read()
    for name in ("HSD_MAX_Q_LEN", "HSD_MAX_TREE_ROWS", "HSD_MAX_WINDOW", "HSD_DSV_MAX_CANDIDATES", "HSD_KV_BLOCK", "HSD_NOALLOC_MAX_ROWS", "HSD_FLAG_SIMT_DEBUG", "HSD_FLAG_SIMT_ATTENTION",
                 "HSD_FLAG_DETERMINISTIC", "HSD_FLAG_NO_PDL", "HSD_FLAG_NO_PAIR", "HSD_FLAG_NO_HOST_GRAPH"):
        m = re.search(rf"#define\s+{name}\s+(-?\d+)", text)
        assert m and int(m.group(1)) == getattr(B, name), name
    for k, name in enumerate(("X", "H_ATTN", "H_FFN", "Q", "ATTN", "ACT", "X_MID")):
        m = re.search(rf"#define\s+HSD_TAP_{name}\s+(\d+)", text)
        assert m and int(m.group(1)) == k == getattr(B, "HSD_TAP_" + name), name
    for name in ("INVALID_ARG", "SHAPE", "TOO_LONG", "WORKSPACE", "KV_CAPACITY", "CUDA", "DEVICE_CHECK", "NO_DEVICE"):
        m = re.search(rf"#define\s+HSD_ERR_{name}\s+\((-\d+)\)", text)
        assert m and int(m.group(1)) == getattr(B, "HSD_ERR_" + name), name


def test_host_side_argument_checks_need_no_device(B):
    from paper_2602_12957_b200 import inputs as I
    st, ctx = B.hsd_create(None, None)
    assert st == B.HSD_ERR_INVALID_ARG and not ctx
    cfg = B.make_config(I.TINY)
    w = B.hsd_weights()                                   # all null pointers
    st, ctx = B.hsd_create(cfg, w)
    assert st == B.HSD_ERR_INVALID_ARG
    bad = B.make_config(I.ModelConfig(1, 256, 4, 4, 96, 1024, 4096))    # head_dim is 64 or 128
    assert B.hsd_create(bad, w)[0] == B.HSD_ERR_SHAPE
    simt128 = B.make_config(I.ModelConfig(1, 256, 2, 2, 128, 1024, 4096), B.HSD_FLAG_SIMT_ATTENTION)
    assert B.hsd_create(simt128, w)[0] == B.HSD_ERR_SHAPE              # the plain cross-check kernels: head_dim 64 only
    bad = B.make_config(I.ModelConfig(1, 256, 4, 3, 64, 1024, 4096))     # heads not a multiple of kv heads
    assert B.hsd_create(bad, w)[0] == B.HSD_ERR_SHAPE
    # calls on a null context
    assert B.hsd_destroy(None) == B.HSD_ERR_INVALID_ARG
    assert B.hsd_workspace_bytes(None, 10, 1) == 0
    assert B.hsd_launch_count(None) == 0
    assert B.hsd_kv_commit(None, None, 1, None, None, None, None) == B.HSD_ERR_INVALID_ARG
    assert B.hsd_verify_regions(None, None, 1, None, None, None, 1, 1, 0.0, None, None, None, None, None, None,
                                None, 0, None) == B.HSD_ERR_INVALID_ARG
    assert B.hsd_verify_page(None, None, 0, None, None, 0, 0.0, None, None, None, None, None, None, None, 0,
                             None) == B.HSD_ERR_INVALID_ARG
    assert B.hsd_verify_tree(None, None, 1, None, None, None, None, 1, 1, 0.0, None, None, None, None, None, None, None,
                             None, 0, None) == B.HSD_ERR_INVALID_ARG
    assert B.hsd_kv_commit_tree(None, None, 1, None, None, None, 1, None, None) == B.HSD_ERR_INVALID_ARG
    assert B.hsd_debug_tap(None, 0, 0, None, 0) == B.HSD_ERR_INVALID_ARG
    assert B.hsd_dsv_build(None, 1, 3, None, None, None, 0, None, 0, None, 0, None, 128, None, None, None, None,
                           None) == B.HSD_ERR_INVALID_ARG


def test_binding_refuses_to_import_without_the_library(tmp_path, B):
    """No CPU fallback: with the shared library absent the binding raises instead of degrading."""
    import importlib.util
    src = os.path.join(ROOT, "paper_2602_12957_b200", "binding.py")
    dst = tmp_path / "binding_copy.py"
    dst.write_text(open(src).read())
    spec = importlib.util.spec_from_file_location("binding_copy", dst)
    mod = importlib.util.module_from_spec(spec)
    with pytest.raises(ImportError):
        spec.loader.exec_module(mod)
