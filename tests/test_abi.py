"""The shared library loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

from paper_2607_11136_b200 import binding as xb

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "xema.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(xema_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    names = _declared()
    assert len(names) >= 20
    L = ctypes.CDLL(xb.LIB_PATH)
    for n in names:
        assert hasattr(L, n), n
    assert sorted(xb.EXPORTS) == names


def test_struct_sizes_match_the_header():
    # 13 int32 + 3 float + 1 int32; name[24] + 4 x 4 + 8 + 2 x 4; 12 pointers; gemm args
    assert ctypes.sizeof(xb.xema_config) == 68
    assert ctypes.sizeof(xb.xema_tensor) == 56
    assert ctypes.sizeof(xb.xema_block_weights) == 96
    assert ctypes.sizeof(xb.xema_gemm_args) == 168


def test_error_paths_without_gpu():
    assert xb.version().startswith("xema-b200")
    assert xb.strerror(0) == "ok" and "budget" in xb.strerror(xb.XEMA_EBUDGET)
    from xema_inputs import template
    cfg = xb.make_config(template("tiny"))
    for bad in (0, -1, 289):
        try:
            xb.xema_trace(cfg, bad)
            raise AssertionError("expected XEMA_EINVAL")
        except xb.XemaError as e:
            assert e.status == xb.XEMA_EINVAL
    bad_cfg = xb.make_config(template("tiny"))
    bad_cfg.rope_dim_t = 15
    try:
        xb.xema_trace(bad_cfg, 1)
        raise AssertionError("expected XEMA_EINVAL")
    except xb.XemaError as e:
        assert e.status == xb.XEMA_EINVAL
    bad_cfg = xb.make_config(template("tiny"))
    bad_cfg.heads = 7
    try:
        xb.Plan(bad_cfg, 1)
        raise AssertionError("expected XEMA_EINVAL")
    except xb.XemaError as e:
        assert e.status == xb.XEMA_EINVAL
    # forward on an unbound plan is refused, not crashed
    p = xb.Plan(cfg, 2)
    assert p.launch_count() == 0
    try:
        p.block_forward(0)
        raise AssertionError("expected XEMA_ESTATE")
    except xb.XemaError as e:
        assert e.status == xb.XEMA_ESTATE
    # arena too small / misaligned / null weights are refused before any CUDA call
    w = [{k: 16 for k in xb._WEIGHT_FIELDS}]
    for arena_ptr, nbytes, want in ((256, p.peak_bytes - 1, xb.XEMA_ENOSPC), (257, p.peak_bytes, xb.XEMA_EALIGN)):
        try:
            p.bind(arena_ptr, nbytes, w, 256)
            raise AssertionError("expected an error")
        except xb.XemaError as e:
            assert e.status == want
    p.close()
