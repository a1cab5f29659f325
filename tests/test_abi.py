"""CPU-side checks of the C-ABI library: it loads, exports every symbol the header declares, and rejects bad
arguments before touching a device. No compute call is made here."""
import ctypes
import re
from pathlib import Path

import numpy as np
import pytest

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def B():
    from paper_2609_22755_b200 import build

    build.build_library()
    from paper_2609_22755_b200 import binding

    return binding


def test_header_symbols_are_exported(B):
    header = (ROOT / "include" / "nsp.h").read_text()
    # what the header declares only for the checked build belongs to libnsp_checked.so
    checked_part = "".join(re.findall(r"#ifdef NSP_CHECKED(.*?)#endif", header, flags=re.S))
    header = re.sub(r"#ifdef NSP_CHECKED.*?#endif", "", header, flags=re.S)
    declared = set(re.findall(r"\b(nsp_[a-z0-9_]+)\s*\(", header))
    assert {"nsp_plan_tiles", "nsp_attn_fwd", "nsp_attn_bwd"} <= declared
    lib = ctypes.CDLL(str(B.LIB_PATH))
    for name in sorted(declared):
        assert hasattr(lib, name), f"{name} is declared in include/nsp.h but not exported"
    assert declared == set(B.EXPORTS)
    declared_checked = set(re.findall(r"\b(nsp_[a-z0-9_]+)\s*\(", checked_part))
    assert declared_checked == set(B.CHECKED_EXPORTS)
    checked = ctypes.CDLL(str(B.LIB_PATH.parent / "libnsp_checked.so"))
    for name in sorted(declared | declared_checked):
        assert hasattr(checked, name), f"{name} is missing from the checked build"
    for name in declared_checked:
        assert not hasattr(lib, name), f"{name} must not be in the regular library"


def test_status_strings(B):
    assert B.status_string(B.NSP_OK) == "ok"
    for code in range(1, 9):
        assert B.status_string(code) not in ("ok", "unknown status")
    assert B.status_string(99) == "unknown status"


def test_error_codes_match_the_header(B):
    """The binding's constants are the header's enum, value by value (DEVICE_ASSERT keeps code 7, the planner's
    INFEASIBLE has its own)."""
    header = (ROOT / "include" / "nsp.h").read_text()
    enum = dict((m.group(1), int(m.group(2))) for m in re.finditer(r"\b(NSP_(?:OK|ERR_[A-Z_]+))\s*=\s*(\d+)", header))
    assert enum["NSP_ERR_DEVICE_TIMEOUT"] == 5 and enum["NSP_ERR_DEVICE_ASSERT"] == 7 and enum["NSP_ERR_INFEASIBLE"] == 8
    for name, value in enum.items():
        assert getattr(B, name) == value, name
    assert len(set(enum.values())) == len(enum)


def _plan_rc(B, cu, hq, hkv, head_dim=128, opts=None, null=None):
    cu, hq, hkv = (np.asarray(x, np.int32) for x in (cu, hq, hkv))
    handle = ctypes.c_void_p()
    o = B.PlanOpts(*opts) if opts else None
    args = [B._ptr(cu), B._ptr(hq), B._ptr(hkv)]
    if null is not None:
        args[null] = None
    rc = B.lib().nsp_plan_tiles(*args, len(hq), head_dim, ctypes.byref(o) if o else None, None, ctypes.byref(handle))
    if rc == B.NSP_OK:
        B.lib().nsp_plan_destroy(handle)
    else:
        assert not handle.value
    return rc


def test_plan_argument_validation(B):
    good = ([0, 4, 9], [4, 4], [2, 2])
    assert _plan_rc(B, [1, 4, 9], good[1], good[2]) == B.NSP_ERR_INVALID_ARG  # cu_seqlens[0] != 0
    assert _plan_rc(B, [0, 9, 4], good[1], good[2]) == B.NSP_ERR_INVALID_ARG  # decreasing
    assert _plan_rc(B, good[0], [4, 0], good[2]) == B.NSP_ERR_INVALID_ARG  # hq <= 0
    assert _plan_rc(B, good[0], good[1], [2, -1]) == B.NSP_ERR_INVALID_ARG  # hkv <= 0
    assert _plan_rc(B, good[0], [4, 3], good[2]) == B.NSP_ERR_INVALID_ARG  # hq % hkv != 0
    for null in (0, 1, 2):
        assert _plan_rc(B, *good, null=null) == B.NSP_ERR_INVALID_ARG
    assert _plan_rc(B, *good, head_dim=96) == B.NSP_ERR_UNSUPPORTED  # built: 128 and 64
    assert _plan_rc(B, *good, opts=(64, 128, 1, 0)) == B.NSP_ERR_UNSUPPORTED  # tile size not built
    assert _plan_rc(B, *good, opts=(0, 128, 1, 0)) == B.NSP_ERR_INVALID_ARG
    assert _plan_rc(B, *good, opts=(128, 128, 2, 0)) == B.NSP_ERR_UNSUPPORTED  # unknown order version
    assert _plan_rc(B, good[0], [512, 512], good[2]) == B.NSP_ERR_UNSUPPORTED  # > 256 heads
    # too many runs: alternating head counts
    n = B.NSP_MAX_RUNS + 1
    assert _plan_rc(B, np.arange(n + 1) * 8, [4, 8] * (n // 2) + [4], [1] * n) == B.NSP_ERR_UNSUPPORTED
    rc = B.lib().nsp_plan_tiles(None, None, None, -1, 128, None, None, ctypes.byref(ctypes.c_void_p()))
    assert rc == B.NSP_ERR_INVALID_ARG
    rc = B.lib().nsp_plan_tiles(B._ptr(np.zeros(1, np.int32)), None, None, 0, 128, None, None, None)
    assert rc == B.NSP_ERR_INVALID_ARG  # null out pointer


def test_null_plan_is_rejected(B):
    L = B.lib()
    assert L.nsp_plan_sizes(None, None, None, None, None, None) == B.NSP_ERR_INVALID_ARG
    assert L.nsp_attn_fwd(None, None, None, None, None, None, 1.0, None, 0, None) == B.NSP_ERR_INVALID_ARG
    assert L.nsp_attn_bwd(None, None, None, None, None, None, None, None, None, None, 0, 1, 1.0, None, 0,
                          None) == B.NSP_ERR_INVALID_ARG
    n = ctypes.c_size_t()
    assert L.nsp_plan_step_host_ws_bytes(None, 0, 1, ctypes.byref(n)) == B.NSP_ERR_INVALID_ARG
    assert L.nsp_attn_step_host(None, None, None, None, None, None, None, None, None, None, 0, 1, 1.0, None, 0,
                                None) == B.NSP_ERR_INVALID_ARG
    assert L.nsp_plan_destroy(None) == B.NSP_OK
    assert L.nsp_launch_count() >= 0


def test_no_device_means_an_error_not_a_fallback(B):
    import torch

    if torch.cuda.is_available():
        pytest.skip("a device is present")
    assert _plan_rc(B, [0, 4, 9], [4, 4], [2, 2]) in (B.NSP_ERR_CUDA, B.NSP_ERR_UNSUPPORTED)


def test_layout_and_selftest_calls_reject_bad_arguments_without_a_device(B):
    lib = ctypes.CDLL(str(B.LIB_PATH))
    fh = (ctypes.c_int32 * 4)(0, 2, 4, 6)
    buf = ctypes.c_void_p(256)  # never dereferenced: every case below is refused first
    for fn in (lib.nsp_a2a_gather_heads, lib.nsp_a2a_scatter_heads):
        fn.restype = ctypes.c_int
        fn.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
                       ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p]
        args = lambda **kw: [kw.get("src", buf), kw.get("dst", buf), kw.get("tokens", 8), kw.get("heads", 8),
                             kw.get("hpb", 2), kw.get("n", 4), kw.get("D", 128), kw.get("dtype", B.NSP_BF16),
                             kw.get("fh", fh), None]
        assert fn(*args(tokens=-1)) == B.NSP_ERR_INVALID_ARG
        assert fn(*args(hpb=0)) == B.NSP_ERR_INVALID_ARG
        assert fn(*args(hpb=3)) == B.NSP_ERR_INVALID_ARG  # block 3 would reach past the last head
        assert fn(*args(n=65)) == B.NSP_ERR_INVALID_ARG
        assert fn(*args(dtype=7)) == B.NSP_ERR_INVALID_ARG
        assert fn(*args(fh=None)) == B.NSP_ERR_INVALID_ARG
        assert fn(*args(D=4)) == B.NSP_ERR_UNSUPPORTED  # 8-byte rows
        assert fn(*args(src=ctypes.c_void_p(260))) == B.NSP_ERR_INVALID_ARG  # misaligned
        assert fn(*args(src=None)) == B.NSP_ERR_INVALID_ARG
        assert fn(*args(tokens=0, src=None, dst=None)) == B.NSP_OK  # nothing to move
    lib.nsp_selftest_wait_timeout.restype = ctypes.c_int
    lib.nsp_selftest_wait_timeout.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p]
    assert lib.nsp_selftest_wait_timeout(None, 1000, None) == B.NSP_ERR_INVALID_ARG
    lib.nsp_attn_bwd_recompute.restype = ctypes.c_int
    assert lib.nsp_plan_recompute_ws_bytes(None, None) == B.NSP_ERR_INVALID_ARG
