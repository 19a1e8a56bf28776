"""The C-ABI shared library loads without a GPU, exports every symbol that include/attn.h
declares, and rejects bad arguments before touching a device."""
import ctypes
import os
import re

import pytest

import paper_2603_24517_b200 as lib
from paper_2603_24517_b200 import binding
from paper_2603_24517_b200 import build as lib_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def cdll():
    lib_build.build()
    return lib.load_library()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "attn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(attn_[a-z_0-9]+)\s*\(", text)))


def test_header_symbols_are_exported(cdll):
    names = declared_functions()
    assert "attn_fwd" in names and "attn_fwd_host" in names and len(names) >= 9
    for name in names:
        assert hasattr(cdll, name), f"{name} declared in include/attn.h but not exported"
    assert set(names) == set(binding.EXPORTED_SYMBOLS)


def test_version_and_status_strings(cdll):
    assert lib.attn_version() >= 100
    for code, name in binding.STATUS_NAMES.items():
        assert lib.attn_status_str(code) == name
    assert lib.attn_status_str(99) == "ATTN_ERR_UNKNOWN"


def _fwd(cdll, q=16, k=16, v=16, o=16, lse=0, B=1, Hq=2, Hkv=2, Sq=128, Sk=128, D=128, causal=0, scale=0.1):
    return cdll.attn_fwd(q, k, v, o, lse or None, B, Hq, Hkv, Sq, Sk, D, causal, scale, None)


def test_argument_errors_need_no_device(cdll):
    assert _fwd(cdll, q=0) == 1            # ATTN_ERR_NULL
    assert _fwd(cdll, o=0) == 1
    assert _fwd(cdll, B=0) == 2            # ATTN_ERR_SHAPE
    assert _fwd(cdll, Sk=-5) == 2
    assert _fwd(cdll, Hq=3, Hkv=2) == 2
    assert _fwd(cdll, D=64) == 3           # ATTN_ERR_UNSUPPORTED
    assert _fwd(cdll, scale=float("nan")) == 3
    assert _fwd(cdll, scale=float("inf")) == 3
    assert _fwd(cdll, scale=-1.0) == 3
    assert _fwd(cdll, scale=0.0) == 3
    assert _fwd(cdll, q=24) == 4           # ATTN_ERR_ALIGN
    assert _fwd(cdll, lse=18) == 4
    # host entry point: same shape checks, no alignment requirement
    assert cdll.attn_fwd_host(None, 16, 16, 16, None, 1, 2, 2, 128, 128, 128, 0, 0.1, None) == 1
    assert cdll.attn_fwd_host(16, 16, 16, 16, None, 1, 2, 2, 128, 128, 96, 0, 0.1, None) == 3


def test_options(cdll):
    assert cdll.attn_set_option(b"scheduler", 3) == 3
    assert cdll.attn_set_option(b"no_such_option", 1) == 3
    assert cdll.attn_set_option(None, 1) == 1
    for v in (0, 1, 2):
        assert cdll.attn_set_option(b"scheduler", v) == 0
    assert cdll.attn_set_option(b"kernel", 4) == 3
    for v in (3, 2, 1, 0):
        assert cdll.attn_set_option(b"kernel", v) == 0
    for name, bad, good in ((b"rescale_threshold", 65, 8), (b"split_p", 2, 1), (b"overlap_epilogue", -1, 1)):
        assert cdll.attn_set_option(name, bad) == 3
        assert cdll.attn_set_option(name, good) == 0
    assert cdll.attn_set_option(b"max_ctas", -1) == 3
    assert cdll.attn_set_option(b"max_ctas", 0) == 0


def test_options_read_back_and_defaults(cdll):
    """attn_get_option returns what attn_set_option stored; the documented defaults hold
    whenever a test module starts (conftest.py checks and restores them after every module)."""
    for name, default in binding.OPTION_DEFAULTS.items():
        assert lib.attn_get_option(name) == default, name
    lib.attn_set_option("rescale_threshold", 3)
    assert lib.attn_get_option("rescale_threshold") == 3
    lib.attn_set_option("rescale_threshold", 8)
    v = ctypes.c_int(-1)
    assert cdll.attn_get_option(b"no_such_option", ctypes.byref(v)) == 3
    assert cdll.attn_get_option(None, ctypes.byref(v)) == 1
    assert cdll.attn_get_option(b"kernel", None) == 1


def test_last_device_status_null(cdll):
    assert cdll.attn_last_device_status(None, None) == 1
    assert cdll.attn_selftest_wait_timeout(0, None) == 3
    assert cdll.attn_selftest_wait_timeout(5000, None) == 3


def test_clock_ring_argument_errors_need_no_device(cdll):
    n = ctypes.c_int(0)
    buf = (ctypes.c_double * 4)()
    assert cdll.attn_launch_clocks(None, 4, ctypes.byref(n)) == 1     # ATTN_ERR_NULL
    assert cdll.attn_launch_clocks(buf, 4, None) == 1
    assert cdll.attn_launch_clocks(buf, 0, ctypes.byref(n)) == 2      # ATTN_ERR_SHAPE
    assert cdll.attn_last_launch_clock(None, None) == 1


def test_variant_build_reports_spills_and_exports_the_abi(tmp_path):
    """Another register split is a build of its own beside the in-tree library (how the register-split
    rows of the ablation are made): it must export the whole ABI and report ptxas's spill figures."""
    out = str(tmp_path / "libattn_b200_176_80_80.so")
    info = lib_build.build_variant(out, ["-DATTN_REGS_SOFTMAX=176", "-DATTN_REGS_EPILOGUE=80", "-DATTN_REGS_OTHER=80"])
    assert info["path"] == out and os.path.exists(out)
    assert isinstance(info["spill_store_bytes"], int) and isinstance(info["spill_load_bytes"], int)
    other = ctypes.CDLL(out)
    for name in binding.EXPORTED_SYMBOLS:
        assert hasattr(other, name)
    with pytest.raises(RuntimeError):   # 8 a + 4 b + 4 c > 2048 is refused at compile time (static_assert)
        lib_build.build_variant(str(tmp_path / "bad.so"), ["-DATTN_REGS_SOFTMAX=200", "-DATTN_REGS_EPILOGUE=128",
                                                           "-DATTN_REGS_OTHER=128"])


def test_missing_library_is_loud(monkeypatch):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", os.path.join(ROOT, "no_such_dir", "libattn_b200.so"))
    with pytest.raises(ImportError):
        binding.load_library()


def test_stride_errors_need_no_device(cdll):
    import ctypes
    arr = lambda *v: (ctypes.c_longlong * 3)(*v)
    ok = arr(128 * 2 * 128, 2 * 128, 128)

    def call(qs=ok, ks=ok, vs=ok, os_=ok):
        return cdll.attn_fwd_strided(16, 16, 16, 16, None, 1, 2, 2, 128, 128, 128, qs, ks, vs, os_, 0, 0.1, None)

    assert call(qs=None) == 1                      # ATTN_ERR_NULL
    assert call(ks=arr(0, 256, 128)) == 2          # ATTN_ERR_SHAPE: stride <= 0
    assert call(vs=arr(32768, 64, 128)) == 2       # rows of 128 elements would overlap
    assert call(os_=arr(32768, 260, 128)) == 4     # ATTN_ERR_ALIGN: not a multiple of 8 elements
    assert call(qs=arr(1 << 40, 256, 128)) == 3    # ATTN_ERR_UNSUPPORTED: beyond the descriptor's range
