"""CPU-only checks of the C-ABI library: it builds, loads, exports every symbol include/mok.h declares, and its
host-side logic (size queries, argument validation that happens before any launch) behaves.  No compute calls."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2609_36070_b200 import build
    path = build.build()
    return ctypes.CDLL(path)


def declared_functions():
    text = open(os.path.join(ROOT, "include", "mok.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mok_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert "mok_moe_forward" in names and "mok_moe_forward_ex" in names and len(names) >= 10
    for n in names:
        assert hasattr(lib, n), n
    from paper_2609_36070_b200 import mok
    assert sorted(mok.EXPORTS) == names                      # the binding covers the same set


def test_version_and_status_strings(lib):
    lib.mok_status_string.restype = ctypes.c_char_p
    assert lib.mok_version() >= 100
    seen = set()
    for s in range(0, -9, -1):
        msg = lib.mok_status_string(s).decode()
        assert msg and msg != "unknown status"
        seen.add(msg)
    assert len(seen) == 9
    assert lib.mok_status_string(-99).decode() == "unknown status"


def test_workspace_size_query(lib):
    lib.mok_workspace_bytes.restype = ctypes.c_size_t
    ws = lib.mok_workspace_bytes
    base = ws(256, 256, 512, 512, 8, 2)
    assert base > 0 and base % 256 == 0
    assert ws(512, 256, 512, 512, 8, 2) > base                # grows with T
    assert ws(256, 256, 512, 0, 8, 2) < base                  # no shared expert -> smaller
    # buffers for the padded dispatch space: T*k rows + up to 255 pad rows per non-empty expert (256-row pair tiles)
    T, H, I, E, k = 16384, 2048, 768, 128, 8
    rows = T * k + 255 * E
    need = 2 * rows * (2 * H + I)
    assert need <= ws(T, H, I, 0, E, k) <= need * 1.1 + (8 << 20)
    for bad in [(256, 250, 512, 0, 8, 2),     # H not a multiple of 8
                (256, 256, 100, 0, 8, 2),     # I not a multiple of 8
                (256, 256, 512, 0, 8, 9),     # k > E
                (256, 256, 512, 0, 8, 0),     # k < 1
                (256, 256, 512, 0, 1024, 2),  # E beyond the limit
                (-1, 256, 512, 0, 8, 2)]:
        assert ws(*bad) == 0, bad
    assert ws(0, 256, 512, 0, 8, 2) > 0                       # T = 0 is legal


def test_argument_validation_needs_no_device(lib):
    from paper_2609_36070_b200 import mok
    assert lib.mok_moe_forward_ex(None) == mok.MOK_ERR_NULL
    a = mok.mok_args()
    a.T, a.H, a.I, a.I_shared, a.E, a.k = 8, 64, 64, 0, 4, 5
    assert lib.mok_moe_forward_ex(ctypes.byref(a)) == mok.MOK_ERR_SHAPE
    a.k = 2
    assert lib.mok_moe_forward_ex(ctypes.byref(a)) == mok.MOK_ERR_NULL        # weights missing
    a.T = 0
    assert lib.mok_moe_forward_ex(ctypes.byref(a)) == mok.MOK_OK              # nothing to do
    lib.mok_launch_count.argtypes = [ctypes.c_int] * 6 + [ctypes.c_void_p]
    assert lib.mok_launch_count(256, 256, 512, 512, 8, 2, None) == lib.mok_launch_count(256, 256, 512, 0, 8, 2, None) + 2
    assert lib.mok_launch_count(0, 256, 512, 0, 8, 2, None) == 0
    # up to 160 experts the router is one kernel less (projection + top-k fused)
    assert lib.mok_launch_count(256, 256, 512, 0, 160, 2, None) + 1 == lib.mok_launch_count(256, 256, 512, 0, 161, 2, None)


def test_launch_state_is_kept_per_device(lib):
    """The shared-memory opt-in and the SM count are cached per device, not per process: a second device configures
    its kernels again, a failed configuration is retried, device ids out of range are refused."""
    assert lib.mok_selftest_per_device() == 0


def test_binding_fails_loudly_without_the_library(tmp_path, monkeypatch):
    """The product path has no fallback: importing the binding without libmok.so raises."""
    import importlib.util
    src = os.path.join(ROOT, "paper_2609_36070_b200", "mok.py")
    dst = tmp_path / "mok_copy.py"
    dst.write_text(open(src).read())
    spec = importlib.util.spec_from_file_location("mok_copy", dst)
    with pytest.raises(ImportError):
        spec.loader.exec_module(importlib.util.module_from_spec(spec))
