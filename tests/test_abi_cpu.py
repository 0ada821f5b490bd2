"""Host-side checks of the C ABI that need no GPU: the library builds and loads, exports every
function include/lory.h declares, validates arguments before touching a device, and its workspace
sizes follow the documented layout."""
import ctypes
import os
import re
import shutil

import pytest

import paper_2405_03133_b200 as lory
from paper_2405_03133_b200 import build as lory_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    if not os.path.exists(lory_build.LIB) and shutil.which("nvcc") is None:
        pytest.skip("liblory.so not built and nvcc not available")
    lory_build.build()
    return lory.binding.load()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "lory.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(lory_[a-z0-9_]+)\s*\(", text)))


def test_exports_every_declared_symbol(lib):
    names = declared_functions()
    assert {"lory_moe_forward", "lory_moe_backward", "lory_moe_ffn", "lory_moe_workspace_bytes",
            "lory_moe_step_host", "lory_check_status"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} declared in lory.h but not exported"
    # and the binding wraps all of them
    assert set(names) == set(lory.binding.exported_symbols())


def test_debug_build_exports_the_same_symbols():
    """The bounds-checking build (-DLORY_DEBUG) has the same ABI and says what it is."""
    if shutil.which("nvcc") is None and not os.path.exists(lory_build.LIB_DEBUG):
        pytest.skip("liblory_debug.so not built and nvcc not available")
    dbg = ctypes.CDLL(lory_build.build(debug=True))
    for n in declared_functions():
        assert hasattr(dbg, n), f"{n} missing from the debug build"
    dbg.lory_debug_build.restype = ctypes.c_int
    assert dbg.lory_debug_build() == 1


def test_release_build_is_not_the_debug_build(lib):
    assert lory.binding.lory_debug_build() == 0


def test_status_strings(lib):
    assert lory.lory_status_string(0) == "LORY_OK"
    for code in range(-9, 0):
        assert lory.lory_status_string(code).startswith("LORY_ERR_")
    assert "unknown" in lory.lory_status_string(-99)


def test_workspace_sizes_follow_layout(lib):
    d = lory.make_dims(8, 4096, 256, 1024, 2752, 32, "bf16")
    fwd, bwd = lory.lory_moe_workspace_bytes(d)
    S, tok, P1 = 128, 8 * 4096, 1024 * 2752
    merged = 3 * S * P1 * 2
    acts = 3 * tok * 2752 * 2
    assert merged + acts <= fwd <= merged + acts + (4 << 20)
    assert fwd + merged + 2 * tok * 2752 * 2 <= bwd <= fwd + merged + 2 * tok * 2752 * 2 + (64 << 20)
    assert fwd % 256 == 0 and bwd % 256 == 0
    d32 = lory.make_dims(2, 512, 128, 256, 688, 4, "fp32")
    f32, b32 = lory.lory_moe_workspace_bytes(d32)
    assert b32 > f32 > 3 * 8 * 256 * 688 * 4


@pytest.mark.parametrize("bad", [
    dict(L=500),              # L % T != 0
    dict(B=0), dict(E=0), dict(d=0), dict(f=0), dict(T=0),
    dict(d=1020),             # bf16 rows must be 16-byte multiples
    dict(E=129),              # bf16 expert limit
])
def test_rejects_bad_shapes_on_the_host(lib, bad):
    kw = dict(B=2, L=512, T=128, d=256, f=688, E=4, dtype="bf16")
    kw.update(bad)
    with pytest.raises(lory.LoryError) as e:
        lory.lory_moe_workspace_bytes(lory.make_dims(**kw))
    assert e.value.status == -2


def test_rejects_bad_dtype_and_null_pointers(lib):
    d = lory.make_dims(2, 512, 128, 256, 688, 4, 7)
    with pytest.raises(lory.LoryError) as e:
        lory.lory_moe_workspace_bytes(d)
    assert e.value.status == -3
    d = lory.make_dims(2, 512, 128, 256, 688, 4, "fp32")
    null = ctypes.c_void_p(0)
    rc = lib.lory_moe_forward(ctypes.byref(d), null, null, null, null, null, null, null, null, null, 0, null)
    assert rc == -1
    rc = lib.lory_moe_backward(ctypes.byref(d), *([null] * 13), 0, null)
    assert rc == -1
    rc = lib.lory_moe_ffn(ctypes.byref(d), *([null] * 7), 0, null)
    assert rc == -1
    # a non-NULL but too small / misaligned workspace is refused before any device call
    one = ctypes.c_void_p(256)
    rc = lib.lory_moe_forward(ctypes.byref(d), one, one, one, one, one, one, one, null, one, 16, null)
    assert rc == -4
    rc = lib.lory_moe_forward(ctypes.byref(d), one, one, one, one, one, one, one, null, ctypes.c_void_p(264),
                              1 << 40, null)
    assert rc == -4


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(lory.binding, "_lib", None)
    monkeypatch.setattr(lory.binding, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(lory.LoryError):
        lory.lory_moe_workspace_bytes(lory.make_dims(1, 8, 8, 8, 8, 1, "fp32"))


def test_library_has_no_unresolved_symbols():
    """Loading with immediate binding fails if any function the library calls is missing from it."""
    import ctypes
    import os
    from paper_2405_03133_b200 import binding
    ctypes.CDLL(binding.LIB_PATH, mode=os.RTLD_NOW)
