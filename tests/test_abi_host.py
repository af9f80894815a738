"""Host-side checks of the C ABI that need no GPU: the library builds and loads, exports every
symbol the header declares, and rejects bad arguments before launching anything."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2606_26453_b200 import build
    build.build_library()
    return ctypes.CDLL(build.LIB_PATH)


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "moe_b200.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(moe_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert len(names) >= 18
    for n in names:
        assert hasattr(lib, n), n
    from paper_2606_26453_b200 import binding
    assert sorted(binding.EXPORTS) == names


def test_status_strings(lib):
    lib.moe_status_string.restype = ctypes.c_char_p
    seen = {lib.moe_status_string(i) for i in (0, 1, 2, 3, 4, 5, 6, 8)}
    assert len(seen) == 8 and all(seen)
    assert lib.moe_status_string(12345)


def test_argument_validation_without_a_device(lib):
    from paper_2606_26453_b200.binding import MoeDims
    lib.moe_permute_workspace_bytes.restype = ctypes.c_size_t
    good = MoeDims(256, 256, 512, 8, 2)
    assert lib.moe_permute_workspace_bytes(ctypes.byref(good)) == ((512 + 255) // 256) * 8 * 4
    for bad, code in ((MoeDims(0, 256, 512, 8, 2), 2), (MoeDims(256, 256, 512, 8, 9), 2),
                      (MoeDims(256, 200, 512, 8, 2), 3), (MoeDims(256, 256, 96, 8, 2), 3),
                      (MoeDims(256, 256, 512, 2048, 2), 3), (MoeDims(2 ** 30, 256, 512, 8, 4), 2)):
        assert lib.moe_permute_workspace_bytes(ctypes.byref(bad)) == 0
        rc = lib.moe_permute_bwd(ctypes.byref(bad), ctypes.c_void_p(256), ctypes.c_void_p(256), ctypes.c_void_p(256), None)
        assert rc == code, (bad.T, bad.H, bad.I, bad.E, bad.K, rc)
    p = ctypes.c_void_p
    # NULL required pointer / misaligned pointer / short workspace: all before any CUDA call
    assert lib.moe_permute_bwd(ctypes.byref(good), None, p(256), p(256), None) == 1
    assert lib.moe_permute_bwd(ctypes.byref(good), p(256), p(264), p(256), None) == 4
    assert lib.moe_grouped_gemm_down(ctypes.byref(good), p(256), p(256), None, p(256), None) == 1
    assert lib.moe_grouped_gemm_gateup_swiglu(ctypes.byref(good), p(256), p(256), p(256), p(256), p(256), p(8), None) == 4
    rc = lib.moe_permute(ctypes.byref(good), p(256), p(256), p(256), p(256), p(256), p(256), p(256), p(256),
                         ctypes.c_size_t(8), None)
    assert rc == 5
    assert lib.moe_unpermute_combine_bwd(ctypes.byref(good), p(256), None, p(256), p(256), p(256), p(256), None) == 1
    assert lib.moe_permute_bwd(None, p(256), p(256), p(256), None) == 1


def test_binding_fails_loudly_without_the_library(monkeypatch, tmp_path):
    from paper_2606_26453_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "missing.so"))
    with pytest.raises(ImportError):
        binding.load_library()
