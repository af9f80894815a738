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


def test_block_scaled_calls_validate_before_launching(lib):
    """The block-scaled FP8 entry points: widths that are not multiples of 128, missing pointers, a token-axis operand
    whose column range does not fit its tensor -- all refused on the host."""
    from paper_2606_26453_b200.binding import MoeDims
    p = ctypes.c_void_p
    good = MoeDims(256, 256, 512, 8, 2)
    narrow = MoeDims(256, 192, 512, 8, 2)          # fine for the bf16 calls (multiple of 64), not for these
    for name in ("moe_mxfp8_act_scale_bytes", "moe_mxfp8_w_down_scale_bytes", "moe_mxfp8_dy_scale_bytes",
                 "moe_mxfp8_w_down_dgrad_scale_bytes", "moe_mxfp8_dgu_scale_bytes", "moe_mxfp8_w_gateup_dgrad_scale_bytes",
                 "moe_mxfp8_x_scale_bytes", "moe_mxfp8_w_gateup_scale_bytes"):
        fn = getattr(lib, name)
        fn.restype = ctypes.c_size_t
        assert fn(ctypes.byref(good)) > 0 and fn(ctypes.byref(narrow)) == 0, name
    R, E = 512, 8
    lib.moe_mxfp8_act_scale_bytes.restype = ctypes.c_size_t
    assert lib.moe_mxfp8_act_scale_bytes(ctypes.byref(good)) == (512 // 128) * R * 4
    for name in ("moe_mxfp8_tokens_codes_bytes", "moe_mxfp8_tokens_scale_bytes"):
        getattr(lib, name).restype = ctypes.c_size_t
        getattr(lib, name).argtypes = [ctypes.POINTER(MoeDims), ctypes.c_int]
    pitch = R + 128 * E
    assert lib.moe_mxfp8_tokens_codes_bytes(ctypes.byref(good), 256) == 256 * pitch
    assert lib.moe_mxfp8_tokens_scale_bytes(ctypes.byref(good), 256) == 8192 + (pitch // 128) * 256 * 4 + 2 * (pitch // 128) * 1024
    assert lib.moe_mxfp8_tokens_codes_bytes(ctypes.byref(good), 200) == 0
    # GEMMs and quantisers: shape first, then pointers
    assert lib.moe_grouped_gemm_down_mxfp8(ctypes.byref(narrow), p(256), p(256), p(256), p(256), p(256), p(256), None) == 3
    assert lib.moe_grouped_gemm_down_mxfp8(ctypes.byref(good), p(256), None, p(256), p(256), p(256), p(256), None) == 1
    assert lib.moe_grouped_gemm_gateup_dgrad_mxfp8(ctypes.byref(good), p(256), p(256), p(256), p(264), p(256), p(256), None) == 4
    assert lib.moe_swiglu_mxfp8(ctypes.byref(good), p(256), p(256), None, p(256), None) == 1
    assert lib.moe_grouped_gemm_gateup_wgrad_mxfp8(ctypes.byref(good), p(256), p(256), p(256), p(256), p(256), p(256), p(256),
                                                   None, None) == 1
    q = lib.moe_mxfp8_quantize_tokens
    q.argtypes = [ctypes.POINTER(MoeDims), p, ctypes.c_int, ctypes.c_int, ctypes.c_int, p, p, p, p]
    assert q(ctypes.byref(good), p(256), 1024, 640, 512, p(256), p(256), p(256), None) == 2      # runs past the row
    assert q(ctypes.byref(good), p(256), 1024, 4, 512, p(256), p(256), p(256), None) == 2        # column offset not a multiple of 8
    assert q(ctypes.byref(good), p(256), 1024, 0, 200, p(256), p(256), p(256), None) == 3        # features not a multiple of 128
    assert q(ctypes.byref(good), None, 1024, 0, 512, p(256), p(256), p(256), None) == 1


def test_binding_fails_loudly_without_the_library(monkeypatch, tmp_path):
    from paper_2606_26453_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "missing.so"))
    with pytest.raises(ImportError):
        binding.load_library()
