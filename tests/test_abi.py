"""The C-ABI library builds, loads, exports every symbol the header declares,
and rejects bad arguments on the host before touching a device."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2607_15810_b200 import build
    return C.CDLL(build.build())


def _declared():
    text = open(os.path.join(ROOT, "include", "quads.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(quads_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert {"quads_quantize_nvfp4", "quads_moe_w4a4_rac", "quads_fake_quant_weights"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_status_strings_and_sizes(lib):
    lib.quads_status_string.restype = C.c_char_p
    for code in range(0, -7, -1):
        assert lib.quads_status_string(code).startswith(b"QUADS_")
    lib.quads_sf_tiled_bytes.restype = C.c_size_t
    lib.quads_sf_tiled_bytes.argtypes = [C.c_int64, C.c_int64]
    assert lib.quads_sf_tiled_bytes(128, 64) == 512
    assert lib.quads_sf_tiled_bytes(129, 65) == 2048
    assert lib.quads_sf_tiled_bytes(1536, 2048) == 12 * 32 * 512
    lib.quads_moe_workspace_bytes.restype = C.c_size_t
    lib.quads_moe_workspace_bytes.argtypes = [C.c_int32] * 6
    small = lib.quads_moe_workspace_bytes(256, 2048, 768, 128, 8, 0)
    big = lib.quads_moe_workspace_bytes(8192, 2048, 768, 128, 8, 0)
    assert 0 < small < big < (1 << 30)


def test_argument_errors_come_back_before_any_launch(lib):
    f = lib.quads_quantize_nvfp4
    f.restype = C.c_int32
    f.argtypes = [C.c_void_p, C.c_int64, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                  C.c_int, C.c_void_p, C.c_size_t, C.c_void_p]
    fake = 0x1000  # never dereferenced: every case fails a host-side check first
    assert f(fake, 4, 40, 40, None, fake, fake, None, 0, fake, 256, None) == -2      # K % 16
    assert f(fake, 4, 64, 32, None, fake, fake, None, 0, fake, 256, None) == -2      # ld < K
    assert f(fake, 4, 64, 64, None, fake, fake, None, 7, fake, 256, None) == -2      # layout
    assert f(fake, 4, 64, 64, None, None, fake, None, 0, fake, 256, None) == -1      # q NULL
    assert f(fake, 4, 64, 64, None, fake, fake, None, 0, None, 0, None) == -3        # workspace
    assert f(fake, 4, 64, 64, None, fake, fake, None, 0, 0x1010, 256, None) == -3    # misaligned
    g = lib.quads_moe_w4a4_rac
    g.restype = C.c_int32
    g.argtypes = [C.c_void_p, C.c_void_p]
    assert g(None, None) == -1
