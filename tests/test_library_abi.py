"""CPU-side checks of the C-ABI library: it builds, loads, exports every symbol the header
declares, and rejects bad arguments on the host before anything is launched."""
import ctypes
import os
import re

import pytest

from paper_2512_00956_b200 import build as wbuild
from paper_2512_00956_b200 import wush

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    wbuild.build()
    return wush.lib()


def test_exports_match_header(L):
    text = open(os.path.join(ROOT, "include", "wush.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = set(re.findall(r"\b(wush_[a-z0-9_]+)\s*\(", text))
    assert declared, "no declarations parsed"
    for name in sorted(declared):
        assert hasattr(L, name), f"{name} declared in wush.h but not exported"
    assert declared >= set(wush.EXPORTS)


def test_header_is_plain_c_and_cpp(tmp_path):
    """include/wush.h is the boundary: it must compile on its own as C99 and as C++ (no torch, no CUDA types)."""
    import shutil
    import subprocess
    hdr = os.path.join(ROOT, "include", "wush.h")
    for cc, flags in (("gcc", ["-std=c99", "-pedantic", "-x", "c"]), ("g++", ["-std=c++11", "-x", "c++"])):
        if shutil.which(cc) is None:
            pytest.skip(f"{cc} not installed")
        res = subprocess.run([cc, "-Wall", "-Werror", "-fsyntax-only"] + flags + [hdr], capture_output=True, text=True)
        assert res.returncode == 0, res.stderr


def test_status_strings(L):
    assert L.wush_status_string(0) == b"ok"
    for code in range(-8, 0):
        assert L.wush_status_string(code) not in (b"ok", b"unknown status")
    assert L.wush_status_string(-99) == b"unknown status"


def test_scale_bytes(L):
    assert L.wush_scale_bytes(128, 2048, 32, wush.SF_LINEAR) == 128 * 64
    assert L.wush_scale_bytes(128, 2048, 32, wush.SF_TILED) == 1 * 16 * 512
    assert L.wush_scale_bytes(129, 64, 32, wush.SF_TILED) == 2 * 1 * 512
    assert L.wush_scale_bytes(1, 64, 16, wush.SF_TILED) == 512
    assert L.wush_scale_bytes(1, 64, 8, wush.SF_TILED) == 0
    assert L.wush_linear_workspace_bytes(128, 2048, 32) == 128 * 1024 + 16 * 512 + 16 + 16   # codes, scales, tensor scale slot, status
    assert L.wush_calib_moments_workspace_bytes(512, 2048, 32) % (2048 * 32 * 4) == 0


def test_workspace_bytes_covers_every_call(L):
    for M, N, K, fmt, g in ((128, 2048, 2048, 0, 32), (2048, 4096, 4096, 1, 16), (1, 28672, 8192, 2, 32), (16384, 28672, 8192, 1, 16)):
        need = L.wush_workspace_bytes(M, N, K, fmt, g)
        assert need >= L.wush_linear_workspace_bytes(M, K, g) > 0
        assert need >= L.wush_quantize_weight_workspace_bytes(N, K, fmt, g) > 0
        assert need >= L.wush_calib_moments_workspace_bytes(N, K, g) > 0
        assert need >= L.wush_calib_moments_workspace_bytes(M, K, g)
        assert need == max(L.wush_linear_workspace_bytes(M, K, g), L.wush_quantize_weight_workspace_bytes(N, K, fmt, g),
                           L.wush_calib_moments_workspace_bytes(max(M, N), K, g))
    assert L.wush_workspace_bytes(128, 128, 128, 0, 16) == 0        # g does not match the format
    assert L.wush_workspace_bytes(128, 128, 100, 0, 32) == 0
    assert L.wush_workspace_bytes(-1, 128, 128, 0, 32) == 0


def test_prepare_module_holds_no_arithmetic():
    """Offline preparation is marshalling only: every matrix it hands to the kernels is made by the library."""
    import ast
    src = open(os.path.join(ROOT, "paper_2512_00956_b200", "prepare.py")).read()
    tree = ast.parse(src)
    assert not any(isinstance(n, (ast.BinOp, ast.AugAssign, ast.For, ast.While)) and not
                   (isinstance(n, ast.BinOp) and isinstance(n.op, ast.FloorDiv)) for n in ast.walk(tree))
    for banned in ("torch.where", "torch.eye", "torch.arange", "math.", "numpy", ".sqrt", "@"):
        assert banned not in src.split('"""', 2)[2], banned


def test_argument_errors_are_found_on_the_host(L):
    p = ctypes.c_void_p(0x1000)         # aligned, never dereferenced: every call below must fail first
    odd = ctypes.c_void_p(0x1004)
    null = None
    q = L.wush_quantize_act
    assert q(null, 16, 64, p, 0, 32, null, p, p, 0, null) == -1                 # NULL X
    assert q(p, 16, 64, p, 1, 16, null, p, p, 0, null) == -1                    # NVFP4 without tensor scale
    assert q(p, 16, 64, p, 0, 16, null, p, p, 0, null) == -3                    # g does not match format
    assert q(p, 16, 64, p, 7, 32, null, p, p, 0, null) == -3                    # unknown format
    assert q(p, 16, 96, p, 0, 32, null, p, p, 0, null) == -2                    # K % 64
    assert q(p, -1, 64, p, 0, 32, null, p, p, 0, null) == -2
    assert q(odd, 16, 64, p, 0, 32, null, p, p, 0, null) == -4                  # misaligned
    assert q(p, 16, 64, p, 0, 32, null, p, p, 5, null) == -3                    # unknown scale layout
    assert q(p, 0, 64, p, 0, 32, null, p, p, 0, null) == 0                      # empty input: no-op
    w = L.wush_quantize_weight
    assert w(p, 16, 64, p, 0, 32, null, p, p, 0, null, 0, null) == -5           # no workspace
    assert w(p, 16, 64, p, 1, 16, null, p, p, 0, p, 4096, null) == -1           # NVFP4 needs w_tensor_scale
    gm = L.wush_gemm_fp4
    assert gm(p, p, p, p, 16, 12, 64, 0, 32, null, null, p, 0, null, null) == -2   # N % 8
    assert gm(p, p, p, p, 16, 16, 64, 0, 32, null, null, p, 3, null, null) == -3   # bad output type
    assert gm(p, p, p, null, 16, 16, 64, 0, 32, null, null, p, 0, null, null) == -1
    lin = L.wush_linear
    assert lin(p, 16, 64, p, p, p, 16, null, null, 0, 32, p, 0, p, 8, null) == -5    # workspace too small
    mo = L.wush_calib_moments
    assert mo(p, 16, 64, 8, p, p, p, 1 << 20, null) == -3
    assert mo(p, 16, 64, 32, p, null, p, 1 << 20, null) == -1
    assert mo(p, 16, 64, 32, p, p, p, 16, null) == -5
    assert mo(p, 16, 64, 32, p, odd, p, 1 << 20, null) == -4                    # count not 8-byte aligned
    assert L.wush_calib_moments_static(p, 16, 64, 32, p, odd, null) == -4
    bk = L.wush_build_transforms_kind
    assert bk(null, 0, null, 0, 64, 32, 0.0, 2, null, p, null, null) == -1      # Hadamard: moments optional, outputs not
    assert bk(null, 0, null, 0, 64, 32, 0.0, 3, p, odd, null, null) == -4
    assert bk(null, 0, null, 0, 60, 32, 0.0, 2, p, p, null, null) == -2
    assert bk(null, 0, null, 0, 64, 32, 0.0, 9, p, p, null, null) == -3         # unknown kind
    assert bk(null, 5, null, 5, 64, 32, 0.0, 0, p, p, null, null) == -1         # WUSH needs the moments
    gq = L.wush_gptq_quantize_weight
    big = L.wush_gptq_workspace_bytes(16, 64, 32)
    assert big >= 8 * (16 * 64 + 2 * 64 * 64)
    wsp = ctypes.c_void_p(0x10000)
    assert gq(p, 16, 64, p, 8, 0, 32, 0.0, null, p, p, p, p, 0, null, wsp, big, null) == -2      # lambda must be positive
    assert gq(p, 16, 64, p, 0, 0, 32, 0.01, null, p, p, p, p, 0, null, wsp, big, null) == -2     # no calibration tokens
    assert gq(p, 16, 64, p, 8, 1, 16, 0.01, null, p, p, p, p, 0, null, wsp, big, null) == -1     # NVFP4 needs the tensor scale
    assert gq(p, 16, 64, p, 8, 0, 32, 0.01, null, p, p, p, p, 0, null, wsp, big - 1, null) == -5
    assert gq(p, 16, 64, p, 8, 0, 32, 0.01, null, p, p, p, p, 0, null, ctypes.c_void_p(0x10010), big, null) == -4
    assert L.wush_quantize_f32(p, 4, 64, 0, 32, null, p, null, 0, null) == -1
    assert L.wush_transform_act_f32(p, 4, 64, p, 24, p, null) == -3


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(wush, "_lib", None)
    monkeypatch.setattr(wush, "LIB_PATH", "/nonexistent/libwush.so")
    with pytest.raises(wush.WushError):
        wush.lib()
