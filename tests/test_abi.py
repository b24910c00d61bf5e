"""The C-ABI library builds, loads and exports what include/nvfp4.h declares; argument checks need no GPU."""
import ctypes
import os
import re

import pytest

from paper_2509_25149_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "nvfp4.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"NVFP4_API[^;(]*?\b(nvfp4_\w+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    L = B.lib()
    names = declared_symbols()
    assert len(names) >= 12 and set(names) == set(B.EXPORTED)
    for n in names:
        assert hasattr(L, n), n


def test_struct_layouts_match_the_header():
    assert ctypes.sizeof(B.CTensor) == 48 and ctypes.sizeof(B.CQuantOpts) == 56
    assert B.CTensor.rows.offset == 24 and B.CQuantOpts.seed.offset == 24


def test_status_strings_and_knobs():
    assert B.status_string(0) == "ok"
    assert "NULL" in B.status_string(1) and "shape" in B.status_string(2)
    B.nvfp4_set_gemm_tile_n(128)
    B.nvfp4_set_gemm_tile_n(0)
    with pytest.raises(ValueError):
        B.nvfp4_set_gemm_tile_n(64)
    assert B.nvfp4_linear_fwd_workspace_bytes(256, 256) >= 256 * 256 // 2 + 256 * 256 // 16 + 8
    assert B.nvfp4_linear_bwd_workspace_bytes(256, 512) >= 2 * (256 * 512 // 2 + 256 * 512 // 16 + 8)


def test_argument_validation_happens_before_any_launch():
    L = B.lib()
    o = B.quant_opts()
    fake = 0x7F0000000000  # never dereferenced: validation fails first
    t = B.CTensor(fake, fake, fake, 128, 128, B.SF_SWIZZLED, 0)
    q = lambda *a: L.nvfp4_quantize(*a)
    assert q(None, 128, 128, 128, ctypes.byref(o), ctypes.byref(t), None, None) == 1          # NULL input
    assert q(fake, 128, 128, 128, ctypes.byref(o), None, None, None) == 1                      # no copy requested
    assert q(fake, 120, 128, 128, ctypes.byref(o), ctypes.byref(t), None, None) == 2           # rows % 16
    assert q(fake, 128, 128, 64, ctypes.byref(o), ctypes.byref(t), None, None) == 2            # ld < cols
    assert q(fake + 2, 128, 128, 128, ctypes.byref(o), ctypes.byref(t), None, None) == 3       # alignment
    bad = B.quant_opts(block_rows=4)
    assert q(fake, 128, 128, 128, ctypes.byref(bad), ctypes.byref(t), None, None) == 4
    bad = B.quant_opts(block_rows=16, rht_colwise=True)
    assert q(fake, 128, 128, 128, ctypes.byref(bad), ctypes.byref(t), None, None) == 4         # no RHT on 2D blocks
    wrong = B.CTensor(fake, fake, fake, 128, 256, B.SF_SWIZZLED, 0)
    assert q(fake, 128, 128, 128, ctypes.byref(o), ctypes.byref(wrong), None, None) == 2       # copy shape
    small = B.CTensor(fake, fake, fake, 64, 128, B.SF_SWIZZLED, 0)
    assert q(fake, 64, 128, 128, ctypes.byref(o), ctypes.byref(small), None, None) == 2        # swizzled needs 128 rows
    a = B.CTensor(fake, fake, fake, 128, 256, B.SF_SWIZZLED, 0)
    b = B.CTensor(fake, fake, fake, 128, 512, B.SF_SWIZZLED, 0)
    assert L.nvfp4_gemm(ctypes.byref(a), ctypes.byref(b), fake, 0, 128, 0, None) == 2          # K mismatch
    b = B.CTensor(fake, fake, fake, 128, 256, B.SF_LINEAR, 0)
    assert L.nvfp4_gemm(ctypes.byref(a), ctypes.byref(b), fake, 0, 128, 0, None) == 4          # needs swizzled scales
    b = B.CTensor(fake, fake, fake, 128, 256, B.SF_SWIZZLED, 0)
    assert L.nvfp4_gemm(ctypes.byref(a), ctypes.byref(b), fake, 0, 128, 1, None) == 4          # accumulate into bf16
    assert L.nvfp4_gemm(ctypes.byref(a), ctypes.byref(b), fake, 0, 64, 0, None) == 2           # ldd < N
    assert L.nvfp4_gemm(ctypes.byref(a), None, fake, 0, 128, 0, None) == 1
    assert L.nvfp4_linear_fwd(fake, fake, 256, 256, 256, ctypes.byref(o), fake, None, ctypes.byref(a), None, 0,
                              None, 0, None) == 5                                              # workspace
    assert L.nvfp4_linear_fwd(fake, fake, 200, 256, 256, ctypes.byref(o), fake, None, ctypes.byref(a), None, 0,
                              fake, 1 << 30, None) == 2
    assert L.nvfp4_linear_bwd(fake, None, None, 256, 256, 256, ctypes.byref(o), None, None, 0, fake, 1 << 30,
                              None) == 1
    # the composed calls validate EVERY step before the first launch: an error found in a later step (an option the
    # X quantizer rejects, a misaligned output of the GEMM) must leave the launch counter where it was
    w_row, w_col = B.CTensor(fake, fake, fake, 256, 256, B.SF_SWIZZLED, 0), B.CTensor(fake, fake, fake, 256, 256, B.SF_SWIZZLED, 0)
    x_col = B.CTensor(fake, fake, fake, 256, 256, B.SF_SWIZZLED, 0)
    before = L.nvfp4_launch_count()
    fwd = lambda opts, y, wr=w_row: L.nvfp4_linear_fwd(fake, fake, 256, 256, 256, ctypes.byref(opts), y, ctypes.byref(x_col),
                                                       ctypes.byref(wr), ctypes.byref(w_col), 0, fake, 1 << 30, None)
    assert fwd(o, fake + 2) == 3                                                               # Y not 16-byte aligned
    mx = [B.CTensor(fake, fake, fake, 256, 256, B.SF_SWIZZLED, 1) for _ in range(3)]
    assert L.nvfp4_linear_fwd(fake, fake, 256, 256, 256, ctypes.byref(B.quant_opts(rht_dim=8)), fake, ctypes.byref(mx[0]),
                              ctypes.byref(mx[1]), ctypes.byref(mx[2]), 0, fake, 1 << 30, None) == 8  # MXFP4 + d = 8
    assert L.nvfp4_linear_bwd(fake, ctypes.byref(x_col), ctypes.byref(w_col), 256, 256, 256, ctypes.byref(o), fake + 2,
                              fake, 0, fake, 1 << 30, None) == 3                               # dX not aligned
    assert L.nvfp4_linear_bwd(fake, ctypes.byref(x_col), ctypes.byref(w_col), 256, 256, 256,
                              ctypes.byref(B.quant_opts(rht_dim=7)), fake, fake, 0, fake, 1 << 30, None) == 4
    assert L.nvfp4_launch_count() == before
    # a row-scaled operand (format 2) pairs with NVFP4 only, and only on 256 x 256 tiles
    ar = B.CTensor(fake, fake, fake, 256, 256, B.SF_SWIZZLED, 2)
    bm = B.CTensor(fake, fake, fake, 256, 256, B.SF_SWIZZLED, 1)
    bn = B.CTensor(fake, fake, fake, 128, 256, B.SF_SWIZZLED, 0)
    assert L.nvfp4_gemm(ctypes.byref(ar), ctypes.byref(bm), fake, 0, 256, 0, None) == 4
    assert L.nvfp4_gemm(ctypes.byref(ar), ctypes.byref(bn), fake, 0, 128, 0, None) == 2
    rs = B.CTensor(fake, fake, fake, 64, 128, B.SF_LINEAR, 2)
    assert q(fake, 64, 128, 128, ctypes.byref(o), ctypes.byref(rs), ctypes.byref(rs), None) == 4   # no transposed copy
    g16 = lambda M, N, K, lda=None, ldb=None, ldd=None, al=0, bl=0, fp32=0, acc=0, A=fake: L.nvfp4_gemm_bf16(
        A, al, lda or K, fake, bl, ldb or K, M, N, K, fake, fp32, ldd or N, acc, None)
    assert g16(256, 256, 64, A=None) == 1
    assert g16(124, 256, 64) == 2 and g16(256, 380, 64) == 2 and g16(256, 256, 36) == 2      # multiples of 8
    assert g16(256, 256, 64, lda=32) == 2 and g16(256, 256, 64, ldd=128) == 2                 # leading dimensions
    assert g16(256, 256, 64, al=1, lda=64) == 2                                                # [K][M] needs lda >= M
    assert g16(256, 256, 64, al=2) == 4 and g16(256, 256, 64, acc=1) == 4                      # layout id; bf16 accumulate
    assert g16(256, 256, 64, lda=68) == 3                                                      # lda % 8
    assert L.nvfp4_linear_bf16_bwd(fake, fake, fake, 256, 256, 256, None, None, 0, None) == 1


def test_header_is_plain_c_and_cxx():
    import subprocess
    hdr = os.path.join(ROOT, "include", "nvfp4.h")
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror", "-fsyntax-only", "-x", "c", hdr], check=True)
    subprocess.run(["g++", "-std=c++17", "-Wall", "-Werror", "-fsyntax-only", "-x", "c++", hdr], check=True)


def test_plain_c_client_compiles_and_links():
    """The C client under tests/c uses nothing but the header, the shared library and the CUDA runtime."""
    import subprocess, tempfile
    B.lib()
    libdir = os.path.join(ROOT, "paper_2509_25149_b200")
    with tempfile.TemporaryDirectory() as tmp:
        exe = os.path.join(tmp, "abi_roundtrip")
        subprocess.run(["gcc", "-std=c99", "-O1", "-Wall", "-Werror", os.path.join(ROOT, "tests", "c", "abi_roundtrip.c"),
                        "-I", os.path.join(ROOT, "include"), "-I", "/usr/local/cuda/include", "-L", libdir,
                        "-lnvfp4_b200", "-L", "/usr/local/cuda/lib64", "-lcudart", f"-Wl,-rpath,{libdir}", "-o", exe],
                       check=True)
        assert os.path.exists(exe)


@pytest.mark.gpu
def test_plain_c_client_runs():
    import subprocess, tempfile
    B.lib()
    libdir = os.path.join(ROOT, "paper_2509_25149_b200")
    with tempfile.TemporaryDirectory() as tmp:
        exe = os.path.join(tmp, "abi_roundtrip")
        subprocess.run(["gcc", "-std=c99", "-O1", os.path.join(ROOT, "tests", "c", "abi_roundtrip.c"),
                        "-I", os.path.join(ROOT, "include"), "-I", "/usr/local/cuda/include", "-L", libdir,
                        "-lnvfp4_b200", "-L", "/usr/local/cuda/lib64", "-lcudart", f"-Wl,-rpath,{libdir}", "-o", exe],
                       check=True)
        r = subprocess.run([exe], capture_output=True, text=True, timeout=120)
        assert r.returncode == 0 and r.stdout.startswith("ok"), (r.returncode, r.stdout, r.stderr)
