"""CPU-only checks of the C-ABI boundary: the library builds, loads without a GPU, exports every
symbol include/muxq.h declares, and its host-side argument validation returns the documented
codes before any CUDA call is made."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    from paper_2604_04701_b200 import build
    build.build()
    import paper_2604_04701_b200 as m
    return m


def test_every_declared_symbol_is_exported(L):
    inc = os.path.join(ROOT, "include")
    hdr = "".join(open(os.path.join(inc, f)).read() for f in sorted(os.listdir(inc)) if f.endswith(".h"))
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = set(re.findall(r"\b(muxq_[a-z0-9_]+)\s*\(", hdr))
    assert {"muxq_detect_outliers", "muxq_build_aux", "muxq_quantize", "muxq_linear"} <= declared
    lib = ctypes.CDLL(L.library_path())
    for name in sorted(declared):
        assert hasattr(lib, name), name
    from paper_2604_04701_b200 import binding
    assert declared == set(binding.EXPORTS)


def test_host_only_helpers(L):
    p = L.MuxqParams()
    assert L.muxq_aux_cols(p) == 256                      # 3 * 64 rounded up to 128
    assert L.muxq_aux_cols(L.MuxqParams(max_outliers=32)) == 128
    assert L.muxq_aux_cols(L.MuxqParams(exp_factor=3, max_outliers=64)) == 512
    assert L.muxq_aux_cols(L.MuxqParams(exp_factor=0)) == 0
    n = L.muxq_workspace_bytes(8192, 768, 2304, p)
    assert n >= 8192 * 768 + 8192 * 256 + 2304 * 256 and n % 1024 == 0
    assert L.muxq_workspace_bytes(0, 768, 768, p) == 0
    assert L.muxq_workspace_bytes(128, 768, 768, L.MuxqParams(max_outliers=8193)) == 0
    assert L.muxq_host_workspace_bytes(128, 768, 768, p, 0) >= L.muxq_workspace_bytes(128, 768, 768, p) + 128 * 768 * 4
    v = L.muxq_workspace_view(128, 768, 768, p)
    assert v.ld_body_q == 768 and v.aux_cols == 256 and v.body_q % 1024 == 0 and v.aux_q > v.body_q
    assert L.muxq_status_string(0) == "ok" and "outlier" in L.muxq_status_string(5)
    assert "wait" in L.muxq_status_string(6)


def test_argument_validation_without_gpu(L):
    lib = L.lib()
    p = L.MuxqParams().c()
    fake = ctypes.c_void_p(0x10000)     # aligned, never dereferenced: every call below fails validation first
    odd = ctypes.c_void_p(0x10004)
    big = 1 << 30
    # NULL pointers / bad sizes
    assert lib.muxq_linear(None, 128, 768, 768, fake, 768, fake, 768, ctypes.byref(p), fake, 768, 0, fake, big, fake, None) == 1
    assert lib.muxq_linear(fake, 0, 768, 768, fake, 768, fake, 768, ctypes.byref(p), fake, 768, 0, fake, big, fake, None) == 1
    assert lib.muxq_linear(fake, 128, 768, 760, fake, 768, fake, 768, ctypes.byref(p), fake, 768, 0, fake, big, fake, None) == 1
    assert lib.muxq_linear(fake, 128, 768, 768, fake, 768, fake, 768, ctypes.byref(p), fake, 768, 3, fake, big, fake, None) == 1
    # unsupported shapes / alignment
    assert lib.muxq_linear(fake, 128, 776, 776, fake, 776, fake, 768, ctypes.byref(p), fake, 768, 0, fake, big, fake, None) == 2
    assert lib.muxq_linear(odd, 128, 768, 768, fake, 768, fake, 768, ctypes.byref(p), fake, 768, 0, fake, big, fake, None) == 2
    assert lib.muxq_linear(fake, 128, 768, 768, fake, 768, fake, 772, ctypes.byref(p), fake, 772, 0, fake, big, fake, None) == 2
    own = L.MuxqParams(aux_scale=1).c()
    # the own-scale reading has no common integer accumulator to return
    assert lib.muxq_linear(fake, 128, 768, 768, fake, 768, fake, 768, ctypes.byref(own), fake, 768, 2, fake, big, fake, None) == 2
    # workspace too small
    assert lib.muxq_linear(fake, 128, 768, 768, fake, 768, fake, 768, ctypes.byref(p), fake, 768, 0, fake, 1024, fake, None) == 3
    # other entry points
    assert lib.muxq_detect_outliers(fake, 128, 768, 768, ctypes.c_float(6.0), fake, fake, fake, 0, fake, big, None) == 1
    assert lib.muxq_detect_outliers(fake, 128, 772, 772, ctypes.c_float(6.0), fake, fake, fake, 8, fake, big, None) == 2
    assert lib.muxq_detect_outliers(fake, 128, 768, 768, ctypes.c_float(6.0), fake, fake, fake, 8, fake, 16, None) == 3
    assert lib.muxq_build_aux(fake, 128, 768, 768, fake, fake, 8, 4, fake, 8, None, 0, None) == 1
    assert lib.muxq_quantize(fake, 128, 768, 768, ctypes.byref(p), 0, None, None, None, fake, 768, None, 0, fake, fake, big, None) == 1
    assert lib.muxq_quantize(fake, 128, 768, 768, ctypes.byref(p), 1, None, None, None, fake, 64, None, 0, fake, fake, big, None) == 1
    assert lib.muxq_quantize(fake, 128, 768, 768, ctypes.byref(p), 1, None, None, None, fake, 128, None, 0, fake, fake, 64, None) == 3
    assert lib.muxq_gemm(fake, 768, None, 0, fake, 768, None, 0, None, 128, 768, 768, ctypes.byref(p), None, None, fake, 768, 0, fake, None) == 1
    assert lib.muxq_gemm(fake, 776, None, 0, fake, 768, None, 0, None, 128, 768, 768, ctypes.byref(p), fake, fake, fake, 768, 0, fake, None) == 2
    assert lib.muxq_read_status(None, None) == 1
    assert lib.muxq_workspace_init(None, big, None) == 1
    assert lib.muxq_workspace_init(fake, 128, None) == 1   # smaller than the control block
    assert lib.muxq_linear_host(None, 128, 768, fake, 768, fake, 768, ctypes.byref(p), fake, 0, fake, big, fake, None) == 1
    assert lib.muxq_linear_host(fake, 128, 768, fake, 768, fake, 768, ctypes.byref(p), fake, 0, fake, 4096, fake, None) == 3


def test_product_does_not_touch_the_oracle():
    """The CUDA package and its sources must not import, include or call anything under oracle/."""
    pkg = os.path.join(ROOT, "paper_2604_04701_b200")
    for dirpath, _, files in os.walk(pkg):
        if "_build" in dirpath:
            continue
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower(), os.path.join(dirpath, f)
    for f in os.listdir(os.path.join(ROOT, "include")):
        assert "oracle" not in open(os.path.join(ROOT, "include", f)).read().lower()
