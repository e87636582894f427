"""CPU checks of the C-ABI boundary: the library loads, exports every symbol the header
declares, its pure host functions behave, and argument validation answers before any
GPU work (no compute is launched here)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2504_14152_b200 import build
    return ctypes.CDLL(build.build())


def declared_functions():
    text = open(os.path.join(ROOT, "include", "fgmp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(fgmp_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_three_entry_points():
    names = declared_functions()
    for must in ("fgmp_quantize_weights", "fgmp_quantize_activations", "fgmp_linear"):
        assert must in names


def test_library_exports_every_declared_symbol(lib):
    for name in declared_functions():
        assert hasattr(lib, name), f"{name} is declared in fgmp.h but not exported"


def test_size_functions(lib):
    import paper_2504_14152_b200 as fg
    assert fg.version() == 1
    assert fg.acts_bytes(64, 100) == 0 and fg.acts_bytes(0, 256) == 0
    # sections: header + codes4 + sf + mask + FP8 plane, each rounded to 1 KiB
    assert fg.acts_bytes(64, 256) == 1024 + 8192 + 2048 + 1024 + 16384
    w0 = fg.weights_bytes(256, 256, 0)
    assert fg.weights_bytes(256, 256, 410) - w0 == 4096          # 12 bytes per FP8 block beyond its slot (the first KiB is there already)
    assert fg.weights_bytes(256, 256, 4097) == 0                 # more blocks than exist
    # algorithmic payload versus the layout: an FP8 block's first half takes the place of the NVFP4 codes, so the
    # blob holds little beyond the payload (per-unit tables, the second copy of the mask bits, padding)
    N, K = 11008, 4096
    B = N * K // 16
    n8 = B // 10
    algorithmic = (B - n8) * 9 + n8 * 16 + B / 8
    stored = fg.weights_bytes(N, K, n8)
    assert 1.0 < stored / algorithmic < 1.07
    assert fg.workspace_bytes(1, 64, 0, 256) == 0
    assert fg.workspace_bytes(2, 64, 256, 256) >= 2 * (64 + 256) * 256
    assert fg.workspace_bytes(0, 0, 256, 250) == 0
    assert "timed out" in fg.status_string(-6)


def test_validation_rejects_bad_arguments_on_the_host(lib):
    import paper_2504_14152_b200.binding as b
    L = b._load()
    sc = b._Scales(1.0, 3)
    # NULL pointers
    assert L.fgmp_quantize_activations(None, 256, None, 4, 256, sc, 0, 0.0, None, 0, None, 0, None) == -1
    assert L.fgmp_linear(None, None, None, 0, 256, 4, 256, 256, None, 0, None) == -1
    assert L.fgmp_unpack(None, 4, 256, None, None, None, None, None) == -1
    # shape: K not a multiple of 64 (pointers are fake but aligned; validation comes first)
    fake = ctypes.c_void_p(0x10000)
    assert L.fgmp_quantize_activations(fake, 96, fake, 4, 96, sc, 0, 0.0, fake, 1 << 20, None, 0, None) == -2
    assert L.fgmp_quantize_activations(fake, 256, fake, 4, 256, b._Scales(-1.0, 3), 0, 0.0, fake, 1 << 20, None, 0, None) == -1
    assert L.fgmp_quantize_activations(fake, 256, fake, 4, 256, sc, 7, 0.0, fake, 1 << 20, None, 0, None) == -1
    # output blob too small
    assert L.fgmp_quantize_activations(fake, 256, fake, 4, 256, sc, 0, 0.0, fake, 100, None, 0, None) == -3
    assert L.fgmp_quantize_weights(fake, 256, fake, 256, 4, 256, sc, 0, 0, 2.0, 0.0, fake, 1 << 20, None, fake, 1 << 20, None) == -1
    assert L.fgmp_quantize_weights(fake, 256, fake, 256, 4, 256, sc, 0, 0, 0.1, 0.0, fake, 10, None, fake, 1 << 20, None) == -3
    assert L.fgmp_linear(fake, fake, fake, 0, 8, 4, 256, 256, fake, 1 << 30, None) == -2    # ldy < N


def test_product_path_never_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_2504_14152_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                assert "oracle" not in open(os.path.join(dirpath, f)).read(), f
    bench = open(os.path.join(ROOT, "bench.py")).read() if os.path.exists(os.path.join(ROOT, "bench.py")) else ""
    # the benchmark may touch the oracle only in its CPU-baseline / reference legs
    for line in bench.splitlines():
        if "import oracle" in line:
            assert line.startswith("    "), "oracle must be imported lazily inside the baseline functions"
