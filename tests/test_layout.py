"""The index maps of the packed layout (csrc/fgmp_common.cuh), run on the host: every map is a
bijection onto its region, and the activation record has the fragment order that include/fgmp.h
documents.  Needs nvcc (host compilation only), no GPU."""
import os
import shutil
import subprocess

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CSRC = os.path.join(ROOT, "paper_2504_14152_b200", "csrc")


@pytest.fixture(scope="module")
def maps(tmp_path_factory):
    nvcc = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(nvcc):
        pytest.skip("nvcc not found")
    exe = str(tmp_path_factory.mktemp("layout") / "layout_probe")
    subprocess.check_call([nvcc, "-std=c++17", "-O1", "-I", CSRC, "-I", os.path.join(ROOT, "include"),
                           "-o", exe, os.path.join(ROOT, "tests", "layout_probe.cu")])
    out = subprocess.check_output([exe], text=True)
    arec, rec, const = {}, {}, None
    for line in out.splitlines():
        f = line.split()
        if f[0] == "arec":
            arec[(int(f[1]), int(f[2]), int(f[3]))] = int(f[4])
        elif f[0] == "rec":
            rec[(int(f[1]), int(f[2]))] = (int(f[3]), int(f[4]))
        else:
            const = [int(x) for x in f[1:]]
    return arec, rec, const


def test_activation_record_is_a_bijection_in_fragment_order(maps):
    arec, _, const = maps
    arec_bytes = const[0]
    assert arec_bytes == 16 * 256 * 2                       # 16 tokens x 256 elements, fp16
    offs = sorted(arec.values())
    assert offs == list(range(0, arec_bytes, 16))           # every 16-byte slot exactly once
    for (m, j, half), off in arec.items():
        # elements 16j + 8half .. +7 of token m: lane (g, t) = (m % 8, j // 4) owns elements 64t + 8sp ..,
        # so sp = 2 (j % 4) + half; piece 2 sp + (m // 8) of 512 bytes; slot 4g + (t ^ (g & 3)) of 16 bytes
        g, t, sp, octet = m % 8, j // 4, 2 * (j % 4) + half, m // 8
        assert 64 * t + 8 * sp == 16 * j + 8 * half
        assert off == (2 * sp + octet) * 512 + (4 * g + (t ^ (g & 3))) * 16
    # eight tokens of one block column (what an FP8-weight warp reads at once) spread over four
    # different 16-byte bank groups of a 128-byte line, two tokens each
    for j in range(16):
        groups = [(arec[(m, j, 0)] // 16) % 8 for m in range(8)]
        assert sorted(groups.count(x) for x in set(groups)) == [2, 2, 2, 2]


def test_weight_record_maps_are_bijections(maps):
    _, rec, const = maps
    _, rec_w4, rec_sf, rec_kbcnt, rec_kbstart, rec_rowid = const
    assert (rec_w4, rec_sf, rec_kbcnt) == (0, 16384, 18432) and rec_kbstart == rec_kbcnt + 16 and rec_rowid == rec_kbstart + 48
    w4 = sorted(v[0] for v in rec.values())
    assert w4 == list(range(0, 16384, 8))                   # 8 bytes of codes per block, all distinct
    sf = sorted(v[1] for v in rec.values())
    assert sf == list(range(2048))                          # one microscale byte per block
    for (r, j), (o4, osf) in rec.items():
        assert o4 // 128 == r and osf == 16 * r + j          # codes stay in their row; microscales row-major
        assert (o4 % 128) // 16 == (j // 2) ^ (r % 8)        # 16-byte pieces XOR-ed with r % 8
