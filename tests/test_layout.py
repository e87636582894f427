"""The index maps of the packed layout (csrc/fgmp_common.cuh), run on the host: every map is a
bijection onto its region, and the records have the fragment order that include/fgmp.h
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
    arec, rec, pow2, const = {}, {}, {}, None
    for line in out.splitlines():
        f = line.split()
        if f[0] == "arec":
            arec[(int(f[1]), int(f[2]), int(f[3]))] = int(f[4])
        elif f[0] == "rec":
            rec[(int(f[1]), int(f[2]))] = tuple(int(x) for x in f[3:])
        elif f[0] == "pow2":
            pow2[int(f[1])] = int(f[2])
        else:
            const = [int(x) for x in f[1:]]
    return arec, rec, pow2, const


def test_activation_record_is_a_bijection_in_fragment_order(maps):
    arec, _, _, const = maps
    arec_bytes = const[0]
    assert arec_bytes == 16 * 256 * 2                       # 16 tokens x 256 elements, fp16
    offs = sorted(arec.values())
    assert offs == list(range(0, arec_bytes, 16))           # every 16-byte slot exactly once
    for (m, j, half), off in arec.items():
        # token octet m // 8 in its own 4096 bytes; there piece 2 (j % 4) + half of 512 bytes holds, for lane
        # (g, t) = (m % 8, j // 4) of the warps with hq = j % 4, elements 8 half .. 8 half + 7 of block column j
        g, t, hq, octet = m % 8, j // 4, j % 4, m // 8
        assert off == octet * 4096 + (2 * hq + half) * 512 + (4 * g + t) * 16
    # a batch of at most eight tokens lives in the first half of the record
    assert max(off for (m, _, _), off in arec.items() if m < 8) < 4096


def test_weight_record_maps_are_bijections(maps):
    _, rec, _, const = maps
    _, rec_w4, rec_sf, rec_wstart, rec_bytes = const
    assert (rec_w4, rec_sf, rec_wstart, rec_bytes) == (0, 16384, 18432, 18560) and rec_bytes % 128 == 0
    assert sorted(v[0] for v in rec.values()) == list(range(0, 16384, 8))     # 8 bytes per block, all distinct
    assert sorted(v[1] for v in rec.values()) == list(range(2048))            # one scale byte per block
    assert sorted(v[2] for v in rec.values()) == list(range(2048))            # ranks of the overflow order
    for (r, j), (o4, osf, order, w, lane, k, r_back, j_back) in rec.items():
        # warp (jr, hq) = (r // 32, j % 4); lane (g, t) = (r % 8, j // 4); slot k = (r // 8) % 4
        assert w == 4 * (r // 32) + j % 4 and lane == 4 * (r % 8) + j // 4 and k == (r // 8) % 4
        assert (r_back, j_back) == (r, j)
        # a warp's slots: 1 KiB, two 512-byte halves (k // 2) of 16 bytes per lane (two slots side by side)
        assert o4 == w * 1024 + (k // 2) * 512 + lane * 16 + (k % 2) * 8
        assert osf == (w // 4) * 512 + lane * 16 + (w % 4) * 4 + k     # a lane's sixteen scale bytes of a row group: one 16-byte load
        assert order == (w * 32 + lane) * 4 + k
    # one warp-wide 16-byte load per half reads 512 contiguous bytes: no bank conflicts
    for w in range(16):
        for kh in range(2):
            offs = sorted(o4 for (o4, _, _, ww, _, k, _, _) in rec.values() if ww == w and k // 2 == kh)
            assert offs == list(range(w * 1024 + kh * 512, w * 1024 + kh * 512 + 512, 8))


def test_power_of_two_scale_codes(maps):
    """The scale byte of an FP8 weight block holds 2^ratio as an E4M3 code (2^-7 is subnormal)."""
    _, _, pow2, _ = maps
    def e4m3(code):
        e, m = code >> 3, code & 7
        return (m / 8) * 2.0 ** -6 if e == 0 else (1 + m / 8) * 2.0 ** (e - 7)
    for ratio in range(-7, 8):
        assert 0 < pow2[ratio] < 0x7f and e4m3(pow2[ratio]) == 2.0 ** ratio
