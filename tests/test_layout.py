"""The index maps of the packed layout (csrc/fgmp_common.cuh), run on the host: every map is a
bijection onto its region, and the records have the order that include/fgmp.h documents.  Needs
nvcc (host compilation only), no GPU."""
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
    arec, rec, lists, const = {}, {}, {}, None
    for line in out.splitlines():
        f = line.split()
        if f[0] == "arec":
            arec[(int(f[1]), int(f[2]))] = (int(f[3]), int(f[4]))
        elif f[0] == "rec":
            rec[(int(f[1]), int(f[2]))] = (int(f[3]), int(f[4]))
        elif f[0] == "list":
            lists[int(f[1])] = (int(f[2]), int(f[3]))
        else:
            const = [int(x) for x in f[1:]]
    return arec, rec, lists, const


def test_activation_record_sections_and_maps(maps):
    arec, _, _, const = maps
    arec_bytes, a4, sf, hot, at = const[:5]
    assert (a4, sf, hot, at, arec_bytes) == (0, 2048, 2304, 2560, 2560 + 16 * 256 * 2)
    assert at % 128 == 0 and arec_bytes % 128 == 0            # bulk copies of whole or half records
    # fp16 values: token octet m // 8 in its own 4096 bytes, there 256 bytes per block column, 32 per token
    offs = sorted(v[0] for v in arec.values())
    assert offs == list(range(at, arec_bytes, 32))
    for (m, j), (o_at, o_a4) in arec.items():
        assert o_at == at + (m // 8) * 4096 + j * 256 + (m % 8) * 32
        # the E2M1 codes: a 16-row x 128-byte tile with 16-byte pieces XOR-swizzled by the row
        assert o_a4 == m * 128 + (((j // 2) ^ (m % 8)) * 16) + (j % 2) * 8
    assert sorted(v[1] for v in arec.values()) == list(range(0, 2048, 8))
    # a batch of at most eight tokens needs the first 2560 + 4096 bytes only
    assert max(v[0] for (m, _), v in arec.items() if m < 8) + 32 == at + 4096


def test_weight_record_maps_are_bijections(maps):
    _, rec, _, const = maps
    rec_w4, rec_sf, rec_kbstart, rec_bytes = const[5:]
    assert (rec_w4, rec_sf, rec_kbstart, rec_bytes) == (0, 16384, 18432, 18560) and rec_bytes % 128 == 0
    assert sorted(v[0] for v in rec.values()) == list(range(0, 16384, 8))     # 8 bytes per block, all distinct
    assert sorted(v[1] for v in rec.values()) == list(range(2048))            # one scale byte per block
    for (r, j), (o4, osf) in rec.items():
        assert o4 // 128 == r and (o4 % 128) // 16 == (j // 2) ^ (r % 8)      # codes stay in their row; swizzled pieces
        # scale tiles in the order the scales go to tensor memory: one 512-byte tile per MMA step (64 elements);
        # lane r % 32 holds 16 bytes: 4 bytes for each of the rows r % 32 + 32c, one byte per block of the step
        assert osf == (j // 4) * 512 + (r % 32) * 16 + (r // 32) * 4 + j % 4


def test_fp8_list_sizes(maps):
    _, _, lists, _ = maps
    for cnt, (halves, steps) in lists.items():
        assert halves % 16 == 0 and halves >= 4 * cnt and halves - 4 * cnt < 16     # one word per block, padded to 16 bytes
        assert steps * 16 >= halves + 8 * cnt and steps * 16 - (halves + 8 * cnt) < 16
