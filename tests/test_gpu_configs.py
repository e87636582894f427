"""GPU parity at the full sizes of the five benchmark configurations: sampled GEMM outputs against the
oracle (after the packed operands have been compared with the oracle's bit for bit), the clip-search packer
at full width, and the hand-derived tie cases of the clip search."""
import numpy as np
import pytest
import torch

import fgmp_inputs as gi
import oracle
from test_gpu_parity import GEMM_TOL, compare_packed, fg, quantize_both, _sampled_linear_check  # noqa: F401
from test_oracle_quant import clip_tie_case

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("M", [2, 4, 8])
def test_config2_llama2_7b_fc1_decode_token_counts(fg, M):
    """Config 2 says M = 1..16 tokens: the counts between the two that the other tests use."""
    _sampled_linear_check(fg, gi.llama("cfg2", M, 11008, 4096, seed=8), 0.1, 4000, 10 + M)


@pytest.mark.parametrize("N,K", [(11008, 4096), (4096, 11008)])
def test_config3_llama2_7b_prefill_fc1_and_fc2(fg, N, K):
    """Config 3 at M = 4096: FC1 / gate (4096 -> 11008) and FC2 (11008 -> 4096); the 4096 x 4096 projections are
    test_linear_prefill_shape_sampled."""
    _sampled_linear_check(fg, gi.llama("cfg3", 4096, N, K, seed=9), 0.1, 2500, 20)


@pytest.mark.parametrize("N,K", [(13824, 5120), (5120, 13824)])
def test_config4_llama2_13b_at_ten_percent(fg, N, K):
    """Config 4 at M = 2048: both layers at the 10 % point of the sweep (0 / 20 / 30 % of FC1 are swept elsewhere)."""
    _sampled_linear_check(fg, gi.llama("cfg4", 2048, N, K, seed=10), 0.1, 2500, 21)


def test_config5_llama2_70b_prefill(fg):
    """Config 5 at M = 8192: the 8192 x 8192 activations through the quantizer and the 28672 x 8192 FC1 GEMM."""
    _sampled_linear_check(fg, gi.llama("cfg5", 8192, 28672, 8192, seed=11), 0.1, 2500, 22)


def test_config3_fc2_activation_quantizer_full_size(fg):
    """The activation quantizer on the 4096 x 11008 input of FC2, every block against the oracle."""
    wl = gi.llama("cfg3a", 4096, 1, 11008, seed=12)
    x, fx = wl.x(), wl.fx()
    s4 = gi.tensor_scale(x)
    xb = gi.bf16_bits(x)
    scores = oracle.quantize_activations(xb, fx.numpy(), s4, tau=np.inf).scores
    k = int(np.floor(0.1 * scores.size + 0.5))
    srt = np.sort(scores)[::-1]
    tau = float(np.float32(0.5) * (srt[k - 1] + srt[k]))
    q = oracle.quantize_activations(xb, fx.numpy(), s4, tau=tau)
    p = fg.quantize_activations(x.cuda(), fx.cuda(), scale_fp4=s4, tau=tau)
    compare_packed(fg, p, q, tau, "4096 x 11008")


def test_config5_clip_search_packer_at_full_width(fg):
    """The packer with the Eq. 11 clip search on a full-width tensor (11008 x 4096, threshold mode, tensor scale
    given, so that every block's outcome depends on that block alone): the blocks of the first 512 rows against
    the oracle run on those rows."""
    wl = gi.llama("cfg5w", 1, 11008, 4096, seed=13)
    w, fw = wl.w(), wl.fw()
    rows = 512
    s4 = float(np.float32(w.float().abs().max().item() / 2688.0))
    q0 = oracle.quantize_weights(gi.bf16_bits(w)[:rows].copy(), fw.numpy()[:rows].copy(), scale_fp4=s4, clip=True, fp8_fraction=0.0)
    tau = float(np.sort(q0.scores)[::-1][int(0.1 * q0.scores.size)])
    q = oracle.quantize_weights(gi.bf16_bits(w)[:rows].copy(), fw.numpy()[:rows].copy(), scale_fp4=s4, clip=True,
                                fp8_fraction=-1.0, tau=tau)
    p = fg.quantize_weights(w.cuda(), fw.cuda(), scale_fp4=s4, clip_mode=1, fp8_fraction=-1.0, tau=tau)
    assert p.header()["error"] == 0
    c4, c8, sc, mk = [t.cpu().numpy() for t in fg.unpack(p)]
    K, KB = 4096, 256
    MW = KB // 32
    g = oracle.Quantized(rows, K, c4[: rows * K // 2], c8[: rows * K], sc[: rows * KB], mk.view(np.uint32)[: rows * MW],
                         q.scores, s4, 3)
    excused = np.abs(q.scores.reshape(rows, KB) - np.float32(tau)) <= 1e-6 * tau
    keep = ~excused
    assert ((g.mask_bits() == q.mask_bits()) | excused).all()
    assert np.array_equal(g.scales.reshape(rows, KB)[keep], q.scales.reshape(rows, KB)[keep])
    assert not ((g.codes4.reshape(rows, KB, 8) != q.codes4.reshape(rows, KB, 8)).any(-1) & keep).any()
    assert not ((g.codes8.reshape(rows, KB, 16) != q.codes8.reshape(rows, KB, 16)).any(-1) & keep).any()
    assert 0.05 < q.mask_bits().mean() < 0.2


def test_clip_search_tie_cases_on_the_gpu(fg):
    """The two tie cases whose outcome is derived by hand in tests/test_oracle_quant.py (an all-zero block; a block
    that four scale codes represent exactly): the GPU packer gives the derived codes and scales."""
    w, bits, codes4, scales = clip_tie_case()
    wt = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16)
    p = fg.quantize_weights(wt.cuda(), torch.ones(2, 64).cuda(), scale_fp4=1.0, clip_mode=1, fp8_fraction=0.0)
    c4, c8, sc, mk = [t.cpu().numpy() for t in fg.unpack(p)]
    assert np.array_equal(sc, scales) and np.array_equal(c4, codes4)
    assert not c8.any() and not mk.any()


@pytest.mark.parametrize("M,N,K", [(64, 256, 256), (77, 300, 1024), (129, 136, 64), (384, 1000, 2048), (1000, 640, 320)])
def test_all_nvfp4_operands_take_the_fp4_tensor_core_kernel(fg, M, N, K):
    """With no FP8 block on either side (threshold +inf, fraction 0) the prefill GEMM runs on the NVFP4 tensor-core
    kind straight from the packed operands (word 2 of the workspace status says which kernel produced Y): every
    output against the oracle, fp32 and bf16; one FP8 block anywhere sends the call down the general path."""
    wl = gi.llama("n4", M, N, K, seed=50 + M)
    qa, qw, pa, pw = quantize_both(fg, wl, 0.0, 0.0, clip=True)
    Y, S = oracle.linear(qa, qw)
    y = fg.linear(pa, pw)
    ws = fg.linear.last_workspace
    fg.check(ws)
    assert int(ws[8:12].view(torch.int32).item()) == 1, "the NVFP4 kernel did not take the call"
    err = np.abs(y.cpu().numpy().astype(np.float64) - Y)
    assert (err <= 1e-5 * S + 1e-30).all(), f"max err/S = {(err / np.maximum(S, 1e-300)).max():.3e}"
    assert torch.equal(fg.linear(pa, pw), y)
    yb = fg.linear(pa, pw, out_dtype=torch.bfloat16).float().cpu().numpy().astype(np.float64)
    assert (np.abs(yb - Y) <= GEMM_TOL * S + np.abs(Y) * 2.0 ** -8 + 1e-30).all()
    # FP8 blocks in the weights: the general path, same bar
    qa2, qw2, pa2, pw2 = quantize_both(fg, wl, 0.0, 0.1, clip=True)
    y2 = fg.linear(pa2, pw2)
    ws2 = fg.linear.last_workspace
    fg.check(ws2)
    assert int(ws2[8:12].view(torch.int32).item()) == 0
    Y2, S2 = oracle.linear(qa2, qw2)
    assert (np.abs(y2.cpu().numpy().astype(np.float64) - Y2) <= 1e-5 * S2 + 1e-30).all()


# ------------------------------------------------------------ the other model families of Section 5.1

# FC1 / FC2 shapes (N, K) of the GPT3 and Nemotron-4 models that Section 5.1 evaluates beside Llama-2; hidden and
# feed-forward widths as in the models' public descriptions (the paper gives the names only)
OTHER_FAMILIES = {
    "gpt3-1.3b": (2048, 8192),
    "gpt3-8.3b": (3072, 12288),
    "gpt3-22b": (6144, 24576),
    "nemotron4-15b": (6144, 24576),
}


@pytest.mark.parametrize("model,M", [("gpt3-1.3b", 16), ("gpt3-8.3b", 3), ("gpt3-22b", 16), ("nemotron4-15b", 1)])
def test_section_5_1_other_families_decode(fg, model, M):
    """GPT3 and Nemotron-4 feed-forward layers at decode size: FC1 and FC2, sampled outputs against the oracle
    (packed operands compared bit for bit first)."""
    h, f = OTHER_FAMILIES[model]
    _sampled_linear_check(fg, gi.llama(model + "-fc1", M, f, h, seed=60), 0.1, 3000, 30)
    _sampled_linear_check(fg, gi.llama(model + "-fc2", M, h, f, seed=61), 0.1, 3000, 31)


@pytest.mark.parametrize("model,M", [("gpt3-8.3b", 2048), ("nemotron4-15b", 1024)])
def test_section_5_1_other_families_prefill(fg, model, M):
    h, f = OTHER_FAMILIES[model]
    _sampled_linear_check(fg, gi.llama(model + "-fc1p", M, f, h, seed=62), 0.1, 2500, 32)


# ------------------------------------------------------------ guard bands

CANARY = 0xA5


class Guarded:
    """A device buffer with 4 KiB of canary bytes before and after the part that is handed to the library."""

    def __init__(self, nbytes, device="cuda", fill=None):
        self.n = int(nbytes)
        self.raw = torch.full((self.n + 2 * 4096 + 1024,), CANARY, dtype=torch.uint8, device=device)
        off = 4096 + ((-(self.raw.data_ptr() + 4096)) % 1024)
        self.off = off
        self.view = self.raw[off:off + self.n]
        if fill is not None:
            self.view.fill_(fill)

    def intact(self):
        before, after = self.raw[: self.off], self.raw[self.off + self.n:]
        return bool((before == CANARY).all().item()) and bool((after == CANARY).all().item())


@pytest.mark.parametrize("M,N,K", [(16, 1000, 1024), (200, 392, 512)])
def test_no_call_writes_outside_its_buffers(fg, M, N, K):
    """Every buffer a call writes (packed activations, packed weights, workspaces, Y) sits between canary bytes
    that must be unchanged afterwards: the packer, the activation quantizer, fgmp_linear at decode and prefill
    size and the fused decode step, with results equal to those of the same calls on ordinary buffers."""
    wl = gi.llama("guard", M, N, K, seed=70)
    x, fx, w, fw = wl.x().cuda(), wl.fx().cuda(), wl.w().cuda(), wl.fw().cuda()
    s4 = gi.tensor_scale(wl.x())
    tau = float(fg.calibrate_tau(x, fx, scale_fp4=s4, fp8_fraction=0.1))
    B = N * K // 16
    n8 = int(0.1 * B + 0.5) + 1
    gw = Guarded(fg.weights_bytes(N, K, n8))
    gws = Guarded(fg.workspace_bytes(fg.OP_QUANTIZE_WEIGHTS, 0, N, K))
    pw = fg.quantize_weights(w, fw, fp8_fraction=0.1, out=gw.view, workspace=gws.view)
    ga = Guarded(fg.acts_bytes(M, K))
    pa = fg.quantize_activations(x, fx, scale_fp4=s4, tau=tau, out=ga.view)
    gy = Guarded(M * N * 4)
    gl = Guarded(fg.workspace_bytes(fg.OP_LINEAR, M, N, K), fill=0)
    fg.workspace_init(gl.view)
    y = fg.linear(pa, pw, out=gy.view.view(torch.float32).view(M, N), workspace=gl.view)
    fg.check(gl.view)
    torch.cuda.synchronize()
    for name, g in (("packed weights", gw), ("packer workspace", gws), ("packed activations", ga), ("Y", gy), ("workspace", gl)):
        assert g.intact(), f"bytes around {name} were written"
    pw0 = fg.quantize_weights(w, fw, fp8_fraction=0.1)
    pa0 = fg.quantize_activations(x, fx, scale_fp4=s4, tau=tau)
    assert torch.equal(fg.linear(pa0, pw0), y)
    if M <= 16:
        gy2 = Guarded(M * N * 2)
        gf = Guarded(fg.workspace_bytes(fg.OP_LINEAR_FUSED, M, N, K), fill=0)
        gp = Guarded(fg.acts_bytes(M, K))
        fg.workspace_init(gf.view)
        y2, _ = fg.linear_fused(x, fx, pw, scale_fp4=s4, tau=tau, out=gy2.view.view(torch.bfloat16).view(M, N),
                                packed_out=gp.view, workspace=gf.view)
        fg.check(gf.view)
        torch.cuda.synchronize()
        for name, g in (("Y (bf16)", gy2), ("fused workspace", gf), ("packed activations of the fused call", gp), ("packed weights", gw)):
            assert g.intact(), f"bytes around {name} were written"
        assert torch.equal(y2.float(), fg.linear(pa0, pw0, out_dtype=torch.bfloat16).float())
