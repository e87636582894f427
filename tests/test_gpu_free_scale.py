"""GPU parity for operands whose FP8 blocks carry a tensor scale of their own (Section 5.1: FP8 blocks have no
microscale, only a per-tensor scale; here amax / 448 beside amax / (6 * 448) for the NVFP4 part, a ratio of 6):
both quantizers bit for bit against the oracle, the per-class GEMM against the oracle's fp64 result, and the refusal
of the single-accumulator entry points."""
import numpy as np
import pytest
import torch

import fgmp_inputs as gi
import oracle
from test_gpu_parity import GEMM_TOL, compare_packed, fg, tau_for_fraction  # noqa: F401

pytestmark = pytest.mark.gpu


def free_scales(t):
    a = float(t.float().abs().max())
    return float(np.float32(a / 2688.0)), float(np.float32(a / 448.0))


def quantize_both_free(fg, wl, frac, mode=0, clip=True, free_w=True, free_a=True):
    x, fx, w, fw = wl.x(), wl.fx(), wl.w(), wl.fw()
    as4, as8 = free_scales(x)
    ws4, ws8 = free_scales(w)
    if not free_a:
        as8 = 0.0
    if not free_w:
        ws8 = 0.0
    xb = gi.bf16_bits(x)
    scores = oracle.quantize_activations(xb, fx.numpy(), as4, tau=np.inf, mode=mode, scale_fp8=as8).scores
    tau = tau_for_fraction(scores, frac)
    qa = oracle.quantize_activations(xb, fx.numpy(), as4, tau=tau, mode=mode, scale_fp8=as8)
    pa = fg.quantize_activations(x.cuda(), fx.cuda(), scale_fp4=as4, scale_fp8=as8, score_mode=mode, tau=tau)
    compare_packed(fg, pa, qa, tau, "activations, free FP8 scale")
    qw = oracle.quantize_weights(gi.bf16_bits(w), fw.numpy(), scale_fp4=ws4, scale_fp8=ws8, clip=clip, mode=mode, fp8_fraction=frac)
    pw = fg.quantize_weights(w.cuda(), fw.cuda(), scale_fp4=ws4, scale_fp8=ws8, clip_mode=int(clip), score_mode=mode, fp8_fraction=frac)
    compare_packed(fg, pw, qw, None, "weights, free FP8 scale")
    ha, hw = pa.header(), pw.header()
    assert ha["fp8_scale_free"] == int(free_a) and hw["fp8_scale_free"] == int(free_w)
    if free_a:
        assert np.float32(ha["scale_fp8"]) == np.float32(as8)
    if free_w:
        assert np.float32(hw["scale_fp8"]) == np.float32(ws8)
    return qa, qw, pa, pw


@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("frac", [0.1, 1.0])
def test_tiny_config_with_free_fp8_scales(fg, mode, frac):
    """Config 1 with free scales on both operands: packed operands bit for bit (mode 1 puts s8 into every score),
    every output of the per-class GEMM within the GEMM tolerance, and the run repeats bit for bit."""
    wl = gi.tiny(0)
    qa, qw, pa, pw = quantize_both_free(fg, wl, frac, mode=mode)
    Y, S = oracle.linear(qa, qw)
    y = fg.linear(pa, pw)                      # routed to the per-class entry by the binding
    fg.check(fg.linear.last_workspace)
    err = np.abs(y.cpu().numpy().astype(np.float64) - Y)
    assert (err <= 1e-5 * S + 1e-30).all(), f"max err/S = {(err / np.maximum(S, 1e-300)).max():.3e}"
    assert torch.equal(fg.linear_classes(pa, pw), y)


@pytest.mark.parametrize("M,N,K,free_a,free_w", [(16, 1000, 1024, True, True), (3, 392, 512, True, False),
                                                 (200, 392, 512, False, True), (640, 1100, 2048, True, True)])
def test_per_class_gemm_against_the_oracle(fg, M, N, K, free_a, free_w):
    """Decode-sized and prefill-sized shapes with ragged tiles, a free scale on one or both operands."""
    wl = gi.llama("free", M, N, K, seed=80 + M)
    qa, qw, pa, pw = quantize_both_free(fg, wl, 0.1, clip=False, free_a=free_a, free_w=free_w)
    Y, S = oracle.linear(qa, qw)
    y = fg.linear_classes(pa, pw)
    fg.check(fg.linear.last_workspace)
    err = np.abs(y.cpu().numpy().astype(np.float64) - Y)
    assert (err <= 1e-5 * S + 1e-30).all(), f"max err/S = {(err / np.maximum(S, 1e-300)).max():.3e}"


def test_per_class_gemm_equals_the_single_accumulator_for_tied_scales(fg):
    """Operands with tied scales are accepted by the per-class entry too and give the oracle's result; fgmp_linear
    on the same operands agrees within the tolerance of both."""
    wl = gi.llama("tied", 130, 392, 512, seed=90)
    x, fx, w, fw = wl.x(), wl.fx(), wl.w(), wl.fw()
    s4 = gi.tensor_scale(x)
    tau = float(fg.calibrate_tau(x.cuda(), fx.cuda(), scale_fp4=s4, fp8_fraction=0.1))
    pa = fg.quantize_activations(x.cuda(), fx.cuda(), scale_fp4=s4, tau=tau)
    pw = fg.quantize_weights(w.cuda(), fw.cuda(), fp8_fraction=0.1)
    qa = oracle.quantize_activations(gi.bf16_bits(x), fx.numpy(), s4, tau=tau)
    qw = oracle.quantize_weights(gi.bf16_bits(w), fw.numpy(), fp8_fraction=0.1)
    Y, S = oracle.linear(qa, qw)
    for y in (fg.linear_classes(pa, pw), fg.linear(pa, pw)):
        fg.check(fg.linear.last_workspace)
        assert (np.abs(y.cpu().numpy().astype(np.float64) - Y) <= 1e-5 * S + 1e-30).all()


def test_single_accumulator_entries_refuse_a_free_scale(fg):
    """fgmp_linear needs the power-of-two tie: on an operand packed with a free scale its kernels record
    FGMP_ERR_INVALID_ARG (fgmp_check) at both sizes, the fused decode step refuses the scale on the host, and the
    workspace serves a normal call after being cleared."""
    import paper_2504_14152_b200.binding as b
    for M in (8, 200):
        wl = gi.llama("refuse", M, 392, 512, seed=91)
        qa, qw, pa, pw = quantize_both_free(fg, wl, 0.1, clip=False, free_a=False, free_w=True)
        y = torch.empty(M, 392, device="cuda")
        ws = fg.alloc_workspace(fg.OP_LINEAR, M, 392, 512, "cuda")
        L = b._load()
        rc = L.fgmp_linear(pa.blob.data_ptr(), pw.blob.data_ptr(), y.data_ptr(), 0, 392, M, 392, 512, ws.data_ptr(), ws.numel(), None)
        assert rc == 0
        with pytest.raises(fg.FgmpError) as e:
            fg.check(ws)
        assert e.value.code == -1
    x, fx = wl.x().cuda(), wl.fx().cuda()
    with pytest.raises(fg.FgmpError) as e:
        fg.linear_fused(x[:8].contiguous(), fx, pw, scale_fp4=1.0, tau=1.0)      # free-scale weights: caught on the device
        fg.check(fg.linear.last_workspace)
    assert e.value.code == -1
    rc = b._load().fgmp_linear_fused(x.data_ptr(), 512, fx.data_ptr(), b._Scales(1.0, 3, 0.5), 0, 1.0, pw.blob.data_ptr(),
                                     y.data_ptr(), 0, 392, 8, 392, 512, None, 0, ws.data_ptr(), ws.numel(), None)
    assert rc == -1
