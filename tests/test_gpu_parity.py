"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle, element by element.

Bars: codes, microscales and masks bit-exact (a block whose fp32 score lies within
1e-6*tau of tau is excused); GEMM outputs within 2e-3 * sum|a||w| of the oracle's fp64 result.
"""
import numpy as np
import pytest
import torch

import fgmp_inputs as gi
import oracle

pytestmark = pytest.mark.gpu

GEMM_TOL = 2e-3


@pytest.fixture(scope="module")
def fg():
    import paper_2504_14152_b200 as fg_
    assert torch.cuda.is_available()
    assert torch.cuda.get_device_capability()[0] == 10, "these kernels are sm_100a only"
    return fg_


def tau_for_fraction(scores: np.ndarray, frac: float) -> float:
    k = int(np.floor(frac * scores.size + 0.5))
    if k == 0:
        return float("inf")
    if k == scores.size:
        return -1.0
    s = np.sort(scores.ravel())[::-1]
    return float(np.float32(0.5) * (s[k - 1] + s[k]))


def compare_packed(fg, packed, q: oracle.Quantized, tau=None, what=""):
    c4, c8, sc, mk = [t.cpu().numpy() for t in fg.unpack(packed)]
    mk = mk.view(np.uint32)
    KB = q.K // 16
    excused = np.zeros((q.rows, KB), bool)
    if tau is not None and np.isfinite(tau) and tau > 0:
        excused = np.abs(q.scores.reshape(q.rows, KB) - np.float32(tau)) <= 1e-6 * tau
    g = oracle.Quantized(q.rows, q.K, c4, c8, sc, mk, q.scores, q.scale_fp4, q.ratio)
    ok_mask = (g.mask_bits() == q.mask_bits()) | excused
    assert ok_mask.all(), f"{what}: {np.count_nonzero(~ok_mask)} mask bits differ"
    keep = ~excused
    assert np.array_equal(sc.reshape(q.rows, KB)[keep], q.scales.reshape(q.rows, KB)[keep]), f"{what}: microscales differ"
    d4 = (c4.reshape(q.rows, KB, 8) != q.codes4.reshape(q.rows, KB, 8)).any(-1) & keep
    assert not d4.any(), f"{what}: {d4.sum()} NVFP4 blocks differ, first at {np.argwhere(d4)[:3].tolist()}"
    d8 = (c8.reshape(q.rows, KB, 16) != q.codes8.reshape(q.rows, KB, 16)).any(-1) & keep
    assert not d8.any(), f"{what}: {d8.sum()} FP8 blocks differ, first at {np.argwhere(d8)[:3].tolist()}"
    return int(excused.sum())


def gpu_quant_acts(fg, x, fx, s4, tau, mode=0, ratio=3):
    return fg.quantize_activations(x.cuda(), fx.cuda(), scale_fp4=s4, ratio=ratio, score_mode=mode, tau=tau)


# ------------------------------------------------------------------ conversions

@pytest.mark.parametrize("order", ["sorted", "shuffled"])
def test_every_bf16_value_converts_like_the_oracle(fg, order):
    """All 65 536 bf16 bit patterns (non-finite ones replaced by zero) through the quantizer,
    as NVFP4 (codes + microscales) and as FP8, for several tensor scales."""
    bits = np.arange(65536, dtype=np.uint32)
    f = (bits << 16).view(np.float32)
    bits = np.where(np.isfinite(f), bits, 0).astype(np.uint16)
    if order == "shuffled":
        bits = np.random.default_rng(3).permutation(bits)
    xb = bits.reshape(64, 1024)
    x = torch.from_numpy(xb.view(np.int16)).view(torch.bfloat16)
    fx = torch.ones(1024)
    for s4 in (1.0, 2.0 ** -7 * 1.37, 3.1e-5, 41.0):
        for tau in (float("inf"), -1.0):
            for mode in (0, 1):
                q = oracle.quantize_activations(xb, fx.numpy(), s4, tau=tau, mode=mode)
                p = gpu_quant_acts(fg, x, fx, s4, tau, mode)
                compare_packed(fg, p, q, what=f"s4={s4} tau={tau} mode={mode}")
                if tau == float("inf"):
                    sg = fg.activation_scores(x.cuda(), fx.cuda(), scale_fp4=s4, score_mode=mode).cpu().numpy()
                    assert np.array_equal(sg.ravel().view(np.uint32), q.scores.view(np.uint32))


# ------------------------------------------------------------------ activations

@pytest.mark.parametrize("mode", [0, 1])
def test_activations_tiny_config(fg, mode):
    wl = gi.tiny(0)
    x, fx = wl.x(), wl.fx()
    s4 = gi.tensor_scale(x)
    xb = gi.bf16_bits(x)
    scores = oracle.quantize_activations(xb, fx.numpy(), s4, tau=np.inf, mode=mode).scores
    sg = fg.activation_scores(x.cuda(), fx.cuda(), scale_fp4=s4, score_mode=mode).cpu().numpy()
    assert np.array_equal(sg.ravel().view(np.uint32), scores.view(np.uint32))
    tau = tau_for_fraction(scores, wl.fp8_fraction)
    q = oracle.quantize_activations(xb, fx.numpy(), s4, tau=tau, mode=mode)
    p = gpu_quant_acts(fg, x, fx, s4, tau, mode)
    compare_packed(fg, p, q, tau, "tiny")
    assert q.mask_bits().sum() == int(np.floor(0.1 * scores.size + 0.5))
    # calibration entry point reproduces the threshold (Eq. 9)
    tg = fg.calibrate_tau(x.cuda(), fx.cuda(), scale_fp4=s4, score_mode=mode, fp8_fraction=wl.fp8_fraction)
    assert np.float32(tg.item()) == np.float32(tau)
    h = p.header()
    assert h["magic"] == 0x504D4746 and h["rows"] == wl.M and h["K"] == wl.K and h["kind"] == 0


@pytest.mark.parametrize("M,K", [(1, 4096), (16, 4096), (77, 11008), (300, 5120), (129, 64), (2048, 1024)])
def test_activations_ragged_shapes(fg, M, K):
    wl = gi.llama("a", M, 1, K, seed=M + K)
    x, fx = wl.x(), wl.fx()
    s4 = gi.tensor_scale(x)
    xb = gi.bf16_bits(x)
    scores = oracle.quantize_activations(xb, fx.numpy(), s4, tau=np.inf).scores
    for frac in (0.1, 0.0, 1.0):
        tau = tau_for_fraction(scores, frac)
        q = oracle.quantize_activations(xb, fx.numpy(), s4, tau=tau)
        p = gpu_quant_acts(fg, x, fx, s4, tau)
        compare_packed(fg, p, q, tau, f"M={M} K={K} frac={frac}")


def test_activations_strided_input_and_zero_blocks(fg):
    wl = gi.llama("a", 40, 1, 1024, seed=9)
    big = torch.zeros(40, 2048, dtype=torch.bfloat16)
    x = wl.x()
    x[:, 64:96] = 0                      # all-zero blocks
    x[3, 70] = -0.0
    big[:, :1024] = x
    fx = wl.fx()
    s4 = gi.tensor_scale(x)
    q = oracle.quantize_activations(gi.bf16_bits(x), fx.numpy(), s4, tau=1e-3)
    xg = big.cuda()[:, :1024]            # row stride 2048
    assert xg.stride(0) == 2048
    p = fg.quantize_activations(xg, fx.cuda(), scale_fp4=s4, tau=1e-3)
    compare_packed(fg, p, q, 1e-3, "strided")


def test_argument_validation(fg):
    x = torch.zeros(4, 100, dtype=torch.bfloat16, device="cuda")       # K % 64 != 0
    with pytest.raises(fg.FgmpError) as e:
        fg.quantize_activations(x, torch.ones(100, device="cuda"), scale_fp4=1.0, tau=0.0)
    assert e.value.code == -2
    x = torch.zeros(4, 128, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(fg.FgmpError) as e:
        fg.quantize_activations(x, torch.ones(128, device="cuda"), scale_fp4=0.0, tau=0.0)
    assert e.value.code == -1
    with pytest.raises(fg.FgmpError) as e:
        fg.quantize_activations(x, torch.ones(128, device="cuda"), scale_fp4=1.0, tau=0.0,
                                out=torch.empty(2048, dtype=torch.uint8, device="cuda"))
    assert e.value.code in (-2, -3)


# ---------------------------------------------------------------------- weights

@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("clip", [False, True])
def test_weights_tiny_config(fg, mode, clip):
    wl = gi.tiny(0)
    w, fw = wl.w(), wl.fw()
    wb = gi.bf16_bits(w)
    for frac in (0.1, 0.0, 0.3, 1.0):
        q = oracle.quantize_weights(wb, fw.numpy(), clip=clip, mode=mode, fp8_fraction=frac)
        p = fg.quantize_weights(w.cuda(), fw.cuda(), clip_mode=int(clip), score_mode=mode, fp8_fraction=frac)
        compare_packed(fg, p, q, None, f"tiny clip={clip} mode={mode} frac={frac}")
        h = p.header()
        assert h["n_fp8"] == q.mask_bits().sum() == int(np.floor(frac * 4096 + 0.5))
        assert np.float32(h["scale_fp4"]) == np.float32(q.scale_fp4) and h["error"] == 0
        if 0 < frac:
            assert np.float32(h["tau_eff"]) == np.float32(q.tau_eff)
    # threshold mode with the oracle's effective threshold selects the strictly larger ones
    q = oracle.quantize_weights(wb, fw.numpy(), clip=clip, mode=mode, fp8_fraction=0.1)
    qt = oracle.quantize_weights(wb, fw.numpy(), clip=clip, mode=mode, fp8_fraction=-1.0, tau=q.tau_eff)
    pt = fg.quantize_weights(w.cuda(), fw.cuda(), clip_mode=int(clip), score_mode=mode, fp8_fraction=-1.0,
                             tau=q.tau_eff)
    compare_packed(fg, pt, qt, None, "threshold mode")
    # given tensor scale
    q = oracle.quantize_weights(wb, fw.numpy(), scale_fp4=3e-5, clip=clip, mode=mode, fp8_fraction=0.2)
    p = fg.quantize_weights(w.cuda(), fw.cuda(), scale_fp4=3e-5, clip_mode=int(clip), score_mode=mode, fp8_fraction=0.2)
    compare_packed(fg, p, q, None, "given scale")


def test_weights_ties_take_the_lower_block_index(fg):
    row = gi.weights(1, 64, 5)
    w = row.repeat(96, 1)                                   # every row identical -> massive ties
    w = torch.cat([w[:, :16]] * 4, dim=1).contiguous()      # and every block identical
    fw = torch.ones(96, 64)
    for frac in (0.37, 0.5, 0.011):
        q = oracle.quantize_weights(gi.bf16_bits(w), fw.numpy(), clip=False, fp8_fraction=frac)
        p = fg.quantize_weights(w.cuda(), fw.cuda(), clip_mode=0, fp8_fraction=frac)
        compare_packed(fg, p, q, None, f"ties frac={frac}")
        k = int(np.floor(frac * 96 * 4 + 0.5))
        assert q.mask_bits().ravel()[:k].all() and not q.mask_bits().ravel()[k:].any()


@pytest.mark.parametrize("N,K,clip", [(11008, 4096, False), (384, 4096, True), (200, 11008, True), (5120, 1024, False)])
def test_weights_llama_shapes(fg, N, K, clip):
    wl = gi.llama("w", 1, N, K, seed=1)
    w, fw = wl.w(), wl.fw()
    q = oracle.quantize_weights(gi.bf16_bits(w), fw.numpy(), clip=clip, fp8_fraction=0.1)
    p = fg.quantize_weights(w.cuda(), fw.cuda(), clip_mode=int(clip), fp8_fraction=0.1)
    compare_packed(fg, p, q, None, f"N={N} K={K}")
    assert p.header()["n_fp8"] == int(np.floor(0.1 * N * K / 16 + 0.5))


# ------------------------------------------------------------------------- GEMM

_last_weights = {}      # the most recent weight tensor, quantized on both sides (large shapes are reused across M)


def quantize_both(fg, wl, frac_a, frac_w, mode=0, clip=True):
    x, fx = wl.x(), wl.fx()
    s4 = gi.tensor_scale(x)
    xb = gi.bf16_bits(x)
    scores = oracle.quantize_activations(xb, fx.numpy(), s4, tau=np.inf, mode=mode).scores
    tau = tau_for_fraction(scores, frac_a)
    qa = oracle.quantize_activations(xb, fx.numpy(), s4, tau=tau, mode=mode)
    pa = fg.quantize_activations(x.cuda(), fx.cuda(), scale_fp4=s4, score_mode=mode, tau=tau)
    key = (wl.name, wl.N, wl.K, wl.seed, frac_w, mode, clip)
    if key not in _last_weights:
        _last_weights.clear()
        w, fw = wl.w(), wl.fw()
        qw = oracle.quantize_weights(gi.bf16_bits(w), fw.numpy(), clip=clip, mode=mode, fp8_fraction=frac_w)
        pw = fg.quantize_weights(w.cuda(), fw.cuda(), clip_mode=int(clip), score_mode=mode, fp8_fraction=frac_w)
        # the GEMM tests below must not be able to hide a wrong block inside their tolerance
        compare_packed(fg, pw, qw, None, f"weights of {wl.name}")
        _last_weights[key] = (qw, pw)
    qw, pw = _last_weights[key]
    compare_packed(fg, pa, qa, tau, f"activations of {wl.name}")
    return qa, qw, pa, pw


@pytest.mark.parametrize("frac_a,frac_w", [(0.1, 0.1), (0.0, 0.0), (1.0, 1.0), (0.0, 1.0), (1.0, 0.0), (0.3, 0.2)])
def test_linear_tiny_config(fg, frac_a, frac_w):
    wl = gi.tiny(0)
    qa, qw, pa, pw = quantize_both(fg, wl, frac_a, frac_w)
    Y, S = oracle.linear(qa, qw)
    y = fg.linear(pa, pw)
    fg.check(fg.linear.last_workspace)
    err = np.abs(y.cpu().numpy().astype(np.float64) - Y)
    assert (err <= GEMM_TOL * S + 1e-30).all(), f"max err/S = {(err / np.maximum(S, 1e-300)).max():.3e}"
    # the common-container path is exact up to fp32 accumulation: far inside the bar
    assert (err <= 1e-5 * S + 1e-30).all()
    # bf16 output: the oracle's value rounded to bf16, within one bf16 step plus the bar
    yb = fg.linear(pa, pw, out_dtype=torch.bfloat16).float().cpu().numpy().astype(np.float64)
    assert (np.abs(yb - Y) <= GEMM_TOL * S + np.abs(Y) * 2.0 ** -8 + 1e-30).all()


@pytest.mark.parametrize("M,N,K", [(1, 256, 256), (16, 11008, 4096), (77, 300, 1024), (129, 136, 64), (384, 1000, 2048)])
def test_linear_ragged_shapes(fg, M, N, K):
    wl = gi.llama("l", M, N, K, seed=2)
    qa, qw, pa, pw = quantize_both(fg, wl, 0.1, 0.1, clip=False)
    y = fg.linear(pa, pw).cpu().numpy().astype(np.float64)
    fg.check(fg.linear.last_workspace)
    rng = np.random.default_rng(0)
    ns = 4000
    ms = np.r_[rng.integers(0, M, ns), [0, M - 1, 0, M - 1]]
    nn = np.r_[rng.integers(0, N, ns), [0, N - 1, N - 1, 0]]
    Y, S = oracle.linear_sampled(qa, qw, ms, nn)
    err = np.abs(y[ms, nn] - Y)
    assert (err <= GEMM_TOL * S + 1e-30).all(), f"max err/S = {(err / np.maximum(S, 1e-300)).max():.3e}"
    assert np.isfinite(y).all()


def test_linear_prefill_shape_sampled(fg):
    """Llama-2-7B o_proj at M=4096 (one of the prefill benchmark shapes), sampled outputs."""
    wl = gi.llama("o_proj", 4096, 4096, 4096, seed=0)
    qa, qw, pa, pw = quantize_both(fg, wl, 0.1, 0.1, clip=False)
    y = fg.linear(pa, pw).cpu().numpy().astype(np.float64)
    fg.check(fg.linear.last_workspace)
    rng = np.random.default_rng(1)
    ms, nn = rng.integers(0, 4096, 3000), rng.integers(0, 4096, 3000)
    Y, S = oracle.linear_sampled(qa, qw, ms, nn)
    err = np.abs(y[ms, nn] - Y)
    assert (err <= GEMM_TOL * S + 1e-30).all(), f"max err/S = {(err / np.maximum(S, 1e-300)).max():.3e}"
    # two runs give the same bits
    y2 = fg.linear(pa, pw).cpu().numpy().astype(np.float64)
    assert np.array_equal(y, y2)


# ------------------------------------------------------------ decode kernel (M <= 16)

@pytest.mark.parametrize("frac_a,frac_w", [(0.0, 0.0), (0.1, 0.1), (0.0, 0.1), (0.1, 0.0), (1.0, 1.0), (0.0, 1.0),
                                            (1.0, 0.0), (0.3, 0.3)])
@pytest.mark.parametrize("M", [16, 5])
def test_decode_kernel_block_pair_cases(fg, M, frac_a, frac_w):
    """Weight-streaming path: every combination of block formats, full output against the oracle.
    30% FP8 exceeds the staged FP8 capacity of a pipeline stage and takes the global-memory route."""
    wl = gi.llama("d", M, 640, 1024, seed=11)
    qa, qw, pa, pw = quantize_both(fg, wl, frac_a, frac_w, clip=False)
    Y, S = oracle.linear(qa, qw)
    y = fg.linear(pa, pw)
    fg.check(fg.linear.last_workspace)
    err = np.abs(y.cpu().numpy().astype(np.float64) - Y)
    assert (err <= GEMM_TOL * S + 1e-30).all(), f"max err/S = {(err / np.maximum(S, 1e-300)).max():.3e}"
    assert (err <= 1e-5 * S + 1e-30).all(), f"max err/S = {(err / np.maximum(S, 1e-300)).max():.3e}"
    y2 = fg.linear(pa, pw)
    assert torch.equal(y, y2), "stream-K reduction must be deterministic"
    yb = fg.linear(pa, pw, out_dtype=torch.bfloat16).float().cpu().numpy().astype(np.float64)
    assert (np.abs(yb - Y) <= GEMM_TOL * S + np.abs(Y) * 2.0 ** -8 + 1e-30).all()


@pytest.mark.parametrize("M,N,K", [(1, 11008, 4096), (16, 4096, 11008), (8, 300, 256), (2, 129, 5120), (16, 13824, 5120)])
def test_decode_kernel_shapes(fg, M, N, K):
    wl = gi.llama("d", M, N, K, seed=4)
    qa, qw, pa, pw = quantize_both(fg, wl, 0.1, 0.1, clip=False)
    y = fg.linear(pa, pw).cpu().numpy().astype(np.float64)
    fg.check(fg.linear.last_workspace)
    rng = np.random.default_rng(0)
    ms = np.r_[rng.integers(0, M, 6000), [0, M - 1, 0, M - 1]]
    nn = np.r_[rng.integers(0, N, 6000), [0, N - 1, N - 1, 0]]
    Y, S = oracle.linear_sampled(qa, qw, ms, nn)
    err = np.abs(y[ms, nn] - Y)
    assert (err <= GEMM_TOL * S + 1e-30).all(), f"max err/S = {(err / np.maximum(S, 1e-300)).max():.3e}"
    assert np.isfinite(y).all()


def test_decode_workspace_is_left_clear_for_the_next_call(fg):
    """One workspace, cleared once, serves calls of different shapes back to back (the tile counters
    reset themselves); every result equals that of a call with a fresh workspace and the oracle."""
    shapes = [(16, 640, 1024), (5, 1408, 512), (16, 640, 1024), (1, 300, 2048)]
    big = max(fg.workspace_bytes(fg.binding.OP_LINEAR, M, N, K) for M, N, K in shapes)
    ws = fg.workspace_init(fg.binding._alloc_aligned(big, torch.device("cuda")))
    for i, (M, N, K) in enumerate(shapes):
        wl = gi.llama("d", M, N, K, seed=20 + i)
        qa, qw, pa, pw = quantize_both(fg, wl, 0.1, 0.1, clip=False)
        Y, S = oracle.linear(qa, qw)
        y_shared = fg.linear(pa, pw, workspace=ws)
        fg.check(ws)
        y_fresh = fg.linear(pa, pw)
        assert torch.equal(y_shared, y_fresh), f"call {i}: a reused workspace changed the result"
        err = np.abs(y_shared.cpu().numpy().astype(np.float64) - Y)
        assert (err <= 1e-5 * S + 1e-30).all()
    # the control area is zero again
    assert int(ws[: 1024 + 32 * 16].to(torch.int32).abs().sum().item()) == 0


def test_prefill_call_between_decode_calls_on_one_workspace(fg):
    """A prefill-shaped call keeps its scratch behind the control area, so decode-shaped calls before and
    after it on the same workspace (cleared once) still find their tile counters at zero."""
    shapes = [(16, 640, 1024), (77, 300, 1024), (16, 640, 1024), (200, 256, 512), (3, 1408, 512)]
    big = max(fg.workspace_bytes(fg.binding.OP_LINEAR, M, N, K) for M, N, K in shapes)
    ws = fg.workspace_init(fg.binding._alloc_aligned(big, torch.device("cuda")))
    for i, (M, N, K) in enumerate(shapes):
        wl = gi.llama("d", M, N, K, seed=40 + i)
        qa, qw, pa, pw = quantize_both(fg, wl, 0.1, 0.1, clip=False)
        Y, S = oracle.linear(qa, qw)
        y_shared = fg.linear(pa, pw, workspace=ws)
        fg.check(ws)
        assert torch.equal(y_shared, fg.linear(pa, pw)), f"call {i}: a reused workspace changed the result"
        err = np.abs(y_shared.cpu().numpy().astype(np.float64) - Y)
        assert (err <= 1e-5 * S + 1e-30).all(), f"call {i}"
    assert int(ws[: 65536].to(torch.int32).abs().sum().item()) == 0


# ------------------------------------------------------------ quantizer + GEMM in one launch

@pytest.mark.parametrize("M,N,K,mode", [(16, 640, 1024, 0), (5, 1408, 512, 1), (1, 300, 2048, 0), (9, 129, 256, 0),
                                        (16, 11008, 4096, 0), (8, 4096, 11008, 1), (16, 1000, 7424, 0)])
def test_fused_decode_step_equals_the_two_calls_and_the_oracle(fg, M, N, K, mode):
    """fgmp_linear_fused: packed activations bit-equal to the oracle's (and so to fgmp_quantize_activations'),
    Y bit-equal to fgmp_linear on them and within the bar of the oracle; twice on one workspace."""
    wl = gi.llama("f", M, N, K, seed=60 + M)
    qa, qw, pa, pw = quantize_both(fg, wl, 0.1, 0.1, mode=mode, clip=False)
    x, fx = wl.x(), wl.fx()
    s4 = gi.tensor_scale(x)
    tau = tau_for_fraction(qa.scores, 0.1)
    ws = fg.alloc_workspace(fg.binding.OP_LINEAR_FUSED, M, N, K, torch.device("cuda"))
    y_two = fg.linear(pa, pw)
    for rep in range(2):
        y, pf = fg.linear_fused(x.cuda(), fx.cuda(), pw, scale_fp4=s4, score_mode=mode, tau=tau, want_packed=True, workspace=ws)
        fg.check(ws)
        compare_packed(fg, pf, qa, tau, f"fused rep {rep}")
        assert torch.equal(y, y_two), f"rep {rep}: fused Y differs from the two calls"
    # without the packed output (records in the workspace only)
    y3 = fg.linear_fused(x.cuda(), fx.cuda(), pw, scale_fp4=s4, score_mode=mode, tau=tau, workspace=ws)
    fg.check(ws)
    assert torch.equal(y3, y_two)
    rng = np.random.default_rng(0)
    ms = np.r_[rng.integers(0, M, 3000), [0, M - 1, 0, M - 1]]
    nn = np.r_[rng.integers(0, N, 3000), [0, N - 1, N - 1, 0]]
    Y, S = oracle.linear_sampled(qa, qw, ms, nn)
    err = np.abs(y3.cpu().numpy().astype(np.float64)[ms, nn] - Y)
    assert (err <= 1e-5 * S + 1e-30).all(), f"max err/S = {(err / np.maximum(S, 1e-300)).max():.3e}"
    # a plain fgmp_linear on the same workspace afterwards still works (control area as it expects)
    assert torch.equal(fg.linear(pa, pw, workspace=ws), y_two)
    fg.check(ws)


@pytest.mark.parametrize("M,N,K,mode,frac", [(40, 300, 512, 0, 0.1), (333, 520, 1024, 1, 0.1), (130, 136, 320, 0, 1.0),
                                             (12, 300, 320, 0, 0.1), (200, 392, 512, 0, 0.0)])
def test_fused_step_for_a_prefill_sized_batch(fg, M, N, K, mode, frac):
    """Beyond the decode kernel's shapes the fused call runs the two calls: packed activations bit for bit as the
    oracle's, Y bit for bit as the two calls give (all-FP8, mixed, and the all-NVFP4 operands that take the FP4
    tensor-core kernel)."""
    wl = gi.llama("f", M, N, K, seed=70)
    qa, qw, pa, pw = quantize_both(fg, wl, frac, frac, mode=mode, clip=False)
    x, fx = wl.x(), wl.fx()
    s4 = gi.tensor_scale(x)
    tau = tau_for_fraction(qa.scores, frac)
    y, pf = fg.linear_fused(x.cuda(), fx.cuda(), pw, scale_fp4=s4, score_mode=mode, tau=tau, want_packed=True)
    fg.check(fg.linear.last_workspace)
    compare_packed(fg, pf, qa, tau, "fused prefill-sized")
    assert torch.equal(y, fg.linear(pa, pw))
    Y, S = oracle.linear(qa, qw)
    assert (np.abs(y.cpu().numpy().astype(np.float64) - Y) <= 1e-5 * S + 1e-30).all()


def test_weight_blob_that_does_not_match_the_call_is_refused_on_the_device(fg):
    """Threshold mode with too little room: the packer flags the blob, fgmp_unpack refuses it, and fgmp_linear
    reads none of it (status FGMP_ERR_INVALID_ARG) -- on both GEMM paths.  So does a blob of another shape."""
    wl = gi.llama("cap", 16, 640, 1024, seed=5)
    w, fw = wl.w(), wl.fw()
    qa, qw, pa, pw_ok = quantize_both(fg, wl, 0.1, 0.1, clip=False)
    pw = fg.quantize_weights(w.cuda(), fw.cuda(), clip_mode=0, fp8_fraction=-1.0, tau=0.0, max_fp8_blocks=100)
    assert pw.header()["error"] == -7
    with pytest.raises(fg.FgmpError):
        fg.unpack(pw)
    y = fg.linear(pa, pw)
    with pytest.raises(fg.FgmpError) as e:
        fg.check(fg.linear.last_workspace)
    assert e.value.code == -1
    # a blob packed for another N
    other = fg.quantize_weights(wl.w()[:512].contiguous().cuda(), fw[:512].contiguous().cuda(), clip_mode=0, fp8_fraction=0.1)
    other.rows = 640                                           # the caller claims a shape the blob does not have
    big = fg.binding._alloc_aligned(pw_ok.blob.numel(), torch.device("cuda"))
    big[: other.blob.numel()] = other.blob                     # inside an allocation large enough for the claimed shape
    other.blob = big
    fg.linear(pa, other)
    with pytest.raises(fg.FgmpError) as e:
        fg.check(fg.linear.last_workspace)
    assert e.value.code == -1
    # the good blob still works afterwards
    y = fg.linear(pa, pw_ok)
    fg.check(fg.linear.last_workspace)


@pytest.mark.parametrize("kind", [0, 1, 2, 4, 5, 6])
def test_tensor_peak_loop_runs(fg, kind):
    """Kinds 0-2: one CTA per SM; kinds 4-6: the same operand kinds on CTA pairs (cta_group::2)."""
    ws = fg.binding._alloc_aligned(1024, torch.device("cuda"))
    ws.zero_()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    fg.tensor_peak(kind, 1000, ws)
    e0.record()
    fg.tensor_peak(kind, 50000, ws)
    e1.record()
    torch.cuda.synchronize()
    fg.check(ws)
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    if kind >= 4:
        sms, kind = (sms // 2) * 2, kind - 4
    tflops = 2.0 * 128 * 256 * (16, 32, 64)[kind] * 50000 * sms / (e0.elapsed_time(e1) * 1e-3) / 1e12
    # far below the rate means the loop did not run on the tensor cores, far above that it did not run at all
    assert 0.3 * (2250, 4500, 9000)[kind] < tflops < 1.05 * (2250, 4500, 9000)[kind], tflops


def _sampled_linear_check(fg, wl, frac, n_samples, seed):
    qa, qw, pa, pw = quantize_both(fg, wl, frac, frac, clip=False)
    M, N = qa.rows, qw.rows
    y = fg.linear(pa, pw).cpu().numpy().astype(np.float64)
    fg.check(fg.linear.last_workspace)
    rng = np.random.default_rng(seed)
    ms = np.r_[rng.integers(0, M, n_samples), [0, M - 1, 0, M - 1]]
    nn = np.r_[rng.integers(0, N, n_samples), [0, N - 1, N - 1, 0]]
    Y, S = oracle.linear_sampled(qa, qw, ms, nn)
    err = np.abs(y[ms, nn] - Y)
    assert (err <= GEMM_TOL * S + 1e-30).all(), f"max err/S = {(err / np.maximum(S, 1e-300)).max():.3e}"
    assert np.isfinite(y).all()
    # packed size against the closed form: blocks * [(1 - p) * 9 + p * 16] bytes of codes and scales
    blocks = N * qw.K // 16
    n8 = int(qw.mask_bits().sum())
    assert n8 == int(np.floor(frac * blocks + 0.5))


@pytest.mark.parametrize("frac", [0.0, 0.2, 0.3])
def test_linear_llama2_13b_fc1_fraction_sweep_sampled(fg, frac):
    """Llama-2-13B FC1 (13824 x 5120) at M = 2048 with 0 / 20 / 30 % of the blocks of both operands in FP8
    (10 % is the setting of every other test): sampled outputs against the oracle."""
    _sampled_linear_check(fg, gi.llama("fc1_13b", 2048, 13824, 5120, seed=5), frac, 2500, 2)


@pytest.mark.parametrize("M", [1, 16])
def test_decode_llama2_70b_fc1_sampled(fg, M):
    """Llama-2-70B FC1 (28672 x 8192), the largest decode shape that is benchmarked: sampled outputs."""
    _sampled_linear_check(fg, gi.llama("fc1_70b", M, 28672, 8192, seed=6), 0.1, 4000, 3)


def test_decode_llama2_70b_fc2_sampled(fg):
    """The K of Llama-2-70B FC2 (28672: 112 chunks per tile, every tile shared by several thread blocks) with
    1024 of its 8192 output rows."""
    _sampled_linear_check(fg, gi.llama("fc2_70b", 16, 1024, 28672, seed=7), 0.1, 4000, 4)


# ------------------------------------------------------------ global threshold (Eq. 10)

def test_global_threshold_over_several_tensors(fg):
    """One tau for two weight tensors and one for two activation batches: GPU scores equal the oracle's bit
    for bit, the pooled threshold equals the oracle's, and packing with it gives each tensor exactly the
    blocks whose score exceeds it (their total is the budget; the per-tensor shares differ)."""
    wls = [gi.llama("g0", 48, 384, 1024, seed=31), gi.llama("g1", 32, 256, 2048, seed=32)]
    frac = 0.1
    # weights
    ws_gpu, ws_cpu, fws = [], [], []
    for i, wl in enumerate(wls):
        w, fw = wl.w(), wl.fw() * (1.0 if i == 0 else 6.0)          # the second tensor is the more sensitive one
        fws.append(fw)
        ws_gpu.append(fg.weight_scores(w.cuda(), fw.cuda(), clip_mode=1))
        q = oracle.quantize_weights(gi.bf16_bits(w), fw.numpy(), clip=True, mode=0, fp8_fraction=0.0)
        ws_cpu.append(q.scores)
        assert np.array_equal(ws_gpu[-1].cpu().numpy().ravel().view(np.uint32), q.scores.view(np.uint32))
    tau_w = oracle.global_threshold(ws_cpu, frac)
    tau_w_gpu = float(fg.global_tau(ws_gpu, frac).item())
    assert np.float32(tau_w_gpu) == np.float32(tau_w)
    total8 = 0
    shares = []
    for wl, fw, sc in zip(wls, fws, ws_cpu):
        w = wl.w()
        q = oracle.quantize_weights(gi.bf16_bits(w), fw.numpy(), clip=True, mode=0, fp8_fraction=-1.0, tau=tau_w)
        pw = fg.quantize_weights(w.cuda(), fw.cuda(), clip_mode=1, fp8_fraction=-1.0, tau=tau_w_gpu)
        compare_packed(fg, pw, q, tau=tau_w, what=wl.name)
        n8 = int(q.mask_bits().sum())
        assert n8 == int((sc > np.float32(tau_w)).sum())
        total8 += n8
        shares.append(n8 / sc.size)
    B = sum(s.size for s in ws_cpu)
    assert total8 == int(np.floor(frac * B + 0.5))
    assert shares[1] > frac > shares[0]
    # activations
    xs_gpu, xs_cpu = [], []
    for wl in wls:
        x, fx = wl.x(), wl.fx()
        s4 = gi.tensor_scale(x)
        xs_gpu.append(fg.activation_scores(x.cuda(), fx.cuda(), scale_fp4=s4))
        xs_cpu.append(oracle.quantize_activations(gi.bf16_bits(x), fx.numpy(), s4, tau=np.inf).scores)
    tau_a = oracle.global_threshold(xs_cpu, frac)
    assert np.float32(float(fg.global_tau(xs_gpu, frac).item())) == np.float32(tau_a)
    for f, want in ((0.0, float("inf")), (1.0, -1.0)):
        assert float(fg.global_tau(xs_gpu, f).item()) == want


# ------------------------------------------------------------ baseline policies (Eq. 12, 13)

def test_baseline_policies_as_weight_substitutions(fg):
    """Quantization Error (ones as sensitivity weights) and Output Error (mean squared channel magnitude of
    the other operand, computed on the GPU) run through the same kernels: packed tensors equal the oracle's."""
    wl = gi.llama("pol", 40, 256, 1024, seed=41)
    x, w = wl.x(), wl.w()
    xb, wb = gi.bf16_bits(x), gi.bf16_bits(w)
    s4 = gi.tensor_scale(x)
    # Output Error weights: bit-exact against the oracle
    ax_cpu, aw_cpu = oracle.channel_mean_sq(xb), oracle.channel_mean_sq(wb)
    ax_gpu, aw_gpu = fg.channel_mean_sq(x.cuda()), fg.channel_mean_sq(w.cuda())
    assert np.array_equal(ax_gpu.cpu().numpy().view(np.uint32), ax_cpu.view(np.uint32))
    assert np.array_equal(aw_gpu.cpu().numpy().view(np.uint32), aw_cpu.view(np.uint32))
    ones_k = torch.ones(wl.K, dtype=torch.float32)
    for name, fa, fwv in (("QE", ones_k, ones_k), ("OE", torch.from_numpy(aw_cpu), torch.from_numpy(ax_cpu))):
        fwm = fwv.expand(wl.N, wl.K).contiguous()
        # weights: local threshold = fraction mode
        qw = oracle.quantize_weights(wb, fwm.numpy(), clip=False, mode=1, fp8_fraction=0.1)
        pw = fg.quantize_weights(w.cuda(), fwm.cuda(), clip_mode=0, score_mode=1, fp8_fraction=0.1)
        compare_packed(fg, pw, qw, what=name + " weights")
        # activations: threshold from this batch's own scores
        scores = oracle.quantize_activations(xb, fa.numpy(), s4, tau=np.inf, mode=1).scores
        tau = tau_for_fraction(scores, 0.1)
        qa = oracle.quantize_activations(xb, fa.numpy(), s4, tau=tau, mode=1)
        pa = fg.quantize_activations(x.cuda(), fa.cuda(), scale_fp4=s4, score_mode=1, tau=tau)
        compare_packed(fg, pa, qa, tau=tau, what=name + " activations")
        assert qa.mask_bits().sum() == int(np.floor(0.1 * scores.size + 0.5))


# ------------------------------------------------------------ quantizer in the GEMM's epilogue (Section 4.2)

@pytest.mark.parametrize("M,N,K,mode", [(300, 1024, 512, 0), (4096, 4096, 1024, 0), (77, 320, 256, 1), (2048, 11008, 256, 0),
                                         (16, 1024, 512, 0), (5, 320, 256, 1), (8, 192, 320, 0)])
def test_linear_with_next_layer_quantizer_in_the_epilogue(fg, M, N, K, mode):
    """fgmp_linear_quantize against the two calls it fuses (bit for bit) and against the oracle's quantizer
    run on the same bf16 outputs; the bf16 outputs themselves against the oracle's GEMM."""
    wl = gi.llama("fuse", M, N, K, seed=51)
    qa, qw, pa, pw = quantize_both(fg, wl, 0.1, 0.1, clip=False)
    y16 = fg.linear(pa, pw, out_dtype=torch.bfloat16)
    fg.check(fg.linear.last_workspace)
    # next layer's calibrated constants: sensitivity per output channel, tensor scale, threshold for 10 % FP8
    g = torch.Generator().manual_seed(7)
    f_next = torch.exp(1.5 * torch.randn(N, generator=g)).float()
    s4n = gi.tensor_scale(y16.float().cpu())
    yb = gi.bf16_bits(y16.cpu())
    scores = oracle.quantize_activations(yb, f_next.numpy(), s4n, tau=np.inf, mode=mode).scores
    tau = tau_for_fraction(scores, 0.1)
    q_ref = oracle.quantize_activations(yb, f_next.numpy(), s4n, tau=tau, mode=mode)
    fused = fg.linear_quantize(pa, pw, f_next.cuda(), scale_fp4=s4n, score_mode=mode, tau=tau)
    fg.check(fg.linear.last_workspace)
    two_step = fg.quantize_activations(y16, f_next.cuda(), scale_fp4=s4n, score_mode=mode, tau=tau)
    for a, b in zip(fg.unpack(fused), fg.unpack(two_step)):
        assert torch.equal(a, b), "the fused epilogue and the two separate calls must agree bit for bit"
    compare_packed(fg, fused, q_ref, tau=tau, what="epilogue quantizer")
    assert int(q_ref.mask_bits().sum()) == int(np.floor(0.1 * scores.size + 0.5))
    # and the GEMM outputs that were quantized are the oracle's, within the bar (bf16 output)
    rng = np.random.default_rng(3)
    ms, nn = rng.integers(0, M, 2000), rng.integers(0, N, 2000)
    Y, S = oracle.linear_sampled(qa, qw, ms, nn)
    got = y16.float().cpu().numpy().astype(np.float64)[ms, nn]
    assert (np.abs(got - Y) <= GEMM_TOL * S + np.abs(Y) * 2.0 ** -8 + 1e-30).all()


def test_bounded_wait_runs_out_and_the_workspace_recovers(fg):
    """The failure path of the kernels' waits, made to happen safely: one thread block waits 1 ms for a barrier
    that nothing completes; the status word then says FGMP_ERR_TIMEOUT, clearing the workspace removes it, and
    the same workspace serves a correct fgmp_linear afterwards."""
    M, N, K = 16, 640, 1024
    wl = gi.llama("d", M, N, K, seed=11)
    qa, qw, pa, pw = quantize_both(fg, wl, 0.1, 0.1, clip=False)
    ws = fg.alloc_workspace(fg.binding.OP_LINEAR, M, N, K, torch.device("cuda"))
    y0 = fg.linear(pa, pw, workspace=ws)
    fg.check(ws)
    fg.selftest_wait_timeout(ws, 1_000_000)
    with pytest.raises(fg.FgmpError) as e:
        fg.check(ws)
    assert e.value.code == -6 and "timed out" in str(e.value)
    fg.workspace_init(ws)
    fg.check(ws)
    assert torch.equal(fg.linear(pa, pw, workspace=ws), y0)
    fg.check(ws)
