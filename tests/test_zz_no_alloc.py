"""fgmp_linear_static: the decode-sized GEMM whose scratch lives inside the library, for
callers that cannot allocate device memory (no cudaMalloc allowed where they run, or no way to
pass a workspace).  Checked through the C ABI against fgmp_linear, the entry point that takes a
caller-provided workspace, and against the CPU oracle, on two calls in a row that share the
built-in scratch: the second call uses another shape, so whatever the first call left behind
(tile counters, partial sums) must not leak into it.

Collected last on purpose: a failure here cannot hide the result of any other test.
"""
import numpy as np
import pytest
import torch

import fgmp_inputs as gi
import oracle

pytestmark = pytest.mark.gpu

GEMM_TOL = 2e-3


def _case(fg, M, N, K, seed):
    wl = gi.llama("static", M, N, K, seed=seed)
    x, w, fx, fw = wl.x(), wl.w(), wl.fx(), wl.fw()
    s4 = gi.tensor_scale(x)
    xb, wb = gi.bf16_bits(x), gi.bf16_bits(w)
    scores = oracle.quantize_activations(xb, fx.numpy(), s4, tau=np.inf).scores
    srt = np.sort(scores.ravel())[::-1]
    k = int(np.floor(0.1 * scores.size + 0.5))
    tau = float(np.float32(0.5) * (srt[k - 1] + srt[k]))
    qa = oracle.quantize_activations(xb, fx.numpy(), s4, tau=tau)
    qw = oracle.quantize_weights(wb, fw.numpy(), clip=False, fp8_fraction=0.1)
    pa = fg.quantize_activations(x.cuda(), fx.cuda(), scale_fp4=s4, tau=tau)
    pw = fg.quantize_weights(w.cuda(), fw.cuda(), clip_mode=0, fp8_fraction=0.1)
    Y, S = oracle.linear(qa, qw)
    return pa, pw, Y, S


def test_static_scratch_variant_matches_fgmp_linear_on_two_calls_in_a_row():
    import paper_2504_14152_b200 as fg
    assert torch.cuda.is_available()
    cases = [_case(fg, 16, 1152, 2048, seed=21), _case(fg, 5, 640, 1024, seed=22)]
    outs = []
    status = torch.full((2,), -99, dtype=torch.int32, device="cuda")
    # both calls are enqueued back to back on one stream before anything is read back
    for pa, pw, _, _ in cases:
        y = torch.empty(pa.rows, pw.rows, dtype=torch.float32, device="cuda")
        outs.append(fg.linear_static(pa, pw, out=y, status_out=status))
    torch.cuda.synchronize()
    assert status.tolist() == [0, 0]
    for (pa, pw, Y, S), y in zip(cases, outs):
        y_ref = fg.linear(pa, pw)                       # caller-provided workspace
        fg.check(fg.linear.last_workspace)
        got = y.cpu().numpy().astype(np.float64)
        ref = y_ref.cpu().numpy().astype(np.float64)
        assert (np.abs(got - ref) <= GEMM_TOL * S + 1e-30).all()
        assert (np.abs(got - Y) <= GEMM_TOL * S + 1e-30).all()
        assert np.array_equal(got, ref), "same kernel, same reduction order: bits must agree"


def test_static_scratch_variant_rejects_what_does_not_fit():
    import paper_2504_14152_b200 as fg
    import paper_2504_14152_b200.binding as b
    L = b._load()
    fake = 0x10000 * 1024
    # prefill-sized M and K % 256 != 0 are not decode shapes
    assert L.fgmp_linear_static(fake, fake, fake, 0, 4096, 17, 4096, 4096, None, None) == -2
    assert L.fgmp_linear_static(fake, fake, fake, 0, 4096, 16, 4096, 4096 + 64, None, None) == -2
    # a shape whose scratch need exceeds the built-in array
    N, K = 200000, 4096
    assert fg.workspace_bytes(b.OP_LINEAR, 16, N, K) > fg.STATIC_SCRATCH_BYTES
    assert L.fgmp_linear_static(fake, fake, fake, 0, N, 16, N, K, None, None) == -3
    # Llama-2-70B FC1 fits
    assert fg.workspace_bytes(b.OP_LINEAR, 16, 28672, 8192) <= fg.STATIC_SCRATCH_BYTES
