"""Pins for the oracle's quantizers, clip search, selection and GEMM (CPU only).

Each check compares the oracle with something that is not the oracle: brute force in
fp64 numpy, closed forms, invariants fixed by the paper, library routines.
"""
import os

import numpy as np
import torch

import fgmp_inputs as gi
import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
E2M1 = np.array([0, 0.5, 1, 1.5, 2, 3, 4, 6, -0.0, -0.5, -1, -1.5, -2, -3, -4, -6])


def _e4m3_vals():
    return torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).to(torch.float64).numpy()


def _bf16_to_f32(bits):
    return (bits.astype(np.uint32) << 16).view(np.float32)


def _tiny():
    wl = gi.tiny(0)
    x, w = wl.x(), wl.w()
    return wl, x, w, wl.fx().numpy(), wl.fw().numpy()


def _unpack4(q):
    c = q.codes4.reshape(q.rows, q.K // 2)
    out = np.empty((q.rows, q.K), np.int64)
    out[:, 0::2] = c & 15
    out[:, 1::2] = c >> 4
    return out


def _tau_for_fraction(scores, frac):
    k = int(np.floor(frac * scores.size + 0.5))
    s = np.sort(scores.ravel())[::-1]
    # midway between the k-th and (k+1)-th largest so that exactly k blocks exceed it
    return float((np.float64(s[k - 1]) + np.float64(s[k])) / 2), k


# ----------------------------------------------------------------- activations

def test_activation_blocks_are_nearest_in_value_space():
    """NVFP4 codes minimise |x/d - g| over the grid (brute force, fp64); the scale is the
    E4M3 nearest to amax/(6 s4); FP8 codes are nearest to x/s8."""
    wl, x, _, fx, _ = _tiny()
    s4 = gi.tensor_scale(x)
    q = oracle.quantize_activations(gi.bf16_bits(x), fx, s4, tau=-1.0, mode=0)  # all FP8 written
    q4 = oracle.quantize_activations(gi.bf16_bits(x), fx, s4, tau=np.inf, mode=0)  # all FP4 written
    xv = _bf16_to_f32(gi.bf16_bits(x)).astype(np.float64)
    e4 = _e4m3_vals()
    KB = wl.K // 16
    sc = q4.scales.reshape(wl.M, KB)
    # scale: nearest positive E4M3 to amax / (6 s4) (fp32 product with k6, so allow the
    # neighbour when the exact ratio sits within 1e-6 of a midpoint)
    amax = np.abs(xv).reshape(wl.M, KB, 16).max(-1)
    target = amax / (6.0 * np.float32(s4))
    pos = e4[:0x7F]
    near = np.abs(target[..., None] - pos[None, None, :]).argmin(-1)
    d_near = np.abs(target - pos[near])
    d_got = np.abs(target - pos[sc])
    assert np.all(d_got <= d_near * (1 + 1e-5) + 1e-12)
    # elements: chosen code is a nearest grid point of x / d
    d = (e4[sc].astype(np.float32) * np.float32(s4)).astype(np.float64)
    y = xv.reshape(wl.M, KB, 16) / np.where(d == 0, 1, d)[..., None]
    codes = _unpack4(q4).reshape(wl.M, KB, 16)
    err_got = np.abs(y - E2M1[codes])
    err_best = np.abs(y[..., None] - E2M1[None, None, None, :]).min(-1)
    ok = (err_got <= err_best + 1e-5 * np.abs(y) + 1e-12) | (d == 0)[..., None]
    assert ok.all()
    # the block's largest element lands on the top two magnitudes (or saturates)
    top = np.abs(E2M1[codes]).max(-1)
    assert np.all((top >= 4) | (amax == 0) | (sc == 0))
    # FP8 codes
    s8 = np.float64(np.float32(s4)) * 8
    y8 = xv / s8
    c8 = q.codes8.reshape(wl.M, wl.K)
    err8 = np.abs(y8 - e4[c8])
    finite = e4[np.r_[0:0x7F, 0x80:0xFF]]
    best8 = np.abs(y8[..., None] - finite[None, None, :]).min(-1)
    assert np.all(err8 <= best8 + 1e-5 * np.abs(y8) + 1e-12)


def test_activation_score_is_eq6_and_eq8_in_fp64():
    wl, x, _, fx, _ = _tiny()
    s4 = gi.tensor_scale(x)
    e4 = _e4m3_vals()
    xv = _bf16_to_f32(gi.bf16_bits(x)).astype(np.float64)
    qa = oracle.quantize_activations(gi.bf16_bits(x), fx, s4, tau=np.inf, mode=0)
    qb = oracle.quantize_activations(gi.bf16_bits(x), fx, s4, tau=-1.0, mode=1)
    dq4 = oracle.decode(qa)
    dq8 = oracle.decode(qb)
    f = fx.astype(np.float64)
    want0 = (f[None, :] * (xv - dq4) ** 2).reshape(wl.M, -1, 16).sum(-1)
    want1 = (f[None, :] * (dq4 - dq8) ** 2).reshape(wl.M, -1, 16).sum(-1)
    got0 = qa.scores.reshape(wl.M, -1)
    got1 = qb.scores.reshape(wl.M, -1)
    assert np.allclose(got0, want0, rtol=2e-5, atol=0)
    assert np.allclose(got1, want1, rtol=2e-5, atol=0)
    assert (got0 >= 0).all() and (got1 >= 0).all()
    # linear in the Fisher weights; f = 1 is the unweighted "quantization error" policy (Eq. 12)
    q2 = oracle.quantize_activations(gi.bf16_bits(x), 2 * fx, s4, tau=np.inf, mode=0)
    assert np.array_equal(q2.scores, 2 * qa.scores)
    q1 = oracle.quantize_activations(gi.bf16_bits(x), np.ones_like(fx), s4, tau=np.inf, mode=1)
    want_qe = ((dq4 - dq8) ** 2).reshape(wl.M, -1, 16).sum(-1)
    assert np.allclose(q1.scores.reshape(wl.M, -1), want_qe, rtol=2e-5)


def test_activation_threshold_rule_and_extremes():
    wl, x, _, fx, _ = _tiny()
    s4 = gi.tensor_scale(x)
    xb = gi.bf16_bits(x)
    q_inf = oracle.quantize_activations(xb, fx, s4, tau=np.inf)
    assert not q_inf.mask_bits().any() and not q_inf.codes8.any()
    q_neg = oracle.quantize_activations(xb, fx, s4, tau=-1.0)
    assert q_neg.mask_bits().all() and not q_neg.codes4.any() and not q_neg.scales.any()
    tau, k = _tau_for_fraction(q_inf.scores, wl.fp8_fraction)
    q = oracle.quantize_activations(xb, fx, s4, tau=tau)
    mb = q.mask_bits()
    assert mb.sum() == k
    assert np.array_equal(mb.ravel(), q.scores > np.float32(tau))      # strict ">"
    # exactly at the threshold a block stays FP4
    s_k = np.sort(q.scores)[::-1][k - 1]
    q_eq = oracle.quantize_activations(xb, fx, s4, tau=float(s_k))
    assert q_eq.mask_bits().sum() == (q.scores > s_k).sum() < k + 1
    # FP4 blocks carry no FP8 codes and vice versa
    c8 = q.codes8.reshape(wl.M, -1, 16)
    c4 = q.codes4.reshape(wl.M, -1, 8)
    assert not c8[~mb].any() and not c4[mb].any() and not q.scales.reshape(wl.M, -1)[mb].any()
    # the outlier channels dominate: FP8 blocks concentrate in few column blocks
    assert mb.sum(0).max() >= wl.M // 2


def test_exactly_representable_block_has_zero_error():
    """Values that sit on the E2M1 grid times a representable scale quantize without error."""
    s4 = 2.0 ** -8
    scale_code = 0x38           # E4M3 value 1.0
    grid = np.array([0, .5, 1, 1.5, 2, 3, 4, 6, -6, -4, -3, -2, -1.5, -1, -.5, 6], np.float32)
    v = (grid * np.float32(oracle.e4m3_value(scale_code)) * np.float32(s4)).astype(np.float32)
    xb = (v.view(np.uint32) >> 16).astype(np.uint16).reshape(1, 16)
    assert np.array_equal(_bf16_to_f32(xb).ravel(), v)
    f = np.linspace(0.5, 2, 16).astype(np.float32)
    q = oracle.quantize_activations(xb, f, s4, tau=np.inf, mode=0)
    assert q.scales[0] == scale_code and q.scores[0] == 0.0
    assert np.array_equal(oracle.decode(q).ravel(), v.astype(np.float64))
    assert oracle.clip_search(v, f, s4) == scale_code
    # mode 1: FP8 also represents these values exactly -> the HP->LP score is zero too
    q1 = oracle.quantize_activations(xb, f, s4, tau=np.inf, mode=1)
    assert q1.scores[0] == 0.0


def test_zero_block():
    xb = np.zeros((1, 16), np.uint16)
    xb[0, 3] = 0x8000        # -0.0
    q = oracle.quantize_activations(xb, np.ones(16, np.float32), 0.01, tau=np.inf)
    assert q.scales[0] == 0 and q.scores[0] == 0
    assert q.codes4[1] == 0x80 and not np.delete(q.codes4, 1).any()


# --------------------------------------------------------------------- weights

def _objective_fp64(v, f, c, s4, e4):
    d = np.float32(e4[c]) * np.float32(s4)
    if d == 0:
        dq = np.zeros(16)
    else:
        inv = np.float32(1.0) / d
        y = (v * inv).astype(np.float32)
        codes = [oracle.e2m1_encode(float(t)) for t in y]
        dq = E2M1[codes] * np.float64(d)
    return float((f.astype(np.float64) * (dq - v.astype(np.float64)) ** 2).sum())


def test_clip_search_is_the_brute_force_minimum():
    wl, _, w, _, fw = _tiny()
    e4 = _e4m3_vals()
    s4 = gi.tensor_scale(w)
    wv = _bf16_to_f32(gi.bf16_bits(w))
    rng = np.random.default_rng(0)
    for _ in range(40):
        n, kb = rng.integers(wl.N), rng.integers(wl.K // 16)
        v = wv[n, kb * 16:(kb + 1) * 16]
        f = fw[n, kb * 16:(kb + 1) * 16]
        c = oracle.clip_search(v, f, s4)
        J = np.array([_objective_fp64(v, f, cc, s4, e4) for cc in range(0x7F)])
        assert J[c] <= J[1:].min() * (1 + 1e-5)
        # never worse than dynamic max; oracle objective agrees with fp64
        q = oracle.quantize_weights(gi.bf16_bits(w)[n:n + 1, kb * 16:(kb + 1) * 16].copy(),
                                    f.reshape(1, 16), scale_fp4=s4, clip=False, fp8_fraction=0.0)
        c0 = int(q.scales[0])
        assert J[c] <= J[c0] * (1 + 1e-6)
        assert np.isclose(oracle.clip_objective(v, f, c, s4), J[c], rtol=1e-5)
        # constant Fisher weights: same scale as the plain squared-error search
        cu = oracle.clip_search(v, np.full(16, 3.0, np.float32), s4)
        Ju = np.array([_objective_fp64(v, np.ones(16, np.float32), cc, s4, e4) for cc in range(0x7F)])
        assert Ju[cu] <= Ju[1:].min() * (1 + 1e-5)


def test_clipping_lowers_the_weighted_error_of_the_tensor():
    wl, _, w, _, fw = _tiny()
    wb = gi.bf16_bits(w)
    wv = _bf16_to_f32(wb).astype(np.float64)
    q0 = oracle.quantize_weights(wb, fw, clip=False, fp8_fraction=0.0)
    q1 = oracle.quantize_weights(wb, fw, clip=True, fp8_fraction=0.0)
    e0 = (fw * (oracle.decode(q0) - wv) ** 2).sum()
    e1 = (fw * (oracle.decode(q1) - wv) ** 2).sum()
    assert e1 < e0
    assert q0.scale_fp4 == q1.scale_fp4 == np.float32(np.abs(wv).max()) / np.float32(2688.0)
    # mode-0 score of every block is that block's weighted error under the chosen scale
    per_block = (fw * (oracle.decode(q1) - wv) ** 2).reshape(wl.N, -1, 16).sum(-1)
    assert np.allclose(q1.scores.reshape(wl.N, -1), per_block, rtol=2e-5)


def test_weight_fraction_invariant_and_selection():
    wl, _, w, _, fw = _tiny()
    wb = gi.bf16_bits(w)
    B = wl.N * wl.K // 16
    for frac in (0.0, 0.1, 0.2, 0.3, 0.25001, 1.0):
        q = oracle.quantize_weights(wb, fw, clip=False, fp8_fraction=frac)
        k = int(np.floor(frac * B + 0.5))
        mb = q.mask_bits().ravel()
        assert mb.sum() == k
        if 0 < k < B:
            # the selected blocks are exactly the k largest scores (stable in block order)
            order = np.lexsort((np.arange(B), -q.scores.astype(np.float64)))
            assert np.array_equal(np.sort(order[:k]), np.nonzero(mb)[0])
            assert q.tau_eff == q.scores[order[k - 1]]
            assert q.scores[mb].min() >= q.scores[~mb].max()
    # threshold mode: strict comparison
    q = oracle.quantize_weights(wb, fw, clip=False, fp8_fraction=0.1)
    qt = oracle.quantize_weights(wb, fw, clip=False, fp8_fraction=-1.0, tau=q.tau_eff)
    assert np.array_equal(qt.mask_bits().ravel(), q.scores > np.float32(q.tau_eff))


def test_ties_go_to_the_lower_block_index():
    wb = np.tile(gi.bf16_bits(gi.weights(1, 16, 5)), (8, 1))     # 8 identical blocks
    f = np.ones((8, 16), np.float32)
    q = oracle.quantize_weights(wb, f, clip=False, fp8_fraction=0.375)
    assert q.mask_bits().ravel().tolist() == [True, True, True] + [False] * 5


def test_memory_closed_form_matches_the_paper():
    """Payload = 9 bytes per NVFP4 block, 16 per FP8 block, 1 bit per block; the saving versus
    all-FP8 is what the paper prints."""
    wl, _, w, _, fw = _tiny()
    rows = [l.split() for l in open(os.path.join(GOLDEN, "memory_savings.txt")) if not l.startswith("#")]
    B = wl.N * wl.K // 16
    for frac4, printed in rows:
        p = 1.0 - float(frac4)
        q = oracle.quantize_weights(gi.bf16_bits(w), fw, clip=False, fp8_fraction=p)
        n8 = int(q.mask_bits().sum())
        payload_bits = (B - n8) * 72 + n8 * 128 + B
        bits_per_elt = payload_bits / (wl.N * wl.K)
        closed = (1 - n8 / B) * 4.5 + (n8 / B) * 8 + 1 / 16
        assert abs(bits_per_elt - closed) < 1e-12
        saving = 100 * (1 - bits_per_elt / 8)
        assert round(saving) == int(printed)
        # what is stored is what the count says: non-zero payload only where the mask allows
        mb = q.mask_bits()
        assert not q.codes8.reshape(wl.N, -1, 16)[~mb].any()
        assert not q.codes4.reshape(wl.N, -1, 8)[mb].any()


# ------------------------------------------------------------------------ GEMM

def _quantize_tiny(frac_a, frac_w, mode=0):
    wl, x, w, fx, fw = _tiny()
    s4 = gi.tensor_scale(x)
    xb, wb = gi.bf16_bits(x), gi.bf16_bits(w)
    if frac_a <= 0:
        tau = np.inf
    elif frac_a >= 1:
        tau = -1.0
    else:
        sc = oracle.quantize_activations(xb, fx, s4, tau=np.inf, mode=mode).scores
        tau, _ = _tau_for_fraction(sc, frac_a)
    qa = oracle.quantize_activations(xb, fx, s4, tau=tau, mode=mode)
    qw = oracle.quantize_weights(wb, fw, clip=True, fp8_fraction=frac_w, mode=mode)
    return wl, x, w, qa, qw


def test_linear_matches_library_matmul_in_fp64():
    for fa, fw_ in ((0.1, 0.1), (0.0, 0.0), (1.0, 1.0), (0.0, 1.0), (1.0, 0.0)):   # mixed + 4 pure pairs
        wl, x, w, qa, qw = _quantize_tiny(fa, fw_)
        Y, S = oracle.linear(qa, qw)
        A = torch.from_numpy(oracle.decode(qa))
        Wd = torch.from_numpy(oracle.decode(qw))
        Yt = (A @ Wd.T).numpy()
        St = (A.abs() @ Wd.abs().T).numpy()
        assert np.allclose(Y, Yt, rtol=0, atol=1e-12 * St.max())
        assert np.allclose(S, St, rtol=1e-12)
        # sampled variant agrees with the full one
        ms = np.array([0, 5, 63, 17]); ns = np.array([0, 255, 128, 3])
        Ys, Ss = oracle.linear_sampled(qa, qw, ms, ns)
        assert np.allclose(Ys, Y[ms, ns], rtol=0, atol=1e-12 * St.max()) and np.allclose(Ss, S[ms, ns])
        # and the quantized layer approximates the bf16 layer
        ref = x.double() @ w.double().T
        rel = np.abs(Y - ref.numpy()).sum() / np.abs(ref.numpy()).sum()
        assert rel < (0.05 if fa == 1.0 and fw_ == 1.0 else 0.25)


def test_all_fp8_equals_plain_fp8_gemm():
    """tau < 0 and fraction 1: the layer is a per-tensor-scaled E4M3 GEMM, computed here with
    torch's own cast and an fp64 matmul."""
    wl, x, w, qa, qw = _quantize_tiny(1.0, 1.0)
    sa8 = np.float64(np.float32(qa.scale_fp4)) * 8
    sw8 = np.float64(np.float32(qw.scale_fp4)) * 8
    xa = (x.float() * (np.float32(1.0) / np.float32(sa8))).to(torch.float8_e4m3fn).double() * sa8
    ww = (w.float() * (np.float32(1.0) / np.float32(sw8))).to(torch.float8_e4m3fn).double() * sw8
    Y, _ = oracle.linear(qa, qw)
    assert np.allclose(Y, (xa @ ww.T).numpy(), rtol=0, atol=1e-12 * np.abs(Y).max())


def test_decoded_values_follow_the_format_definitions():
    wl, x, w, qa, qw = _quantize_tiny(0.1, 0.1)
    e4 = _e4m3_vals()
    for q in (qa, qw):
        mb = np.repeat(q.mask_bits(), 16, axis=1)
        sc = np.repeat(q.scales.reshape(q.rows, -1), 16, axis=1)
        s4 = np.float64(np.float32(q.scale_fp4))
        v4 = E2M1[_unpack4(q)] * e4[sc] * s4
        v8 = e4[q.codes8.reshape(q.rows, q.K)] * s4 * 2.0 ** q.ratio
        assert np.array_equal(oracle.decode(q), np.where(mb, v8, v4))


# ------------------------------------------------------------------ global threshold (Eq. 10)

def test_global_threshold_counts_and_layer_shares():
    """Pins of oracle.global_threshold: against a brute-force rank count on small pools; exactly k blocks
    of the pool exceed it; with one tensor it is the local threshold of Eq. 9; a tensor with uniformly
    larger scores takes a larger share of the FP8 budget than its size (the point of Eq. 10)."""
    rng = np.random.default_rng(5)
    a = rng.lognormal(0.0, 1.0, 300).astype(np.float32)
    b = (4.0 * rng.lognormal(0.0, 1.0, 100)).astype(np.float32)
    for frac in (0.05, 0.1, 0.25, 0.5):
        tau = oracle.global_threshold([a, b], frac)
        pool = np.concatenate([a, b])
        k = int(np.floor(frac * pool.size + 0.5))
        assert int((pool > np.float32(tau)).sum()) == k
        # brute force: tau lies strictly below exactly k pooled scores and at or above all others
        assert sum(1 for v in pool if v > np.float32(tau)) == k
        assert np.float32(tau) in (np.float32(tau),) and np.sort(pool)[::-1][k] <= np.float32(tau) < np.sort(pool)[::-1][k - 1]
        # the sensitive tensor gets more than its proportional share
        share_b = (b > np.float32(tau)).mean()
        share_a = (a > np.float32(tau)).mean()
        assert share_b > frac > share_a
    # one tensor: the same value as sorting that tensor alone
    s = np.sort(a)[::-1]
    k = int(np.floor(0.1 * a.size + 0.5))
    assert oracle.global_threshold([a], 0.1) == float(np.float32(0.5) * (s[k - 1] + s[k]))
    # extremes and ties
    assert oracle.global_threshold([a, b], 0.0) == float("inf")
    assert oracle.global_threshold([a, b], 1.0) == -1.0
    t = np.array([3, 3, 3, 1, 1], np.float32)
    assert oracle.global_threshold([t], 0.4) == 2.0       # k = 2 falls inside the tie at 3: next distinct value below is 1
    assert (t > 2.0).sum() == 3                            # ties across the boundary all go to FP8


def test_channel_mean_sq_against_float64():
    """Pins of oracle.channel_mean_sq: exact on small integers, within fp32 rounding of the fp64 mean of
    squares on random data, and a transposed or unsquared version fails."""
    xi = torch.tensor([[1, -2, 3], [3, 2, -1], [2, 2, 2], [0, 4, 1]], dtype=torch.float32).to(torch.bfloat16)
    got = oracle.channel_mean_sq(gi.bf16_bits(xi))
    assert got.tolist() == [14 / 4, 28 / 4, 15 / 4]
    x = gi.activations(200, 64, 3, 0.05, 30.0)
    ref = (x.double() ** 2).mean(0).numpy()
    got = oracle.channel_mean_sq(gi.bf16_bits(x))
    assert got.shape == (64,)
    assert np.all(np.abs(got - ref) <= 200 * 2.0 ** -24 * ref)
    assert not np.allclose((x.double().abs()).mean(0).numpy(), ref)


# ------------------------------------------------------------------ tie rule of the clip search

def clip_tie_case():
    """Weights whose clip objective (Eq. 11) ties, with the outcome derived by hand.  Tensor scale 1.
    * An all-zero block: every scale code gives J = 0; the incumbent is the dynamic-max code E4M3(0) = 0x00 and
      a candidate replaces it only on strict improvement, so the scale stays 0x00 and all codes are +0.
    * A block of +-2 and 0: amax / 6 = 0.3333 rounds to the E4M3 value 0.34375 (code 0x2b), under which 2 becomes
      6 * 0.34375 = 2.0625 (J > 0).  J = 0 exactly for the scales 0.5, 1, 2 and 4 (2 / d in the E2M1 set); the
      ascending scan meets 0.5 = code 0x30 first and later ties do not replace it: scale 0x30, 2 -> 2 / 0.5 = 4 =
      E2M1 index 6 (code 0x6, negative 0xe), 0 -> code 0x0."""
    pattern = np.array([2, -2, 2, 2, 0, -2, 0, 2, -2, -2, 2, 0, 2, 2, -2, 2], np.float32)
    w = np.zeros((2, 64), np.float32)
    w[0, 16:32] = pattern
    w[1, 48:64] = pattern[::-1]
    bits = (w.view(np.uint32) >> 16).astype(np.uint16)
    codes = np.where(w == 2, 0x6, np.where(w == -2, 0xE, 0x0)).astype(np.uint8)
    packed = (codes[:, 0::2] | (codes[:, 1::2] << 4)).astype(np.uint8)          # even element in the low nibble
    scales = np.zeros((2, 4), np.uint8)
    scales[0, 1] = 0x30
    scales[1, 3] = 0x30
    return w, bits, packed.ravel(), scales.ravel()


def test_clip_search_ties_keep_the_incumbent_then_the_lowest_code():
    w, bits, codes4, scales = clip_tie_case()
    f = np.ones_like(w)
    q = oracle.quantize_weights(bits, f, scale_fp4=1.0, clip=True, fp8_fraction=0.0)
    assert np.array_equal(q.scales, scales), (q.scales, scales)
    assert np.array_equal(q.codes4, codes4)
    assert not q.mask_bits().any() and (q.scores == 0).all()
    # the single-block entry point agrees, and the objective really ties where the derivation says
    assert oracle.clip_search(w[0, 16:32], f[0, 16:32], 1.0) == 0x30
    assert oracle.clip_search(np.zeros(16, np.float32), np.ones(16, np.float32), 1.0) == 0x00
    for c in (0x30, 0x38, 0x40, 0x48):
        assert oracle.clip_objective(w[0, 16:32], f[0, 16:32], c, 1.0) == 0.0
    assert oracle.clip_objective(w[0, 16:32], f[0, 16:32], 0x2B, 1.0) > 0.0
    # without the search the dynamic-max code stays
    q0 = oracle.quantize_weights(bits, f, scale_fp4=1.0, clip=False, fp8_fraction=0.0)
    assert q0.scales[1] == 0x2B and q0.scales[0] == 0x00


# ------------------------------------------------------------------ FP8 tensor scale given on its own (Section 5.1)

def _free_scales(x, w):
    """amax / 448 for the FP8 part, amax / (6 * 448) for the NVFP4 part: a ratio of 6, not a power of two."""
    ax, aw = float(x.float().abs().max()), float(w.float().abs().max())
    return (np.float32(ax / 2688.0), np.float32(ax / 448.0)), (np.float32(aw / 2688.0), np.float32(aw / 448.0))


def test_free_fp8_scale_rounds_to_nearest_under_that_scale():
    """FP8 codes are the E4M3 values nearest to x / s8 (brute force over the 253 finite values, fp64) for an s8 that
    is not s4 times a power of two; the NVFP4 side does not depend on s8; mode-1 scores are Eq. 8 in fp64 with
    this s8."""
    wl, x, _, fx, _ = _tiny()
    (s4, s8), _ = _free_scales(x, x)
    q = oracle.quantize_activations(gi.bf16_bits(x), fx, s4, tau=-1.0, mode=1, scale_fp8=s8)
    xv = _bf16_to_f32(gi.bf16_bits(x)).astype(np.float64)
    e4 = _e4m3_vals()
    y8 = xv / np.float64(s8)
    c8 = q.codes8.reshape(wl.M, wl.K)
    finite = e4[np.r_[0:0x7F, 0x80:0xFF]]
    best8 = np.abs(y8[..., None] - finite[None, None, :]).min(-1)
    assert np.all(np.abs(y8 - e4[c8]) <= best8 + 1e-5 * np.abs(y8) + 1e-12)
    assert np.abs(e4[c8]).max() > 224          # the scale uses the E4M3 range (amax lands near 448)
    q4 = oracle.quantize_activations(gi.bf16_bits(x), fx, s4, tau=np.inf, mode=0, scale_fp8=s8)
    q4t = oracle.quantize_activations(gi.bf16_bits(x), fx, s4, tau=np.inf, mode=0)
    assert np.array_equal(q4.codes4, q4t.codes4) and np.array_equal(q4.scales, q4t.scales) and np.array_equal(q4.scores, q4t.scores)
    # Eq. 8 with this s8: sum f (Q4(x) - Q8(x))^2
    d4 = oracle.decode(q4)
    d8 = e4[c8] * np.float64(s8)
    ref = (fx.astype(np.float64)[None, :] * (d4 - d8) ** 2).reshape(wl.M, -1, 16).sum(-1)
    assert np.allclose(q.scores.reshape(wl.M, -1), ref, rtol=2e-5, atol=1e-30)


def test_free_fp8_scale_equal_to_the_tied_one_changes_nothing():
    """Passing s8 = s4 * 2^3 explicitly gives the arrays of the tied default, and decode / linear use the given value."""
    wl, x, w, fx, fw = _tiny()
    s4 = gi.tensor_scale(x)
    a = oracle.quantize_activations(gi.bf16_bits(x), fx, s4, tau=1e-4, mode=1)
    b = oracle.quantize_activations(gi.bf16_bits(x), fx, s4, tau=1e-4, mode=1, scale_fp8=float(np.float32(s4) * np.float32(8)))
    for n in ("codes4", "codes8", "scales", "mask", "scores"):
        assert np.array_equal(getattr(a, n), getattr(b, n)), n
    assert np.array_equal(oracle.decode(a), oracle.decode(b))


def test_free_fp8_scale_decode_and_linear():
    """Decoded FP8 blocks are e4m3 * s8 with the given s8 (NVFP4 blocks unchanged); the layer is the fp64 library
    matmul of the decoded operands; with every block in FP8 it is the plain per-tensor-scaled E4M3 GEMM through
    torch's own cast."""
    wl, x, w, fx, fw = _tiny()
    (as4, as8), (ws4, ws8) = _free_scales(x, w)
    e4 = _e4m3_vals()
    for frac in (0.1, 1.0):
        sa = oracle.quantize_activations(gi.bf16_bits(x), fx, as4, tau=np.inf, scale_fp8=as8).scores
        tau = -1.0 if frac == 1.0 else _tau_for_fraction(sa, frac)[0]
        qa = oracle.quantize_activations(gi.bf16_bits(x), fx, as4, tau=tau, scale_fp8=as8)
        qw = oracle.quantize_weights(gi.bf16_bits(w), fw, scale_fp4=ws4, fp8_fraction=frac, scale_fp8=ws8)
        for q, s8 in ((qa, as8), (qw, ws8)):
            mb = np.repeat(q.mask_bits(), 16, axis=1)
            sc = np.repeat(q.scales.reshape(q.rows, -1), 16, axis=1)
            v4 = E2M1[_unpack4(q)] * e4[sc] * np.float64(np.float32(q.scale_fp4))
            v8 = e4[q.codes8.reshape(q.rows, q.K)] * np.float64(s8)
            assert np.array_equal(oracle.decode(q), np.where(mb, v8, v4))
        Y, S = oracle.linear(qa, qw)
        A, Wd = torch.from_numpy(oracle.decode(qa)), torch.from_numpy(oracle.decode(qw))
        assert np.allclose(Y, (A @ Wd.T).numpy(), rtol=0, atol=1e-12 * S.max())
        ms = np.array([0, 5, 63, 17]); ns = np.array([0, 255, 128, 3])
        Ys, _ = oracle.linear_sampled(qa, qw, ms, ns)
        assert np.allclose(Ys, Y[ms, ns], rtol=0, atol=1e-12 * S.max())
        if frac == 1.0:
            xa = (x.float() * (np.float32(1.0) / as8)).to(torch.float8_e4m3fn).double() * np.float64(as8)
            ww = (w.float() * (np.float32(1.0) / ws8)).to(torch.float8_e4m3fn).double() * np.float64(ws8)
            assert np.allclose(Y, (xa @ ww.T).numpy(), rtol=0, atol=1e-12 * np.abs(Y).max())
            # a free scale uses the whole E4M3 range: the FP8 layer is closer to the bf16 layer than with s8 = 8 s4 > amax / 448
            ref = (x.double() @ w.double().T).numpy()
            assert np.abs(Y - ref).sum() / np.abs(ref).sum() < 0.05
