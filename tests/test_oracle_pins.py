"""Pins for the CPU oracle: every function is checked against something other
than itself -- an SVD, exact rational iterates, closed forms, invariants,
brute force on tiny inputs.  No GPU needed."""
import math
import os

import numpy as np
import pytest

from oracle import muloco_oracle as O
from paper_2505_23725_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")
A, B, C = O.NS_COEFFS


def p5(x):
    x = np.asarray(x, dtype=np.float64)
    for _ in range(5):
        x = x * (A + x * x * (B + C * x * x))
    return x


def relfro(x, y):
    return np.linalg.norm(x - y) / np.linalg.norm(y)


# ---- P1: Newton-Schulz == U diag(p^(5)(s/||X||_F)) V^T ----------------------
@pytest.mark.parametrize("m,n", [(8, 8), (16, 40), (40, 16), (1, 7), (7, 1), (33, 32)])
def test_ns_matches_svd_closed_form(m, n):
    rng = np.random.default_rng(100 + m * 64 + n)
    r = min(m, n)
    U, V = synth.haar(rng, m, r), synth.haar(rng, n, r)
    s = np.sort(rng.uniform(0.05, 3.0, r))[::-1]
    X = (U * s) @ V.T
    got = O.newton_schulz(X, eps=0.0)
    # library routine: numpy's SVD of the input, scalar map on the singular values
    Us, ss, Vts = np.linalg.svd(X, full_matrices=False)
    want = (Us * p5(ss / np.linalg.norm(ss))) @ Vts
    assert relfro(got, want) < 1e-12
    # and the singular values of the output are the mapped ones (order-free check)
    sv = np.sort(np.linalg.svd(got, compute_uv=False))
    assert np.allclose(sv, np.sort(np.abs(p5(s / np.linalg.norm(s)))), rtol=1e-10, atol=1e-12)


# ---- P2: scalar recurrence against exact rational iterates ------------------
def test_ns_scalar_iterates_golden():
    rows = [l.split() for l in open(os.path.join(GOLD, "ns_scalar_iterates.txt")) if not l.startswith("#")]
    assert len(rows) == 5
    for row in rows:
        x0 = float(row[0])
        for steps in range(1, 6):
            want = float(row[steps])
            # 1x1 matrix [x0]: normalisation makes it 1, so scale by hand: use a 1x2
            # matrix [x0, sqrt(1-x0^2)] whose only singular value is 1 ... instead
            # pin the scalar map through a 2x2 diagonal with known normalised spectrum.
            y = math.sqrt(max(0.0, 1.0 - x0 * x0))
            X = np.diag([x0, y]) if y > 0 else np.array([[x0]])
            got = O.newton_schulz(X, steps=steps, eps=0.0)
            assert abs(got[0, 0] - want) <= 1e-12 * max(1.0, abs(want))
            if y > 0:
                assert abs(got[0, 1]) < 1e-15 and abs(got[1, 0]) < 1e-15


def test_ns_coefficients_are_the_papers():
    assert O.NS_COEFFS == (3.4445, -4.7750, 2.0315)
    # p(1) = a + b + c
    got = O.newton_schulz(np.array([[2.5]]), steps=1, eps=0.0)
    assert abs(got[0, 0] - 0.7010) < 1e-12


def test_ns_equivariance_and_transpose():
    rng = np.random.default_rng(7)
    X = rng.standard_normal((12, 20))
    Q = synth.haar(rng, 12, 12)
    R = synth.haar(rng, 20, 20)
    base = O.newton_schulz(X)
    assert relfro(O.newton_schulz(Q @ X @ R.T), Q @ base @ R.T) < 1e-11
    assert relfro(O.newton_schulz(X.T), base.T) < 1e-13
    assert relfro(O.newton_schulz(-X), -base) < 1e-15
    # scale invariance (up to eps): the input is normalised first
    assert relfro(O.newton_schulz(1e3 * X), base) < 1e-7


def test_ns_zero_input_and_eps():
    Z = np.zeros((4, 6))
    out = O.newton_schulz(Z)
    assert np.all(out == 0) and np.all(np.isfinite(out))
    # eps enters as ||U||_F + eps
    X = np.array([[1e-7, 0.0], [0.0, 0.0]])
    got = O.newton_schulz(X, steps=1, eps=1e-7)
    assert abs(got[0, 0] - float(p1(0.5))) < 1e-12


def p1(x):
    return x * (A + x * x * (B + C * x * x))


def test_ns_output_spectrum_band():
    # singular values of a well-conditioned input land in about [0.68, 1.21]
    rng = np.random.default_rng(3)
    X = rng.standard_normal((24, 64))
    sv = np.linalg.svd(O.newton_schulz(X), compute_uv=False)
    assert sv.min() > 0.6 and sv.max() < 1.25
    r = 24
    assert 0.68 * math.sqrt(r) < np.linalg.norm(O.newton_schulz(X)) < 1.21 * math.sqrt(r)


# ---- P3: Muon step on a rank-1 gradient (closed form) -----------------------
@pytest.mark.parametrize("m,n", [(6, 10), (10, 6)])
@pytest.mark.parametrize("nesterov", [True, False])
def test_muon_rank1_closed_form(m, n, nesterov):
    rng = np.random.default_rng(11)
    # small-integer factors: the outer product is exact in float32, so the stored
    # gradient is exactly rank 1 (rounding noise would be amplified by the iteration)
    u = rng.integers(-4, 5, m).astype(np.float64); u[0] = 3.0
    v = rng.integers(-4, 5, n).astype(np.float64); v[0] = -2.0
    G = np.outer(u, v).astype(np.float32)
    assert np.array_equal(G.astype(np.float64), np.outer(u, v))
    W0 = (0.02 * rng.standard_normal((m, n))).astype(np.float32)
    W = W0.copy(); M = np.zeros_like(W)
    lr, beta, wd = 0.02, 0.95, 0.01
    O.muon_step(W, M, G, lr=lr, beta=beta, wd=wd, nesterov=nesterov, eps=0.0)
    # after the first step M = G; U is a positive multiple of G either way, rank 1,
    # so O = p^(5)(1) * u v^T computed from the float32 G that the step saw
    Gd = G.astype(np.float64)
    uv = Gd / np.linalg.norm(Gd)
    eta = lr * math.sqrt(n / m)
    want = W0.astype(np.float64) * (1 - eta * wd) - eta * float(p5(1.0)) * uv
    assert np.allclose(W, want, rtol=0, atol=2e-7 * np.abs(want).max() + 1e-9)
    assert np.array_equal(M, G)


def test_muon_momentum_and_nesterov_input():
    # two steps: check M and the NS input by recomputing O from an SVD
    rng = np.random.default_rng(5)
    m, n = 5, 9
    W = np.zeros((m, n), np.float32); M = np.zeros_like(W)
    g1 = rng.standard_normal((m, n)).astype(np.float32)
    g2 = rng.standard_normal((m, n)).astype(np.float32)
    beta = 0.5
    O.muon_step(W, M, g1, lr=0.0, beta=beta, wd=0.0)
    Oret = O.muon_step(W, M, g2, lr=0.1, beta=beta, wd=0.0, nesterov=True, lr_mult=1.0, eps=0.0)
    assert np.allclose(M, beta * g1.astype(np.float64) + g2, rtol=1e-7)
    Uin = g2.astype(np.float64) + beta * M.astype(np.float64)
    Us, ss, Vt = np.linalg.svd(Uin, full_matrices=False)
    want = (Us * p5(ss / np.linalg.norm(ss))) @ Vt
    assert relfro(Oret, want) < 1e-12
    assert np.allclose(W, -0.1 * want, atol=1e-7)


def test_muon_lr_mult_is_sqrt_cols_over_rows():
    assert O.muon_lr_mult(128, 352) == pytest.approx(math.sqrt(352 / 128))
    assert O.muon_lr_mult(352, 128) == pytest.approx(math.sqrt(128 / 352))
    rng = np.random.default_rng(0)
    G = rng.standard_normal((4, 16)).astype(np.float32)
    W1 = np.zeros((4, 16), np.float32); W2 = np.zeros((4, 16), np.float32)
    O.muon_step(W1, np.zeros_like(W1), G, lr=0.1, beta=0.9, wd=0.0)
    O.muon_step(W2, np.zeros_like(W2), G, lr=0.1, beta=0.9, wd=0.0, lr_mult=1.0)
    assert np.allclose(W1, 2.0 * W2.astype(np.float64), rtol=1e-6)


def test_muon_weight_decay_scaling_flag():
    G = np.zeros((4, 16), np.float32)          # zero gradient: only decay acts
    W0 = np.full((4, 16), 1.0, np.float32)
    Wa = W0.copy(); Wb = W0.copy()
    O.muon_step(Wa, np.zeros_like(Wa), G, lr=0.1, beta=0.9, wd=0.5, wd_uses_scaled_lr=True)
    O.muon_step(Wb, np.zeros_like(Wb), G, lr=0.1, beta=0.9, wd=0.5, wd_uses_scaled_lr=False)
    assert np.allclose(Wa, 1 - 0.1 * 2.0 * 0.5, rtol=1e-6)
    assert np.allclose(Wb, 1 - 0.1 * 0.5, rtol=1e-6)


# ---- P7: AdamW ---------------------------------------------------------------
def test_adamw_first_step_closed_form():
    rng = np.random.default_rng(2)
    g = rng.standard_normal(50).astype(np.float32)
    th0 = rng.standard_normal(50).astype(np.float32)
    th = th0.copy(); m = np.zeros_like(th); v = np.zeros_like(th)
    lr, wd, eps = 1e-2, 0.1, 1e-8
    O.adamw_step(th, m, v, g, t=1, lr=lr, beta1=0.9, beta2=0.99, eps=eps, wd=wd)
    gd = g.astype(np.float64)
    want = th0 - lr * (gd / (np.abs(gd) + eps) + wd * th0)
    assert np.allclose(th, want, rtol=2e-6, atol=1e-7)
    assert np.allclose(m, 0.1 * gd, rtol=1e-6)
    assert np.allclose(v, 0.01 * gd * gd, rtol=1e-6)
    # where eps is felt: |g| = eps gives a half step, |g| << eps an almost vanishing one
    # (eps is added to sqrt(v^), outside the root)
    g2 = np.array([1e-8, -1e-8, 1e-10, 0.0], np.float32)
    th = np.zeros(4, np.float32); m = np.zeros(4, np.float32); v = np.zeros(4, np.float32)
    O.adamw_step(th, m, v, g2, t=1, lr=1.0, beta1=0.9, beta2=0.99, eps=1e-8, wd=0.0)
    g2d = g2.astype(np.float64)
    assert np.allclose(th, -(g2d / (np.abs(g2d) + 1e-8)), rtol=1e-5, atol=1e-12)
    assert abs(th[0] + 0.5) < 1e-5 and abs(th[2]) < 0.0101


def test_adamw_constant_gradient_and_no_bias_correction():
    g = np.array([0.5, -2.0, 1e-3], np.float32)
    th = np.zeros(3, np.float32); m = np.zeros(3, np.float32); v = np.zeros(3, np.float32)
    for t in range(1, 6):
        O.adamw_step(th, m, v, g, t=t, lr=0.1, beta1=0.9, beta2=0.99, eps=0.0, wd=0.0)
        # bias-corrected moments equal g and g^2 under a constant gradient: unit steps
        assert np.allclose(th, -0.1 * t * np.sign(g), rtol=1e-5)
    th2 = np.zeros(3, np.float32); m2 = np.zeros(3, np.float32); v2 = np.zeros(3, np.float32)
    O.adamw_step(th2, m2, v2, g, t=1, lr=0.1, beta1=0.9, beta2=0.99, eps=0.0, wd=0.0,
                 bias_correction=False)
    # without correction: m/sqrt(v) = 0.1 g / (0.1 |g|) = sign(g) as well at t=1 for b2=.99
    assert np.allclose(th2, -0.1 * (0.1 / math.sqrt(0.01)) * np.sign(g), rtol=1e-5)


def test_adamw_against_textbook_loop():
    rng = np.random.default_rng(9)
    n = 40
    th = rng.standard_normal(n).astype(np.float32)
    m = np.zeros(n, np.float32); v = np.zeros(n, np.float32)
    ref_th = th.astype(np.float64); ref_m = np.zeros(n); ref_v = np.zeros(n)
    b1, b2, lr, wd, eps = 0.9, 0.99, 3e-3, 0.05, 1e-8
    for t in range(1, 8):
        g = rng.standard_normal(n).astype(np.float32)
        O.adamw_step(th, m, v, g, t=t, lr=lr, beta1=b1, beta2=b2, eps=eps, wd=wd)
        for i in range(n):      # scalar loop, element by element
            ref_m[i] = b1 * ref_m[i] + (1 - b1) * float(g[i])
            ref_v[i] = b2 * ref_v[i] + (1 - b2) * float(g[i]) ** 2
            mh = ref_m[i] / (1 - b1 ** t); vh = ref_v[i] / (1 - b2 ** t)
            ref_th[i] = ref_th[i] - lr * (mh / (math.sqrt(vh) + eps) + wd * ref_th[i])
    assert np.allclose(th, ref_th, rtol=1e-5, atol=1e-6)


# ---- P8: outer Nesterov closed forms ----------------------------------------
def test_outer_step_closed_forms():
    th0 = np.array([1.0, -2.0, 0.5], np.float32)
    psi = np.array([0.25, 0.5, -1.0], np.float64)
    # mu = 0: plain SGD on the pseudogradient
    th = th0.copy(); u = np.zeros(3, np.float32)
    O.outer_nesterov(th, u, psi, outer_lr=0.5, outer_momentum=0.0)
    assert np.allclose(th, th0 - 0.5 * psi) and np.allclose(u, 0.5 * psi)
    # psi = 0: theta unchanged apart from -mu*u drift, u decays
    th = th0.copy(); u = np.array([1.0, 1.0, 1.0], np.float32)
    O.outer_nesterov(th, u, np.zeros(3), outer_lr=0.7, outer_momentum=0.5)
    assert np.allclose(u, 0.5) and np.allclose(th, th0 - 0.25)
    # two syncs with a constant psi (powers of two keep fp32 exact)
    th = th0.copy(); u = np.zeros(3, np.float32)
    eta, mu = 0.5, 0.5
    for _ in range(2):
        O.outer_nesterov(th, u, psi, outer_lr=eta, outer_momentum=mu)
    assert np.allclose(u, eta * (1 + mu) * psi)
    assert np.allclose(th, th0 - eta * psi * (2 + 2 * mu + mu * mu))


def test_pseudogradient_definitions():
    rng = np.random.default_rng(4)
    tg = rng.standard_normal((3, 5)).astype(np.float32)
    reps = [tg + rng.standard_normal((3, 5)).astype(np.float32) * 0.1 for _ in range(4)]
    psi = O.pseudogradient(tg, reps)
    # theta_global - mean_k theta_k
    want = tg.astype(np.float64) - np.mean([r.astype(np.float64) for r in reps], axis=0)
    assert np.allclose(psi, want, rtol=1e-12, atol=1e-15)
    psi32 = O.pseudogradient_f32(tg, reps)
    assert psi32.dtype == np.float32
    assert np.allclose(psi32, want, rtol=0, atol=4 * 6e-8 * 0.5)


# ---- P9: quantiser -----------------------------------------------------------
@pytest.mark.parametrize("bits", [8, 4])
def test_quantiser_properties(bits):
    rng = np.random.default_rng(21)
    qmax = (1 << (bits - 1)) - 1
    x = (rng.standard_normal((7, 352)) * np.exp(rng.standard_normal((7, 1)) * 3)).astype(np.float32)
    x[2, 128:256] = 0.0                         # an all-zero block
    codes, scales, deq = O.quantize_blocks(x, bits, 128)
    assert codes.dtype == np.int8 and scales.shape == (7, 3)
    assert np.abs(codes).max() <= qmax
    for r in range(7):
        for j in range(3):
            lo, hi = j * 128, min(352, (j + 1) * 128)
            xb = x[r, lo:hi]; cb = codes[r, lo:hi]
            amax = np.abs(xb).max()
            if amax == 0:
                assert scales[r, j] == 0 and not cb.any() and not deq[r, lo:hi].any()
                continue
            # the absmax element takes the extreme code; error at most half a step
            assert abs(int(cb[np.argmax(np.abs(xb))])) == qmax
            sc = float(scales[r, j])
            assert sc == pytest.approx(amax / qmax, rel=1e-6)
            err = np.abs(deq[r, lo:hi].astype(np.float64) - xb.astype(np.float64))
            assert err.max() <= 0.5 * sc * (1 + 1e-5) + 1e-6 * amax
    # idempotent: quantising the dequantised values gives the same codes
    codes2, _, deq2 = O.quantize_blocks(deq, bits, 128)
    assert np.array_equal(codes, codes2) and np.array_equal(deq, deq2)


def test_quantiser_round_half_to_even_and_brute_force():
    # block with amax = 127 (int8): inv = 1, so x itself is rounded; ties go to even
    x = np.zeros((1, 128), np.float32)
    x[0, 0] = 127.0
    x[0, 1:9] = [0.5, 1.5, 2.5, -0.5, -1.5, -2.5, 3.5, 0.49999997]
    codes, scales, _ = O.quantize_blocks(x, 8, 128)
    assert scales[0, 0] == 1.0
    assert codes[0, 1:9].tolist() == [0, 2, 2, 0, -2, -2, 4, 0]
    # int4: amax = 7
    x4 = np.zeros((1, 16), np.float32); x4[0, 0] = -7.0; x4[0, 1:5] = [0.5, 1.5, 6.5, -6.5]
    c4, s4, d4 = O.quantize_blocks(x4, 4, 128)
    assert s4[0, 0] == 1.0 and c4[0, :5].tolist() == [-7, 0, 2, 6, -6]
    # brute force against Python's exact round-half-even on float32-exact products
    rng = np.random.default_rng(8)
    xb = rng.standard_normal(128).astype(np.float32)
    codes, scales, deq = O.quantize_blocks(xb, 8, 128)
    amax = np.float32(np.abs(xb).max()); inv = np.float32(127.0) / amax
    for i in range(128):
        prod = float(np.float32(xb[i] * inv))     # the float32 product, exactly
        assert int(codes[0, i]) == max(-127, min(127, round(prod)))
        assert deq[0, i] == np.float32(np.float32(codes[0, i]) * (amax / np.float32(127.0)))


def test_quantiser_blocks_do_not_span_rows_and_vectors_are_one_row():
    x = np.ones((2, 96), np.float32); x[1] *= 100.0
    _, scales, deq = O.quantize_blocks(x, 8, 128)
    assert scales.shape == (2, 1) and scales[0, 0] != scales[1, 0]
    assert np.allclose(deq, x, rtol=1e-6)
    v = np.arange(300, dtype=np.float32)
    c, s, d = O.quantize_blocks(v, 8, 128)
    assert c.shape == (1, 300) and s.shape == (1, 3)


def test_int4_packing():
    c = np.array([[1, -1, 7, -7, 0]], np.int8)
    p = O.pack_int4(c)
    assert p.tolist() == [[0x1 | (0xF << 4), 0x7 | (0x9 << 4), 0x0]]


# ---- P10: streaming schedule -------------------------------------------------
def test_fragments_due_schedule():
    H, J = 12, 4
    seen = {j: [] for j in range(J)}
    for t in range(1, 3 * H + 1):
        for f in O.fragments_due(t, H, J):
            seen[f].append(t)
    # fragment j (1-based) at multiples j*H/J within each interval
    assert seen[0] == [3, 15, 27] and seen[1] == [6, 18, 30]
    assert seen[2] == [9, 21, 33] and seen[3] == [12, 24, 36]
    assert O.fragments_due(0, H, J) == []
    assert O.fragments_due(H, H, 1) == [0] and O.fragments_due(H - 1, H, 1) == []
    with pytest.raises(ValueError):
        O.fragments_due(1, 10, 4)


# ---------------------------------------------------------------------------
# Algorithm 2: two-stage compression and error feedback
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("bits", [8, 4, 2])
def test_two_stage_compression_collapses_for_one_worker(bits):
    # K = 1: mean of one dequantised delta is that delta, and quantising a dequantised block
    # again reproduces it (idempotence), so two stages equal one stage bit for bit
    rng = np.random.default_rng(31 + bits)
    tg = rng.standard_normal((5, 300)).astype(np.float32)
    th = (tg - 0.01 * rng.standard_normal((5, 300))).astype(np.float32)
    two = O.compressed_pseudogradient(tg, [th], bits, 128)
    _, _, one = O.quantize_blocks((tg - th).astype(np.float32), bits, 128)
    assert np.array_equal(two, one)


@pytest.mark.parametrize("bits", [8, 4])
def test_two_stage_compression_error_bound(bits):
    # each quantisation moves a value by at most half a step of its block: the result is within
    # (mean of the workers' half steps) + (half step of the second stage) of the exact mean
    rng = np.random.default_rng(7)
    K, qmax = 4, (1 << (bits - 1)) - 1
    tg = rng.standard_normal((3, 256)).astype(np.float32)
    ths = [(tg - 0.02 * rng.standard_normal((3, 256))).astype(np.float32) for _ in range(K)]
    psi = O.compressed_pseudogradient(tg, ths, bits, 128).astype(np.float64)
    exact = np.mean([tg.astype(np.float64) - t for t in ths], axis=0)
    for j in range(2):
        sl = slice(128 * j, 128 * (j + 1))
        half1 = np.mean([np.abs(tg[:, sl].astype(np.float64) - t[:, sl]).max(axis=1) / qmax / 2 for t in ths], axis=0)
        half2 = (np.abs(exact[:, sl]).max(axis=1) + half1) / qmax / 2
        bound = (half1 + half2)[:, None] * (1 + 1e-5) + 1e-7
        assert np.all(np.abs(psi[:, sl] - exact[:, sl]) <= bound)


def test_error_feedback_conserves_what_was_not_sent():
    # beta = 1: after every sync  E_i + (sum of everything sent so far) = sum of the deltas so far,
    # up to one float32 rounding per operation; and |E_i| is at most half a quantisation step
    rng = np.random.default_rng(11)
    K, bits = 2, 4
    tg = np.zeros((2, 128), dtype=np.float32)
    ef = [np.zeros_like(tg) for _ in range(K)]
    sent = [np.zeros(tg.shape) for _ in range(K)]
    total = [np.zeros(tg.shape) for _ in range(K)]
    for rnd in range(6):
        ths = [(-(0.1 * rng.standard_normal(tg.shape))).astype(np.float32) for _ in range(K)]   # delta_i = -theta_i
        before = [e.copy() for e in ef]
        O.compressed_pseudogradient(tg, ths, bits, 128, ef, 1.0)
        for i in range(K):
            e_in = (before[i] + (tg - ths[i])).astype(np.float32)
            c = e_in.astype(np.float64) - ef[i]                     # what worker i sent this round
            _, sc, deq = O.quantize_blocks(e_in, bits, 128)
            assert np.allclose(c, deq, rtol=0, atol=1e-6 * np.abs(e_in).max())
            assert np.all(np.abs(ef[i]) <= sc[:, :1] / 2 * (1 + 1e-5) + 1e-7)
            sent[i] += c
            total[i] += (tg - ths[i]).astype(np.float64)
            assert np.allclose(sent[i] + ef[i], total[i], rtol=0, atol=1e-5)


def test_error_feedback_changes_nothing_when_nothing_is_lost():
    # values that the quantiser represents exactly (multiples of the step, absmax = 7 steps)
    # leave E = 0, and the sync equals the uncompressed mean
    steps = np.array([[7, -3, 0, 1, 5, -7, 2, 4]], dtype=np.float32)
    tg = np.zeros((1, 8), dtype=np.float32)
    ths = [-(0.25 * steps), -(0.5 * steps[:, ::-1].copy())]
    ef = [np.zeros_like(tg) for _ in range(2)]
    psi = O.compressed_pseudogradient(tg, [t.astype(np.float32) for t in ths], 4, 8, ef, 0.9)
    assert all(np.all(e == 0) for e in ef)
    mean = (0.25 * steps + 0.5 * steps[:, ::-1]) / 2
    _, _, want = O.quantize_blocks(mean.astype(np.float32), 4, 8)
    assert np.array_equal(psi, want)


def test_row_wise_quantisation_is_one_block_per_row():
    rng = np.random.default_rng(3)
    x = rng.standard_normal((4, 300)).astype(np.float32)
    codes, scales, deq = O.quantize_blocks(x, 8, 300)
    assert scales.shape == (4, 1)
    assert np.array_equal(scales[:, 0], (np.abs(x).max(axis=1) / np.float32(127)).astype(np.float32))
    assert np.all(np.abs(codes).max(axis=1) == 127)


# ---- top-k sparsification (Section 2, "Compressed Communication") ------------
def _topk_brute(x, kk):
    """Plain selection: walk the entries from the largest magnitude down, keep the first kk and
    everything tied with the kk-th."""
    flat = [float(v) for v in np.asarray(x, dtype=np.float32).reshape(-1)]
    order = sorted(range(len(flat)), key=lambda i: -abs(flat[i]))
    tau = abs(flat[order[kk - 1]])
    return np.array([v if abs(v) >= tau else 0.0 for v in flat], dtype=np.float32).reshape(np.shape(x))


@pytest.mark.parametrize("shape,frac", [((7, 9), 0.1), ((1, 50), 0.5), ((33, 4), 0.02), ((5, 5), 1.0),
                                        ((64, 3), 0.005), ((12, 12), 0.25)])
def test_topk_matches_brute_force_selection(shape, frac):
    rng = np.random.default_rng(700 + shape[0])
    x = rng.standard_normal(shape).astype(np.float32)
    n = x.size
    kk = min(n, max(1, int(math.floor(float(np.float32(frac)) * n))))
    assert O.topk_count(n, frac) == kk
    got = O.topk_sparsify(x, frac)
    assert np.array_equal(got, _topk_brute(x, kk))
    kept = got != 0
    assert kept.sum() == kk                                   # no ties in continuous data
    assert np.array_equal(got[kept], x[kept])                 # kept entries unchanged, sign included
    if kk < n:
        assert np.abs(x[kept]).min() > np.abs(x[~kept]).max() # every kept entry beats every dropped one
    if frac == 1.0:
        assert np.array_equal(got, x)


def test_topk_is_the_best_k_term_approximation():
    """Among all arrays with at most kk non-zeros, keeping the kk largest magnitudes is the
    closest to x in the Frobenius norm: checked by enumerating every support for small n."""
    import itertools
    rng = np.random.default_rng(701)
    for n, frac in [(6, 0.5), (8, 0.25), (7, 0.3), (5, 0.2)]:
        x = rng.standard_normal(n).astype(np.float32)
        kk = O.topk_count(n, frac)
        best = min(float(np.sum(np.delete(x.astype(np.float64), list(sup)) ** 2))
                   for sup in itertools.combinations(range(n), kk))
        got = O.topk_sparsify(x.reshape(1, n), frac).reshape(-1)
        assert np.count_nonzero(got) == kk
        assert abs(float(np.sum((x.astype(np.float64) - got) ** 2)) - best) < 1e-12


def test_topk_ties_counts_and_degenerate_inputs():
    # ties with the kk-th magnitude are all kept, whatever their sign or position
    x = np.array([[3.0, -1.0, 1.0, 0.5, -3.0, 1.0, 0.25, -1.0]], dtype=np.float32)
    assert np.array_equal(O.topk_sparsify(x, 3 / 8), np.array([[3, -1, 1, 0, -3, 1, 0, -1]], dtype=np.float32))
    assert np.array_equal(O.topk_sparsify(x, 2 / 8), np.array([[3, 0, 0, 0, -3, 0, 0, 0]], dtype=np.float32))
    # a fraction that selects less than one entry still keeps one; the selection is over the whole tensor,
    # not per row
    y = np.array([[1.0, 2.0], [9.0, 3.0], [4.0, 8.0]], dtype=np.float32)
    assert np.array_equal(O.topk_sparsify(y, 0.01), np.array([[0, 0], [9, 0], [0, 0]], dtype=np.float32))
    assert np.array_equal(O.topk_sparsify(y, 0.5), np.array([[0, 0], [9, 0], [4, 8]], dtype=np.float32))
    assert O.topk_count(1000, 0.0005) == 1 and O.topk_count(1000, 0.0025) == 2 and O.topk_count(8, 1.0) == 8
    # all-zero input stays zero; an empty tensor stays empty
    assert not O.topk_sparsify(np.zeros((3, 4), np.float32), 0.1).any()
    assert O.topk_sparsify(np.zeros((0, 4), np.float32), 0.1).shape == (0, 4)


def test_sparsified_pseudogradient_definitions_and_error_feedback():
    rng = np.random.default_rng(702)
    tg = rng.standard_normal((9, 14)).astype(np.float32)
    K, frac = 3, 0.2
    thetas = [(tg - 0.1 * rng.standard_normal(tg.shape)).astype(np.float32) for _ in range(K)]
    # one worker: Psi is the sparsified delta itself; fraction 1: the plain float32 pseudogradient
    assert np.array_equal(O.sparsified_pseudogradient(tg, thetas[:1], frac), O.topk_sparsify(tg - thetas[0], frac))
    assert np.array_equal(O.sparsified_pseudogradient(tg, thetas, 1.0), O.pseudogradient_f32(tg, thetas))
    # K workers: the mean of the individually sparsified deltas (float64 reference of the same sum)
    want = sum(O.topk_sparsify(tg - th, frac).astype(np.float64) for th in thetas) / K
    got = O.sparsified_pseudogradient(tg, thetas, frac)
    assert np.abs(got - want).max() < 1e-6
    # error feedback with beta = 1: what was not sent stays in E, entry by entry and exactly
    # (a kept entry leaves 0 behind, a dropped entry is carried whole)
    ef = [np.zeros_like(tg) for _ in range(K)]
    sent_total = [np.zeros(tg.shape, np.float64) for _ in range(K)]
    delta_total = [np.zeros(tg.shape, np.float64) for _ in range(K)]
    for rnd in range(4):
        thetas = [(tg - 0.1 * rng.standard_normal(tg.shape)).astype(np.float32) for _ in range(K)]
        before = [e.copy() for e in ef]
        O.sparsified_pseudogradient(tg, thetas, frac, ef, 1.0)
        for k in range(K):
            e_in = (before[k] + (tg - thetas[k])).astype(np.float32)
            sent = O.topk_sparsify(e_in, frac)
            assert np.array_equal(ef[k], np.where(sent != 0, 0, e_in).astype(np.float32))
            assert np.count_nonzero(ef[k]) == tg.size - O.topk_count(tg.size, frac)
            sent_total[k] += sent
            delta_total[k] += (tg - thetas[k]).astype(np.float32)
    for k in range(K):
        assert np.abs(ef[k] + sent_total[k] - delta_total[k]).max() < 1e-5
    # beta = 0: the accumulator is overwritten, so the sent part equals that of the run without it
    ef0 = [rng.standard_normal(tg.shape).astype(np.float32) for _ in range(K)]
    assert np.array_equal(O.sparsified_pseudogradient(tg, thetas, frac, ef0, 0.0),
                          O.sparsified_pseudogradient(tg, thetas, frac))


def test_oracle_sync_with_topk_runs_algorithm_2():
    rng = np.random.default_rng(703)
    specs = [O.TensorSpec("a", 6, 10), O.TensorSpec("b", 1, 17, kind="adamw")]
    init = [rng.standard_normal((s.rows, s.cols)).astype(np.float32) for s in specs]
    cfg = O.OracleConfig(K=2, H=1, outer_lr=0.5, outer_momentum=0.0, topk_fraction=0.25, error_feedback=True)
    orc = O.MuLoCoOracle(cfg, specs, init)
    for k in range(2):
        for i in range(2):
            orc.theta_k[k][i] += rng.standard_normal(init[i].shape).astype(np.float32)
    tg0 = [w.copy() for w in orc.theta_g]
    d = [[(tg0[i] - orc.theta_k[k][i]).astype(np.float32) for i in range(2)] for k in range(2)]
    orc.outer_sync()
    for i in range(2):
        psi = (O.topk_sparsify(d[0][i], 0.25).astype(np.float64) + O.topk_sparsify(d[1][i], 0.25)) / 2
        assert np.abs(orc.theta_g[i] - (tg0[i] - 0.5 * psi)).max() < 1e-6     # mu = 0: plain SGD outer step
        assert np.array_equal(orc.theta_k[0][i], orc.theta_g[i])
        assert np.count_nonzero(orc.ef[0][i]) == init[i].size - O.topk_count(init[i].size, 0.25)
    with pytest.raises(ValueError):
        O.MuLoCoOracle(O.OracleConfig(K=2, H=1, topk_fraction=0.1, quant_bits=8), specs, init)
