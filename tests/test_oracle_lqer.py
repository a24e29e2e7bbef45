"""Pins for the oracle's weight preparation and inference layer."""
import os
from fractions import Fraction

import numpy as np
import pytest

import lqer_inputs as gen
from oracle import lqer, mxint

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "calibration_example.txt")


def test_calibration_hand_example():
    samples, want = [], None
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            parts = [p.strip() for p in line.split(";")]
            rows = [[float(x) for x in p.split()] for p in parts[1:]]
            if parts[0] == "sample":
                samples.append(np.array(rows))
            else:
                want = np.array(rows[0])
    s = lqer.calibration_scale(samples)
    assert np.allclose(s, want, rtol=0, atol=1e-15)


def test_calibration_normalisation_and_order():
    g = np.random.default_rng(0)
    xs = [np.abs(g.standard_normal((r, 12))) + 0.1 for r in (5, 9, 3)]
    s = lqer.calibration_scale(xs)
    assert np.isclose(s.min() * s.max(), 1.0, rtol=1e-14)
    # mean is over tokens within a sample, max is across samples: not the other way round
    a = np.stack([x.mean(axis=0) for x in xs]).max(axis=0)
    assert np.allclose(s / s[0], a / a[0], rtol=1e-14)
    wrong = np.concatenate(xs).mean(axis=0)
    assert not np.allclose(s / s[0], wrong / wrong[0], rtol=1e-6)
    with pytest.raises(ValueError):
        lqer.calibration_scale([np.array([[1.0, 0.0], [2.0, 0.0]])])


def _small_layer(K=64, N=48, seed=1, outliers=3):
    spec = gen.LayerSpec("t", M=8, K=K, N=N, k=8, calib_rows=32, outlier_frac=0, n_outliers=outliers,
                         outlier_scale=20.0, seed=seed)
    return spec, gen.make_weight(spec), gen.make_activations(spec), gen.make_calibration(spec)


def test_full_rank_identity():
    # At k = min(K, N) the correction reproduces E_q, so W_q + A_k B_k = W (Section 3.1, 3.2).
    spec, W, X, calib = _small_layer()
    Wm, We = lqer.quantize_weight(W)
    E = lqer.quantization_error(W, Wm, We)
    assert np.abs(E).max() > 1e-4                       # the quantiser did lose something
    s = lqer.calibration_scale(calib)
    for scale in (None, s):
        A, B, _ = lqer.lqer_factors(E, min(W.shape), scale)
        assert np.abs(mxint.dequantize(Wm, We, 4, 0) + A @ B - W.astype(np.float64)).max() < 1e-10


def test_weighted_residual_closed_form_and_monotone():
    # Eckart-Young on S E_q: ||S (E_q - A_k B_k)||_F^2 = sum_{i>k} sigma'_i^2, hence non-increasing in k.
    spec, W, X, calib = _small_layer(seed=2)
    Wm, We = lqer.quantize_weight(W)
    E = lqer.quantization_error(W, Wm, We)
    s = lqer.calibration_scale(calib)
    prev = np.inf
    for k in (0, 1, 4, 8, 16, 32, 48):
        A, B, sig = lqer.lqer_factors(E, k, s)
        res = np.sum((s[:, None] * (E - A @ B)) ** 2)
        assert np.isclose(res, np.sum(sig[k:] ** 2), rtol=1e-9, atol=1e-18)
        assert res <= prev * (1 + 1e-12)
        prev = res
        # B = U'_k^T (S E_q): the rows of B are the projections on the left singular vectors
        U = A * s[:, None]
        assert np.allclose(B, U.T @ (s[:, None] * E), atol=1e-12)
    # plain LQER (S = I): the unweighted error norm is monotone too
    prev = np.inf
    for k in (0, 2, 8, 24, 48):
        A, B, sig = lqer.lqer_factors(E, k, None)
        res = np.sum((E - A @ B) ** 2)
        assert np.isclose(res, np.sum(sig[k:] ** 2), rtol=1e-9, atol=1e-18)
        assert res <= prev * (1 + 1e-12)
        prev = res
        assert np.abs(A.T @ A - np.eye(k)).max() < 1e-12 if k else True


def test_scaling_steepens_the_spectrum():
    # With outlier channels S concentrates the spectrum of S E_q in its first components (Section 1, 3.2).
    spec, W, X, calib = _small_layer(K=128, N=96, seed=3, outliers=4)
    Wm, We = lqer.quantize_weight(W)
    E = lqer.quantization_error(W, Wm, We)
    s = lqer.calibration_scale(calib)
    _, _, sig_plain = lqer.lqer_factors(E, 4, None)
    _, _, sig_scaled = lqer.lqer_factors(E, 4, s)
    frac = lambda sg: np.sum(sg[:4] ** 2) / np.sum(sg ** 2)
    assert frac(sig_scaled) > 2 * frac(sig_plain)
    # and the activation-weighted output error is smaller with the scaled factors
    A0, B0, _ = lqer.lqer_factors(E, 4, None)
    A1, B1, _ = lqer.lqer_factors(E, 4, s)
    Xd = X.astype(np.float64)
    err0 = np.linalg.norm(Xd @ (E - A0 @ B0))
    err1 = np.linalg.norm(Xd @ (E - A1 @ B1))
    assert err1 < err0


def test_approximation_error_and_average_bits():
    E = np.array([[1.0, -2.0], [0.5, 0.0]])
    assert lqer.approximation_error(E, np.zeros((2, 1)), np.zeros((1, 2))) == pytest.approx(0.875)
    # Appendix D bookkeeping: 4-bit mantissa + 4-bit exponent per 16 = 4.25 bits for W_q alone;
    # with the k = 32 factors the paper's table reports 4.3 for LLaMA-sized layers.
    assert lqer.average_weight_bits(4096, 4096, 0) == 4.25
    for K, N in ((4096, 4096), (4096, 11008), (11008, 4096), (5120, 13824)):
        assert round(lqer.average_weight_bits(K, N, 32), 1) in (4.3, 4.4)
    assert abs(lqer.average_weight_bits(4096, 11008, 32) - 4.3) < 0.05
    # extra multiplies of the correction: (m + n) k / (m n) ~ 0.01 k % for OPT-175B FFN shapes (Section 3.1)
    m, n, k = 12288, 49152, 32
    assert abs((m + n) * k / (m * n) * 100 - 0.01 * k) < 0.01 * k * 0.05


def _exact_forward(Xm, Xe, P, Tm, Te, w_bits=4):
    """Y from integer mantissas in exact rational arithmetic (definition of the MXINT dot, Section 2.2)."""
    M, K = Xm.shape
    Y = [[Fraction(0)] * P.N for _ in range(M)]
    for i in range(M):
        for j in range(P.N):
            acc = Fraction(0)
            for kk in range(K):
                acc += int(Xm[i, kk]) * int(P.Wm[kk, j]) * Fraction(2) ** (int(Xe[i, kk // 16]) - 6 + int(P.We[kk // 16, j]) - (w_bits - 2))
            for r in range(P.k_pad):
                acc += int(Tm[i, r]) * int(P.Bm[r, j]) * Fraction(2) ** (int(Te[i, r // 16]) - 6 + int(P.Be[r // 16, j]) - 6)
            Y[i][j] = acc
    return Y


def test_forward_against_exact_rational_brute_force():
    spec = gen.LayerSpec("t", M=3, K=48, N=20, k=5, calib_rows=16, outlier_frac=0, n_outliers=2,
                         outlier_scale=20.0, seed=7)
    W, X, calib = gen.make_weight(spec), gen.make_activations(spec), gen.make_calibration(spec)
    Wm, We = lqer.quantize_weight(W)
    A, B, _ = lqer.lqer_factors(lqer.quantization_error(W, Wm, We), spec.k, lqer.calibration_scale(calib))
    P = lqer.prepare_weights(W, A, B)
    assert P.k_pad == 16 and not P.Bm[5:].any()
    out = lqer.forward(X, P)
    # T itself, exactly
    for i in range(spec.M):
        for r in range(spec.k):
            t = sum(int(out.Xm[i, kk]) * int(P.Am[kk, r]) * Fraction(2) ** (int(out.Xe[i, kk // 16]) - 6 + int(P.Ae[kk // 16, r]) - 6)
                    for kk in range(spec.K))
            assert Fraction(float(out.T[i, r])) == t
    Yex = _exact_forward(out.Xm, out.Xe, P, out.Tm, out.Te)
    for i in range(spec.M):
        for j in range(spec.N):
            assert abs(float(Yex[i][j]) - out.Y[i, j]) <= 1e-13 * max(1.0, abs(out.Y[i, j]))
    # the corrected layer is closer to X W than the uncorrected one (what the method is for)
    ref = X.astype(np.float64) @ W.astype(np.float64)
    P0 = lqer.prepare_weights(W, None, None)
    assert np.linalg.norm(out.Y - ref) < np.linalg.norm(lqer.forward(X, P0).Y - ref)


def test_forward_special_cases():
    spec, W, X, calib = _small_layer(seed=4)
    Wm, We = lqer.quantize_weight(W)
    E = lqer.quantization_error(W, Wm, We)
    A, B, _ = lqer.lqer_factors(E, 8, lqer.calibration_scale(calib))
    P = lqer.prepare_weights(W, A, B)
    out = lqer.forward(X, P)
    # k = 0: a plain MXINT GEMM
    out0 = lqer.forward(X, lqer.prepare_weights(W, None, None))
    Xdq = mxint.dequantize(out.Xm, out.Xe, 8, 1)
    assert np.array_equal(out0.Y, Xdq @ mxint.dequantize(Wm, We, 4, 0))
    # the correction term is linear in B_q: doubling B (a pure exponent shift) doubles it
    P2 = lqer.prepare_weights(W, A, 2 * B)
    assert np.array_equal(P2.Bm, P.Bm) and np.array_equal(P2.Be, P.Be + 1)
    out2 = lqer.forward(X, P2)
    assert np.allclose(out2.Y - out0.Y, 2 * (out.Y - out0.Y), rtol=1e-12, atol=1e-15)
    # rows are independent: row i of Y depends on row i of X only
    Xp = X.copy(); Xp[2] *= 3.0
    outp = lqer.forward(Xp, P)
    keep = [i for i in range(X.shape[0]) if i != 2]
    assert np.array_equal(outp.Y[keep], out.Y[keep]) and not np.array_equal(outp.Y[2], out.Y[2])
    # X is quantised once: a sign flip of X flips Y exactly
    outn = lqer.forward(-X, P)
    assert np.array_equal(outn.Y, -out.Y)
    # tolerance map is the stated formula and positive
    Tdq = mxint.dequantize(out.Tm, out.Te, 8, 1)
    want = 1e-4 * (np.abs(Xdq) @ np.abs(mxint.dequantize(P.Wm, P.We, 4, 0))
                   + np.abs(Tdq) @ np.abs(mxint.dequantize(P.Bm, P.Be, 8, 0)))
    assert np.allclose(out.tol, want, rtol=1e-14) and np.all(out.tol > 0)


def test_exact_integer_regime():
    # Inputs already on the MXINT grid with equal exponents: every partial sum is a small
    # integer multiple of one step, so the result is exact in any accumulation order.
    g = np.random.default_rng(12)
    K, N, M = 64, 32, 4
    X = g.integers(-127, 128, size=(M, K)).astype(np.float32) / 64.0
    X[:, ::16] = 127 / 64.0                                   # pin every block's exponent to 0
    W = g.integers(-7, 8, size=(K, N)).astype(np.float32) / 4.0
    W[::16, :] = 7 / 4.0
    P = lqer.prepare_weights(W, None, None)
    out = lqer.forward(X, P)
    assert np.array_equal(mxint.dequantize(out.Xm, out.Xe, 8, 1), X)
    assert np.array_equal(mxint.dequantize(P.Wm, P.We, 4, 0), W)
    want = (X.astype(np.float64) * 64).astype(np.int64) @ (W.astype(np.float64) * 4).astype(np.int64)
    assert np.array_equal(out.Y * 256.0, want.astype(np.float64))


def test_prepare_weights_exponent_window():
    # the window of W_q, A_k, B_k is passed through to every one of the three quantisers and nowhere else
    g = np.random.default_rng(5)
    W = (g.standard_normal((64, 24)) * 0.02).astype(np.float32)
    W[:16, 0] = 2.0 ** -20           # a block below the window [-12, 3]
    A = (g.standard_normal((64, 8)) * 0.1).astype(np.float32)
    B = (g.standard_normal((8, 24)) * 0.05).astype(np.float32)
    B[:, 1] = 300.0                   # a block above it
    wide = lqer.prepare_weights(W, A, B)
    narrow = lqer.prepare_weights(W, A, B, exp_min=-12, exp_max=3)
    for name, bits, axis in (("W", 4, 0), ("A", 8, 0), ("B", 8, 0)):
        src = {"W": W, "A": A, "B": mxint.pad_axis(B, axis=0)}[name]
        m, e = mxint.quantize(src, bits, axis=axis, exp_min=-12, exp_max=3)
        assert np.array_equal(getattr(narrow, name + "m"), m) and np.array_equal(getattr(narrow, name + "e"), e)
    assert narrow.We.min() == -12 and narrow.We[0, 0] == -12 and wide.We[0, 0] == -20
    assert narrow.Be.max() == 3 and narrow.Be[0, 1] == 3 and wide.Be[0, 1] == 8
    # blocks inside the window are untouched
    inside = (wide.We >= -12) & (wide.We <= 3)
    assert np.array_equal(np.repeat(inside, 16, axis=0) * narrow.Wm, np.repeat(inside, 16, axis=0) * wide.Wm)
    # the forward pass reads the stored exponents: X keeps its own, wide window
    X = (g.standard_normal((3, 64)) * np.exp2(g.integers(-30, 20, size=(3, 1)))).astype(np.float32)
    ref = lqer.forward(X, narrow)
    assert ref.Xe.min() < -12 or ref.Xe.max() > 3
    Xdq = mxint.dequantize(ref.Xm, ref.Xe, 8, axis=1)
    Wdq = mxint.dequantize(narrow.Wm, narrow.We, 4, axis=0)
    Tdq = mxint.dequantize(ref.Tm, ref.Te, 8, axis=1)
    Bdq = mxint.dequantize(narrow.Bm, narrow.Be, 8, axis=0)
    assert np.allclose(ref.Y, Xdq @ Wdq + Tdq @ Bdq, rtol=1e-13, atol=0)


def test_tiny_config_end_to_end():
    # Config 1 end to end on the oracle alone: the factors come out of the full Jacobi SVD.
    spec = gen.config_tiny()
    W, X, calib = gen.make_weight(spec), gen.make_activations(spec), gen.make_calibration(spec)
    assert X.shape == (16, 256) and W.shape == (256, 256) and calib[0].shape == (128, 256)
    ch = gen.outlier_channels(spec)
    assert ch.size == 4 and np.abs(X[:, ch]).mean() > 8 * np.abs(X).mean() / 2
    Wm, We = lqer.quantize_weight(W)
    E = lqer.quantization_error(W, Wm, We)
    s = lqer.calibration_scale(calib)
    A, B, sig = lqer.lqer_factors(E, spec.k, s)
    P = lqer.prepare_weights(W, A, B)
    out = lqer.forward(X, P)
    ref = X.astype(np.float64) @ W.astype(np.float64)
    e_corr = np.linalg.norm(out.Y - ref)
    e_plain = np.linalg.norm(lqer.forward(X, lqer.prepare_weights(W, None, None)).Y - ref)
    assert e_corr < 0.8 * e_plain


def test_forward_requantises_t_per_rank_block_hand_worked():
    # T = X_q A_q has 20 rank columns -> two blocks of 16 after zero padding, each with its own shared exponent.
    # Worked by hand: X = e_0 (quantises to exactly 1), A's row 0 = a (every entry a multiple of 2^(e-6) of its own
    # block, so A_q = A), hence T row = a.
    #   block 0: a = 0.75, -0.5, 0.3125, 2^-7, 0...   max 0.75 -> e = -1, step 2^-7: m = 96, -64, 40, 1
    #   block 1: a = 40, -3.25, 0.25, 10.75, pad 0... max 40   -> e = 5,  step 2^-1: m = 80, -6 (6.5 -> even), 0 (0.5 -> even), 22 (21.5 -> even)
    # One exponent for the whole padded row (e = 5) would turn block 0 into 1, -1, 1 (0.3125 / 0.5 = 0.625), 0.
    K, N, k = 16, 8, 20
    X = np.zeros((1, K), np.float32); X[0, 0] = 1.0
    A = np.zeros((K, k), np.float32)
    A[0, :4] = [0.75, -0.5, 0.3125, 2.0 ** -7]
    A[0, 16:20] = [40.0, -3.25, 0.25, 10.75]
    B = np.zeros((k, N), np.float32)
    B[:, 0] = 1.0            # sums both blocks
    B[16:, 1] = 1.0          # the second block alone
    B[:16, 2] = 1.0          # the first block alone
    P = lqer.prepare_weights(np.zeros((K, N), np.float32), A, B)
    assert P.k_pad == 32
    r = lqer.forward(X, P)
    assert r.Tm.shape == (1, 32) and r.Te.shape == (1, 2)
    assert r.Te.tolist() == [[-1, 5]]
    assert r.Tm[0, :4].tolist() == [96, -64, 40, 1] and not r.Tm[0, 4:16].any()
    assert r.Tm[0, 16:20].tolist() == [80, -6, 0, 22] and not r.Tm[0, 20:].any()
    first, second = 73.0 / 128.0, 48.0
    assert r.Y[0, 0] == first + second and r.Y[0, 1] == second and r.Y[0, 2] == first
    assert not r.Y[0, 3:].any()


def test_two_bit_weights_with_a_large_rank():
    # W2A8 with k = 256 (Section 4.4): the same layer with 2-bit mantissas for W_q.  The full-rank identity, the exact
    # rational forward pass and the bookkeeping of Appendix D must hold for this width too.
    spec = gen.LayerSpec("w2", M=5, K=64, N=48, k=32, calib_rows=32, outlier_frac=0.0, n_outliers=2, outlier_scale=20.0, seed=21)
    W = gen.make_weight(spec)
    Wm, We = lqer.quantize_weight(W, w_bits=2)
    assert set(np.unique(Wm)) <= {-1, 0, 1}
    E = lqer.quantization_error(W, Wm, We, w_bits=2)
    A, B, _ = lqer.lqer_factors(E, min(spec.K, spec.N), None)             # plain LQER (S = I), full rank
    assert np.allclose(mxint.dequantize(Wm, We, 2, axis=0) + A @ B, W, rtol=0, atol=1e-10)
    s = lqer.calibration_scale(gen.make_calibration(spec))
    A, B, _ = lqer.lqer_factors(E, spec.k, s)
    P = lqer.prepare_weights(W, A.astype(np.float32), B.astype(np.float32), w_bits=2)
    X = gen.make_activations(spec)
    r = lqer.forward(X, P, w_bits=2)
    exact = _exact_forward(r.Xm, r.Xe, P, r.Tm, r.Te, w_bits=2)
    assert np.array_equal(np.array([[float(v) for v in row] for row in exact]), r.Y)
    # a coarser W_q leaves a larger error for the same rank
    E4 = lqer.quantization_error(W, *lqer.quantize_weight(W, w_bits=4), w_bits=4)
    assert np.linalg.norm(E) > 2.0 * np.linalg.norm(E4)
    # 2 + 4/16 bits for W_q alone; with k = 256 on a 13B-shaped layer the factors add about 1.1 bits
    assert lqer.average_weight_bits(5120, 5120, 0, w_bits=2) == 2.25
    assert abs(lqer.average_weight_bits(5120, 13824, 256, w_bits=2) - (2.25 + 256 * (5120 + 13824) * 8.25 / (5120 * 13824))) < 1e-12
