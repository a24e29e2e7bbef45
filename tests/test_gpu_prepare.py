"""Factor preparation on the GPU (Section 3.1, Section 3.2, Appendix A) against the oracle's.

Singular vectors are unique only up to sign (and rotation inside a cluster of equal singular values), and the GPU's
truncated SVD is an iteration, so factors are never compared entry by entry.  What is unique and fixed by the
paper is held instead: W_q bit for bit; the S-weighted residual ||S (E_q - A B)||_F against the optimum that the
oracle's exact SVD gives (Eckart-Young: the root of the sum of the discarded sigma^2), from above and within
one per cent (the error of a quantiser is close to white noise, so its spectrum is flat and a subspace iteration
of four rounds stops a few parts in a thousand above the optimum; with outlier-scaled rows it is much closer); the orthonormality of S A; and the layer built from the GPU's factors against the oracle's
forward pass with those same factors.
"""
import numpy as np
import pytest
import torch

import lqer_inputs as gen
import paper_2402_02446_b200 as L
from oracle import lqer as olqer
from oracle import mxint
from helpers import exp_bytes, worst_ratio

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _t(a):
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


def _samples(spec, rows):
    # several calibration samples of different lengths with the layer's outlier channels
    return [gen.make_activations(gen.LayerSpec(spec.name, M=r, K=spec.K, N=spec.N, k=spec.k, calib_rows=r,
                                               outlier_frac=spec.outlier_frac, outlier_scale=spec.outlier_scale,
                                               weight_law=spec.weight_law, seed=spec.seed + 100 * i, n_outliers=spec.n_outliers))
            for i, r in enumerate(rows)]


CASES = [
    ("l2qer_mid", gen.LayerSpec("pp_a", M=40, K=512, N=384, k=16, calib_rows=64, outlier_frac=0.02, outlier_scale=20.0, seed=501), (96, 33, 128), 4),
    ("plain_lqer", gen.LayerSpec("pp_b", M=40, K=256, N=320, k=24, calib_rows=64, outlier_frac=0.02, outlier_scale=20.0, seed=502), (), 4),
    ("w2_rank256", gen.LayerSpec("pp_c", M=40, K=512, N=320, k=256, calib_rows=64, outlier_frac=0.01, outlier_scale=50.0,
                                 weight_law="student_t4", seed=503), (200,), 2),
    ("odd_rank", gen.LayerSpec("pp_d", M=40, K=320, N=136, k=5, calib_rows=64, outlier_frac=0.0, n_outliers=3, outlier_scale=20.0, seed=504), (50, 50), 4),
]


@pytest.mark.parametrize("name,spec,rows,w_bits", CASES, ids=[c[0] for c in CASES])
def test_prepare_from_calibration_against_the_exact_svd(name, spec, rows, w_bits):
    W = gen.make_weight(spec)
    samples = _samples(spec, rows)
    cfg = L.default_config()
    cfg.w_bits = w_bits
    Pg, A, B, code = L.prepare_from_calibration(_t(W), [_t(x) for x in samples], spec.k, cfg=cfg, seed=spec.seed)
    assert code == 0
    A = A.cpu().numpy().astype(np.float64)
    B = B.cpu().numpy().astype(np.float64)
    # the oracle's side: W_q, E_q, S, the exact spectrum of S E_q
    Wm, We = olqer.quantize_weight(W, w_bits=w_bits)
    ex = L.export_weights(Pg)
    assert np.array_equal(ex["Wm"].cpu().numpy(), Wm) and np.array_equal(ex["We"].cpu().numpy(), exp_bytes(We))
    E = olqer.quantization_error(W, Wm, We, w_bits=w_bits)
    s = olqer.calibration_scale(samples) if rows else np.ones(spec.K)
    _, sig, _ = olqer.jacobi_svd(s[:, None] * E)
    optimum = float(np.sqrt(np.sum(sig[spec.k:] ** 2)))
    got = float(np.linalg.norm(s[:, None] * (E - A @ B)))
    assert optimum * (1 - 1e-6) <= got <= optimum * (1 + 1e-2), (got, optimum)
    # S A has orthonormal columns (A = S^-1 U_k), and B = (S A)^T (S E_q) (B = Sigma_k V_k^T = U_k^T S E_q)
    SA = s[:, None] * A
    assert np.max(np.abs(SA.T @ SA - np.eye(spec.k))) < 1e-5
    assert np.max(np.abs(B - SA.T @ (s[:, None] * E))) < 1e-5 * float(np.abs(B).max())
    # singular values: the row norms of B are the leading sigma of S E_q
    assert np.allclose(np.linalg.norm(B, axis=1), sig[:spec.k], rtol=2e-2)
    # the packed layer: quantised factors bit for bit, forward pass within the layer's tolerance
    P = olqer.prepare_weights(W, A.astype(np.float32), B.astype(np.float32), w_bits=w_bits)
    assert np.array_equal(ex["Am"].cpu().numpy(), P.Am) and np.array_equal(ex["Bm"].cpu().numpy(), P.Bm)
    assert np.array_equal(ex["Ae"].cpu().numpy(), exp_bytes(P.Ae)) and np.array_equal(ex["Be"].cpu().numpy(), exp_bytes(P.Be))
    X = gen.make_activations(spec)
    ref = olqer.forward(X, P, w_bits=w_bits)
    ws = L.new_workspace(spec.M, Pg)
    for M in (1, 9, spec.M):
        r = olqer.forward(X[:M], P, w_bits=w_bits)
        assert worst_ratio(L.linear(_t(X[:M]), Pg, ws).cpu().numpy(), r) <= 1.0, M
    # the correction does what the paper builds it for: a smaller output error than W_q alone
    Yfull = X.astype(np.float64) @ W.astype(np.float64)
    Xdq = mxint.dequantize(ref.Xm, ref.Xe, 8, axis=1)
    Yq = Xdq @ mxint.dequantize(Wm, We, w_bits, axis=0)
    assert np.linalg.norm(ref.Y - Yfull) < np.linalg.norm(Yq - Yfull)
    Pg.release()


def test_prepare_reports_a_dead_calibration_channel():
    spec = CASES[0][1]
    W = gen.make_weight(spec)
    x = _samples(spec, (64,))[0]
    x[:, 7] = 0.0                                 # S would not be invertible (Section 3.2 assumes this never happens)
    Pg, A, B, code = L.prepare_from_calibration(_t(W), [_t(x)], spec.k, seed=1)
    assert code == 1
    with pytest.raises(ValueError):
        olqer.calibration_scale([x])
    Pg.release()
