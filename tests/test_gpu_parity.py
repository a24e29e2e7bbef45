"""GPU parity: the CUDA path against the CPU oracle, element by element, through the C ABI."""
import numpy as np
import pytest
import torch

import lqer_inputs as gen
import paper_2402_02446_b200 as L
from paper_2402_02446_b200 import binding
from oracle import lqer as olqer
from oracle import mxint
from helpers import exp_bytes, oracle_layer, worst_ratio

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _t(a):
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


def _prepare(spec, method="jacobi"):
    W, A, B, P = oracle_layer(spec, method)
    Pg = L.prepare_weights(_t(W), None if A is None else _t(A), None if B is None else _t(B))
    return W, A, B, P, Pg


SMALL_SPECS = [
    gen.config_tiny(),
    gen.LayerSpec("odd", M=37, K=80, N=136, k=5, calib_rows=48, outlier_frac=0, n_outliers=2, outlier_scale=20.0, seed=11),
    gen.LayerSpec("k0", M=20, K=192, N=256, k=0, calib_rows=32, outlier_frac=0, n_outliers=2, outlier_scale=20.0, seed=12),
    gen.LayerSpec("wide_rank", M=150, K=320, N=392, k=72, calib_rows=64, outlier_frac=0.02, outlier_scale=50.0,
                  weight_law="student_t4", seed=13),
]


@pytest.mark.parametrize("spec", SMALL_SPECS, ids=lambda s: s.name)
def test_prepare_weights_bit_exact(spec):
    W, A, B, P, Pg = _prepare(spec)
    ex = L.export_weights(Pg)
    torch.cuda.synchronize()
    assert np.array_equal(ex["Wm"].cpu().numpy(), P.Wm)
    assert np.array_equal(ex["We"].cpu().numpy(), exp_bytes(P.We))
    if spec.k:
        assert np.array_equal(ex["Am"].cpu().numpy(), P.Am)
        assert np.array_equal(ex["Ae"].cpu().numpy(), exp_bytes(P.Ae))
        assert np.array_equal(ex["Bm"].cpu().numpy(), P.Bm)
        assert np.array_equal(ex["Be"].cpu().numpy(), exp_bytes(P.Be))
    Pg.release()


def test_prepare_weights_every_nibble_position():
    # one-hot columns: each K position of a 64-slab lands in its own nibble and comes back
    K, N = 128, 128
    W = np.zeros((K, N), np.float32)
    for kk in range(K):
        W[kk, kk] = (1 + kk % 7) * (-1.0) ** kk * 0.25
    Pg = L.prepare_weights(_t(W), None, None)
    ex = L.export_weights(Pg)
    Wm, We = olqer.quantize_weight(W)
    assert np.array_equal(ex["Wm"].cpu().numpy(), Wm)
    assert np.array_equal(ex["We"].cpu().numpy(), exp_bytes(We))
    Pg.release()


def _adversarial_x():
    g = np.random.default_rng(21)
    X = g.standard_normal((64, 256)).astype(np.float32)
    X *= np.exp2(g.integers(-30, 30, size=(64, 16))).repeat(16, axis=1).astype(np.float32)
    X[0, :16] = 0.0                                     # all-zero block
    X[1, :16] = [1, 0.0234375, 0.0390625, 0.0078125, 0.0546875, -0.0078125, -0.0234375] + [0] * 9   # ties
    X[2, 0] = 3.99; X[2, 1:16] = 0.01                   # clipped maximum
    X[3, :16] = np.float32(1e-40)                       # subnormal block
    X[4, 0] = np.float32(3e38); X[4, 1] = -1.0          # above the window
    X[5, 0] = np.inf; X[5, 1] = -np.inf; X[5, 2] = 1.0
    X[6, 0] = np.nan; X[6, 1] = 0.75
    X[7, :16] = np.nextafter(np.float32(2.0), np.float32(0))  # just below a power of two
    X[8, :16] = 2.0 ** -60                              # below the window
    X[9, :16] = np.arange(16, dtype=np.float32) * 0.5 / 64.0  # exact half-step ties at e=... many
    return X


def test_quantize_activations_bit_exact():
    for X in (_adversarial_x(), gen.make_activations(gen.config_tiny()), gen.make_activations(gen.config_decode(4))):
        Xm, Xe = L.quantize_activations(_t(X))
        om, oe = mxint.quantize(X, 8, axis=1)
        assert np.array_equal(Xm.cpu().numpy(), om)
        assert np.array_equal(Xe.cpu().numpy(), exp_bytes(oe))


@pytest.mark.parametrize("spec", [s for s in SMALL_SPECS if s.k], ids=lambda s: s.name)
def test_project_lowrank_bit_exact(spec):
    W, A, B, P, Pg = _prepare(spec)
    X = gen.make_activations(spec)
    ref = olqer.forward(X, P)
    ws = L.new_workspace(spec.M, Pg)
    Tm, Te = L.project_lowrank(_t(X), Pg, ws)
    assert np.array_equal(Tm.cpu().numpy(), ref.Tm)
    assert np.array_equal(Te.cpu().numpy(), exp_bytes(ref.Te))
    assert L.poll_status(ws) == 0
    Pg.release()


@pytest.mark.parametrize("spec", SMALL_SPECS, ids=lambda s: s.name)
def test_linear_reference_kernel(spec):
    W, A, B, P, Pg = _prepare(spec)
    X = gen.make_activations(spec)
    ref = olqer.forward(X, P)
    ws = L.new_workspace(spec.M, Pg)
    L.set_path(binding.PATH_SIMT)
    try:
        Y = L.linear(_t(X), Pg, ws).cpu().numpy()
    finally:
        L.set_path(binding.PATH_AUTO)
    assert worst_ratio(Y, ref) <= 1.0
    assert L.poll_status(ws) == 0
    Pg.release()


MID_SPECS = [
    gen.LayerSpec("mid_odd_tiles", M=300, K=1024, N=640, k=40, calib_rows=128, outlier_frac=0.01, outlier_scale=20.0, seed=31),
    gen.LayerSpec("mid_k0", M=129, K=512, N=384, k=0, calib_rows=64, outlier_frac=0.01, outlier_scale=20.0, seed=32),
    gen.LayerSpec("mid_rank96", M=257, K=2048, N=512, k=96, calib_rows=128, outlier_frac=0.005, outlier_scale=50.0,
                  weight_law="student_t4", seed=33),
]


@pytest.mark.parametrize("path", [binding.PATH_TENSOR, binding.PATH_TENSOR_PAIR], ids=["cta1", "cta2"])
@pytest.mark.parametrize("spec", SMALL_SPECS + MID_SPECS, ids=lambda s: s.name)
def test_linear_tensor_core_kernel(spec, path):
    W, A, B, P, Pg = _prepare(spec, "jacobi" if spec.K <= 320 else "subspace")
    X = gen.make_activations(spec)
    ref = olqer.forward(X, P)
    ws = L.new_workspace(spec.M, Pg)
    L.set_path(path)
    try:
        Y = L.linear(_t(X), Pg, ws).cpu().numpy()
        Y2 = L.linear(_t(X), Pg, ws).cpu().numpy()
    finally:
        L.set_path(binding.PATH_AUTO)
    assert L.poll_status(ws) == 0
    assert worst_ratio(Y, ref) <= 1.0
    assert np.array_equal(Y, Y2)          # fixed reduction order: bit-identical run to run
    Pg.release()
