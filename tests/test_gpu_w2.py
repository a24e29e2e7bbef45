"""W2A8 (Section 4.4): 2-bit mantissas for W_q, ranks up to 256, against the oracle through the C ABI."""
import numpy as np
import pytest
import torch

import lqer_inputs as gen
import paper_2402_02446_b200 as L
from paper_2402_02446_b200 import binding
from oracle import lqer as olqer
from helpers import exp_bytes, worst_ratio

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _t(a):
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


def _cfg():
    cfg = L.default_config()
    cfg.w_bits = 2
    return cfg


def _layer(spec, plain_lqer=False):
    """Factors by the oracle's own preparation from the 2-bit quantisation error where that is quick (plain LQER,
    S = I, or L2QER), seeded stand-ins otherwise."""
    W = gen.make_weight(spec)
    if spec.k == 0:
        return W, None, None
    if spec.K * spec.N <= 1024 * 640:
        Wm, We = olqer.quantize_weight(W, w_bits=2)
        E = olqer.quantization_error(W, Wm, We, w_bits=2)
        s = None if plain_lqer else olqer.calibration_scale(gen.make_calibration(spec))
        A, B, _ = olqer.lqer_factors(E, spec.k, s, method="subspace", rng=np.random.default_rng(spec.seed))
        return W, np.ascontiguousarray(A, dtype=np.float32), np.ascontiguousarray(B, dtype=np.float32)
    A, B = gen.make_random_factors(spec)
    return W, A, B


SPECS = [
    gen.LayerSpec("w2_tiny", M=16, K=256, N=256, k=8, calib_rows=64, outlier_frac=0.0, n_outliers=4, outlier_scale=20.0, seed=401),
    gen.LayerSpec("w2_odd", M=37, K=80, N=136, k=5, calib_rows=48, outlier_frac=0, n_outliers=2, outlier_scale=20.0, seed=402),
    gen.LayerSpec("w2_k0", M=129, K=512, N=384, k=0, calib_rows=64, outlier_frac=0.01, outlier_scale=20.0, seed=403),
    gen.LayerSpec("w2_rank256", M=300, K=1024, N=640, k=256, calib_rows=128, outlier_frac=0.01, outlier_scale=20.0,
                  weight_law="student_t4", seed=404),
]


@pytest.mark.parametrize("spec", SPECS, ids=lambda s: s.name)
def test_two_bit_weights_pack_and_layer(spec, ratio_log):
    W, A, B = _layer(spec, plain_lqer=spec.name == "w2_tiny")
    P = olqer.prepare_weights(W, A, B, w_bits=2)
    Pg = L.prepare_weights(_t(W), None if A is None else _t(A), None if B is None else _t(B), _cfg())
    assert L.packed_bytes(spec.K, spec.N, spec.k, _cfg()) < L.packed_bytes(spec.K, spec.N, spec.k)
    ex = L.export_weights(Pg)
    torch.cuda.synchronize()
    assert np.array_equal(ex["Wm"].cpu().numpy(), P.Wm) and set(np.unique(P.Wm)) <= {-1, 0, 1}
    assert np.array_equal(ex["We"].cpu().numpy(), exp_bytes(P.We))
    if spec.k:
        assert np.array_equal(ex["Bm"].cpu().numpy(), P.Bm) and np.array_equal(ex["Am"].cpu().numpy(), P.Am)
    ws = L.new_workspace(spec.M, Pg)
    # every path: the checking kernel, the small-batch kernels (1 .. 100 rows; path 5 at up to 16 rows: the register-operand
    # GEMM on crumbs), the large-batch GEMM with either prologue
    for M, path in ((spec.M, binding.PATH_SIMT), (1, binding.PATH_AUTO), (4, binding.PATH_AUTO), (9, binding.PATH_AUTO),
                    (9, binding.PATH_SMALL), (16, binding.PATH_SMALL), (100, binding.PATH_AUTO), (spec.M, binding.PATH_TENSOR), (spec.M, binding.PATH_TENSOR_PAIR),
                    (spec.M, binding.PATH_AUTO)):
        if M > spec.M:
            continue
        X = gen.make_activations(spec, M=M)
        ref = olqer.forward(X, P, w_bits=2)
        L.set_path(path)
        try:
            Y = L.linear(_t(X), Pg, ws).cpu().numpy()
        finally:
            L.set_path(binding.PATH_AUTO)
        assert L.poll_status(ws) == 0
        assert ratio_log(spec.name, worst_ratio(Y, ref)) <= 1.0, (M, path)
    Pg.release()


def test_two_bit_every_crumb_position():
    # one-hot columns: each K position of a 64-slab lands in its own crumb and comes back
    K, N = 128, 128
    W = np.zeros((K, N), np.float32)
    for kk in range(K):
        W[kk, kk] = (-1.0) ** kk * 0.25 * (1 + kk % 3)
        W[(kk + 5) % K, kk] = 0.25 * (-1.0) ** (kk // 3)
    Pg = L.prepare_weights(_t(W), None, None, _cfg())
    ex = L.export_weights(Pg)
    Wm, We = olqer.quantize_weight(W, w_bits=2)
    assert np.array_equal(ex["Wm"].cpu().numpy(), Wm)
    assert np.array_equal(ex["We"].cpu().numpy(), exp_bytes(We))
    Pg.release()


def test_two_bit_full_size_sampled_rows(ratio_log):
    # the 13B-shaped layer with rank 256 (Section 4.4's setting): prefill rows sampled per tile, and a decode batch
    spec = gen.config_sweep(5120, 512, 256)
    W = gen.make_weight(spec)
    A, B = gen.make_random_factors(spec)
    P = olqer.prepare_weights(W, A, B, w_bits=2)
    Pg = L.prepare_weights(_t(W), _t(A), _t(B), _cfg())
    X = gen.make_activations(spec)
    rows = [0, 130, 259, 300, 511]
    ref = olqer.forward(X[rows], P, w_bits=2)
    ws = L.new_workspace(spec.M, Pg)
    Y = L.linear(_t(X), Pg, ws)
    assert L.poll_status(ws) == 0
    assert ratio_log(spec.name + "_w2", worst_ratio(Y[torch.tensor(rows, device=DEV)].cpu().numpy(), ref)) <= 1.0
    for M in (1, 16):
        r1 = olqer.forward(X[:M], P, w_bits=2)
        y1 = L.linear(_t(X[:M]), Pg, ws).cpu().numpy()
        assert worst_ratio(y1, r1) <= 1.0, M
    Pg.release()


@pytest.mark.parametrize("M", [1, 3])
def test_two_bit_batched_decode_shares_launches(M):
    # the column-owner decode kernel on crumbs: a stretch of independent calls shares launches (activations quantised
    # ahead by one kernel), and every result equals the single call's bit for bit and the oracle's within the tolerance
    specs = [gen.LayerSpec("w2_dec_a", M=M, K=1024, N=640, k=40, calib_rows=32, outlier_frac=0.01, outlier_scale=20.0, seed=411),
             gen.LayerSpec("w2_dec_b", M=M, K=2112, N=264, k=72, calib_rows=32, outlier_frac=0.01, outlier_scale=20.0, seed=412)]
    layers = []
    for s in specs:
        W = gen.make_weight(s)
        A, B = gen.make_random_factors(s)
        layers.append((olqer.prepare_weights(W, A, B, w_bits=2), L.prepare_weights(_t(W), _t(A), _t(B), _cfg())))
    order = [0, 1] * 10                                   # 20 calls: more than one launch of 16
    Xs = [gen.make_activations(specs[i], M=M) + 0.125 * j for j, i in enumerate(order)]
    Xd = [_t(X) for X in Xs]
    Yb = [torch.full((M, specs[i].N), float("nan"), dtype=torch.float32, device=DEV) for i in order]
    calls = L.make_calls([(x, layers[i][1], y) for x, i, y in zip(Xd, order, Yb)])
    ws = torch.zeros(L.batched_workspace_bytes(calls), dtype=torch.uint8, device=DEV)
    before = L.launch_count()
    L.linear_batched(calls, ws)
    torch.cuda.synchronize()
    assert L.launch_count() - before == 3                 # activations ahead + two decode launches (16 + 4 layers)
    assert L.poll_status(ws) == 0
    for x, X, i, y in zip(Xd, Xs, order, Yb):
        single = L.linear(x, layers[i][1], ws)
        assert torch.equal(single, y)
        assert worst_ratio(y.cpu().numpy(), olqer.forward(X, layers[i][0], w_bits=2)) <= 1.0
    for _, Pg in layers:
        Pg.release()


@pytest.mark.parametrize("M", [6, 16])
def test_two_bit_small_batches_share_launches(M):
    # twelve independent calls above the column-owner kernel's range: one launch of the small prologue and one of the
    # register-operand GEMM (crumbs converted in registers), every result within the tolerance of the oracle's and
    # the second run of the batch equal to the first bit for bit
    specs = [gen.LayerSpec("w2_sm_a", M=M, K=1024, N=640, k=40, calib_rows=32, outlier_frac=0.01, outlier_scale=20.0, seed=421),
             gen.LayerSpec("w2_sm_b", M=M, K=2112, N=264, k=72, calib_rows=32, outlier_frac=0.01, outlier_scale=20.0, seed=422)]
    layers = []
    for s in specs:
        W = gen.make_weight(s)
        A, B = gen.make_random_factors(s)
        layers.append((olqer.prepare_weights(W, A, B, w_bits=2), L.prepare_weights(_t(W), _t(A), _t(B), _cfg())))
    order = [0, 1] * 6
    Xs = [gen.make_activations(specs[i], M=M) + 0.125 * j for j, i in enumerate(order)]
    Xd = [_t(X) for X in Xs]
    Yb = [torch.full((M, specs[i].N), float("nan"), dtype=torch.float32, device=DEV) for i in order]
    calls = L.make_calls([(x, layers[i][1], y) for x, i, y in zip(Xd, order, Yb)])
    ws = torch.zeros(L.batched_workspace_bytes(calls), dtype=torch.uint8, device=DEV)
    first = None
    for rep in range(2):
        before = L.launch_count()
        L.linear_batched(calls, ws)
        torch.cuda.synchronize()
        assert L.launch_count() - before == 2
        assert L.poll_status(ws) == 0
        if first is None:
            first = [y.clone() for y in Yb]
        else:
            assert all(torch.equal(a, b) for a, b in zip(first, Yb))
    for X, i, y in zip(Xs, order, Yb):
        assert worst_ratio(y.cpu().numpy(), olqer.forward(X, layers[i][0], w_bits=2)) <= 1.0
    for _, Pg in layers:
        Pg.release()
