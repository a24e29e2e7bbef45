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


TC_PROLOGUE_SPECS = [
    gen.config_tiny(),
    gen.LayerSpec("odd", M=37, K=80, N=136, k=5, calib_rows=48, outlier_frac=0, n_outliers=2, outlier_scale=20.0, seed=11),
    gen.LayerSpec("tp_rank40", M=300, K=1024, N=640, k=40, calib_rows=128, outlier_frac=0.01, outlier_scale=20.0, seed=31),
    gen.LayerSpec("tp_rank64_tail", M=1100, K=2112, N=256, k=64, calib_rows=128, outlier_frac=0.005, outlier_scale=50.0,
                  weight_law="student_t4", seed=34),     # K = 16.5 panels of 128: a half panel at the end; nine row tiles
    gen.LayerSpec("tp_rank32_k4096", M=260, K=4096, N=256, k=32, calib_rows=128, outlier_frac=0.01, outlier_scale=20.0, seed=35),
]


@pytest.mark.parametrize("spec", TC_PROLOGUE_SPECS, ids=lambda s: s.name)
def test_project_lowrank_tensor_core_prologue_bit_exact(spec):
    # the prologue whose projection runs on the int8 tensor cores, forced at every batch size
    W, A, B, P, Pg = _prepare(spec, "jacobi" if spec.K <= 320 else "subspace")
    X = gen.make_activations(spec)
    ref = olqer.forward(X, P)
    ws = L.new_workspace(spec.M, Pg)
    L.set_path(binding.PATH_TENSOR_PROLOGUE)
    try:
        Tm, Te = L.project_lowrank(_t(X), Pg, ws)
        Y = L.linear(_t(X), Pg, ws).cpu().numpy()
    finally:
        L.set_path(binding.PATH_AUTO)
    assert L.poll_status(ws) == 0
    assert np.array_equal(Tm.cpu().numpy(), ref.Tm)
    assert np.array_equal(Te.cpu().numpy(), exp_bytes(ref.Te))
    assert worst_ratio(Y, ref) <= 1.0
    Pg.release()


@pytest.mark.parametrize("path", [binding.PATH_AUTO, binding.PATH_TENSOR, binding.PATH_TENSOR_PROLOGUE, binding.PATH_SIMT],
                         ids=["auto_small", "mma_sync_prologue", "tensor_prologue", "checking_kernel"])
def test_adversarial_activations_through_every_prologue(path, ratio_log):
    # zero, tie, clipped-maximum, subnormal, out-of-window, infinite and NaN blocks (the quantisers' slow path) through
    # each prologue of the layer: X_q feeds T (bit-exact against the oracle) and Y (within the tolerance)
    spec = gen.LayerSpec("adversarial", M=64, K=256, N=136, k=20, calib_rows=32, outlier_frac=0.01, outlier_scale=20.0, seed=61)
    W, A, B, P, Pg = _prepare(spec)
    X = _adversarial_x()
    ref = olqer.forward(X, P)
    assert np.isfinite(ref.Y).all()
    ws = L.new_workspace(spec.M, Pg)
    L.set_path(path)
    try:
        Tm, Te = L.project_lowrank(_t(X), Pg, ws)
        Y = L.linear(_t(X), Pg, ws).cpu().numpy()
    finally:
        L.set_path(binding.PATH_AUTO)
    assert L.poll_status(ws) == 0
    assert np.array_equal(Tm.cpu().numpy(), ref.Tm)
    assert np.array_equal(Te.cpu().numpy(), exp_bytes(ref.Te))
    assert ratio_log(f"adversarial_path{path}", worst_ratio(Y, ref)) <= 1.0
    Pg.release()


@pytest.mark.parametrize("a_bits", [6, 4])
def test_activation_mantissa_width_option(a_bits):
    # W4A6 (Section 4.3) and a narrower width: X and T = X_q A_q take a_bits mantissa bits, everything else as before.
    # Every path: the decode kernels (M = 1, 3 and 9), the GEMM with either prologue (M = 37, 300), and a stretch of
    # batched decode calls whose activations are quantised ahead.
    cfg = L.default_config()
    cfg.a_bits = a_bits
    for X in (_adversarial_x(), gen.make_activations(gen.config_tiny())):
        Xm, Xe = L.quantize_activations(_t(X), cfg)
        om, oe = mxint.quantize(X, a_bits, axis=1)
        assert np.array_equal(Xm.cpu().numpy(), om)
        assert np.array_equal(Xe.cpu().numpy(), exp_bytes(oe))
    for spec, Ms in ((SMALL_SPECS[1], (2, 37)), (TC_PROLOGUE_SPECS[2], (1, 3, 9, 300))):
        W, A, B, P = oracle_layer(spec, "jacobi" if spec.K <= 320 else "subspace")
        Pg = L.prepare_weights(_t(W), _t(A), _t(B), cfg)
        ws = L.new_workspace(max(Ms), Pg)
        for M in Ms:
            X = gen.make_activations(spec, M=M)
            ref = olqer.forward(X, P, a_bits=a_bits)
            for path in (binding.PATH_AUTO, binding.PATH_TENSOR_PROLOGUE):
                if path != binding.PATH_AUTO and M <= 16:
                    continue
                L.set_path(path)
                try:
                    Tm, Te = L.project_lowrank(_t(X), Pg, ws)
                    Y = L.linear(_t(X), Pg, ws).cpu().numpy()
                finally:
                    L.set_path(binding.PATH_AUTO)
                assert L.poll_status(ws) == 0
                assert np.array_equal(Tm.cpu().numpy(), ref.Tm), (spec.name, M, path)
                assert np.array_equal(Te.cpu().numpy(), exp_bytes(ref.Te)), (spec.name, M, path)
                assert worst_ratio(Y, ref) <= 1.0, (spec.name, M, path)
        if spec.N >= 32 and 1 in Ms:
            Xs = [_t(gen.make_activations(spec, M=1)) + 0.25 * i for i in range(20)]
            Yb = [torch.full((1, spec.N), float("nan"), dtype=torch.float32, device=DEV) for _ in Xs]
            calls = L.make_calls([(x, Pg, y) for x, y in zip(Xs, Yb)])
            wsb = torch.zeros(L.batched_workspace_bytes(calls), dtype=torch.uint8, device=DEV)
            L.linear_batched(calls, wsb)
            torch.cuda.synchronize()
            assert L.poll_status(wsb) == 0
            for i, (x, yb) in enumerate(zip(Xs, Yb)):
                assert torch.equal(L.linear(x, Pg, ws), yb)
                if i in (0, 19):
                    assert worst_ratio(yb.cpu().numpy(), olqer.forward(x.cpu().numpy(), P, a_bits=a_bits)) <= 1.0
        Pg.release()


def test_weight_exponent_window_option():
    # W_q, A_k and B_k with a 4-bit shared exponent (Section 4.1): a window of 16 values, here [-12, 3], while X and T
    # keep the wide one.  Some blocks lie below the window, some above; packing must match the oracle bit for bit and
    # the layer (decode kernels and GEMM) must stay within the tolerance.
    spec = gen.LayerSpec("win", M=40, K=256, N=264, k=24, calib_rows=32, outlier_frac=0.01, outlier_scale=20.0, seed=81)
    W = gen.make_weight(spec)
    W[:, :8] *= np.float32(2.0 ** -12)
    W[:, 8:16] *= np.float32(2.0 ** 9)
    A, B = gen.make_random_factors(spec)
    B[:, 16:24] *= np.float32(2.0 ** 12)
    A[:, :2] *= np.float32(2.0 ** -14)
    cfg = L.default_config()
    cfg.w_exp_min, cfg.w_exp_max = -12, 3
    P = olqer.prepare_weights(W, A, B, exp_min=-12, exp_max=3)
    assert P.We.min() == -12 and P.We.max() == 3 and P.Be.max() == 3 and P.Ae.min() == -12
    Pg = L.prepare_weights(_t(W), _t(A), _t(B), cfg)
    ex = L.export_weights(Pg)
    torch.cuda.synchronize()
    for name in ("Wm", "Am", "Bm"):
        assert np.array_equal(ex[name].cpu().numpy(), getattr(P, name)), name
    for name in ("We", "Ae", "Be"):
        assert np.array_equal(ex[name].cpu().numpy(), exp_bytes(getattr(P, name))), name
    ws = L.new_workspace(spec.M, Pg)
    for M in (1, 5, 40):
        X = gen.make_activations(spec, M=M)
        ref = olqer.forward(X, P)
        Tm, Te = L.project_lowrank(_t(X), Pg, ws)
        Y = L.linear(_t(X), Pg, ws).cpu().numpy()
        assert L.poll_status(ws) == 0
        assert np.array_equal(Tm.cpu().numpy(), ref.Tm) and np.array_equal(Te.cpu().numpy(), exp_bytes(ref.Te)), M
        assert worst_ratio(Y, ref) <= 1.0, M
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


@pytest.mark.parametrize("path", [binding.PATH_TENSOR, binding.PATH_TENSOR_PAIR, binding.PATH_TENSOR_PROLOGUE],
                         ids=["cta1", "cta2", "cta2_tcprologue"])
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


# ---------------------------------------------------------------------------- decode and small-batch kernels (M <= 128)
DECODE_SPECS = SMALL_SPECS + MID_SPECS + [
    gen.LayerSpec("dec_many_tiles", M=16, K=64, N=2048, k=24, calib_rows=32, outlier_frac=0.0, n_outliers=1,
                  outlier_scale=20.0, seed=41),      # few units per column tile: CTAs span several tiles
    gen.LayerSpec("dec_interior", M=16, K=64, N=65536, k=8, calib_rows=32, outlier_frac=0.0, n_outliers=1,
                  outlier_scale=20.0, seed=43),      # CTAs that cover whole column tiles between two partial ones
    gen.LayerSpec("dec_deep", M=16, K=4096, N=128, k=16, calib_rows=32, outlier_frac=0.01, outlier_scale=20.0, seed=42),
]


@pytest.mark.parametrize("M,path", [(1, binding.PATH_DECODE), (3, binding.PATH_DECODE), (4, binding.PATH_DECODE),
                                    (1, binding.PATH_SMALL), (2, binding.PATH_SMALL), (5, binding.PATH_SMALL),
                                    (8, binding.PATH_SMALL), (9, binding.PATH_SMALL), (16, binding.PATH_SMALL),
                                    (1, binding.PATH_SMALL_TMEM), (16, binding.PATH_SMALL_TMEM),
                                    (23, binding.PATH_AUTO), (64, binding.PATH_AUTO), (100, binding.PATH_AUTO),
                                    (128, binding.PATH_AUTO)],
                         ids=["cols_M1", "cols_M3", "cols_M4", "mma_M1", "mma_M2", "mma_M5", "mma_M8", "mma_M9", "mma_M16",
                              "small_M1", "small_M16", "small_M23", "small_M64", "small_M100", "small_M128"])
@pytest.mark.parametrize("spec", DECODE_SPECS, ids=lambda s: s.name)
def test_linear_decode_kernel(spec, M, path):
    W, A, B, P, Pg = _prepare(spec, "jacobi" if spec.K <= 320 else "subspace")
    X = gen.make_activations(spec, M=M)
    ref = olqer.forward(X, P)
    ws = L.new_workspace(M, Pg)
    L.set_path(path)
    try:
        Y = L.linear(_t(X), Pg, ws).cpu().numpy()
        Y2 = L.linear(_t(X), Pg, ws).cpu().numpy()      # same workspace again: the kernel left its counters at zero
    finally:
        L.set_path(binding.PATH_AUTO)
    assert L.poll_status(ws) == 0
    assert worst_ratio(Y, ref) <= 1.0
    assert np.array_equal(Y, Y2)
    Pg.release()


def test_decode_chain_shares_one_workspace():
    # layers of different shapes back to back on one stream (each launch may start while the previous drains)
    specs = [DECODE_SPECS[0], MID_SPECS[0], DECODE_SPECS[3], MID_SPECS[2], DECODE_SPECS[-3]]
    layers = [_prepare(s, "jacobi" if s.K <= 320 else "subspace") for s in specs]
    M = 4
    Xs = [gen.make_activations(s, M=M) for s in specs]
    refs = [olqer.forward(X, lay[3]) for X, lay in zip(Xs, layers)]
    n = max(L.workspace_bytes(M, s.K, s.N, s.k) for s in specs)
    ws = torch.zeros(n, dtype=torch.uint8, device=DEV)
    Xg = [_t(X) for X in Xs]
    Yg = [torch.empty((M, s.N), dtype=torch.float32, device=DEV) for s in specs]
    for _ in range(3):
        L.linear_batched([(x, lay[4], y) for x, lay, y in zip(Xg, layers, Yg)] * 2, ws)
    torch.cuda.synchronize()
    assert L.poll_status(ws) == 0
    for y, ref, s in zip(Yg, refs, specs):
        assert worst_ratio(y.cpu().numpy(), ref) <= 1.0, s.name
    for lay in layers:
        lay[4].release()


@pytest.mark.parametrize("M", [1, 3])
def test_batched_decode_groups_same_shape_calls(M):
    # seven independent calls: five layers of one shape, then two of another; the batched entry point runs them in
    # one launch that divides the SMs among the layers, and must give what single calls give
    spec_a = gen.LayerSpec("grp_a", M=M, K=1024, N=640, k=40, calib_rows=64, outlier_frac=0.01, outlier_scale=20.0, seed=51)
    spec_b = gen.LayerSpec("grp_b", M=M, K=512, N=2048, k=8, calib_rows=64, outlier_frac=0.01, outlier_scale=20.0, seed=52)
    layers = []
    for i, spec in enumerate([spec_a] * 5 + [spec_b] * 2):
        sp = gen.LayerSpec(f"{spec.name}{i}", M=M, K=spec.K, N=spec.N, k=spec.k, calib_rows=spec.calib_rows,
                           outlier_frac=spec.outlier_frac, outlier_scale=spec.outlier_scale, seed=spec.seed + i)
        layers.append((sp,) + _random_factor_layer(sp))
    Xs = [_t(gen.make_activations(sp, M=M)) for sp, _, _ in layers]
    Yb = [torch.full((M, sp.N), float("nan"), dtype=torch.float32, device=DEV) for sp, _, _ in layers]
    calls = L.make_calls([(x, lay[2], y) for x, lay, y in zip(Xs, layers, Yb)])
    ws = torch.zeros(L.batched_workspace_bytes(calls), dtype=torch.uint8, device=DEV)
    launches = L.launch_count()
    L.linear_batched(calls, ws)
    torch.cuda.synchronize()
    assert L.poll_status(ws) == 0
    assert L.launch_count() - launches == 1            # seven layers with one M: one launch
    for x, (sp, P, Pg), yb in zip(Xs, layers, Yb):
        ys = L.linear(x, Pg, ws)
        assert torch.equal(ys, yb), sp.name             # same arithmetic, same order: bit-identical
        assert worst_ratio(yb.cpu().numpy(), olqer.forward(x.cpu().numpy(), P)) <= 1.0, sp.name
    for _, _, Pg in layers:
        Pg.release()


@pytest.mark.parametrize("M", [1, 2])
def test_batched_decode_stretch_quantises_activations_ahead(M):
    # 37 independent decode calls of three shapes (one with no low-rank part): more than one shared launch, so the
    # batched entry point first computes every call's quantised activations and T_q in one launch, then runs the layers
    # in launches of up to 16 that do not wait for one another; it must give what single calls give, bit for bit.
    # With a workspace that has no room for the activations the launches compute them themselves: same results.
    shapes = [gen.LayerSpec("st_a", M=M, K=1024, N=640, k=40, calib_rows=64, outlier_frac=0.01, outlier_scale=20.0, seed=71),
              gen.LayerSpec("st_b", M=M, K=2112, N=264, k=16, calib_rows=64, outlier_frac=0.01, outlier_scale=20.0, seed=72),
              gen.LayerSpec("st_c", M=M, K=512, N=1032, k=0, calib_rows=64, outlier_frac=0.01, outlier_scale=20.0, seed=73)]
    base = []
    for sp in shapes:
        if sp.k:
            base.append((sp,) + _random_factor_layer(sp))
        else:
            W = gen.make_weight(sp)
            base.append((sp, olqer.prepare_weights(W, None, None), L.prepare_weights(_t(W), None, None)))
    order = [0, 1, 0, 2, 1] * 7 + [0, 2]
    Xs = [_t(gen.make_activations(base[j][0], M=M)) + 0.125 * i for i, j in enumerate(order)]
    Yb = [torch.full((M, base[j][0].N), float("nan"), dtype=torch.float32, device=DEV) for j in order]
    calls = L.make_calls([(x, base[j][2], y) for x, j, y in zip(Xs, order, Yb)])
    ws = torch.zeros(L.batched_workspace_bytes(calls), dtype=torch.uint8, device=DEV)
    launches = L.launch_count()
    L.linear_batched(calls, ws)
    torch.cuda.synchronize()
    assert L.poll_status(ws) == 0
    assert L.launch_count() - launches == 1 + 3         # activations ahead, then 16 + 16 + 5 layers
    ws1 = torch.zeros(max(L.workspace_bytes(M, sp.K, sp.N, sp.k) for sp, _, _ in base), dtype=torch.uint8, device=DEV)
    singles = []
    for x, j, yb in zip(Xs, order, Yb):
        ys = L.linear(x, base[j][2], ws1)
        assert torch.equal(ys, yb), base[j][0].name
        singles.append(ys)
    for i in (0, 1, 3, 36):
        sp, P, _ = base[order[i]]
        assert worst_ratio(Yb[i].cpu().numpy(), olqer.forward(Xs[i].cpu().numpy(), P)) <= 1.0, sp.name
    small = torch.zeros(ws1.numel(), dtype=torch.uint8, device=DEV)
    Y2 = [torch.full_like(y, float("nan")) for y in Yb]
    launches = L.launch_count()
    L.linear_batched([(x, base[j][2], y) for x, j, y in zip(Xs, order, Y2)], small)
    torch.cuda.synchronize()
    assert L.poll_status(small) == 0
    for y2, ys in zip(Y2, singles):
        assert torch.equal(y2, ys)
    for _, _, Pg in base:
        Pg.release()


@pytest.mark.parametrize("M", [4, 5, 8, 16, 40])
def test_batched_small_batches_share_two_launches(M):
    # nine independent calls with one M above the column-owner kernel's range (or, at M = 4, enough of them that the
    # small-batch kernels take them all the same): layers of three shapes (one without a
    # low-rank part) run as ONE launch of the small prologue and ONE launch of the small-batch GEMM over the work items
    # of all of them.  Layers that share a launch are cut into fewer K chunks than alone, so a result may differ from
    # the single call's in the last bits: every one is held against the oracle, the quantised operands (which do not
    # depend on the chunks) make the two agree to well within the tolerance, and a second run of the same batch must
    # reproduce the first bit for bit (counters are left at zero, the grouping is a function of the calls alone).
    shapes = [gen.LayerSpec("sg_a", M=M, K=1024, N=640, k=40, calib_rows=64, outlier_frac=0.01, outlier_scale=20.0, seed=171),
              gen.LayerSpec("sg_b", M=M, K=2112, N=264, k=16, calib_rows=64, outlier_frac=0.01, outlier_scale=20.0, seed=172),
              gen.LayerSpec("sg_c", M=M, K=512, N=1032, k=0, calib_rows=64, outlier_frac=0.01, outlier_scale=20.0, seed=173)]
    base = []
    for sp in shapes:
        if sp.k:
            base.append((sp,) + _random_factor_layer(sp))
        else:
            W = gen.make_weight(sp)
            base.append((sp, olqer.prepare_weights(W, None, None), L.prepare_weights(_t(W), None, None)))
    order = [0, 1, 2, 0, 0, 1, 2, 1, 0]
    Xs = [_t(gen.make_activations(base[j][0], M=M)) + 0.125 * i for i, j in enumerate(order)]
    Yb = [torch.full((M, base[j][0].N), float("nan"), dtype=torch.float32, device=DEV) for j in order]
    calls = L.make_calls([(x, base[j][2], y) for x, j, y in zip(Xs, order, Yb)])
    ws = torch.zeros(L.batched_workspace_bytes(calls), dtype=torch.uint8, device=DEV)
    first = None
    for rep in range(2):
        launches = L.launch_count()
        L.linear_batched(calls, ws)
        torch.cuda.synchronize()
        assert L.poll_status(ws) == 0
        assert L.launch_count() - launches == 2
        if first is None:
            first = [y.clone() for y in Yb]
            for y in Yb:
                y.fill_(float("nan"))
        else:
            for a, b in zip(first, Yb):
                assert torch.equal(a, b)
    ws1 = torch.zeros(max(L.workspace_bytes(M, sp.K, sp.N, sp.k) for sp, _, _ in base), dtype=torch.uint8, device=DEV)
    for i, (x, j, yb) in enumerate(zip(Xs, order, Yb)):
        sp, P, Pg = base[j]
        ref = olqer.forward(x.cpu().numpy(), P)
        assert worst_ratio(yb.cpu().numpy(), ref) <= 1.0, (i, sp.name)
        ys = L.linear(x, Pg, ws1)
        assert worst_ratio(ys.cpu().numpy(), ref) <= 1.0, (i, sp.name)
        assert float(np.max(np.abs((ys - yb).cpu().numpy().astype(np.float64)) / ref.tol)) <= 0.5, (i, sp.name)
    for _, _, Pg in base:
        Pg.release()


def test_batched_mixed_stretches_and_prefill():
    # one batched call: a stretch of 18 decode calls with M = 1, three prefill calls (M = 300), then a stretch of 20
    # decode calls with M = 2 that is followed by a lone M = 9 call.  The stretches quantise their activations ahead into
    # the part of the workspace that the prefill group uses in between; every call must give what it gives alone.
    sd = gen.LayerSpec("mx_d", M=1, K=1024, N=640, k=40, calib_rows=64, outlier_frac=0.01, outlier_scale=20.0, seed=91)
    se = gen.LayerSpec("mx_e", M=1, K=512, N=2048, k=8, calib_rows=64, outlier_frac=0.01, outlier_scale=20.0, seed=92)
    Pd, Pe = _random_factor_layer(sd)[1], _random_factor_layer(se)[1]
    plan = [(1, Pd if i % 3 else Pe) for i in range(18)] + [(300, Pd), (300, Pe), (300, Pd)] + \
           [(2, Pe if i % 4 else Pd) for i in range(20)] + [(9, Pd)]
    Xs, Ys = [], []
    for i, (M, P) in enumerate(plan):
        spec = sd if P is Pd else se
        Xs.append(_t(gen.make_activations(spec, M=M)) + 0.0625 * i)
        Ys.append(torch.full((M, spec.N), float("nan"), dtype=torch.float32, device=DEV))
    calls = L.make_calls([(x, P, y) for x, (_, P), y in zip(Xs, plan, Ys)])
    ws = torch.zeros(L.batched_workspace_bytes(calls), dtype=torch.uint8, device=DEV)
    for _ in range(2):                                  # twice: the counters and slots must be left clean
        L.linear_batched(calls, ws)
    torch.cuda.synchronize()
    assert L.poll_status(ws) == 0
    ws1 = torch.zeros(max(L.workspace_bytes(300, sp.K, sp.N, sp.k) for sp in (sd, se)), dtype=torch.uint8, device=DEV)
    for x, (M, P), y in zip(Xs, plan, Ys):
        assert torch.equal(L.linear(x, P, ws1), y), M
    Pd.release()
    Pe.release()


@pytest.mark.parametrize("M", [1, 4, 16])
def test_linear_decode_full_size(M, ratio_log):
    spec = gen.config_decode(M)
    W, A, B, P, Pg = _prepare(spec, "subspace")
    X = gen.make_activations(spec)
    ref = olqer.forward(X, P)
    ws = L.new_workspace(M, Pg)
    Y = L.linear(_t(X), Pg, ws).cpu().numpy()          # automatic path selection: the column-owner kernel (M <= 4) or the small-batch kernels
    assert L.poll_status(ws) == 0
    assert ratio_log(spec.name, worst_ratio(Y, ref)) <= 1.0
    Pg.release()


# ---------------------------------------------------------------------------- full-size layers, sampled rows
def _random_factor_layer(spec):
    """Full-size layer with seeded stand-in factors (the factors are inputs of the layer; deriving them by
    SVD at this size would take minutes on the host)."""
    W = gen.make_weight(spec)
    A, B = gen.make_random_factors(spec)
    P = olqer.prepare_weights(W, A, B)
    Pg = L.prepare_weights(_t(W), _t(A), _t(B))
    return P, Pg


FULL_SPECS = [
    gen.config_prefill(False),                       # M=2048, 4096 x 11008, rank 32
    gen.config_prefill(True),                        # M=2048, 11008 x 4096
    gen.config_sweep(13824, 512, 128),               # 13B-shaped: K=5120, N=13824, M=512, rank 128, Student-t weights
    gen.config_sweep(5120, 64, 256),                 # M=64, rank 256
    # the rest of the 13B sweep's corners: 32 row tiles with the large ranks (the SIMT-style prologue serves ranks above 64),
    # the small ranks at M = 512, and the decode kernel with one to sixteen rank blocks at both widths
    gen.config_sweep(13824, 4096, 256),
    gen.config_sweep(5120, 4096, 128),
    gen.config_sweep(5120, 4096, 32),
    gen.config_sweep(5120, 512, 8),
    gen.config_sweep(5120, 512, 32),
    gen.config_sweep(13824, 512, 64),
    gen.config_sweep(13824, 64, 8),
    gen.config_sweep(5120, 1, 64),
    gen.config_sweep(5120, 1, 256),
    gen.config_sweep(13824, 1, 32),
    gen.config_sweep(13824, 1, 256),
]


@pytest.mark.parametrize("spec", FULL_SPECS, ids=lambda s: s.name)
def test_linear_full_size_sampled_rows(spec, ratio_log):
    # Rows of Y depend only on the same rows of X, so the oracle computes a seeded sample of rows that
    # touches every 128-row tile (and the first and last row); the GPU runs the whole layer as bench.py does.
    P, Pg = _random_factor_layer(spec)
    X = gen.make_activations(spec)
    g = np.random.default_rng(spec.seed)
    rows = sorted({0, spec.M - 1} | {int(t * 128 + g.integers(0, 128)) for t in range((spec.M + 127) // 128) if t * 128 + 127 < spec.M})
    ref = olqer.forward(X[rows], P)
    ws = L.new_workspace(spec.M, Pg)
    Y = L.linear(_t(X), Pg, ws)
    assert L.poll_status(ws) == 0
    Ys = Y[torch.tensor(rows, device=DEV)].cpu().numpy()
    assert ratio_log(spec.name, worst_ratio(Ys, ref)) <= 1.0
    Pg.release()


def test_accumulation_rounding_regime(ratio_log):
    # K = 11008 with the block exponents of every row of X spread over 13 binades (each 16-block scaled by a seeded power
    # of two in [2^-6, 2^6]) and Student-t weights: the exact products differ by up to 2^20 in magnitude, so the fp32
    # accumulation has to round (on N(0,1) inputs the sums stay exact).  The observed |dY| / tol shows how much of
    # the 1e-4 bound the accumulation uses.
    spec = gen.LayerSpec("round_K11008", M=384, K=11008, N=512, k=32, calib_rows=64, outlier_frac=0.005, outlier_scale=50.0,
                         weight_law="student_t4", seed=77)
    P, Pg = _random_factor_layer(spec)
    X = gen.make_activations(spec)
    g = np.random.default_rng(spec.seed)
    X *= np.exp2(g.integers(-6, 7, size=(spec.M, spec.K // 16))).repeat(16, axis=1).astype(np.float32)
    rows = list(range(0, spec.M, 7))
    ref = olqer.forward(X[rows], P)
    spread = ref.Xe.max(axis=1) - ref.Xe.min(axis=1)
    assert spread.min() >= 12
    ws = L.new_workspace(spec.M, Pg)
    Y = L.linear(_t(X), Pg, ws)
    assert L.poll_status(ws) == 0
    ratio = worst_ratio(Y[torch.tensor(rows, device=DEV)].cpu().numpy(), ref)
    assert 0.0 < ratio_log(spec.name, ratio) <= 1.0       # the sums do round, and stay inside the bound
    for M in (1, 9):                                       # the decode kernels on the same layer
        r1 = olqer.forward(X[:M], P)
        y1 = L.linear(_t(X[:M]), Pg, ws).cpu().numpy()
        assert ratio_log(f"{spec.name}_M{M}", worst_ratio(y1, r1)) <= 1.0
    Pg.release()


@pytest.mark.parametrize("which", [0, 6], ids=["q_4096x4096", "down_11008x4096"])
def test_full_size_projection_bit_exact_on_sampled_rows(which):
    # the bench's prefill configuration (M = 2048, rank 32): T_q of the tensor-core prologue, bit for bit, on one
    # seeded row of every 128-row tile plus the first and last row (a row of T depends only on the same row of X)
    spec = gen.config_stack(0, which, 2048)
    P, Pg = _random_factor_layer(spec)
    X = gen.make_activations(spec)
    g = np.random.default_rng(spec.seed)
    rows = sorted({0, spec.M - 1} | {int(t * 128 + g.integers(0, 128)) for t in range(spec.M // 128)})
    ref = olqer.forward(X[rows], P)
    ws = L.new_workspace(spec.M, Pg)
    Tm, Te = L.project_lowrank(_t(X), Pg, ws)
    assert L.poll_status(ws) == 0
    idx = torch.tensor(rows, device=DEV)
    assert np.array_equal(Tm[idx].cpu().numpy(), ref.Tm)
    assert np.array_equal(Te[idx].cpu().numpy(), exp_bytes(ref.Te))
    Pg.release()


def test_batched_prefill_calls_share_gemm_launches():
    # nine independent prefill calls: five of one shape and two of another with M = 300 (one group of seven: long-K
    # tiles first), then two with M = 1100 (large enough for the tensor-core prologue, which takes both layers in one
    # launch); with a workspace of lqer_batched_workspace_bytes each group is one GEMM launch, and every tile is
    # computed as in a single call
    spec_a = gen.LayerSpec("pgrp_a", M=300, K=1024, N=640, k=40, calib_rows=64, outlier_frac=0.01, outlier_scale=20.0, seed=61)
    spec_c = gen.LayerSpec("pgrp_c", M=300, K=2048, N=392, k=8, calib_rows=64, outlier_frac=0.01, outlier_scale=20.0, seed=63)
    spec_b = gen.LayerSpec("pgrp_b", M=1100, K=512, N=1280, k=32, calib_rows=64, outlier_frac=0.01, outlier_scale=20.0, seed=62)
    layers = []
    for i, spec in enumerate([spec_a] * 3 + [spec_c] + [spec_a] * 2 + [spec_c] + [spec_b] * 2):
        sp = gen.LayerSpec(f"{spec.name}{i}", M=spec.M, K=spec.K, N=spec.N, k=spec.k, calib_rows=spec.calib_rows,
                           outlier_frac=spec.outlier_frac, outlier_scale=spec.outlier_scale, seed=spec.seed + i)
        layers.append((sp,) + _random_factor_layer(sp))
    Xs = [_t(gen.make_activations(sp)) for sp, _, _ in layers]
    Yb = [torch.full((sp.M, sp.N), float("nan"), dtype=torch.float32, device=DEV) for sp, _, _ in layers]
    calls = L.make_calls([(x, lay[2], y) for x, lay, y in zip(Xs, layers, Yb)])
    ws = torch.zeros(L.batched_workspace_bytes(calls), dtype=torch.uint8, device=DEV)
    launches = L.launch_count()
    L.linear_batched(calls, ws)
    torch.cuda.synchronize()
    assert L.poll_status(ws) == 0
    assert L.launch_count() - launches == 7 + 1 + 2     # seven prologues (M = 300), one for both M = 1100 layers, two GEMM launches
    for x, (sp, P, Pg), yb in zip(Xs, layers, Yb):
        ys = L.linear(x, Pg, ws)
        assert torch.equal(ys, yb), sp.name              # same tiles, same arithmetic
    for j in (3, 8):
        sp, P, Pg = layers[j]
        assert worst_ratio(Yb[j].cpu().numpy(), olqer.forward(Xs[j].cpu().numpy(), P)) <= 1.0, sp.name
    # a workspace that only fits single calls: no sharing, same results
    ws1 = torch.zeros(max(L.workspace_bytes(sp.M, sp.K, sp.N, sp.k) for sp, _, _ in layers), dtype=torch.uint8, device=DEV)
    Y1 = [torch.empty_like(y) for y in Yb]
    L.linear_batched([(x, lay[2], y) for x, lay, y in zip(Xs, layers, Y1)], ws1)
    for y1, yb in zip(Y1, Yb):
        assert torch.equal(y1, yb)
    for _, _, Pg in layers:
        Pg.release()


def test_batched_prefill_group_with_long_and_short_layers():
    # four prefill calls with M = 4096 (32 row tiles): two short layers (K = 512) and two long ones (K = 4096).  One
    # prologue launch for all of them would leave the long layers a whole row tile per CTA and the CTAs unequal work,
    # so the long layers get launches of their own; T_q and Y must be what single calls give, and within the oracle's
    # tolerance.
    M = 4096
    short = gen.LayerSpec("lg_s", M=M, K=512, N=264, k=32, calib_rows=64, outlier_frac=0.01, outlier_scale=20.0, seed=95)
    long_ = gen.LayerSpec("lg_l", M=M, K=4096, N=136, k=32, calib_rows=64, outlier_frac=0.01, outlier_scale=20.0, seed=96)
    layers = []
    for i, spec in enumerate([short, long_, short, long_]):
        sp = gen.LayerSpec(f"{spec.name}{i}", M=M, K=spec.K, N=spec.N, k=spec.k, calib_rows=spec.calib_rows,
                           outlier_frac=spec.outlier_frac, outlier_scale=spec.outlier_scale, seed=spec.seed + 10 * i)
        layers.append((sp,) + _random_factor_layer(sp))
    Xs = [_t(gen.make_activations(sp)) for sp, _, _ in layers]
    Yb = [torch.full((M, sp.N), float("nan"), dtype=torch.float32, device=DEV) for sp, _, _ in layers]
    calls = L.make_calls([(x, lay[2], y) for x, lay, y in zip(Xs, layers, Yb)])
    ws = torch.zeros(L.batched_workspace_bytes(calls), dtype=torch.uint8, device=DEV)
    launches = L.launch_count()
    for _ in range(2):
        L.linear_batched(calls, ws)
    torch.cuda.synchronize()
    assert L.poll_status(ws) == 0
    assert L.launch_count() - launches == 2 * (3 + 1)    # the short layers together, each long one alone, one GEMM launch
    for x, (sp, P, Pg), yb in zip(Xs, layers, Yb):
        assert torch.equal(L.linear(x, Pg, ws), yb), sp.name
    for j in (0, 1):
        sp, P, Pg = layers[j]
        rows = np.arange(0, M, 37)
        ref = olqer.forward(Xs[j].cpu().numpy()[rows], P)
        assert worst_ratio(Yb[j].cpu().numpy()[rows], ref) <= 1.0, sp.name
    for _, _, Pg in layers:
        Pg.release()


def test_host_buffer_entry_points_match_device_calls():
    # lqer_linear_host (one layer) and lqer_linear_host_batched (copies and layers pipelined, buffers alternate)
    # against the device entry point on the same inputs; five calls so that every buffer is reused
    specs = [MID_SPECS[0], MID_SPECS[2], SMALL_SPECS[1], MID_SPECS[0], MID_SPECS[1]]
    Ms = [300, 3, 37, 1, 129]
    layers = [_prepare(s, "jacobi" if s.K <= 320 else "subspace") for s in specs]
    Xs = [torch.from_numpy(gen.make_activations(s, M=M)).pin_memory() for s, M in zip(specs, Ms)]
    Ys = [torch.full((M, s.N), float("nan")).pin_memory() for s, M in zip(specs, Ms)]
    calls = L.make_host_calls([(x, lay[4], y) for x, lay, y in zip(Xs, layers, Ys)])
    ws = torch.zeros(L.linear_host_batched_bytes(calls), dtype=torch.uint8, device=DEV)
    L.linear_host_batched(calls, ws)
    assert L.poll_status(ws) == 0
    for s, M, lay, x, y in zip(specs, Ms, layers, Xs, Ys):
        wd = L.new_workspace(M, lay[4])
        yd = L.linear(x.to(DEV), lay[4], wd).cpu()
        assert torch.equal(y, yd), s.name
        y1 = torch.empty_like(y)
        wh = L.new_workspace(M, lay[4], extra_bytes=4 * M * (s.K + s.N) + 1024)
        L.linear_host(x, lay[4], wh, y1)
        assert torch.equal(y1, yd), s.name
    assert worst_ratio(Ys[0].numpy(), olqer.forward(Xs[0].numpy(), layers[0][3])) <= 1.0
    for lay in layers:
        lay[4].release()


def test_stack_linears_batched_decode_and_prefill():
    # the q, gate and down linears of one decoder layer of the 7B stack through lqer_linear_batched on one
    # workspace: M = 1 (decode kernels) and then M = 2048 (prologue + GEMM), as bench.py runs them
    specs = [gen.config_stack(0, w, 2048) for w in (0, 4, 6)]
    layers = [_random_factor_layer(s) for s in specs]
    X1 = [gen.make_activations(s, M=1) for s in specs]
    X2 = [gen.make_activations(s, M=2048) for s in specs]
    rows = [0, 777, 2047]
    n = max(L.workspace_bytes(2048, s.K, s.N, s.k) for s in specs)
    ws = torch.zeros(n, dtype=torch.uint8, device=DEV)
    Y1 = [torch.empty((1, s.N), dtype=torch.float32, device=DEV) for s in specs]
    Y2 = [torch.empty((2048, s.N), dtype=torch.float32, device=DEV) for s in specs]
    L.linear_batched([(_t(x), lay[1], y) for x, lay, y in zip(X1, layers, Y1)], ws)
    L.linear_batched([(_t(x), lay[1], y) for x, lay, y in zip(X2, layers, Y2)], ws)
    torch.cuda.synchronize()
    assert L.poll_status(ws) == 0
    for s, lay, x1, x2, y1, y2 in zip(specs, layers, X1, X2, Y1, Y2):
        assert worst_ratio(y1.cpu().numpy(), olqer.forward(x1, lay[0])) <= 1.0, s.name
        assert worst_ratio(y2[torch.tensor(rows, device=DEV)].cpu().numpy(), olqer.forward(x2[rows], lay[0])) <= 1.0, s.name
    for lay in layers:
        lay[1].release()
