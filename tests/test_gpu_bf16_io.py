"""16-bit activations at the layer's boundary (Section 2.1): bf16 X in, bf16 Y out, through lqer_linear_ex /
lqer_linear_batched_ex, against the oracle.

bf16 X: both sides start from the same bf16 values (every bf16 value is an fp32 value), so X_q and T_q stay bit
exact and Y stays within the layer's tolerance.  bf16 Y: the library rounds its fp32 result to nearest even; the
oracle's fp64 result rounded the same way may differ by one bf16 step where the two unrounded values straddle a
tie, so the bound is the layer's tolerance plus half a bf16 spacing at |Y|.
"""
import numpy as np
import pytest
import torch

import lqer_inputs as gen
import paper_2402_02446_b200 as L
from paper_2402_02446_b200 import binding
from oracle import lqer as olqer
from oracle import mxint

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _t(a):
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


def _layer(spec):
    W = gen.make_weight(spec)
    if spec.k == 0:
        return olqer.prepare_weights(W, None, None), L.prepare_weights(_t(W), None, None)
    A, B = gen.make_random_factors(spec)
    return olqer.prepare_weights(W, A, B), L.prepare_weights(_t(W), _t(A), _t(B))


def _bf16_inputs(spec, M):
    X = mxint.round_bf16(gen.make_activations(spec, M=M)).astype(np.float32)      # exact: bf16 values are fp32 values
    return X, _t(X).to(torch.bfloat16)


def _check(Y, ref, y_is_bf16):
    Y = Y.to(torch.float64).cpu().numpy()
    bound = ref.tol + (mxint.bf16_half_ulp(ref.Y) * 1.0000001 if y_is_bf16 else 0.0)
    return float(np.max(np.abs(Y - ref.Y) / bound))


SPECS = [gen.LayerSpec("io_a", M=300, K=1024, N=640, k=40, calib_rows=32, outlier_frac=0.01, outlier_scale=20.0, seed=301),
         gen.LayerSpec("io_k0", M=129, K=512, N=392, k=0, calib_rows=32, outlier_frac=0.01, outlier_scale=20.0, seed=302),
         gen.LayerSpec("io_tc", M=1100, K=2112, N=264, k=64, calib_rows=32, outlier_frac=0.005, outlier_scale=50.0,
                       weight_law="student_t4", seed=303)]


@pytest.mark.parametrize("x_bf16,y_bf16", [(True, True), (True, False), (False, True)], ids=["bf16_bf16", "bf16_f32", "f32_bf16"])
@pytest.mark.parametrize("spec", SPECS, ids=lambda s: s.name)
def test_linear_ex_every_path(spec, x_bf16, y_bf16, ratio_log):
    # every batch-size regime: small-batch kernels (1, 4, 9, 70 rows), split-K-sized (200), and the large-batch path with
    # either prologue (the spec's own M; 1100 rows take the tensor-core prologue)
    P, Pg = _layer(spec)
    ws = L.new_workspace(spec.M, Pg)
    for M in (1, 4, 9, 70, 200, spec.M):
        if M > spec.M:
            continue
        Xf, Xb = _bf16_inputs(spec, M)
        ref = olqer.forward(Xf, P)
        X = Xb if x_bf16 else _t(Xf)
        Y = L.linear_ex(X, Pg, ws, out_dtype=torch.bfloat16 if y_bf16 else torch.float32)
        assert L.poll_status(ws) == 0
        assert Y.dtype == (torch.bfloat16 if y_bf16 else torch.float32)
        assert ratio_log(f"{spec.name}_{'b' if x_bf16 else 'f'}{'b' if y_bf16 else 'f'}", _check(Y, ref, y_bf16)) <= 1.0, M
        if y_bf16:
            # the 16-bit result is the library's own fp32 result, rounded to nearest even
            Yf = L.linear_ex(X, Pg, ws, out_dtype=torch.float32)
            assert torch.equal(Y, Yf.to(torch.bfloat16)), M
        if x_bf16 and spec.k:
            # the quantised operands do not depend on the container type of X
            Tm_b, Te_b = L.project_lowrank(Xb.to(torch.float32), Pg, ws)
            assert np.array_equal(Tm_b.cpu().numpy(), ref.Tm) and np.array_equal(Te_b.cpu().numpy(), mxint.exponent_bytes(ref.Te)), M
    Pg.release()


@pytest.mark.parametrize("x_bf16", [True, False], ids=["bf16_x", "f32_x"])
def test_tensor_core_prologue_on_ragged_shapes(x_bf16):
    # the tensor-core prologue forced on shapes it does not meet by itself: K = 80 (the second 64-column stage is mostly
    # outside X and its TMA boxes read zeros there), 37 and 300 rows (row tiles mostly outside X), ranks 5 and 40
    for spec in (gen.LayerSpec("rag_a", M=37, K=80, N=136, k=5, calib_rows=32, outlier_frac=0, n_outliers=2, outlier_scale=20.0, seed=321),
                 gen.LayerSpec("rag_b", M=300, K=1104, N=264, k=40, calib_rows=32, outlier_frac=0.01, outlier_scale=20.0, seed=322)):
        P, Pg = _layer(spec)
        ws = L.new_workspace(spec.M, Pg)
        Xf, Xb = _bf16_inputs(spec, spec.M)
        ref = olqer.forward(Xf, P)
        X = Xb if x_bf16 else _t(Xf)
        L.set_path(binding.PATH_TENSOR_PROLOGUE)
        try:
            Y = L.linear_ex(X, Pg, ws, out_dtype=torch.float32)
            Tm, Te = L.project_lowrank(_t(Xf), Pg, ws)
        finally:
            L.set_path(binding.PATH_AUTO)
        assert L.poll_status(ws) == 0
        assert np.array_equal(Tm.cpu().numpy(), ref.Tm) and np.array_equal(Te.cpu().numpy(), mxint.exponent_bytes(ref.Te))
        assert _check(Y, ref, False) <= 1.0, spec.name
        Pg.release()


def test_linear_batched_ex_shares_launches_like_fp32():
    # four prefill calls (M = 1100: one prologue launch, one GEMM launch) and five small-batch calls (M = 9: two launches)
    # with bf16 in and out
    big = gen.LayerSpec("iob_big", M=1100, K=512, N=1280, k=32, calib_rows=32, outlier_frac=0.01, outlier_scale=20.0, seed=311)
    small = gen.LayerSpec("iob_small", M=9, K=1024, N=640, k=40, calib_rows=32, outlier_frac=0.01, outlier_scale=20.0, seed=312)
    Pb, Pgb = _layer(big)
    Ps, Pgs = _layer(small)
    plan = [(big, Pgb, 1100)] * 4 + [(small, Pgs, 9)] * 5
    Xs = [(_bf16_inputs(sp, M)[1].to(torch.float32) + 0.125 * i).to(torch.bfloat16) for i, (sp, _, M) in enumerate(plan)]
    Ys = [torch.zeros((M, sp.N), dtype=torch.bfloat16, device=DEV) for sp, _, M in plan]
    calls = L.make_calls([(x, Pg, y) for x, (_, Pg, _), y in zip(Xs, plan, Ys)], torch.bfloat16, torch.bfloat16)
    ws = torch.zeros(L.batched_workspace_bytes(calls), dtype=torch.uint8, device=DEV)
    launches = L.launch_count()
    L.linear_batched_ex(calls, ws, torch.bfloat16, torch.bfloat16)
    torch.cuda.synchronize()
    assert L.poll_status(ws) == 0
    assert L.launch_count() - launches == 2 + 2
    for x, (sp, Pg, M), y in zip(Xs, plan, Ys):
        if M > 128:        # large batches: the same tiles, the same arithmetic
            assert torch.equal(L.linear_ex(x, Pg, ws, out_dtype=torch.bfloat16), y), sp.name
        else:              # small batches that share a launch are cut into fewer K chunks: both are compared with the oracle
            assert _check(y, olqer.forward(x.to(torch.float32).cpu().numpy(), Ps), True) <= 1.0
    ref = olqer.forward(Xs[0].to(torch.float32).cpu().numpy(), Pb)
    assert _check(Ys[0], ref, True) <= 1.0
    Pgb.release()
    Pgs.release()


def test_linear_ex_rejects_unknown_types():
    spec = SPECS[1]
    P, Pg = _layer(spec)
    ws = L.new_workspace(4, Pg)
    X = torch.zeros((4, spec.K), device=DEV)
    Y = torch.zeros((4, spec.N), device=DEV)
    st = L.lib().lqer_linear_ex(X.data_ptr(), 7, 4, Pg.ptr, Y.data_ptr(), 0, ws.data_ptr(), ws.numel(), None)
    assert st == binding.STATUS_NAMES.index("LQER_ERR_CONFIG")
    Pg.release()
