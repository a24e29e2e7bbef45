"""The register-operand small-batch GEMM (up to 16 tokens, 4-bit weights; Section 3.1 / 3.2: Y = [X_q | T_q] . [W_q ; B_q],
Section 2.1: memory bound on the weights) in the launches that several layers share, against the oracle.

Covered here beyond the small-batch cases of test_gpu_parity.py: tiles with a single K chunk (the finished tile goes
through shared memory and is written in every output type), a rank that ends inside a rank slab, a last column tile
of 16 columns, the second call on a workspace that still holds the first call's flags, and the bounded polls.
"""
import numpy as np
import pytest
import torch

import lqer_inputs as gen
import paper_2402_02446_b200 as L
from paper_2402_02446_b200 import binding
from oracle import lqer as olqer
from oracle import mxint
from helpers import worst_ratio
from test_gpu_mxint8_io import _check_against_oracle

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _t(a):
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


def _layer(spec):
    W = gen.make_weight(spec)
    A, B = gen.make_random_factors(spec)
    return olqer.prepare_weights(W, A, B), L.prepare_weights(_t(W), _t(A), _t(B))


@pytest.mark.parametrize("M", [7, 16])
def test_single_chunk_tiles_in_every_output_type(M):
    # K = 256 is too short to be cut, so every 256-column tile is one work item and the kernel writes Y itself:
    # fp32, bf16 (round to nearest even of the same fp32 values) and MXINT8 (blocks of 16 along N)
    spec = gen.LayerSpec("mma_direct", M=M, K=256, N=8208, k=72, calib_rows=32, outlier_frac=0.01, outlier_scale=20.0, seed=701)
    P, Pg = _layer(spec)
    n = 12
    Xs = [gen.make_activations(spec, M=M) + 0.0625 * i for i in range(n)]
    refs = [olqer.forward(X, P) for X in Xs]
    Xd = [_t(X) for X in Xs]
    outs = {}
    for name, y_t in (("f32", torch.float32), ("bf16", torch.bfloat16), ("mx", L.MXINT8)):
        if y_t is L.MXINT8:
            Ys = [torch.zeros(L.mxint8_bytes(M, spec.N), dtype=torch.uint8, device=DEV) for _ in range(n)]
        else:
            Ys = [torch.full((M, spec.N), float("nan"), dtype=y_t, device=DEV) for _ in range(n)]
        calls = L.make_calls([(x, Pg, y) for x, y in zip(Xd, Ys)], torch.float32, y_t)
        ws = torch.zeros(L.batched_workspace_bytes(calls), dtype=torch.uint8, device=DEV)
        for rep in range(2):                                  # the second run finds the first run's flags in the workspace
            before = L.launch_count()
            L.linear_batched_ex(calls, ws, torch.float32, y_t)
            torch.cuda.synchronize()
            assert L.poll_status(ws) == 0
            assert L.launch_count() - before == 2
        outs[name] = Ys
    for i, ref in enumerate(refs):
        assert worst_ratio(outs["f32"][i].cpu().numpy(), ref) <= 1.0, i
        assert torch.equal(outs["bf16"][i], outs["f32"][i].to(torch.bfloat16)), i
        Ym, Ye = L.split_mxint8(outs["mx"][i], M, spec.N)
        _check_against_oracle(Ym.cpu().numpy(), Ye.cpu().numpy(), ref)
    Pg.release()


def test_forced_single_call_equals_itself_and_the_oracle_on_a_long_layer():
    # K = 11008-like: 172 slabs cut into chunks whose lengths are odd, a rank of 40 (2.5 rank blocks' worth of a rank
    # slab), forced on a single call (which by itself would take the tensor-memory kernel)
    spec = gen.LayerSpec("mma_long", M=13, K=11008, N=520, k=40, calib_rows=32, outlier_frac=0.01, outlier_scale=20.0,
                         weight_law="student_t4", seed=702)
    P, Pg = _layer(spec)
    X = gen.make_activations(spec, M=13)
    ref = olqer.forward(X, P)
    ws = L.new_workspace(13, Pg)
    L.set_path(binding.PATH_SMALL)
    try:
        Y1 = L.linear(_t(X), Pg, ws).clone()
        Y2 = L.linear(_t(X), Pg, ws)
    finally:
        L.set_path(binding.PATH_AUTO)
    assert L.poll_status(ws) == 0
    assert worst_ratio(Y1.cpu().numpy(), ref) <= 1.0
    assert torch.equal(Y1, Y2)
    Pg.release()


def test_replays_of_a_captured_graph_follow_their_inputs():
    # a captured batch repeats its launch parameters, the epoch of the prologue's flags among them: every replay must
    # still wait for its own prologue, so a replay on new activations gives the new results
    spec = gen.LayerSpec("mma_graph", M=9, K=1024, N=640, k=40, calib_rows=32, outlier_frac=0.01, outlier_scale=20.0, seed=703)
    P, Pg = _layer(spec)
    n = 8
    Xd = [torch.zeros((9, spec.K), dtype=torch.float32, device=DEV) for _ in range(n)]
    Ys = [torch.zeros((9, spec.N), dtype=torch.float32, device=DEV) for _ in range(n)]
    calls = L.make_calls([(x, Pg, y) for x, y in zip(Xd, Ys)])
    ws = torch.zeros(L.batched_workspace_bytes(calls), dtype=torch.uint8, device=DEV)
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        L.linear_batched(calls, ws, stream=s)              # first use of the kernels outside the capture
    s.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=s):
        L.linear_batched(calls, ws, stream=torch.cuda.current_stream())
    for rep in range(3):
        Xs = [gen.make_activations(spec, M=9) * (1.0 + rep) + 0.25 * i for i in range(n)]
        for x, X in zip(Xd, Xs):
            x.copy_(_t(X))
        torch.cuda.synchronize()
        g.replay()
        torch.cuda.synchronize()
        assert L.poll_status(ws) == 0
        for X, y in zip(Xs, Ys):
            assert worst_ratio(y.cpu().numpy(), olqer.forward(X, P)) <= 1.0, rep
    Pg.release()
