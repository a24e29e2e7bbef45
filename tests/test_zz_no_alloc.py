"""lqer_linear_static: the layer for callers that cannot allocate device memory.

Some users of the library run inside another component's memory plan (a plugin of a runtime
that owns the whole device, a latency path where cudaMalloc's device-wide synchronisation is
not acceptable) and have no workspace to hand over.  For them the scratch is a fixed array in
the library image.  The array is shared by every call and keeps the previous call's contents,
so the check runs the entry point twice in a row - with different shapes, the second smaller
than the first, so that stale bytes of the first call lie behind the second one's data - and
compares each result with the ordinary entry point's, which gets a fresh workspace.

The file name sorts last on purpose: a run that stops at the first failure has then already
run every other test.  The test builds its own inputs and passes alone in a fresh process as
well as after the rest of the suite.
"""
import ctypes as C

import numpy as np
import pytest
import torch

import lqer_inputs as gen
import paper_2402_02446_b200 as L
from paper_2402_02446_b200 import binding

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _layer(spec):
    W = torch.from_numpy(gen.make_weight(spec)).to(DEV)
    A, B = gen.make_random_factors(spec)
    return L.prepare_weights(W, torch.from_numpy(A).to(DEV), torch.from_numpy(B).to(DEV))


def test_static_scratch_matches_workspace_entry_point_twice_in_a_row():
    specs = [gen.LayerSpec("static_a", M=300, K=1024, N=640, k=40, calib_rows=32, outlier_frac=0.01, outlier_scale=20.0, seed=91),
             gen.LayerSpec("static_b", M=9, K=512, N=384, k=16, calib_rows=32, outlier_frac=0.01, outlier_scale=20.0, seed=92)]
    for spec in specs:
        P = _layer(spec)
        X = torch.from_numpy(gen.make_activations(spec)).to(DEV)
        ws = L.new_workspace(spec.M, P)
        Y_ref = L.linear(X, P, ws)
        assert L.poll_status(ws) == 0
        Y = torch.full((spec.M, spec.N), float("nan"), dtype=torch.float32, device=DEV)
        L.linear_static(X, P, Y)
        torch.cuda.synchronize()
        # both entry points run the same kernels in the same fixed reduction order
        assert torch.equal(Y, Y_ref), spec.name
        # and the tolerance the parity tests use holds trivially: |dY| <= 1e-4 (|X_q| |W_q| + |T_q| |B_q|)
        assert float((Y - Y_ref).abs().max()) == 0.0
        P.release()


def test_static_scratch_rejects_what_does_not_fit():
    spec = gen.LayerSpec("static_big", M=4096, K=2048, N=256, k=16, calib_rows=32, outlier_frac=0.0, outlier_scale=1.0, seed=93)
    P = _layer(spec)
    assert L.workspace_bytes(spec.M, spec.K, spec.N, spec.k) > binding.STATIC_SCRATCH_BYTES
    X = torch.zeros((spec.M, spec.K), dtype=torch.float32, device=DEV)
    Y = torch.zeros((spec.M, spec.N), dtype=torch.float32, device=DEV)
    launches = L.launch_count()
    st = L.lib().lqer_linear_static(X.data_ptr(), spec.M, P.ptr, Y.data_ptr(), None)
    assert st == binding.STATUS_NAMES.index("LQER_ERR_STATIC_SCRATCH")
    assert L.launch_count() == launches          # refused on the host, nothing was launched
    assert L.lib().lqer_linear_static(None, 1, P.ptr, Y.data_ptr(), None) == binding.STATUS_NAMES.index("LQER_ERR_NULL")
    P.release()
