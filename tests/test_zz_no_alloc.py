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


def test_static_scratch_boundary_on_a_4096_layer_and_no_allocation():
    # K = N = 4096, rank 32: the call's own need decides.  M = 57 is the largest small batch that fits (the partial
    # sums of the GEMM's K chunks grow with M), M = 58 is the first that is refused, and M = 300 fits again (no
    # split of K above 256 rows).  The calls that run must not change the amount of device memory in use.
    spec = gen.LayerSpec("static_4096", M=300, K=4096, N=4096, k=32, calib_rows=32, outlier_frac=0.01, outlier_scale=20.0, seed=94)
    P = _layer(spec)
    Xall = torch.from_numpy(gen.make_activations(spec)).to(DEV)
    ws = L.new_workspace(spec.M, P)
    refused = binding.STATUS_NAMES.index("LQER_ERR_STATIC_SCRATCH")
    for M, fits in ((57, True), (58, False), (300, True), (16, True)):
        assert (L.call_workspace_bytes(M, spec.K, spec.N, spec.k) <= binding.STATIC_SCRATCH_BYTES) == fits
        X = Xall[:M].contiguous()
        Y = torch.full((M, spec.N), float("nan"), dtype=torch.float32, device=DEV)
        if not fits:
            assert L.lib().lqer_linear_static(X.data_ptr(), M, P.ptr, Y.data_ptr(), None) == refused
            continue
        Y_ref = L.linear(X, P, ws)
        torch.cuda.synchronize()
        free0, _ = torch.cuda.mem_get_info()
        held0 = torch.cuda.memory_allocated()
        L.linear_static(X, P, Y)
        torch.cuda.synchronize()
        free1, _ = torch.cuda.mem_get_info()
        assert torch.cuda.memory_allocated() == held0 and free1 >= free0      # nothing was allocated, by torch or by the library
        assert torch.equal(Y, Y_ref), M
    P.release()
