"""Device-side error reporting, save / restore of packed buffers, and the host checks around them.

Every wait of a kernel on another CTA, warp or copy is bounded.  These tests make such a wait run out in the
allowed way: the bound is shortened to about a millisecond and the next launch of one kernel family is told
(host-side hook) to expect an arrival that never comes, or has its last operand stage withheld.  Nothing is
accessed out of bounds and nothing spins for ever: every CTA gives up, the kernel writes LQER_ERR_TIMEOUT to the
status word and returns.  Then the workspace is re-initialised and an ordinary call must give the ordinary result.
"""
import ctypes as C

import numpy as np
import pytest
import torch

import lqer_inputs as gen
import paper_2402_02446_b200 as L
from paper_2402_02446_b200 import binding
from oracle import lqer as olqer
from helpers import worst_ratio

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
E = binding.STATUS_NAMES.index
FAM_PROLOGUE, FAM_GEMM, FAM_DECODE = 3, 6, 7


def _t(a):
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


def _layer(spec):
    W = gen.make_weight(spec)
    A, B = gen.make_random_factors(spec)
    return olqer.prepare_weights(W, A, B), L.prepare_weights(_t(W), _t(A), _t(B))


CASES = [
    # (name, family, forced path, M, K, N, k)
    ("decode_cols_T_exchange", FAM_DECODE, binding.PATH_AUTO, 2, 2112, 264, 72),   # 132 K blocks x 3 rank tiles: T is exchanged
    ("small_gemm_ring", FAM_DECODE, binding.PATH_AUTO, 9, 1024, 640, 40),
    ("small_mma_flags", FAM_DECODE, binding.PATH_SMALL, 9, 1024, 640, 40),      # the polls of the prologue's flags
    ("prologue_tc_row_tile", FAM_PROLOGUE, binding.PATH_TENSOR_PROLOGUE, 300, 1024, 640, 32),
    ("gemm_pair_ring", FAM_GEMM, binding.PATH_AUTO, 300, 1024, 640, 40),
]


@pytest.mark.parametrize("name,family,path,M,K,N,k", CASES, ids=[c[0] for c in CASES])
def test_bounded_wait_runs_out_and_the_workspace_recovers(name, family, path, M, K, N, k):
    spec = gen.LayerSpec(name, M=M, K=K, N=N, k=k, calib_rows=32, outlier_frac=0.01, outlier_scale=20.0, seed=201)
    P, Pg = _layer(spec)
    X = _t(gen.make_activations(spec))
    ws = L.new_workspace(M, Pg)
    L.set_path(path)
    try:
        Y_good = L.linear(X, Pg, ws).clone()
        assert L.poll_status(ws) == 0
        L.set_wait_limit_cycles(2_000_000)              # about a millisecond
        L.inject_stall(family)
        try:
            Y_bad = torch.zeros_like(Y_good)
            L.linear(X, Pg, ws, Y_bad)
            torch.cuda.synchronize()                    # the launch ends by itself
        finally:
            L.inject_stall(-1)
            L.set_wait_limit_cycles(4_000_000_000)
        assert L.poll_status(ws) == E("LQER_ERR_TIMEOUT")
        # an interrupted call may leave counters behind: the documented recovery is lqer_workspace_init
        assert L.lib().lqer_workspace_init(ws.data_ptr(), ws.numel(), None) == 0
        assert L.poll_status(ws) == 0
        for _ in range(2):
            Y_again = L.linear(X, Pg, ws)
            assert L.poll_status(ws) == 0
            assert torch.equal(Y_again, Y_good)
    finally:
        L.set_path(binding.PATH_AUTO)
    assert worst_ratio(Y_good.cpu().numpy(), olqer.forward(X.cpu().numpy(), P)) <= 1.0
    Pg.release()


def test_hooks_validate_their_arguments():
    lib = L.lib()
    assert lib.lqer_set_wait_limit_cycles(0) == E("LQER_ERR_CONFIG")
    assert lib.lqer_inject_stall(99) == E("LQER_ERR_CONFIG")
    assert lib.lqer_inject_stall(-1) == 0


def test_packed_buffer_moves_to_a_new_address():
    # save / restore: the header travels with the buffer, so a byte-for-byte copy at another address is a packed
    # buffer too - with lqer_attach_packed, or without (the first call reads the header back once)
    spec = gen.LayerSpec("moved", M=37, K=320, N=392, k=24, calib_rows=32, outlier_frac=0.01, outlier_scale=20.0, seed=202)
    P, Pg = _layer(spec)
    X = _t(gen.make_activations(spec))
    ws = L.new_workspace(spec.M, Pg)
    Y0 = L.linear(X, Pg, ws).clone()
    saved = Pg.buf.cpu()                                               # "file"
    for attach in (False, True):
        buf = saved.to(DEV)
        assert buf.data_ptr() != Pg.ptr
        if attach:
            assert L.lib().lqer_attach_packed(buf.data_ptr(), buf.numel(), None) == 0
        moved = binding.PackedWeights(buf, spec.K, spec.N, spec.k, Pg.k_pad)
        Kq, Nq, kq = C.c_int(), C.c_int(), C.c_int()
        assert L.lib().lqer_packed_shape(buf.data_ptr(), C.byref(Kq), C.byref(Nq), C.byref(kq), None) == 0
        assert (Kq.value, Nq.value, kq.value) == (spec.K, spec.N, spec.k)
        assert torch.equal(L.linear(X, moved, ws), Y0)
        for M in (1, 9):
            assert torch.equal(L.linear(X[:M].contiguous(), moved, ws), L.linear(X[:M].contiguous(), Pg, ws))
        moved.release()
    # a corrupt header is refused, by either route, before anything is launched
    for byte in (0, 9, 40, 131):
        bad = saved.clone()
        bad[byte] ^= 0x5A
        bad = bad.to(DEV)
        launches = L.launch_count()
        assert L.lib().lqer_attach_packed(bad.data_ptr(), bad.numel(), None) == E("LQER_ERR_BAD_PACKED")
        Y = torch.empty((spec.M, spec.N), dtype=torch.float32, device=DEV)
        st = L.lib().lqer_linear_stream(X.data_ptr(), spec.M, bad.data_ptr(), Y.data_ptr(), ws.data_ptr(), ws.numel(), None)
        assert st == E("LQER_ERR_BAD_PACKED")
        assert L.launch_count() == launches
    # too short a buffer for what its header describes
    short = saved[: saved.numel() // 2].to(DEV)
    assert L.lib().lqer_attach_packed(short.data_ptr(), short.numel(), None) == E("LQER_ERR_BUFFER_TOO_SMALL")
    assert worst_ratio(Y0.cpu().numpy(), olqer.forward(X.cpu().numpy(), P)) <= 1.0
    Pg.release()
