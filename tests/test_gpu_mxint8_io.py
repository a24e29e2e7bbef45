"""MXINT8 activations at the layer's boundary (Section 2.1, w&a setting: the activations between layers are quantised;
Section 4.1: MXINT8, blocks [1,16]).  Output: with y_dtype LQER_MXINT8 the epilogue quantises Y in blocks of 16 along N,
as the next layer's prologue would.  Input (second half of the file): X given in the same layout is taken at its value.

Parity against the oracle.  The oracle quantises its fp64 Y, the library its fp32 Y; the two Y differ by at most the
layer's tolerance, and a quantised code is a decision taken on that value.  So:
  * every dequantised element lies within tol + half a quantisation step of the oracle's Y (a whole step where the
    symmetric clamp holds the block's maximum at 2^(b-1) - 1);
  * a block's shared exponent equals the oracle's unless the block maximum lies within tol of a power of two
    (then it may be the neighbouring exponent);
  * where the exponents agree, a mantissa equals the oracle's unless the oracle's scaled value lies within tol of
    a rounding tie (then it may differ by one).
The quantiser itself is also checked in the kernel's own precision: the codes are exactly what round-to-nearest-even
with the block's exponent gives on the fp32 Y the same path writes.
"""
import ctypes as C

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
E = binding.STATUS_NAMES.index


def _t(a):
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


def _layer(spec):
    W = gen.make_weight(spec)
    if spec.k == 0:
        return olqer.prepare_weights(W, None, None), L.prepare_weights(_t(W), None, None)
    A, B = gen.make_random_factors(spec)
    return olqer.prepare_weights(W, A, B), L.prepare_weights(_t(W), _t(A), _t(B))


def _check_against_oracle(Ym, Ye, ref, a_bits=8):
    """Ym int8 [M, N], Ye exponent bytes [M, N/16] from the library; ref: the oracle's forward result."""
    M, N = ref.Y.shape
    e_gpu = Ye.astype(np.int64) - 127
    om, oe = mxint.quantize(ref.Y, a_bits, axis=1)
    oe = np.asarray(oe, dtype=np.int64)
    shift = a_bits - 2
    step = np.repeat(np.exp2((e_gpu - shift).astype(np.float64)), 16, axis=1)
    dq = Ym.astype(np.float64) * step
    # (1) every element within tol + half a step (a whole step where the symmetric clamp holds a block maximum at qmax)
    qmax = 2 ** (a_bits - 1) - 1
    room = np.where(np.abs(Ym.astype(np.int64)) == qmax, 1.0, 0.5) * step
    assert np.all(np.abs(dq - ref.Y) <= ref.tol + room * (1 + 1e-12))
    # (2) exponents: the oracle's, or the neighbour where the block maximum is within tol of a power of two
    tol_blk = ref.tol.reshape(M, N // 16, 16).max(axis=2)
    amax = np.abs(ref.Y).reshape(M, N // 16, 16).max(axis=2)
    lo = np.floor(np.log2(np.maximum(amax - tol_blk, 2.0 ** -60)))
    hi = np.floor(np.log2(np.maximum(amax + tol_blk, 2.0 ** -60)))
    lo, hi = np.clip(lo, -56, 55), np.clip(hi, -56, 55)
    assert np.all((e_gpu >= lo) & (e_gpu <= hi))
    # (3) mantissas where the exponents agree: equal, or one apart next to a tie
    same = np.repeat(e_gpu == oe, 16, axis=1)
    diff = Ym.astype(np.int64) - om.astype(np.int64)
    assert np.all(np.abs(diff[same]) <= 1)
    off = same & (diff != 0)
    if off.any():
        scaled = ref.Y[off] / step[off]
        to_tie = np.abs(np.abs(scaled - np.floor(scaled)) - 0.5)
        assert np.all(to_tie <= ref.tol[off] / step[off] + 1e-9)
    return float(np.mean(same)), int(off.sum())


def _check_own_precision(Ym, Ye, Y32, a_bits=8):
    """The codes against the fp32 Y of the same path, in the kernel's precision: exponent from the block's maximum,
    round to nearest even, symmetric clamp."""
    M, N = Y32.shape
    blk = Y32.reshape(M, N // 16, 16).astype(np.float64)
    amax = np.abs(blk).max(axis=2)
    e = np.clip(np.floor(np.log2(np.maximum(amax, 2.0 ** -100))), -56, 55)
    assert np.array_equal(Ye.astype(np.int64) - 127, e.astype(np.int64))
    q = 2 ** (a_bits - 1) - 1
    m = np.clip(np.rint(blk / np.exp2(e - (a_bits - 2))[:, :, None]), -q, q)       # rint: half to even
    assert np.array_equal(Ym.reshape(M, N // 16, 16).astype(np.int64), m.astype(np.int64))


SPECS = [gen.LayerSpec("q_a", M=300, K=1024, N=640, k=40, calib_rows=32, outlier_frac=0.01, outlier_scale=20.0, seed=401),
         gen.LayerSpec("q_k0", M=129, K=512, N=400, k=0, calib_rows=32, outlier_frac=0.01, outlier_scale=20.0, seed=402),
         gen.LayerSpec("q_tc", M=1100, K=2112, N=272, k=64, calib_rows=32, outlier_frac=0.005, outlier_scale=50.0,
                       weight_law="student_t4", seed=403)]


@pytest.mark.parametrize("spec", SPECS, ids=lambda s: s.name)
def test_mxint8_output_every_path(spec):
    # the column-owner decode kernel (1, 4 rows), the small-batch kernels (9, 70 rows; the chunks of a tile meet in the
    # last arriver's reduction or the tile is written directly), the pair GEMM without split K (200) and behind either prologue (the spec's own M)
    P, Pg = _layer(spec)
    ws = L.new_workspace(spec.M, Pg)
    for M in (1, 4, 9, 70, 200, spec.M):
        if M > spec.M:
            continue
        X = gen.make_activations(spec, M=M)
        ref = olqer.forward(X, P)
        Yq = L.linear_ex(_t(X), Pg, ws, out_dtype=L.MXINT8)
        assert L.poll_status(ws) == 0
        Ym, Ye = L.split_mxint8(Yq, M, spec.N)
        _check_against_oracle(Ym.cpu().numpy(), Ye.cpu().numpy(), ref)
        # the same path with an fp32 Y (for 128 < M <= 256 the fp32 call would cut K, which an MXINT8 Y does not)
        Y32 = L.linear(_t(X), Pg, ws).cpu().numpy() if not (128 < M <= 256) else None
        if Y32 is not None:
            _check_own_precision(Ym.cpu().numpy(), Ye.cpu().numpy(), Y32)
    Pg.release()


def test_mxint8_output_where_the_sums_round():
    # long K, all terms of one sign: the fp32 sums differ from the oracle's fp64 sums, so codes next to ties and block
    # maxima next to powers of two may legitimately differ; the three rules above must still hold
    spec = gen.LayerSpec("q_round", M=40, K=11008, N=256, k=32, calib_rows=32, outlier_frac=0.01, outlier_scale=20.0, seed=404)
    W = np.abs(gen.make_weight(spec))
    A, B = gen.make_random_factors(spec)
    P, Pg = olqer.prepare_weights(W, A, B), L.prepare_weights(_t(W), _t(A), _t(B))
    X = np.abs(gen.make_activations(spec))
    ref = olqer.forward(X, P)
    ws = L.new_workspace(spec.M, Pg)
    Yq = L.linear_ex(_t(X), Pg, ws, out_dtype=L.MXINT8)
    Ym, Ye = L.split_mxint8(Yq, spec.M, spec.N)
    same, off = _check_against_oracle(Ym.cpu().numpy(), Ye.cpu().numpy(), ref)
    assert same > 0.9
    Pg.release()


def test_mxint8_output_of_shared_launches_and_host_buffers():
    # three prefill layers in one GEMM launch, three small-batch layers in one launch, and the host-buffer entry point
    specs = [gen.LayerSpec("q_g0", M=300, K=512, N=256, k=16, calib_rows=32, outlier_frac=0.01, outlier_scale=20.0, seed=411),
             gen.LayerSpec("q_g1", M=300, K=1024, N=384, k=32, calib_rows=32, outlier_frac=0.01, outlier_scale=20.0, seed=412),
             gen.LayerSpec("q_g2", M=300, K=320, N=512, k=16, calib_rows=32, outlier_frac=0.01, outlier_scale=20.0, seed=413)]
    layers = [_layer(s) for s in specs]
    for M in (300, 24, 12, 3):
        Xs = [gen.make_activations(s, M=M) for s in specs]
        refs = [olqer.forward(X, P) for X, (P, _) in zip(Xs, layers)]
        Yq = [torch.zeros(L.mxint8_bytes(M, s.N), dtype=torch.uint8, device=DEV) for s in specs]
        Xd = [_t(X) for X in Xs]                          # the calls hold pointers only: keep the tensors alive
        calls = L.make_calls([(x, Pg, y) for x, (_, Pg), y in zip(Xd, layers, Yq)], torch.float32, L.MXINT8)
        ws = torch.zeros(L.batched_workspace_bytes(calls), dtype=torch.uint8, device=DEV)
        before = L.launch_count()
        L.linear_batched_ex(calls, ws, torch.float32, L.MXINT8)
        torch.cuda.synchronize()
        assert L.launch_count() - before <= 4           # shared launches: prologue(s) + one GEMM, not one pair per layer
        assert L.poll_status(ws) == 0
        for s, y, ref in zip(specs, Yq, refs):
            Ym, Ye = L.split_mxint8(y, M, s.N)
            _check_against_oracle(Ym.cpu().numpy(), Ye.cpu().numpy(), ref)
        # host buffers
        Xh = [torch.from_numpy(X).pin_memory() for X in Xs]
        Yh = [torch.zeros(L.mxint8_bytes(M, s.N), dtype=torch.uint8).pin_memory() for s in specs]
        hcalls = L.make_host_calls([(x, Pg, y) for x, (_, Pg), y in zip(Xh, layers, Yh)], torch.float32, L.MXINT8)
        wsh = torch.zeros(L.linear_host_batched_bytes(hcalls), dtype=torch.uint8, device=DEV)
        L.linear_host_batched_ex(hcalls, wsh, torch.float32, L.MXINT8)
        for y_dev, y_host in zip(Yq, Yh):
            assert torch.equal(y_dev.cpu(), y_host)
    for _, Pg in layers:
        Pg.release()


def test_mxint8_output_is_refused_where_it_cannot_be_written():
    spec = gen.LayerSpec("q_n8", M=8, K=64, N=136, k=0, calib_rows=32, outlier_frac=0, n_outliers=1, outlier_scale=20.0, seed=421)
    P, Pg = _layer(spec)                                  # N = 136 is a multiple of 8, not of 16
    ws = L.new_workspace(spec.M, Pg)
    X = _t(gen.make_activations(spec))
    Y = torch.zeros(L.mxint8_bytes(spec.M, 144), dtype=torch.uint8, device=DEV)
    launches = L.launch_count()
    st = L.lib().lqer_linear_ex(X.data_ptr(), 0, spec.M, Pg.ptr, Y.data_ptr(), 2, ws.data_ptr(), ws.numel(), None)
    assert st == E("LQER_ERR_SHAPE")
    st = L.lib().lqer_linear_ex(X.data_ptr(), 7, spec.M, Pg.ptr, Y.data_ptr(), 0, ws.data_ptr(), ws.numel(), None)
    assert st == E("LQER_ERR_CONFIG")                     # no such element type
    assert L.launch_count() == launches
    Pg.release()


# ---------------------------------------------------------------------------- MXINT8 input
# X given as mantissas + exponent bytes (the layout of the MXINT8 output): the layer takes it at its value, so it must
# compute exactly what it computes on the fp32 tensor of those values - compared bit for bit with the library's own
# fp32-input result (same path, same X_q) and, through that input, with the oracle.


def _mx_buffer(Xm, Xe):
    return L.to_mxint8(_t(Xm), _t(mxint.exponent_bytes(Xe)))


@pytest.mark.parametrize("spec", SPECS + [gen.LayerSpec("q_ragged", M=300, K=80, N=144, k=5, calib_rows=32, outlier_frac=0, n_outliers=2,
                                                        outlier_scale=20.0, seed=431)], ids=lambda s: s.name)
def test_mxint8_input_every_path(spec):
    P, Pg = _layer(spec)
    ws = L.new_workspace(spec.M, Pg)
    for M in (1, 4, 9, 70, 200, spec.M):
        if M > spec.M:
            continue
        X = gen.make_activations(spec, M=M)
        Xm, Xe = mxint.quantize(X, 8, axis=1)                     # what a previous layer's MXINT8 output would hold
        Xq = _mx_buffer(Xm, Xe)
        ref = olqer.forward(X, P)                                  # the oracle quantises X itself: the same X_q
        assert np.array_equal(ref.Xm, Xm)
        for path in (binding.PATH_AUTO, binding.PATH_TENSOR_PROLOGUE, binding.PATH_TENSOR):
            if path != binding.PATH_AUTO and M < 70:
                continue
            L.set_path(path)
            try:
                Y = L.linear_ex(Xq, Pg, ws, M=M)
                Yf = L.linear(_t(X), Pg, ws)
            finally:
                L.set_path(binding.PATH_AUTO)
            assert L.poll_status(ws) == 0
            assert torch.equal(Y, Yf), (M, path)
            assert float(np.max(np.abs(Y.cpu().numpy().astype(np.float64) - ref.Y) / ref.tol)) <= 1.0, (M, path)
    Pg.release()


def test_mxint8_input_blocks_that_are_not_normalised():
    # blocks a quantiser would not have produced (small mantissas under a large exponent, the extreme -127 beside odd
    # mantissas, all-zero blocks under any exponent): the layer must compute on their values, i.e. what it computes on the fp32 tensor of these values
    spec = gen.LayerSpec("q_raw", M=40, K=512, N=256, k=16, calib_rows=32, outlier_frac=0.01, outlier_scale=20.0, seed=432)
    P, Pg = _layer(spec)
    g = np.random.default_rng(432)
    Xm = g.integers(-20, 21, size=(spec.M, spec.K)).astype(np.int8)
    Xm[:, ::37] = -127
    Xm[3, 16:48] = 0
    Xe = g.integers(-8, 9, size=(spec.M, spec.K // 16)).astype(np.int64)
    X = mxint.dequantize(Xm, Xe, 8, axis=1).astype(np.float32)     # exact: at most 8 significant bits
    ref = olqer.forward(X, P)
    ws = L.new_workspace(spec.M, Pg)
    for M, path in ((2, binding.PATH_AUTO), (spec.M, binding.PATH_AUTO), (spec.M, binding.PATH_TENSOR),
                    (spec.M, binding.PATH_TENSOR_PROLOGUE)):       # the last takes the mantissas as they stand
        L.set_path(path)
        try:
            Y = L.linear_ex(L.to_mxint8(_t(Xm[:M]), _t(mxint.exponent_bytes(Xe[:M]))), Pg, ws, M=M)
            Yf = L.linear(_t(X[:M]), Pg, ws)
        finally:
            L.set_path(binding.PATH_AUTO)
        assert L.poll_status(ws) == 0
        assert torch.equal(Y, Yf), (M, path)
        assert float(np.max(np.abs(Y.cpu().numpy().astype(np.float64) - ref.Y[:M]) / ref.tol[:M])) <= 1.0
    Pg.release()


def test_mxint8_chain_of_two_layers_equals_the_fp32_hand_over():
    # layer 1 writes MXINT8, layer 2 reads it: bit for bit what layer 2 gives on layer 1's fp32 output, because the
    # hand-over quantisation is the one layer 2's prologue would have done itself
    s1 = gen.LayerSpec("q_c1", M=300, K=512, N=1024, k=16, calib_rows=32, outlier_frac=0.01, outlier_scale=20.0, seed=441)
    s2 = gen.LayerSpec("q_c2", M=300, K=1024, N=384, k=32, calib_rows=32, outlier_frac=0.01, outlier_scale=20.0, seed=442)
    (_, Pg1), (_, Pg2) = _layer(s1), _layer(s2)
    for M in (1, 3, 24, 300):
        X = _t(gen.make_activations(s1, M=M))
        ws = L.new_workspace(M, Pg1 if L.workspace_bytes(M, s1.K, s1.N, s1.k) > L.workspace_bytes(M, s2.K, s2.N, s2.k) else Pg2)
        Y1 = L.linear(X, Pg1, ws)
        Y2 = L.linear(Y1, Pg2, ws)
        H = L.linear_ex(X, Pg1, ws, out_dtype=L.MXINT8)            # the hand-over buffer: 17 bytes per 16 activations
        Y2q = L.linear_ex(H, Pg2, ws, M=M)
        assert L.poll_status(ws) == 0
        assert torch.equal(Y2q, Y2), M
    Pg1.release()
    Pg2.release()


def test_mxint8_input_of_shared_launches_and_host_buffers():
    spec = gen.LayerSpec("q_in_b", M=1, K=1024, N=640, k=40, calib_rows=32, outlier_frac=0.01, outlier_scale=20.0, seed=451)
    P, Pg = _layer(spec)
    for M, n in ((1, 20), (24, 3), (300, 3)):
        Xs = [gen.make_activations(spec, M=M) + 0.125 * j for j in range(n)]
        Xq = [_mx_buffer(*mxint.quantize(X, 8, axis=1)) for X in Xs]
        Ys = [torch.zeros((M, spec.N), dtype=torch.float32, device=DEV) for _ in Xs]
        calls = L.make_calls([(x, Pg, y) for x, y in zip(Xq, Ys)], L.MXINT8, torch.float32)
        ws = torch.zeros(L.batched_workspace_bytes(calls), dtype=torch.uint8, device=DEV)
        L.linear_batched_ex(calls, ws, L.MXINT8, torch.float32)
        torch.cuda.synchronize()
        assert L.poll_status(ws) == 0
        for X, y in zip(Xs, Ys):
            ref = olqer.forward(X, P)
            assert float(np.max(np.abs(y.cpu().numpy().astype(np.float64) - ref.Y) / ref.tol)) <= 1.0
            if M != 24:        # (small-batch groups cut K into fewer chunks than single calls: compared with the oracle only)
                assert torch.equal(y, L.linear(_t(X), Pg, ws))
        Xh = [x.cpu().pin_memory() for x in Xq]
        Yh = [torch.zeros((M, spec.N), dtype=torch.float32).pin_memory() for _ in Xs]
        hcalls = L.make_host_calls([(x, Pg, y) for x, y in zip(Xh, Yh)], L.MXINT8, torch.float32)
        wsh = torch.zeros(L.linear_host_batched_bytes(hcalls), dtype=torch.uint8, device=DEV)
        L.linear_host_batched_ex(hcalls, wsh, L.MXINT8, torch.float32)
        for X, yh in zip(Xs, Yh):
            assert torch.equal(yh, L.linear(_t(X), Pg, wsh).cpu())
    Pg.release()


def test_mxint8_both_ways_with_two_bit_weights():
    # W2A8 (Section 4.4) with the quantised hand-over on both sides: the decode kernel on crumbs (1 and 3 rows), the
    # small-batch kernels (40) and the pair GEMM (300)
    spec = gen.LayerSpec("q_w2", M=300, K=1024, N=640, k=72, calib_rows=32, outlier_frac=0.01, outlier_scale=20.0, seed=461)
    cfg = L.default_config()
    cfg.w_bits = 2
    W = gen.make_weight(spec)
    A, B = gen.make_random_factors(spec)
    P = olqer.prepare_weights(W, A, B, w_bits=2)
    Pg = L.prepare_weights(_t(W), _t(A), _t(B), cfg)
    ws = L.new_workspace(spec.M, Pg)
    for M in (1, 3, 40, spec.M):
        X = gen.make_activations(spec, M=M)
        ref = olqer.forward(X, P, w_bits=2)
        Xq = _mx_buffer(*mxint.quantize(X, 8, axis=1))
        Yq = L.linear_ex(Xq, Pg, ws, out_dtype=L.MXINT8, M=M)
        assert L.poll_status(ws) == 0
        Ym, Ye = L.split_mxint8(Yq, M, spec.N)
        _check_against_oracle(Ym.cpu().numpy(), Ye.cpu().numpy(), ref)
        _check_own_precision(Ym.cpu().numpy(), Ye.cpu().numpy(), L.linear(_t(X), Pg, ws).cpu().numpy())
    Pg.release()
