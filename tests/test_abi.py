"""The C-ABI library loads, exports every declared symbol, and validates arguments on the host."""
import ctypes as C
import os
import re

import pytest

import paper_2402_02446_b200 as L
from paper_2402_02446_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    names = set()
    inc = os.path.join(ROOT, "include")
    for fn in os.listdir(inc):
        if fn.endswith(".h"):
            text = open(os.path.join(inc, fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(lqer_[a-z_0-9]+)\s*\(", text))
    return sorted(names)


def test_every_declared_symbol_is_exported():
    lib = C.CDLL(L.lib_path())
    names = _declared()
    assert len(names) >= 18
    for n in names:
        assert hasattr(lib, n), n


def test_binding_covers_every_symbol():
    L.lib()
    src = open(os.path.join(ROOT, "paper_2402_02446_b200", "binding.py")).read()
    for n in _declared():
        assert f'"{n}"' in src, n


def test_status_strings_and_defaults():
    lib = L.lib()
    seen = {lib.lqer_status_string(i) for i in range(11)}
    assert len(seen) == 11 and lib.lqer_status_string(0) == b"ok"
    cfg = L.default_config()
    assert (cfg.w_bits, cfg.a_bits, cfg.lr_bits, cfg.block, cfg.exp_min, cfg.exp_max) == (4, 8, 8, 16, -56, 55)
    assert (cfg.w_exp_min, cfg.w_exp_max, cfg.deterministic) == (-56, 55, 1)


def test_size_queries_follow_the_format():
    # Section 4.1 storage: 4 bits + 1 exponent byte per 16 for W_q; 8 bits + 1 byte per 16 for A_k, B_k
    K = N = 4096
    k = 32
    algorithmic = K * N * 0.5625 + 1.0625 * (k * K + k * N)
    got = L.packed_bytes(K, N, k)
    assert algorithmic <= got <= algorithmic + 1024
    assert L.packed_bytes(256, 256, 8) >= 256 * 256 * 0.5625 + 1.0625 * 16 * 512
    # workspace: a zeroed head (status, counters, accumulator) + bf16 [X_q | T_q] and the fp64 partial sums of
    # the tensor-core prologue (at most 148 CTAs x [128, k_pad]), or the decode slots
    xcat = 2048 * (4096 + 32) * 2
    partials = 148 * 128 * 32 * 8
    head = 168192                                     # one size for every layer
    assert head + xcat <= L.workspace_bytes(2048, 4096, 11008, 32) <= head + xcat + partials + 16384
    assert L.workspace_bytes(1, 4096, 4096, 0) >= head + 4096 * 2
    assert L.workspace_bytes(1, 4096, 4096, 32) <= 4 << 20


def test_host_side_argument_errors():
    lib = L.lib()
    cfg = L.default_config()
    out = C.c_size_t()
    E = binding.STATUS_NAMES.index
    assert lib.lqer_packed_bytes(100, 256, 8, C.byref(cfg), C.byref(out)) == E("LQER_ERR_SHAPE")   # K % 16
    assert lib.lqer_packed_bytes(256, 100, 8, C.byref(cfg), C.byref(out)) == E("LQER_ERR_SHAPE")   # N % 8
    assert lib.lqer_packed_bytes(256, 256, 512, C.byref(cfg), C.byref(out)) == E("LQER_ERR_SHAPE")  # rank
    assert lib.lqer_packed_bytes(256, 256, 8, None, C.byref(out)) == E("LQER_ERR_NULL")
    assert lib.lqer_packed_bytes(256, 256, 8, C.byref(cfg), None) == E("LQER_ERR_NULL")
    bad = L.default_config(); bad.w_bits = 3
    assert lib.lqer_packed_bytes(256, 256, 8, C.byref(bad), C.byref(out)) == E("LQER_ERR_CONFIG")
    two = L.default_config(); two.w_bits = 2           # W2A8 (Section 4.4): 2 bits + 1 exponent byte per 16
    assert lib.lqer_packed_bytes(4096, 4096, 0, C.byref(two), C.byref(out)) == 0
    assert 4096 * 4096 * 0.3125 <= out.value <= 4096 * 4096 * 0.3125 + 1024
    bad = L.default_config(); bad.exp_min = -100
    assert lib.lqer_packed_bytes(256, 256, 8, C.byref(bad), C.byref(out)) == E("LQER_ERR_CONFIG")
    bad = L.default_config(); bad.w_exp_max = 56
    assert lib.lqer_packed_bytes(256, 256, 8, C.byref(bad), C.byref(out)) == E("LQER_ERR_CONFIG")
    bad = L.default_config(); bad.w_exp_min, bad.w_exp_max = 4, 3
    assert lib.lqer_packed_bytes(256, 256, 8, C.byref(bad), C.byref(out)) == E("LQER_ERR_CONFIG")
    for a_bits, ok in ((2, False), (3, True), (6, True), (8, True), (9, False)):   # activation mantissa width
        c6 = L.default_config(); c6.a_bits = a_bits
        want = E("LQER_OK") if ok else E("LQER_ERR_CONFIG")
        assert lib.lqer_packed_bytes(256, 256, 8, C.byref(c6), C.byref(out)) == want
    # null / unknown buffers are refused before anything is launched
    assert lib.lqer_linear(None, 1, None, None, None, 0) == E("LQER_ERR_NULL")
    assert lib.lqer_linear_stream(4096, 1, 8192, 4096, 4096, 1 << 20, None) == E("LQER_ERR_BAD_PACKED")
    assert lib.lqer_linear_stream(4096 + 4, 1, 8192, 4096, 4096, 1 << 20, None) == E("LQER_ERR_ALIGN")
    assert lib.lqer_linear_stream(4096, 0, 8192, 4096, 4096, 1 << 20, None) == E("LQER_ERR_SHAPE")
    assert lib.lqer_prepare_weights(None, None, None, 256, 256, 0, C.byref(cfg), None, 0, None) == E("LQER_ERR_NULL")
    assert lib.lqer_prepare_weights(4096, None, None, 256, 256, 8, C.byref(cfg), 4096, 1 << 20, None) == E("LQER_ERR_NULL")
    assert lib.lqer_prepare_weights(4096, None, None, 256, 256, 0, C.byref(cfg), 4096, 16, None) == E("LQER_ERR_BUFFER_TOO_SMALL")
    assert lib.lqer_prepare_weights(4096, None, None, 256, 256, 0, C.byref(cfg), 4096 + 16, 1 << 20, None) == E("LQER_ERR_ALIGN")
    assert lib.lqer_release_packed(12345 * 256) == E("LQER_ERR_BAD_PACKED")
    assert lib.lqer_linear_batched(None, 1, 4096, 4096, None) == E("LQER_ERR_NULL")
    assert lib.lqer_set_path(9) == E("LQER_ERR_CONFIG")
    assert lib.lqer_set_path(0) == 0
    st = C.c_int()
    assert lib.lqer_poll_status(None, None, C.byref(st)) == E("LQER_ERR_NULL")
    assert lib.lqer_workspace_init(4096, 16, None) == E("LQER_ERR_BUFFER_TOO_SMALL")
    assert L.launch_count() == 0


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "_LIB_PATH", "/nonexistent/liblqer.so")
    with pytest.raises(ImportError):
        binding.lib()


def test_workspace_bound_covers_every_smaller_batch():
    # lqer_workspace_bytes(M_max) must fit the call with any M <= M_max, whichever path that call takes: the
    # small-batch kernels (M <= 128), the split-K GEMM (M <= 256), the tensor-core prologue's partial sums (row tiles x K ranges,
    # which grows past one CTA per SM once there are more than 148 row tiles)
    Ms = [1, 4, 16, 17, 64, 127, 128, 129, 255, 256, 257, 300, 511, 512, 1023, 1024, 2048, 4096, 18944, 19072,
          32768, 65536]
    for K, N, k in [(4096, 256, 64), (4096, 4096, 32), (11008, 4096, 32), (5120, 13824, 256), (256, 256, 8),
                    (2112, 264, 16), (4096, 4096, 0), (1024, 640, 40)]:
        need = [L.call_workspace_bytes(M, K, N, k) for M in Ms]
        for i, M_max in enumerate(Ms):
            total = L.workspace_bytes(M_max, K, N, k)
            assert total >= max(need[: i + 1]), (K, N, k, M_max)


def test_static_scratch_limits_follow_the_call_need():
    # the figures the header states for lqer_linear_static at K = N = 4096, rank 32
    fits = lambda M: L.call_workspace_bytes(M, 4096, 4096, 32) <= binding.STATIC_SCRATCH_BYTES
    assert all(fits(M) for M in (1, 16, 17, 57, 257, 487))
    assert not fits(58) and not fits(128) and not fits(256) and not fits(488)
    # decode-sized calls fit for every K up to 131072, and whatever N
    assert L.call_workspace_bytes(16, 131072, 4096, 256) <= binding.STATIC_SCRATCH_BYTES
    assert L.call_workspace_bytes(16, 4096, 1 << 22, 256) <= binding.STATIC_SCRATCH_BYTES
