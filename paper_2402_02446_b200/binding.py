"""ctypes binding of include/lqer.h.  Argument marshalling only.

torch is used for device memory and streams; tensors are passed to the library
as raw device pointers.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# LQER_DEBUG_BOUNDS=1 in the environment selects the checked build of the library (see include/lqer.h).
DEBUG_BOUNDS = os.environ.get("LQER_DEBUG_BOUNDS", "0") not in ("", "0")
_LIB_PATH = os.path.join(_HERE, "lib", "liblqer_dbg.so" if DEBUG_BOUNDS else "liblqer.so")
_lib = None

STATUS_NAMES = ["LQER_OK", "LQER_ERR_NULL", "LQER_ERR_SHAPE", "LQER_ERR_ALIGN", "LQER_ERR_CONFIG",
                "LQER_ERR_BUFFER_TOO_SMALL", "LQER_ERR_BAD_PACKED", "LQER_ERR_ARCH", "LQER_ERR_CUDA",
                "LQER_ERR_TIMEOUT", "LQER_ERR_BOUNDS", "LQER_ERR_STATIC_SCRATCH"]

PATH_AUTO, PATH_SIMT, PATH_DECODE, PATH_TENSOR, PATH_TENSOR_PAIR, PATH_SMALL, PATH_TENSOR_PROLOGUE, PATH_SMALL_TMEM = 0, 1, 2, 3, 4, 5, 6, 7


class LqerError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        name = STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else str(status)
        super().__init__(f"{what}: {name} ({lib().lqer_status_string(status).decode()})")


class Config(C.Structure):
    _fields_ = [("w_bits", C.c_int), ("a_bits", C.c_int), ("lr_bits", C.c_int), ("block", C.c_int),
                ("exp_min", C.c_int), ("exp_max", C.c_int), ("deterministic", C.c_int),
                ("w_exp_min", C.c_int), ("w_exp_max", C.c_int)]


KERNEL_FAMILIES = ["pack", "export", "quantize", "prologue", "gemm_simt", "prepare", "gemm_tc_pair", "decode"]


class KernelTimes(C.Structure):
    _fields_ = [("launches", C.c_ulonglong * len(KERNEL_FAMILIES)), ("milliseconds", C.c_double * len(KERNEL_FAMILIES))]


class Call(C.Structure):
    _fields_ = [("X", C.c_void_p), ("M", C.c_int), ("packed", C.c_void_p), ("Y", C.c_void_p)]


def lib_path() -> str:
    return _LIB_PATH


def lib() -> C.CDLL:
    """The loaded CUDA library.  Raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise ImportError(f"{_LIB_PATH} is missing: build it with `python -m paper_2402_02446_b200.build` "
                              "(there is no CPU fallback)")
        L = C.CDLL(_LIB_PATH)
        vp, sz, i = C.c_void_p, C.c_size_t, C.c_int
        cfgp = C.POINTER(Config)
        sig = {
            "lqer_status_string": (C.c_char_p, [i]),
            "lqer_default_config": (i, [cfgp]),
            "lqer_packed_bytes": (i, [i, i, i, cfgp, C.POINTER(sz)]),
            "lqer_workspace_bytes": (i, [i, i, i, i, cfgp, C.POINTER(sz)]),
            "lqer_call_workspace_bytes": (i, [i, i, i, i, cfgp, C.POINTER(sz)]),
            "lqer_set_wait_limit_cycles": (i, [C.c_longlong]),
            "lqer_inject_stall": (i, [i]),
            "lqer_debug_bounds_shrink": (i, [C.c_longlong]),
            "lqer_prepare_weights": (i, [vp, vp, vp, i, i, i, cfgp, vp, sz, vp]),
            "lqer_factor_sketch_columns": (i, [i, i, i, C.POINTER(i)]),
            "lqer_prepare_workspace_bytes": (i, [i, i, i, C.POINTER(sz)]),
            "lqer_prepare_from_calibration": (i, [vp, C.POINTER(vp), C.POINTER(i), i, vp, i, i, i, cfgp, vp, sz, vp, vp, vp, sz, vp]),
            "lqer_prepare_status": (i, [vp, i, i, i, vp, C.POINTER(i)]),
            "lqer_attach_packed": (i, [vp, sz, vp]),
            "lqer_release_packed": (i, [vp]),
            "lqer_packed_shape": (i, [vp, C.POINTER(i), C.POINTER(i), C.POINTER(i), C.POINTER(i)]),
            "lqer_export_weights": (i, [vp, vp, vp, vp, vp, vp, vp, vp]),
            "lqer_quantize_activations": (i, [vp, i, i, cfgp, vp, vp, vp]),
            "lqer_project_lowrank": (i, [vp, i, vp, vp, vp, vp, sz, vp]),
            "lqer_linear": (i, [vp, i, vp, vp, vp, sz]),
            "lqer_linear_stream": (i, [vp, i, vp, vp, vp, sz, vp]),
            "lqer_linear_static": (i, [vp, i, vp, vp, vp]),
            "lqer_linear_ex": (i, [vp, i, i, vp, vp, i, vp, sz, vp]),
            "lqer_linear_batched_ex": (i, [C.POINTER(Call), i, i, i, vp, sz, vp]),
            "lqer_linear_batched": (i, [C.POINTER(Call), i, vp, sz, vp]),
            "lqer_batched_workspace_bytes": (i, [C.POINTER(Call), i, C.POINTER(sz)]),
            "lqer_linear_host": (i, [vp, i, vp, vp, vp, sz, vp]),
            "lqer_linear_host_batched_bytes": (i, [C.POINTER(Call), i, C.POINTER(sz)]),
            "lqer_linear_host_batched": (i, [C.POINTER(Call), i, vp, sz, vp]),
            "lqer_linear_host_batched_ex": (i, [C.POINTER(Call), i, i, i, vp, sz, vp]),
            "lqer_workspace_init": (i, [vp, sz, vp]),
            "lqer_poll_status": (i, [vp, vp, C.POINTER(i)]),
            "lqer_set_path": (i, [i]),
            "lqer_launch_count": (C.c_ulonglong, []),
            "lqer_profile_enable": (i, [i]),
            "lqer_profile_collect": (i, [C.POINTER(KernelTimes)]),
        }
        for name, (res, args) in sig.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _lib = L
    return _lib


def _check(status: int, what: str) -> None:
    if status != 0:
        raise LqerError(status, what)


def _stream(stream=None) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return int(s.cuda_stream)


def _dev(t: torch.Tensor, dtype=None) -> int:
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    if dtype is not None and t.dtype != dtype:
        raise ValueError(f"expected dtype {dtype}, got {t.dtype}")
    return t.data_ptr()


def default_config() -> Config:
    cfg = Config()
    _check(lib().lqer_default_config(C.byref(cfg)), "lqer_default_config")
    return cfg


def packed_bytes(K: int, N: int, k: int, cfg: Config | None = None) -> int:
    cfg = cfg or default_config()
    out = C.c_size_t()
    _check(lib().lqer_packed_bytes(K, N, k, C.byref(cfg), C.byref(out)), "lqer_packed_bytes")
    return out.value


def workspace_bytes(M_max: int, K: int, N: int, k: int, cfg: Config | None = None) -> int:
    cfg = cfg or default_config()
    out = C.c_size_t()
    _check(lib().lqer_workspace_bytes(M_max, K, N, k, C.byref(cfg), C.byref(out)), "lqer_workspace_bytes")
    return out.value


def call_workspace_bytes(M: int, K: int, N: int, k: int, cfg: Config | None = None) -> int:
    cfg = cfg or default_config()
    out = C.c_size_t()
    _check(lib().lqer_call_workspace_bytes(M, K, N, k, C.byref(cfg), C.byref(out)), "lqer_call_workspace_bytes")
    return out.value


@dataclass
class PackedWeights:
    buf: torch.Tensor   # uint8 device buffer in the kernel layout
    K: int
    N: int
    k: int
    k_pad: int

    @property
    def ptr(self) -> int:
        return self.buf.data_ptr()

    def release(self) -> None:
        lib().lqer_release_packed(self.ptr)


def prepare_weights(W: torch.Tensor, A: torch.Tensor | None, B: torch.Tensor | None,
                    cfg: Config | None = None, stream=None) -> PackedWeights:
    cfg = cfg or default_config()
    K, N = W.shape
    k = 0 if A is None else A.shape[1]
    nbytes = packed_bytes(K, N, k, cfg)
    buf = torch.empty(nbytes, dtype=torch.uint8, device=W.device)
    _check(lib().lqer_prepare_weights(_dev(W, torch.float32), None if k == 0 else _dev(A, torch.float32),
                                      None if k == 0 else _dev(B, torch.float32), K, N, k, C.byref(cfg),
                                      buf.data_ptr(), nbytes, _stream(stream)), "lqer_prepare_weights")
    return PackedWeights(buf, K, N, k, (k + 15) // 16 * 16)


def factor_sketch_columns(K: int, N: int, k: int) -> int:
    out = C.c_int()
    _check(lib().lqer_factor_sketch_columns(K, N, k, C.byref(out)), "lqer_factor_sketch_columns")
    return out.value


def prepare_from_calibration(W: torch.Tensor, samples, k: int, omega: torch.Tensor | None = None,
                             cfg: Config | None = None, seed: int = 0, stream=None):
    """Packed weights from W and calibration samples alone (an empty list gives plain LQER).  Returns
    (PackedWeights, A [K,k], B [k,N], device status code)."""
    cfg = cfg or default_config()
    K, N = W.shape
    cols = factor_sketch_columns(K, N, k)
    if omega is None:
        g = torch.Generator(device=W.device)
        g.manual_seed(seed)
        omega = torch.randn((N, cols), generator=g, device=W.device, dtype=torch.float32)
    nbytes = packed_bytes(K, N, k, cfg)
    buf = torch.empty(nbytes, dtype=torch.uint8, device=W.device)
    wsb = C.c_size_t()
    _check(lib().lqer_prepare_workspace_bytes(K, N, k, C.byref(wsb)), "lqer_prepare_workspace_bytes")
    ws = torch.empty(wsb.value, dtype=torch.uint8, device=W.device)
    A = torch.empty((K, k), dtype=torch.float32, device=W.device)
    B = torch.empty((k, N), dtype=torch.float32, device=W.device)
    samples = list(samples)
    ptrs = (C.c_void_p * max(len(samples), 1))(*[_dev(x, torch.float32) for x in samples])
    rows = (C.c_int * max(len(samples), 1))(*[x.shape[0] for x in samples])
    _check(lib().lqer_prepare_from_calibration(_dev(W, torch.float32), ptrs, rows, len(samples), _dev(omega, torch.float32), K, N, k,
                                               C.byref(cfg), buf.data_ptr(), nbytes, A.data_ptr(), B.data_ptr(), ws.data_ptr(),
                                               ws.numel(), _stream(stream)), "lqer_prepare_from_calibration")
    code = C.c_int()
    _check(lib().lqer_prepare_status(ws.data_ptr(), K, N, k, _stream(stream), C.byref(code)), "lqer_prepare_status")
    return PackedWeights(buf, K, N, k, (k + 15) // 16 * 16), A, B, code.value


def export_weights(P: PackedWeights, stream=None) -> dict:
    dev = P.buf.device
    out = {"Wm": torch.empty((P.K, P.N), dtype=torch.int8, device=dev),
           "We": torch.empty((P.K // 16, P.N), dtype=torch.uint8, device=dev)}
    ptrs = [out["Wm"].data_ptr(), out["We"].data_ptr()]
    if P.k > 0:
        out["Am"] = torch.empty((P.K, P.k), dtype=torch.int8, device=dev)
        out["Ae"] = torch.empty((P.K // 16, P.k), dtype=torch.uint8, device=dev)
        out["Bm"] = torch.empty((P.k_pad, P.N), dtype=torch.int8, device=dev)
        out["Be"] = torch.empty((P.k_pad // 16, P.N), dtype=torch.uint8, device=dev)
        ptrs += [out[n].data_ptr() for n in ("Am", "Ae", "Bm", "Be")]
    else:
        ptrs += [None] * 4
    _check(lib().lqer_export_weights(P.ptr, *ptrs, _stream(stream)), "lqer_export_weights")
    return out


def quantize_activations(X: torch.Tensor, cfg: Config | None = None, stream=None):
    cfg = cfg or default_config()
    M, K = X.shape
    Xm = torch.empty((M, K), dtype=torch.int8, device=X.device)
    Xe = torch.empty((M, K // 16), dtype=torch.uint8, device=X.device)
    _check(lib().lqer_quantize_activations(_dev(X, torch.float32), M, K, C.byref(cfg), Xm.data_ptr(),
                                           Xe.data_ptr(), _stream(stream)), "lqer_quantize_activations")
    return Xm, Xe


def new_workspace(M_max: int, P: PackedWeights, extra_bytes: int = 0, stream=None) -> torch.Tensor:
    n = workspace_bytes(M_max, P.K, P.N, P.k) + extra_bytes
    ws = torch.empty(n, dtype=torch.uint8, device=P.buf.device)
    _check(lib().lqer_workspace_init(ws.data_ptr(), n, _stream(stream)), "lqer_workspace_init")
    return ws


def project_lowrank(X: torch.Tensor, P: PackedWeights, ws: torch.Tensor, stream=None):
    M = X.shape[0]
    Tm = torch.empty((M, P.k_pad), dtype=torch.int8, device=X.device)
    Te = torch.empty((M, P.k_pad // 16), dtype=torch.uint8, device=X.device)
    _check(lib().lqer_project_lowrank(_dev(X, torch.float32), M, P.ptr, Tm.data_ptr(), Te.data_ptr(),
                                      ws.data_ptr(), ws.numel(), _stream(stream)), "lqer_project_lowrank")
    return Tm, Te


def linear(X: torch.Tensor, P: PackedWeights, ws: torch.Tensor, Y: torch.Tensor | None = None, stream=None):
    M = X.shape[0]
    if Y is None:
        Y = torch.empty((M, P.N), dtype=torch.float32, device=X.device)
    _check(lib().lqer_linear_stream(_dev(X, torch.float32), M, P.ptr, _dev(Y, torch.float32), ws.data_ptr(),
                                    ws.numel(), _stream(stream)), "lqer_linear_stream")
    return Y


MXINT8 = "mxint8"       # output type: a flat uint8 buffer, int8 mantissas [M, N] then exponent bytes [M, N / 16]
_DTYPES = {torch.float32: 0, torch.bfloat16: 1, MXINT8: 2}


def _tensor_dtype(dt):
    return torch.uint8 if dt == MXINT8 else dt


def mxint8_bytes(M: int, N: int) -> int:
    return M * N + M * N // 16


def split_mxint8(Y: torch.Tensor, M: int, N: int):
    """Views of an MXINT8 output buffer: (mantissas int8 [M, N], exponent bytes uint8 [M, N / 16])."""
    return Y[: M * N].view(torch.int8).view(M, N), Y[M * N: M * N + M * N // 16].view(M, N // 16)


def linear_ex(X: torch.Tensor, P: PackedWeights, ws: torch.Tensor, Y: torch.Tensor | None = None,
              out_dtype=torch.float32, stream=None, M: int | None = None):
    """The layer with fp32, bf16 or MXINT8 activations in and fp32, bf16 or MXINT8 out.  The input type is taken from X
    (a flat uint8 tensor is an MXINT8 X of M rows: give M), the output type from out_dtype; an MXINT8 Y is a flat uint8
    buffer of mxint8_bytes(M, N), see split_mxint8."""
    x_dtype = MXINT8 if X.dtype == torch.uint8 else X.dtype
    if x_dtype == MXINT8:
        if M is None or X.numel() != mxint8_bytes(M, P.K):
            raise ValueError("an MXINT8 X is a flat uint8 tensor of mxint8_bytes(M, K); pass M")
    else:
        M = X.shape[0]
    if Y is None:
        Y = (torch.empty(mxint8_bytes(M, P.N), dtype=torch.uint8, device=X.device) if out_dtype == MXINT8
             else torch.empty((M, P.N), dtype=out_dtype, device=X.device))
    elif out_dtype != MXINT8:
        out_dtype = Y.dtype
    _check(lib().lqer_linear_ex(_dev(X), _DTYPES[x_dtype], M, P.ptr, _dev(Y, _tensor_dtype(out_dtype)), _DTYPES[out_dtype],
                                ws.data_ptr(), ws.numel(), _stream(stream)), "lqer_linear_ex")
    return Y


def to_mxint8(Xm: torch.Tensor, Xe: torch.Tensor) -> torch.Tensor:
    """The flat MXINT8 buffer of mantissas Xm int8 [M, K] and exponent bytes Xe uint8 [M, K / 16]."""
    return torch.cat([Xm.contiguous().view(torch.uint8).flatten(), Xe.contiguous().flatten()])


def linear_static(X: torch.Tensor, P: PackedWeights, Y: torch.Tensor | None = None, stream=None):
    """The layer without a caller-provided workspace: the scratch is a fixed array inside the
    library (STATIC_SCRATCH_BYTES); nothing is allocated by the call (Y must be given for that to
    hold on the Python side too)."""
    M = X.shape[0]
    if Y is None:
        Y = torch.empty((M, P.N), dtype=torch.float32, device=X.device)
    _check(lib().lqer_linear_static(_dev(X, torch.float32), M, P.ptr, _dev(Y, torch.float32), _stream(stream)),
           "lqer_linear_static")
    return Y


STATIC_SCRATCH_BYTES = 8 << 20


def _rows(X: torch.Tensor, P: "PackedWeights", x_dtype) -> int:
    """Rows of an activation tensor: its first dimension, or, for a flat MXINT8 buffer, what its size says."""
    if x_dtype != MXINT8:
        return X.shape[0]
    M, rest = divmod(X.numel() * 16, 17 * P.K)
    if rest:
        raise ValueError("an MXINT8 X holds mxint8_bytes(M, K) bytes")
    return M


def make_calls(items, x_dtype=torch.float32, y_dtype=torch.float32) -> "C.Array":
    """items: iterable of (X, PackedWeights, Y) -> a host array of lqer_call_t."""
    items = list(items)
    arr = (Call * len(items))()
    for j, (X, P, Y) in enumerate(items):
        arr[j] = Call(_dev(X, _tensor_dtype(x_dtype)), _rows(X, P, x_dtype), P.ptr, _dev(Y, _tensor_dtype(y_dtype)))
    return arr


def batched_workspace_bytes(calls) -> int:
    """Workspace size with which lqer_linear_batched can run same-shape neighbours in shared launches."""
    arr = calls if isinstance(calls, C.Array) else make_calls(calls)
    out = C.c_size_t()
    _check(lib().lqer_batched_workspace_bytes(arr, len(arr), C.byref(out)), "lqer_batched_workspace_bytes")
    return out.value


def linear_batched(calls, ws: torch.Tensor, stream=None) -> None:
    arr = calls if isinstance(calls, C.Array) else make_calls(calls)
    _check(lib().lqer_linear_batched(arr, len(arr), ws.data_ptr(), ws.numel(), _stream(stream)),
           "lqer_linear_batched")


def linear_batched_ex(calls, ws: torch.Tensor, x_dtype, y_dtype, stream=None) -> None:
    """linear_batched with every X of x_dtype (fp32 or bf16) and every Y of y_dtype (fp32, bf16 or MXINT8); `calls` from
    make_calls(..., x_dtype, y_dtype)."""
    _check(lib().lqer_linear_batched_ex(calls, len(calls), _DTYPES[x_dtype], _DTYPES[y_dtype], ws.data_ptr(), ws.numel(),
                                        _stream(stream)), "lqer_linear_batched_ex")


def linear_host(X_host: torch.Tensor, P: PackedWeights, ws: torch.Tensor, Y_host: torch.Tensor, stream=None):
    """X_host / Y_host are (pinned) CPU tensors; copies both ways happen inside the call."""
    if X_host.is_cuda or Y_host.is_cuda or not X_host.is_contiguous() or not Y_host.is_contiguous():
        raise ValueError("expected contiguous CPU tensors")
    _check(lib().lqer_linear_host(X_host.data_ptr(), X_host.shape[0], P.ptr, Y_host.data_ptr(), ws.data_ptr(),
                                  ws.numel(), _stream(stream)), "lqer_linear_host")
    return Y_host


def make_host_calls(items, x_dtype=torch.float32, y_dtype=torch.float32) -> "C.Array":
    """items: iterable of (X_cpu, PackedWeights, Y_cpu), contiguous CPU tensors of the given types -> a host array of lqer_call_t."""
    items = list(items)
    arr = (Call * len(items))()
    for j, (X, P, Y) in enumerate(items):
        for t, dt in ((X, _tensor_dtype(x_dtype)), (Y, _tensor_dtype(y_dtype))):
            if t.is_cuda or t.dtype != dt or not t.is_contiguous():
                raise ValueError("expected contiguous CPU tensors of the stated types")
        arr[j] = Call(X.data_ptr(), _rows(X, P, x_dtype), P.ptr, Y.data_ptr())
    return arr


def linear_host_batched_bytes(calls) -> int:
    arr = calls if isinstance(calls, C.Array) else make_host_calls(calls)
    out = C.c_size_t()
    _check(lib().lqer_linear_host_batched_bytes(arr, len(arr), C.byref(out)), "lqer_linear_host_batched_bytes")
    return out.value


def linear_host_batched(calls, ws: torch.Tensor, stream=None) -> None:
    """Independent layers with host buffers; copies in, layers and copies out overlap.  Returns when all Y are on the host."""
    arr = calls if isinstance(calls, C.Array) else make_host_calls(calls)
    _check(lib().lqer_linear_host_batched(arr, len(arr), ws.data_ptr(), ws.numel(), _stream(stream)),
           "lqer_linear_host_batched")


def linear_host_batched_ex(calls, ws: torch.Tensor, x_dtype, y_dtype, stream=None) -> None:
    """linear_host_batched with host X of x_dtype and host Y of y_dtype; `calls` from make_host_calls(..., x_dtype, y_dtype)."""
    _check(lib().lqer_linear_host_batched_ex(calls, len(calls), _DTYPES[x_dtype], _DTYPES[y_dtype], ws.data_ptr(), ws.numel(),
                                             _stream(stream)), "lqer_linear_host_batched_ex")


def poll_status(ws: torch.Tensor, stream=None) -> int:
    out = C.c_int()
    _check(lib().lqer_poll_status(ws.data_ptr(), _stream(stream), C.byref(out)), "lqer_poll_status")
    return out.value


def set_path(path: int) -> None:
    _check(lib().lqer_set_path(path), "lqer_set_path")


def set_wait_limit_cycles(cycles: int) -> None:
    _check(lib().lqer_set_wait_limit_cycles(cycles), "lqer_set_wait_limit_cycles")


def inject_stall(kernel_family: int) -> None:
    """Test hook: the next launch of that kernel family waits for something that never comes (-1 disarms)."""
    _check(lib().lqer_inject_stall(kernel_family), "lqer_inject_stall")


def debug_bounds_shrink(nbytes: int) -> None:
    """Test hook of the checked build: the declared extent of every Y shrinks by nbytes for the launches that follow, so the
    bounds checks at the end of Y fire (their stores are skipped); 0 restores.  The ordinary build refuses."""
    _check(lib().lqer_debug_bounds_shrink(nbytes), "lqer_debug_bounds_shrink")


def launch_count() -> int:
    return int(lib().lqer_launch_count())


def profile_enable(on: bool) -> None:
    _check(lib().lqer_profile_enable(1 if on else 0), "lqer_profile_enable")


def profile_collect() -> dict:
    """{family: (launches, milliseconds)} of the launches recorded since the last collect."""
    out = KernelTimes()
    _check(lib().lqer_profile_collect(C.byref(out)), "lqer_profile_collect")
    return {name: (int(out.launches[j]), float(out.milliseconds[j])) for j, name in enumerate(KERNEL_FAMILIES)
            if out.launches[j]}
