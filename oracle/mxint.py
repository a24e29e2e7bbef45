"""MXINT block quantisation (Section 2.2; formats of Section 4.1), fp64 numpy.

TEST INFRASTRUCTURE ONLY - see the package docstring.

An MXINT block is `block` fixed-point mantissas that share one power-of-two
exponent (Section 2.2).  Section 4.1 fixes block size 16, taken along the
contraction dimension: [1, 16] for the activations X_q and [16, 1] for W_q,
A_k and B_k; 8-bit mantissas for X, A_k, B_k and 4-bit for W_q.

The paper does not print how the shared exponent is chosen, the rounding mode
or the clamp.  The reading used here (listed with the other readings in the
design notes) is:

  e     = clamp(floor(log2(max_i |v_i|)), exp_min, exp_max)
  step  = 2 ** (e - (bits - 2))
  m_i   = clamp(round_half_even(v_i / step), -(2**(bits-1) - 1), 2**(bits-1) - 1)
  dq_i  = m_i * step

so the largest magnitude of a block lands in [2**(bits-2), 2**(bits-1)) before
rounding, the mantissa range is symmetric, and a block maximum that rounds up
to 2**(bits-1) is clipped.  A block whose maximum is below 2**exp_min (all-zero
blocks included) takes e = exp_min.  +-Inf saturates at e = exp_max; NaN
elements are ignored by the maximum and quantise to mantissa 0.
"""
from __future__ import annotations

import numpy as np

BLOCK = 16
EXP_MIN = -56
EXP_MAX = 55
EXP_BIAS = 127  # exponent byte = e + 127


def _blocked(v: np.ndarray, axis: int, block: int) -> np.ndarray:
    """Move `axis` last and split it into [n_blocks, block]."""
    v = np.moveaxis(np.asarray(v, dtype=np.float64), axis, -1)
    if v.shape[-1] % block != 0:
        raise ValueError(f"length {v.shape[-1]} along the block axis is not a multiple of {block}")
    return v.reshape(v.shape[:-1] + (v.shape[-1] // block, block))


def shared_exponent(amax: np.ndarray, exp_min: int = EXP_MIN, exp_max: int = EXP_MAX) -> np.ndarray:
    """floor(log2(amax)) clamped to the window; amax >= 0 (may be 0 or inf)."""
    amax = np.asarray(amax, dtype=np.float64)
    frac, p = np.frexp(amax)            # amax = frac * 2**p, frac in [0.5, 1)
    e = p.astype(np.int64) - 1          # floor(log2(amax)) for finite amax > 0
    e = np.where(amax == 0.0, exp_min, e)
    e = np.where(np.isinf(amax), exp_max, e)
    return np.clip(e, exp_min, exp_max).astype(np.int64)


def quantize(v: np.ndarray, bits: int, axis: int, block: int = BLOCK,
             exp_min: int = EXP_MIN, exp_max: int = EXP_MAX) -> tuple[np.ndarray, np.ndarray]:
    """Quantise `v` to MXINT with `bits`-bit mantissas, blocks of `block` along `axis`.

    Returns (mantissas int8 shaped like v, exponents int16 shaped like v with
    `axis` shrunk by `block`).  Section 2.2 / Section 4.1.
    """
    if not 2 <= bits <= 8:
        raise ValueError("mantissa width must be 2..8 bits")
    vb = _blocked(v, axis, block)
    mag = np.abs(vb)
    amax = np.fmax.reduce(mag, axis=-1)          # fmax ignores NaN
    amax = np.where(np.isnan(amax), 0.0, amax)   # an all-NaN block
    e = shared_exponent(amax, exp_min, exp_max)
    step = np.ldexp(1.0, (e - (bits - 2)).astype(np.int64))[..., None]
    qmax = float(2 ** (bits - 1) - 1)
    with np.errstate(invalid="ignore", over="ignore"):
        r = np.rint(vb / step)                   # round half to even
    r = np.where(np.isnan(r), 0.0, r)
    m = np.clip(r, -qmax, qmax)
    m = m.reshape(m.shape[:-2] + (m.shape[-2] * block,))
    mant = np.moveaxis(m, -1, axis).astype(np.int8)
    exps = np.moveaxis(e, -1, axis).astype(np.int16)
    return np.ascontiguousarray(mant), np.ascontiguousarray(exps)


def dequantize(mant: np.ndarray, exps: np.ndarray, bits: int, axis: int, block: int = BLOCK) -> np.ndarray:
    """dq = m * 2**(e - (bits - 2)), fp64 (exact)."""
    e = np.repeat(np.asarray(exps, dtype=np.int64), block, axis=axis)
    return np.ldexp(np.asarray(mant, dtype=np.float64), e - (bits - 2))


def exponent_bytes(exps: np.ndarray) -> np.ndarray:
    """The one-byte storage form of a shared exponent: e + 127."""
    return (np.asarray(exps, dtype=np.int64) + EXP_BIAS).astype(np.uint8)


def pad_axis(v: np.ndarray, axis: int, multiple: int = BLOCK) -> np.ndarray:
    """Zero-pad `axis` up to a multiple (rank k -> k_pad; padding never changes a block maximum)."""
    n = v.shape[axis]
    n_pad = (n + multiple - 1) // multiple * multiple
    if n_pad == n:
        return v
    width = [(0, 0)] * v.ndim
    width[axis] = (0, n_pad - n)
    return np.pad(v, width)


def round_bf16(v: np.ndarray) -> np.ndarray:
    """Nearest bfloat16 value (8 significant bits, round half to even) of each element, as fp64.

    The layer may take its activations and hand over its output in 16 bits (Section 2.1: FP16 activations in
    the w-only setting); this is the rounding of that boundary, written out from the format's definition:
    v = f * 2**p with f in [0.5, 1) keeps the eight leading bits of f.  Values inside bfloat16's normal range
    only (the layer's outputs are); zeros, infinities and NaN pass through.
    """
    v = np.asarray(v, dtype=np.float64)
    f, p = np.frexp(v)
    with np.errstate(invalid="ignore"):
        r = np.ldexp(np.rint(f * 256.0), p - 8)
    return np.where(np.isfinite(v), r, v)


def bf16_half_ulp(v: np.ndarray) -> np.ndarray:
    """Half the spacing of bfloat16 values at each |v|: the most a correctly rounded value differs from v."""
    v = np.abs(np.asarray(v, dtype=np.float64))
    _, p = np.frexp(v)
    return np.where(v > 0.0, np.ldexp(1.0, p - 9), 0.0)
