"""Shared helpers of the test-suite: build a layer with the oracle, compare GPU results to it."""
from __future__ import annotations

import functools

import numpy as np

import lqer_inputs as gen
from oracle import lqer as olqer
from oracle import mxint


@functools.lru_cache(maxsize=8)
def oracle_layer(spec: gen.LayerSpec, method: str = "jacobi"):
    """(W, A32, B32, PreparedWeights) for a layer: factors by the oracle's L2QER preparation."""
    W = gen.make_weight(spec)
    Wm, We = olqer.quantize_weight(W)
    if spec.k == 0:
        return W, None, None, olqer.prepare_weights(W, None, None)
    E = olqer.quantization_error(W, Wm, We)
    s = olqer.calibration_scale(gen.make_calibration(spec))
    A, B, _ = olqer.lqer_factors(E, spec.k, s, method=method, rng=np.random.default_rng(spec.seed))
    A32 = np.ascontiguousarray(A, dtype=np.float32)
    B32 = np.ascontiguousarray(B, dtype=np.float32)
    return W, A32, B32, olqer.prepare_weights(W, A32, B32)


def exp_bytes(e):
    return mxint.exponent_bytes(e)


def worst_ratio(Y_gpu: np.ndarray, ref) -> float:
    """max |Y_gpu - Y_oracle| / tol over all elements (<= 1 passes)."""
    return float(np.max(np.abs(Y_gpu.astype(np.float64) - ref.Y) / ref.tol))
