"""Seeded synthetic inputs for the LQER / L2QER linear layer.

This module only draws numbers.  It holds none of the method's arithmetic (no
quantisation, no SVD, no matmul) so that both the CPU oracle's tests and the
CUDA path's tests / benchmark can take their inputs from it without sharing
any code of the method itself.

The paper runs on trained LLM layers whose activations have a few outlier
channels (Section 1, Section 3.2) and calibrates on 32 samples of 2048 tokens
(Section 4.1).  Neither the checkpoints nor the calibration text are available
here, so seeded tensors of the same shapes and the same value structure stand
in for them:

* weights: N(0, 0.02) or Student-t(nu=4) scaled to standard deviation 0.02;
* activations: N(0, 1) with a fixed, seeded subset of input channels scaled
  up (x20 or x50);
* calibration batch: same law and the same outlier channels as the
  activations.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


@dataclass(frozen=True)
class LayerSpec:
    """Shape and distribution recipe of one synthetic linear layer."""

    name: str
    M: int                      # tokens (the paper's t)
    K: int                      # in-features (the paper's m)
    N: int                      # out-features (the paper's n)
    k: int                      # rank of the correction
    calib_rows: int             # rows of the single calibration sample
    outlier_frac: float         # fraction of input channels that are outliers
    outlier_scale: float        # factor applied to those channels
    weight_law: str = "normal"  # "normal" | "student_t4"
    seed: int = 0
    n_outliers: int | None = None  # overrides outlier_frac when given


def _rng(seed: int, stream: int) -> np.random.Generator:
    # Philox is counter based: the same (seed, stream) gives the same numbers
    # on every machine and numpy build.
    return np.random.Generator(np.random.Philox(key=[seed, stream]))


def outlier_channels(spec: LayerSpec) -> np.ndarray:
    """Sorted indices of the outlier input channels (shared by X and calibration)."""
    n = spec.n_outliers if spec.n_outliers is not None else int(round(spec.outlier_frac * spec.K))
    n = max(0, min(spec.K, n))
    if n == 0:
        return np.zeros(0, dtype=np.int64)
    return np.sort(_rng(spec.seed, 1).choice(spec.K, size=n, replace=False))


def make_weight(spec: LayerSpec) -> np.ndarray:
    """W fp32 [K, N]."""
    g = _rng(spec.seed, 2)
    if spec.weight_law == "normal":
        w = g.standard_normal((spec.K, spec.N), dtype=np.float32) * np.float32(0.02)
    elif spec.weight_law == "student_t4":
        # t = Z / sqrt(chi2_4 / 4); Var(t_4) = 2, so 0.02 / sqrt(2) gives std 0.02
        z = g.standard_normal((spec.K, spec.N), dtype=np.float32)
        c = g.chisquare(4.0, size=(spec.K, spec.N)).astype(np.float32)
        w = z / np.sqrt(c / np.float32(4.0)) * np.float32(0.02 / np.sqrt(2.0))
    else:
        raise ValueError(f"unknown weight law {spec.weight_law!r}")
    return np.ascontiguousarray(w, dtype=np.float32)


def _activations(spec: LayerSpec, rows: int, stream: int) -> np.ndarray:
    g = _rng(spec.seed, stream)
    x = g.standard_normal((rows, spec.K), dtype=np.float32)
    ch = outlier_channels(spec)
    if ch.size:
        x[:, ch] *= np.float32(spec.outlier_scale)
    return np.ascontiguousarray(x, dtype=np.float32)


def make_activations(spec: LayerSpec, M: int | None = None) -> np.ndarray:
    """X fp32 [M, K]."""
    return _activations(spec, spec.M if M is None else M, 3)


def make_calibration(spec: LayerSpec) -> list[np.ndarray]:
    """One calibration sample fp32 [calib_rows, K] (a list, as the method takes N samples)."""
    return [_activations(spec, spec.calib_rows, 4)]


def make_random_factors(spec: LayerSpec) -> tuple[np.ndarray, np.ndarray]:
    """Seeded stand-ins for (A_k, B_k) with the magnitudes the real factors have.

    Used where only throughput is measured (224-matrix stacks) and deriving the
    factors by SVD for every matrix would take hours on the host.  A has
    orthonormal-like columns (entries ~ N(0, 1/K)); B rows have the scale of
    sigma * v^T for an error matrix with entries of std 0.004 (about the
    MXINT4 rounding error of N(0, 0.02) weights).
    """
    g = _rng(spec.seed, 5)
    a = g.standard_normal((spec.K, spec.k), dtype=np.float32) * np.float32(1.0 / np.sqrt(spec.K))
    sig = np.float32(0.004) * np.float32(np.sqrt(spec.K) + np.sqrt(spec.N))
    b = g.standard_normal((spec.k, spec.N), dtype=np.float32) * (sig / np.float32(np.sqrt(spec.N)))
    return np.ascontiguousarray(a), np.ascontiguousarray(b)


# ----------------------------------------------------------------------------
# The five workload families
# ----------------------------------------------------------------------------

def config_tiny() -> LayerSpec:
    return LayerSpec("tiny", M=16, K=256, N=256, k=8, calib_rows=128,
                     outlier_frac=0.0, n_outliers=4, outlier_scale=20.0, seed=0)


def config_decode(M: int) -> LayerSpec:
    return LayerSpec(f"decode_M{M}", M=M, K=4096, N=4096, k=32, calib_rows=512,
                     outlier_frac=0.01, outlier_scale=20.0, seed=2000 + M)


def config_prefill(transposed: bool = False) -> LayerSpec:
    K, N = (11008, 4096) if transposed else (4096, 11008)
    return LayerSpec("prefill_down" if transposed else "prefill_up", M=2048, K=K, N=N, k=32,
                     calib_rows=512, outlier_frac=0.01, outlier_scale=20.0,
                     seed=3001 if transposed else 3000)


SWEEP_N = (5120, 13824)
SWEEP_M = (1, 64, 512, 4096)
SWEEP_K_RANK = (8, 32, 64, 128, 256)


def config_sweep(N: int, M: int, k: int) -> LayerSpec:
    idx = (SWEEP_N.index(N) * len(SWEEP_M) + SWEEP_M.index(M)) * len(SWEEP_K_RANK) + SWEEP_K_RANK.index(k)
    return LayerSpec(f"sweep_N{N}_M{M}_k{k}", M=M, K=5120, N=N, k=k, calib_rows=512,
                     outlier_frac=0.005, outlier_scale=50.0, weight_law="student_t4", seed=4000 + idx)


STACK_LINEARS = (("q", 4096, 4096), ("k", 4096, 4096), ("v", 4096, 4096), ("o", 4096, 4096),
                 ("gate", 4096, 11008), ("up", 4096, 11008), ("down", 11008, 4096))


def config_stack(layer: int, which: int, M: int) -> LayerSpec:
    name, K, N = STACK_LINEARS[which]
    return LayerSpec(f"stack_L{layer}_{name}_M{M}", M=M, K=K, N=N, k=32, calib_rows=512,
                     outlier_frac=0.01, outlier_scale=20.0, seed=5000 + layer * 7 + which)


# ----------------------------------------------------------------------------
# Device-side draws for full-size throughput runs
# ----------------------------------------------------------------------------
# A 224-matrix stack holds 6.5 G weights; drawing them with numpy on the host
# would take minutes, so throughput runs draw directly on the device with
# torch's seeded generator.  The law, the shapes and the outlier structure are
# the ones above; the stream of numbers is a different one (kernel speed does
# not depend on the values, and parity is always checked on the numpy draws).

def _torch_gen(spec: LayerSpec, stream: int, device):
    import torch
    g = torch.Generator(device=device)
    g.manual_seed(spec.seed * 8 + stream)
    return g


def make_weight_device(spec: LayerSpec, device):
    import torch
    g = _torch_gen(spec, 2, device)
    if spec.weight_law == "normal":
        return torch.randn((spec.K, spec.N), generator=g, device=device, dtype=torch.float32) * 0.02
    if spec.weight_law == "student_t4":
        z = torch.randn((spec.K, spec.N), generator=g, device=device, dtype=torch.float32)
        c = torch.randn((4, spec.K, spec.N), generator=g, device=device, dtype=torch.float32).square_().sum(0)
        return z / torch.sqrt(c / 4.0) * (0.02 / 2.0 ** 0.5)
    raise ValueError(f"unknown weight law {spec.weight_law!r}")


def make_activations_device(spec: LayerSpec, device, M: int | None = None):
    import torch
    g = _torch_gen(spec, 3, device)
    x = torch.randn((spec.M if M is None else M, spec.K), generator=g, device=device, dtype=torch.float32)
    ch = outlier_channels(spec)
    if ch.size:
        x[:, torch.from_numpy(ch).to(device)] *= spec.outlier_scale
    return x


def make_random_factors_device(spec: LayerSpec, device):
    """Device-side twin of make_random_factors (same magnitudes)."""
    import torch
    g = _torch_gen(spec, 5, device)
    a = torch.randn((spec.K, spec.k), generator=g, device=device, dtype=torch.float32) * (1.0 / spec.K ** 0.5)
    sig = 0.004 * (spec.K ** 0.5 + spec.N ** 0.5)
    b = torch.randn((spec.k, spec.N), generator=g, device=device, dtype=torch.float32) * (sig / spec.N ** 0.5)
    return a, b
