"""L2QER weight preparation and the LQER inference layer, fp64 numpy.

TEST INFRASTRUCTURE ONLY - see the package docstring.

Follows the paper step by step:
  quantisation error      E_q = W - W_q                       (Section 3.1, first equation)
  plain LQER factors      A_k = U_k, B_k = Sigma_k V_k^T      (Section 3.1)
  calibration of S        a_i = mean|X_i| over tokens, a_bar = max_i a_i,
                          s = a_bar / sqrt(min(a_bar) max(a_bar))   (Appendix A)
  L2QER factors           S E_q = U' Sigma' V'^T,
                          A'_k = S^-1 U'_k, B'_k = Sigma'_k V'_k^T (Section 3.2)
  inference layer         Y = X W_q + (X A_k) B_k             (Section 3.1 / 3.2)
with X quantised to MXINT8 on the fly, W_q in MXINT4 and A_k, B_k in MXINT8
(Section 4.1).
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

from . import mxint


# ----------------------------------------------------------------------------
# Calibration (Appendix A)
# ----------------------------------------------------------------------------

def calibration_scale(samples: list[np.ndarray]) -> np.ndarray:
    """Diagonal of S from N calibration samples X_i [tokens, channels] (Appendix A)."""
    a = [np.mean(np.abs(np.asarray(x, dtype=np.float64)), axis=0) for x in samples]
    a_bar = np.max(np.stack(a, axis=0), axis=0)
    lo, hi = float(a_bar.min()), float(a_bar.max())
    if lo <= 0.0:
        # The paper assumes no channel is always zero, so S^-1 exists (Section 3.2).
        raise ValueError("a calibration channel is identically zero: S is not invertible")
    return a_bar / np.sqrt(lo * hi)


# ----------------------------------------------------------------------------
# SVD without LAPACK
# ----------------------------------------------------------------------------

def _round_robin(n: int):
    """Tournament schedule: n-1 (n even) rounds of disjoint column pairs covering all pairs."""
    m = n + (n & 1)
    players = list(range(m))
    for _ in range(m - 1):
        p = np.array(players[: m // 2])
        q = np.array(players[m // 2:][::-1])
        keep = (p < n) & (q < n)
        yield np.minimum(p, q)[keep], np.maximum(p, q)[keep]
        players = [players[0]] + [players[-1]] + players[1:-1]


def jacobi_svd(G: np.ndarray, tol: float = 1e-15, max_sweeps: int = 60):
    """One-sided (Hestenes) Jacobi SVD: G = U diag(s) V^T, s sorted descending.

    Columns are orthogonalised pairwise by plane rotations until every pair
    satisfies |g_p . g_q| <= tol * |g_p| |g_q|; then s_j = |g_j|, u_j = g_j / s_j.
    Returns thin factors U [m, r], s [r], Vt [r, n] with r = min(m, n).
    """
    G = np.array(G, dtype=np.float64)
    m, n = G.shape
    if m < n:
        U, s, Vt = jacobi_svd(G.T, tol, max_sweeps)
        return Vt.T, s, U.T
    V = np.eye(n)
    schedule = list(_round_robin(n))
    for _ in range(max_sweeps):
        rotated = False
        for p, q in schedule:
            gp, gq = G[:, p], G[:, q]
            alpha = np.einsum("ij,ij->j", gp, gp)
            beta = np.einsum("ij,ij->j", gq, gq)
            gamma = np.einsum("ij,ij->j", gp, gq)
            act = np.abs(gamma) > tol * np.sqrt(alpha * beta)
            if not act.any():
                continue
            rotated = True
            g = np.where(act, gamma, 1.0)
            zeta = (beta - alpha) / (2.0 * g)
            t = np.where(zeta >= 0.0, 1.0, -1.0) / (np.abs(zeta) + np.sqrt(1.0 + zeta * zeta))
            c = 1.0 / np.sqrt(1.0 + t * t)
            s_ = c * t
            c = np.where(act, c, 1.0)
            s_ = np.where(act, s_, 0.0)
            G[:, p], G[:, q] = c * gp - s_ * gq, s_ * gp + c * gq
            vp, vq = V[:, p], V[:, q]
            V[:, p], V[:, q] = c * vp - s_ * vq, s_ * vp + c * vq
        if not rotated:
            break
    s = np.sqrt(np.einsum("ij,ij->j", G, G))
    order = np.argsort(-s, kind="stable")
    s, G, V = s[order], G[:, order], V[:, order]
    U = np.zeros_like(G)
    nz = s > 0.0
    U[:, nz] = G[:, nz] / s[nz]
    if not nz.all():
        # complete U for exactly singular matrices so that U^T U = I still holds
        U = _complete_orthonormal(U, nz)
    return U, s, V.T


def _complete_orthonormal(U: np.ndarray, filled: np.ndarray) -> np.ndarray:
    U = U.copy()
    m = U.shape[0]
    basis = [U[:, j] for j in np.nonzero(filled)[0]]
    cand = 0
    for j in np.nonzero(~filled)[0]:
        while True:
            v = np.zeros(m)
            v[cand % m] = 1.0
            cand += 1
            for _ in range(2):
                for b in basis:
                    v -= (b @ v) * b
            nv = np.linalg.norm(v)
            if nv > 1e-8:
                v /= nv
                break
        U[:, j] = v
        basis.append(v)
    return U


def _orthonormalise(Y: np.ndarray) -> np.ndarray:
    """Modified Gram-Schmidt, applied twice."""
    Q = np.array(Y, dtype=np.float64)
    for _ in range(2):
        for j in range(Q.shape[1]):
            for i in range(j):
                Q[:, j] -= (Q[:, i] @ Q[:, j]) * Q[:, i]
            Q[:, j] /= np.linalg.norm(Q[:, j])
    return Q


def subspace_svd(G: np.ndarray, k: int, rng: np.random.Generator, oversample: int = 16, iters: int = 4):
    """Top-k singular triplets by randomised subspace iteration (for full-size layers).

    An approximation of the truncated SVD used where Jacobi on the whole
    matrix would take hours.  The hot-path parity never depends on its
    accuracy because A_k, B_k are inputs of the layer.
    """
    G = np.asarray(G, dtype=np.float64)
    m, n = G.shape
    r = min(k + oversample, m, n)
    Q = _orthonormalise(G @ rng.standard_normal((n, r)))
    for _ in range(iters):
        Z = _orthonormalise(G.T @ Q)
        Q = _orthonormalise(G @ Z)
    Bm = Q.T @ G                      # [r, n]
    Ub, s, Vt = jacobi_svd(Bm)
    return (Q @ Ub)[:, :k], s[:k], Vt[:k]


# ----------------------------------------------------------------------------
# Weight preparation
# ----------------------------------------------------------------------------

def quantization_error(W: np.ndarray, Wm: np.ndarray, We: np.ndarray, w_bits: int = 4) -> np.ndarray:
    """E_q = W - W_q (Section 3.1)."""
    return np.asarray(W, dtype=np.float64) - mxint.dequantize(Wm, We, w_bits, axis=0)


def lqer_factors(E_q: np.ndarray, k: int, s: np.ndarray | None = None,
                 method: str = "jacobi", rng: np.random.Generator | None = None):
    """(A_k, B_k, singular values) of the rank-k correction.

    s is None: plain LQER, A_k = U_k, B_k = Sigma_k V_k^T (Section 3.1).
    otherwise: L2QER, SVD of S E_q, A'_k = S^-1 U'_k, B'_k = Sigma'_k V'_k^T (Section 3.2).
    """
    E_q = np.asarray(E_q, dtype=np.float64)
    K, N = E_q.shape
    if not 0 <= k <= min(K, N):
        raise ValueError("rank out of range")
    s_vec = np.ones(K) if s is None else np.asarray(s, dtype=np.float64)
    G = s_vec[:, None] * E_q
    if method == "jacobi":
        U, sig, Vt = jacobi_svd(G)
    elif method == "subspace":
        U, sig, Vt = subspace_svd(G, k, rng if rng is not None else np.random.default_rng(0))
    else:
        raise ValueError(method)
    A = U[:, :k] / s_vec[:, None]
    B = sig[:k, None] * Vt[:k]
    return A, B, sig


def approximation_error(E_q: np.ndarray, A: np.ndarray, B: np.ndarray) -> float:
    """e_a = mean |E_q - A B| (Appendix B)."""
    return float(np.mean(np.abs(np.asarray(E_q, dtype=np.float64) - A @ B)))


def average_weight_bits(K: int, N: int, k: int, w_bits: int = 4, lr_bits: int = 8,
                        exp_bits: int = 4, block: int = mxint.BLOCK) -> float:
    """Memory bits per weight of W_q, A_k and B_k together (Appendix D bookkeeping)."""
    total = K * N * (w_bits + exp_bits / block) + k * (K + N) * (lr_bits + exp_bits / block)
    return total / (K * N)


@dataclass
class PreparedWeights:
    K: int
    N: int
    k: int
    k_pad: int
    Wm: np.ndarray   # int8 [K, N]       4-bit mantissas, blocks of 16 along K
    We: np.ndarray   # int16 [K/16, N]
    Am: np.ndarray   # int8 [K, k]       8-bit mantissas, blocks of 16 along K
    Ae: np.ndarray   # int16 [K/16, k]
    Bm: np.ndarray   # int8 [k_pad, N]   8-bit mantissas, blocks of 16 along the rank, rows >= k zero
    Be: np.ndarray   # int16 [k_pad/16, N]


def quantize_weight(W: np.ndarray, w_bits: int = 4) -> tuple[np.ndarray, np.ndarray]:
    """W_q = q(W): blocks [16, 1], i.e. 16 along the rows of W [K, N] (Section 4.1)."""
    return mxint.quantize(np.asarray(W, dtype=np.float32), w_bits, axis=0)


def prepare_weights(W: np.ndarray, A: np.ndarray | None, B: np.ndarray | None,
                    w_bits: int = 4, lr_bits: int = 8,
                    exp_min: int = mxint.EXP_MIN, exp_max: int = mxint.EXP_MAX) -> PreparedWeights:
    """Quantise W, A_k, B_k as the layer stores them (Section 3.1, Section 4.1).

    The layer's interface carries fp32 tensors, so A and B are rounded to fp32
    first.  B's rank dimension is zero-padded to a multiple of 16 so that its
    [16, 1] blocks are whole.  [exp_min, exp_max] is the shared-exponent window
    of the three matrices (Section 4.1 gives them a 4-bit shared exponent, i.e.
    16 values, against 8 bits for the activations; where the window sits is left
    to the caller).
    """
    W = np.asarray(W, dtype=np.float32)
    K, N = W.shape
    Wm, We = mxint.quantize(W, w_bits, axis=0, exp_min=exp_min, exp_max=exp_max)
    k = 0 if A is None else A.shape[1]
    if k == 0:
        z8 = np.zeros((0, 0), np.int8)
        return PreparedWeights(K, N, 0, 0, Wm, We, np.zeros((K, 0), np.int8), np.zeros((K // 16, 0), np.int16),
                               np.zeros((0, N), np.int8), np.zeros((0, N), np.int16))
    A32 = np.asarray(A, dtype=np.float32)
    B32 = mxint.pad_axis(np.asarray(B, dtype=np.float32), axis=0)
    Am, Ae = mxint.quantize(A32, lr_bits, axis=0, exp_min=exp_min, exp_max=exp_max)
    Bm, Be = mxint.quantize(B32, lr_bits, axis=0, exp_min=exp_min, exp_max=exp_max)
    return PreparedWeights(K, N, k, B32.shape[0], Wm, We, Am, Ae, Bm, Be)


# ----------------------------------------------------------------------------
# Inference layer (Section 3.1 / 3.2)
# ----------------------------------------------------------------------------

@dataclass
class ForwardResult:
    Xm: np.ndarray    # int8 [M, K]
    Xe: np.ndarray    # int16 [M, K/16]
    T: np.ndarray     # fp64 [M, k]       X_q A_q before re-quantisation
    Tm: np.ndarray    # int8 [M, k_pad]
    Te: np.ndarray    # int16 [M, k_pad/16]
    Y: np.ndarray     # fp64 [M, N]
    tol: np.ndarray   # fp64 [M, N]       elementwise comparison tolerance


def forward(X: np.ndarray, P: PreparedWeights, w_bits: int = 4, a_bits: int = 8, lr_bits: int = 8,
            rel_tol: float = 1e-4) -> ForwardResult:
    """Y = X_q W_q + q(X_q A_q) B_q with every operand in MXINT, sums in fp64.

    X is quantised once (blocks [1, 16] along K) and used by both products.
    T = X_q A_q is re-quantised to the activation format (blocks of 16 along
    the rank, zero-padded to k_pad) before it meets B_q, so that all three
    matmuls run on MXINT operands as the paper's hardware does (Appendix D).
    The tolerance map is rel_tol * (|X_q| |W_q| + |T_q| |B_q|) elementwise.
    """
    X = np.asarray(X, dtype=np.float32)
    M, K = X.shape
    if K != P.K:
        raise ValueError("X and W disagree on K")
    Xm, Xe = mxint.quantize(X, a_bits, axis=1)
    Xdq = mxint.dequantize(Xm, Xe, a_bits, axis=1)
    Wdq = mxint.dequantize(P.Wm, P.We, w_bits, axis=0)
    Y = Xdq @ Wdq
    tol = np.abs(Xdq) @ np.abs(Wdq)
    if P.k > 0:
        Adq = mxint.dequantize(P.Am, P.Ae, lr_bits, axis=0)
        Bdq = mxint.dequantize(P.Bm, P.Be, lr_bits, axis=0)
        T = Xdq @ Adq
        Tm, Te = mxint.quantize(mxint.pad_axis(T, axis=1), a_bits, axis=1)
        Tdq = mxint.dequantize(Tm, Te, a_bits, axis=1)
        Y = Y + Tdq @ Bdq
        tol = tol + np.abs(Tdq) @ np.abs(Bdq)
    else:
        T = np.zeros((M, 0))
        Tm = np.zeros((M, 0), np.int8)
        Te = np.zeros((M, 0), np.int16)
    return ForwardResult(Xm, Xe, T, Tm, Te, Y, rel_tol * tol)
