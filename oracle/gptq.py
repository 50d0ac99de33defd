"""GPTQ rounding of projected weights (Section 5.1: "apply GPTQ for weight quantization") -- part of the CPU
oracle, TEST INFRASTRUCTURE ONLY.

The paper quantizes the projected weights U^T W with GPTQ (Frantar et al., 2022) instead of rounding them to
nearest, and says no more about it; what is restated here is that published algorithm, applied to this layer's
weight format (rows = output channels, split at r into an INT8 and an INT4 segment, one symmetric scale per row
and segment as in Eq. 3):

  * H = (2 / n) X^T X over calibration inputs X (n x K, in the projected basis), damped by 1 % of its mean
    diagonal; a column whose diagonal entry is 0 never influenced an output: its weights are set to 0;
  * U = the upper triangular Cholesky factor of H^-1 (H^-1 = U^T U);
  * the scales are those of round-to-nearest, taken from the unmodified rows (Eq. 1: s = absmax / qmax per segment);
  * columns are visited in order j = 0 .. K-1; each row's weight w_j is rounded to q = clip(rint(w_j / s)) * s, and
    the scaled rounding error e = (w_j - q) / U[j][j] is fed back into the not yet visited columns:
    w[j+1:] -= e * U[j][j+1:].

Everything is fp64 with one rounding per operation in the order written (numpy), on fp32 inputs widened exactly.
Library primitives used as steps: numpy.linalg.cholesky, numpy.linalg.inv.
"""
from __future__ import annotations

import numpy as np

from . import PackedWeights, pack_nibbles, split_quantize


def hessian(X_calib: np.ndarray, percdamp: float = 0.01):
    """Damped H of the layer input X_calib [n][K]; returns (H fp64 [K][K], dead-column mask)."""
    X = np.asarray(X_calib, np.float64)
    H = 2.0 / X.shape[0] * (X.T @ X)
    dead = np.diag(H) == 0.0
    H[dead, dead] = 1.0
    H = H + percdamp * np.mean(np.diag(H)) * np.eye(H.shape[0])
    return H, dead


def inverse_factor(H: np.ndarray) -> np.ndarray:
    """U upper triangular with H^-1 = U^T U."""
    Hinv = np.linalg.inv(np.asarray(H, np.float64))
    Hinv = 0.5 * (Hinv + Hinv.T)
    return np.linalg.cholesky(Hinv).T.copy()


def gptq_codes(W_proj, r: int, U, dead=None, scale_fp16: bool = False):
    """W_proj fp32 [N][K] (rows = output channels), U fp32-representable upper factor [K][K].
    Returns (q8 int8 [N][r], q4 int8 [N][K-r], s8 fp32 [N], s4 fp32 [N])."""
    W_proj = np.ascontiguousarray(W_proj, np.float32)
    N, K = W_proj.shape
    Uf = np.ascontiguousarray(U, np.float32).astype(np.float64)
    W = W_proj.astype(np.float64)
    if dead is not None:
        W[:, np.asarray(dead, bool)] = 0.0
    # round-to-nearest scales of the rows as given (dead columns zeroed first, as they are for the rounding)
    _, _, s8, s4 = split_quantize(W.astype(np.float32), r, scale_fp16)
    code = np.zeros((N, K), np.int8)
    for j in range(K):
        s = (s8 if j < r else s4).astype(np.float64)
        lo, hi = (-128.0, 127.0) if j < r else (-8.0, 7.0)
        w = W[:, j]
        with np.errstate(divide="ignore", invalid="ignore"):
            c = np.where(s > 0.0, np.clip(np.rint(w / s), lo, hi), 0.0)
        code[:, j] = c.astype(np.int8)
        e = (w - c * s) / Uf[j, j]
        if j + 1 < K:
            W[:, j + 1:] -= e[:, None] * Uf[j, j + 1:][None, :]
    return code[:, :r].copy(), code[:, r:].copy(), s8, s4


def pack_weights_gptq(W_proj, r: int, U, dead=None, scale_fp16: bool = False) -> PackedWeights:
    q8, q4, s8, s4 = gptq_codes(W_proj, r, U, dead, scale_fp16)
    N, K = np.asarray(W_proj).shape
    return PackedWeights(K, N, r, q8, q4, pack_nibbles(q4), s8, s4)


def objective(W_proj, pw: PackedWeights, H) -> np.ndarray:
    """Per output channel: (w - w_hat) H (w - w_hat)^T, the layer-output error GPTQ minimises (up to the factor 2/n)."""
    W = np.asarray(W_proj, np.float64)
    W_hat = np.concatenate([pw.q8.astype(np.float64) * pw.s8[:, None], pw.q4.astype(np.float64) * pw.s4[:, None]], axis=1)
    E = W - W_hat
    return np.einsum("nk,kl,nl->n", E, np.asarray(H, np.float64), E)
