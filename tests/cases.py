"""Builders for the parity cases: seeded inputs (synth) + the oracle's fp64 basis.  Test helper only."""
from __future__ import annotations

from dataclasses import dataclass
from functools import lru_cache

import numpy as np

import synth
from oracle import basis


@dataclass
class FoldedCase:
    """A layer whose input already holds the coefficients (projection folded upstream)."""
    T: int
    K: int
    N: int
    r: int
    X: np.ndarray        # raw activations, bf16-valued fp32 [T][K]
    U: np.ndarray        # fp64 [K][K]
    W: np.ndarray        # bf16-valued fp32 [K][N]
    C_bits: np.ndarray   # uint16 [T][K]: bf16(X·U)
    W_proj: np.ndarray   # fp32 [N][K]: (U^T W)^T
    lam: np.ndarray
    P: np.ndarray
    X_calib: np.ndarray


@lru_cache(maxsize=4)
def pca_case(T: int, K: int, N: int, r: int, dist: str, n_calib: int) -> FoldedCase:
    X = synth.activations(T, K, dist, seed=synth.SEED_ACT)
    Xc = synth.activations(n_calib, K, dist, seed=synth.SEED_CALIB)
    G_h = synth.gaussian_matrix(r, synth.SEED_ROT, 0)
    G_l = synth.gaussian_matrix(K - r, synth.SEED_ROT, 1)
    U, P, lam = basis.resq_basis(Xc, r, G_h, G_l)
    W = synth.weights(K, N)
    C = (X.astype(np.float64) @ U).astype(np.float32)
    return FoldedCase(T, K, N, r, X, U, W, synth.f32_to_bf16_bits(C), basis.project_weights(U, W), lam, P, Xc)


def config1() -> FoldedCase:
    """Tiny correctness layer: T=16, d=512, n_out=512, r=64; N(0,1) activations with 5 channels x20;
    PCA on a separate 256-token calibration batch; QR-of-Gaussian rotations 64x64 and 448x448."""
    return pca_case(16, 512, 512, 64, "normal", 256)


def config2_basis() -> FoldedCase:
    """The d = 2048 input dimension of the Llama-3.2-1B-shaped configuration on the real construction: Student-t
    activations with 1 % of the channels x20, PCA on a separate 4096-token calibration batch, QR-of-Gaussian
    rotations 256x256 and 1792x1792; 64 token rows and 512 output channels keep the oracle's layer in seconds."""
    return pca_case(64, 2048, 512, 256, "t4", 4096)


def synthetic_folded(T: int, K: int, N: int, r: int, seed_shift: int = 0):
    """Coefficients and projected weights drawn directly (no basis needed): bf16 t4 coefficients with
    outlier channels, fp32 Gaussian projected weights.  For shape sweeps of the kernels."""
    C = synth.activations(T, K, "t4", seed=synth.SEED_ACT + 100 + seed_shift)
    Wp = synth.projected_weights_direct(N, K, seed=synth.SEED_W + 100 + seed_shift)
    return synth.f32_to_bf16_bits(C), Wp
