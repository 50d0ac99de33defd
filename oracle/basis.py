"""Basis construction of Eq. 5 (Section 4.2) in fp64 -- part of the CPU oracle, TEST INFRASTRUCTURE ONLY.

U = P·blockdiag(R_h, R_l): P holds the eigenvectors of the activations' d x d second-moment matrix,
the r directions of largest eigenvalue forming the high-precision subspace (Theorem 4.2 and the
paragraph after it); R_h (r x r) and R_l ((d-r) x (d-r)) are random orthogonal matrices.

Readings: the paper writes "covariance X X^T" for X of shape n x d; dimensionally that is the d x d
matrix X^T X / n, taken uncentred as written.  The paper orders eigenvalues increasingly and puts the
high-precision block last; here the order is DESCENDING and the high-precision block comes first (a
column permutation of the same U).  The paper states R_l, R_h as d x (d-r) and d x r, which does not
fit the block-diagonal of Eq. 5; they are (d-r) x (d-r) and r x r.

Library primitives used as steps: numpy.linalg.eigh, numpy.linalg.qr.
"""
from __future__ import annotations

import numpy as np


def second_moment(X_calib: np.ndarray) -> np.ndarray:
    X = np.asarray(X_calib, dtype=np.float64)
    return X.T @ X / X.shape[0]


def pca_basis(X_calib: np.ndarray):
    """Eigenpairs of the second-moment matrix, sorted by descending eigenvalue: (lambda [d], P [d][d])."""
    lam, V = np.linalg.eigh(second_moment(X_calib))
    order = np.argsort(-lam, kind="stable")
    return lam[order], V[:, order]


def random_rotation(G: np.ndarray) -> np.ndarray:
    """Q factor of the QR decomposition of a Gaussian matrix, columns sign-fixed so that R has a
    positive diagonal (which makes Q unique and Haar distributed)."""
    Q, R = np.linalg.qr(np.asarray(G, dtype=np.float64))
    sign = np.sign(np.diag(R))
    sign[sign == 0] = 1.0
    return Q * sign


def resq_basis(X_calib: np.ndarray, r: int, G_h: np.ndarray, G_l: np.ndarray):
    """U [d][d] = [P_h P_l]·blockdiag(R_h, R_l); returns (U, P, lambda)."""
    lam, P = pca_basis(X_calib)
    d = P.shape[0]
    assert G_h.shape == (r, r) and G_l.shape == (d - r, d - r)
    U = np.empty_like(P)
    U[:, :r] = P[:, :r] @ random_rotation(G_h)
    U[:, r:] = P[:, r:] @ random_rotation(G_l)
    return U, P, lam


def project_weights(U: np.ndarray, W: np.ndarray) -> np.ndarray:
    """(U^T W)^T in fp64, rounded once to fp32, laid out [N][K] (Eq. 3's argument)."""
    return np.ascontiguousarray((np.asarray(U, np.float64).T @ np.asarray(W, np.float64)).T.astype(np.float32))
