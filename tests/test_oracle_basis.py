"""Pins for the oracle's basis construction (Eq. 5) against invariants and LAPACK-independent facts."""
import numpy as np
import pytest

import synth
from oracle import basis
from tests.cases import config1


def test_U_is_orthogonal_and_layer_is_invariant_without_quantization():
    c = config1()
    U = c.U
    assert np.abs(U.T @ U - np.eye(c.K)).max() < 1e-12
    X, W = c.X.astype(np.float64), c.W.astype(np.float64)
    ref = X @ W
    got = (X @ U) @ (U.T @ W)
    assert np.abs(got - ref).max() / np.abs(ref).max() < 1e-12
    # cross terms vanish: the two same-precision products alone reproduce the output
    r = c.r
    split = (X @ U[:, :r]) @ (U[:, :r].T @ W) + (X @ U[:, r:]) @ (U[:, r:].T @ W)
    assert np.abs(split - ref).max() / np.abs(ref).max() < 1e-12


def test_basis_at_d2048_orthogonal_invariant_and_ordered():
    """The same construction at the 2048-wide input of the Llama-3.2-1B-shaped configuration (4096 calibration
    tokens, r = 256): orthogonality, the unquantized invariance X·U·U^T·W = X·W with vanishing cross terms,
    eigen-residuals, descending order, the trace identity, subspaces kept by the rotations, and the outlier
    channels inside the high-precision subspace."""
    from tests.cases import config2_basis
    c = config2_basis()
    U, r = c.U, c.r
    assert np.abs(U.T @ U - np.eye(c.K)).max() < 1e-12
    X, W = c.X.astype(np.float64), c.W.astype(np.float64)
    ref = X @ W
    assert np.abs((X @ U) @ (U.T @ W) - ref).max() / np.abs(ref).max() < 1e-12
    split = (X @ U[:, :r]) @ (U[:, :r].T @ W) + (X @ U[:, r:]) @ (U[:, r:].T @ W)
    assert np.abs(split - ref).max() / np.abs(ref).max() < 1e-12
    G = basis.second_moment(c.X_calib)
    assert (np.diff(c.lam) <= 1e-9 * c.lam[0]).all()
    assert np.abs(G @ c.P - c.P * c.lam).max() < 1e-9 * c.lam[0]
    assert np.isclose(c.lam.sum(), (c.X_calib.astype(np.float64) ** 2).sum() / c.X_calib.shape[0], rtol=1e-12)
    rq = np.einsum("ij,ij->j", c.P[:, :r], G @ c.P[:, :r])
    assert np.allclose(rq, c.lam[:r], rtol=1e-9)
    assert np.abs(U[:, :r] @ U[:, :r].T - c.P[:, :r] @ c.P[:, :r].T).max() < 1e-11
    out = synth.outlier_channels(c.K, synth.n_outliers(c.K))
    assert ((c.P[out, :r] ** 2).sum(1) > 0.99).all()
    # the coefficient layout the layer receives: bf16(X·U), high-variance block first
    Cf = synth.bf16_bits_to_f32(c.C_bits).astype(np.float64)
    assert (Cf[:, :r] ** 2).mean() > 4 * (Cf[:, r:] ** 2).mean()


def test_pca_eigenpairs_descending_and_residuals():
    c = config1()
    G = basis.second_moment(c.X_calib)
    assert (np.diff(c.lam) <= 1e-9 * c.lam[0]).all()
    resid = G @ c.P - c.P * c.lam
    assert np.abs(resid).max() < 1e-9 * c.lam[0]
    # Rayleigh quotients of the first r columns are the r largest eigenvalues
    rq = np.einsum("ij,ij->j", c.P[:, :c.r], G @ c.P[:, :c.r])
    assert np.allclose(rq, c.lam[:c.r], rtol=1e-10)
    # trace identity: eigenvalues sum to the mean squared row norm of the calibration batch
    assert np.isclose(c.lam.sum(), (c.X_calib.astype(np.float64) ** 2).sum() / c.X_calib.shape[0], rtol=1e-12)


def test_high_subspace_captures_the_most_energy():
    """P_h must maximise ||X P_h||_F (Theorem 4.2): no other r-dimensional coordinate or random
    subspace captures more of the calibration energy, and the outlier channels lie inside it."""
    c = config1()
    Xc = c.X_calib.astype(np.float64)
    e_pca = np.linalg.norm(Xc @ c.P[:, :c.r]) ** 2
    # best axis-aligned choice: the r channels with largest energy
    ch = np.argsort(-(Xc ** 2).sum(0))[:c.r]
    assert e_pca >= (Xc[:, ch] ** 2).sum() * (1 - 1e-12)
    Q = basis.random_rotation(synth.gaussian_matrix(c.K, 77))[:, :c.r]
    assert e_pca > np.linalg.norm(Xc @ Q) ** 2
    out = synth.outlier_channels(c.K, synth.n_outliers(c.K))
    captured = (c.P[out, :c.r] ** 2).sum(1)     # squared length of each outlier axis inside span(P_h)
    assert (captured > 0.99).all()
    # projected variances are monotone in eigenvalue order on the calibration batch
    var = ((Xc @ c.P) ** 2).mean(0)
    assert (np.diff(var) <= 1e-9 * var[0]).all()


def test_rotations_keep_the_subspaces():
    c = config1()
    r = c.r
    # span(U_h) = span(P_h): projectors agree
    assert np.abs(c.U[:, :r] @ c.U[:, :r].T - c.P[:, :r] @ c.P[:, :r].T).max() < 1e-12
    assert np.abs(c.U[:, r:] @ c.U[:, r:].T - c.P[:, r:] @ c.P[:, r:].T).max() < 1e-12


def test_random_rotation_is_sign_fixed_qr():
    G = synth.gaussian_matrix(48, 5)
    Q = basis.random_rotation(G)
    assert np.abs(Q.T @ Q - np.eye(48)).max() < 1e-13
    R = Q.T @ G
    assert np.abs(np.tril(R, -1)).max() < 1e-12 and (np.diag(R) > 0).all()
    # 2x2 closed form: first column is the normalised first column of G
    G2 = np.array([[3.0, 1.0], [4.0, 2.0]])
    Q2 = basis.random_rotation(G2)
    assert np.allclose(Q2[:, 0], [0.6, 0.8]) and np.allclose(Q2[:, 1], [-0.8, 0.6])


def test_project_weights_layout():
    U = basis.random_rotation(synth.gaussian_matrix(16, 6))
    W = synth.weights(16, 4)
    Wp = basis.project_weights(U, W)
    assert Wp.shape == (4, 16) and Wp.dtype == np.float32
    for n in range(4):
        for j in range(16):
            assert np.isclose(Wp[n, j], sum(U[i, j] * float(W[i, n]) for i in range(16)), rtol=1e-6, atol=1e-7)
