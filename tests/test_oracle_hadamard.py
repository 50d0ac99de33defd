"""Pins of the oracle's Hadamard basis (Section 4.3, U_D): the matrices really are Hadamard, the factored
transform equals the dense product with the Kronecker matrix, it is orthogonal (so it leaves X·W unchanged, the
invariance of Section 4.1), and it flattens an outlier channel as the paper intends."""
import numpy as np
import pytest

import oracle
from oracle import hadamard


@pytest.mark.parametrize("H", [hadamard.sylvester(0), hadamard.sylvester(5), hadamard.paley2(5), hadamard.paley2(13)])
def test_hadamard_property(H):
    n = H.shape[0]
    assert set(np.unique(H).tolist()) <= {-1, 1}
    assert (H.astype(np.int64) @ H.astype(np.int64).T == n * np.eye(n, dtype=np.int64)).all()


def test_paley_orders_and_symmetry():
    assert hadamard.paley2(5).shape == (12, 12) and hadamard.paley2(13).shape == (28, 28)
    P = hadamard.paley2(13)
    assert (P == P.T).all()                    # Paley II matrices are symmetric


def test_factorisation_of_the_model_widths():
    assert hadamard.factor(8192) == (13, 1)
    assert hadamard.factor(14336) == (9, 28)
    assert hadamard.factor(28672) == (10, 28)
    assert hadamard.factor(3072) == (8, 12)
    with pytest.raises(ValueError):
        hadamard.factor(1000)


@pytest.mark.parametrize("K", [64, 96, 224, 448])
def test_transform_equals_dense_product(K):
    rng = np.random.default_rng(K)
    C = rng.standard_normal((5, K))
    H = hadamard.hadamard_matrix(K).astype(np.float64)
    want = C @ H / np.sqrt(K)
    got = hadamard.transform(C)
    assert np.abs(got - want).max() <= 1e-6 * np.abs(want).max()
    assert (H @ H.T == K * np.eye(K)).all()


def test_orthogonal_invariance_and_outlier_spreading():
    rng = np.random.default_rng(1)
    K, N, T = 448, 32, 6
    X = rng.standard_normal((T, K))
    X[:, 7] *= 20.0                                   # an outlier channel
    W = rng.standard_normal((K, N)) / np.sqrt(K)
    H = hadamard.hadamard_matrix(K).astype(np.float64) / np.sqrt(K)
    Cx = hadamard.transform(X).astype(np.float64)
    Wp = H.T @ W                                      # U_D^T W
    assert np.abs(Cx @ Wp - X @ W).max() <= 1e-5 * np.abs(X @ W).max()
    assert np.abs(Cx).max(axis=1).mean() < 0.5 * np.abs(X).max(axis=1).mean()   # peaks are spread out


def test_uniform_int4_layer_with_hadamard_beats_plain_int4():
    """Whole down_proj path of the paper (Hadamard U_D, uniform 4-bit weights and activations, r = 0)."""
    rng = np.random.default_rng(2)
    K, N, T = 448, 64, 16
    X = rng.standard_normal((T, K)).astype(np.float32)
    X[:, rng.integers(0, K, 4)] *= 20.0
    W = (rng.standard_normal((K, N)) / np.sqrt(K))
    H = hadamard.hadamard_matrix(K).astype(np.float64) / np.sqrt(K)
    exact = X.astype(np.float64) @ W
    pw_h = oracle.pack_weights((H.T @ W).T.astype(np.float32), 0)
    pw_p = oracle.pack_weights(W.T.astype(np.float32), 0)
    assert pw_h.q8.shape == (N, 0) and pw_h.q4.shape == (N, K)
    y_h = oracle.linear_from_coeff(hadamard.transform(X), pw_h).y32
    y_p = oracle.linear_from_coeff(X, pw_p).y32
    assert np.linalg.norm(y_h - exact) < 0.5 * np.linalg.norm(y_p - exact)
