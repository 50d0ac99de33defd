"""Hadamard basis for the down_proj input (Section 4.3: "we choose U_D to be a hadamard matrix") -- TEST
INFRASTRUCTURE ONLY, part of the CPU oracle.

U_D = H_K / sqrt(K) with H_K a K x K matrix of +-1 entries and H_K H_K^T = K I.  The paper names no
construction; the dimensions it needs are 2^k (Sylvester's doubling) and 2^k * 28 for the Llama-3 feed-forward
widths 14336 and 28672, for which a 28 x 28 factor is required.  Here that factor is Paley's second construction
for q = 13 (and q = 5 gives a 12 x 12 one): with the quadratic character chi of GF(q), q = 1 mod 4, the Jacobsthal
matrix Q[i][j] = chi(i - j) is symmetric, S = [[0, 1^T], [1, Q]] is a symmetric conference matrix of order q + 1,
and  H = S (x) [[1, 1], [1, -1]] + I (x) [[1, -1], [-1, -1]]  is a Hadamard matrix of order 2 (q + 1).
H_K = Sylvester(2^k) (x) H_m, i.e. coefficient index = a * m + b with a the Sylvester index.
"""
from __future__ import annotations

import numpy as np


def sylvester(k: int) -> np.ndarray:
    """2^k x 2^k Hadamard matrix by Sylvester's doubling, entries +-1 (int8)."""
    H = np.ones((1, 1), np.int8)
    for _ in range(k):
        H = np.block([[H, H], [H, -H]]).astype(np.int8)
    return H


def paley2(q: int) -> np.ndarray:
    """Paley's second construction for a prime q = 1 (mod 4): a symmetric Hadamard matrix of order 2 (q + 1)."""
    assert q % 4 == 1 and all(q % p for p in range(2, int(q ** 0.5) + 1)), "q must be a prime = 1 mod 4"
    squares = {(x * x) % q for x in range(1, q)}
    chi = lambda a: 0 if a % q == 0 else (1 if a % q in squares else -1)
    n = q + 1
    S = np.zeros((n, n), np.int64)
    S[0, 1:] = 1
    S[1:, 0] = 1
    for i in range(q):
        for j in range(q):
            S[1 + i, 1 + j] = chi(i - j)
    A = np.array([[1, 1], [1, -1]], np.int64)
    B = np.array([[1, -1], [-1, -1]], np.int64)
    return (np.kron(S, A) + np.kron(np.eye(n, dtype=np.int64), B)).astype(np.int8)


SMALL_FACTORS = {1: None, 12: 5, 28: 13}   # order of the non-Sylvester factor -> q of its Paley construction


def factor(K: int):
    """K = 2^k * m with m in {1, 12, 28}; returns (k, m) with the largest admissible m."""
    for m in (28, 12, 1):
        if K % m == 0:
            a = K // m
            if a & (a - 1) == 0:
                return a.bit_length() - 1, m
    raise ValueError(f"no Hadamard construction here for K = {K}")


def small_factor(m: int) -> np.ndarray:
    return np.ones((1, 1), np.int8) if m == 1 else paley2(SMALL_FACTORS[m])


def hadamard_matrix(K: int) -> np.ndarray:
    """The full K x K matrix (for small K only)."""
    k, m = factor(K)
    return np.kron(sylvester(k), small_factor(m)).astype(np.int8)


def transform(C) -> np.ndarray:
    """Rows of C [T][K] (any real dtype) times H_K / sqrt(K): fp64 sums with the two explicit factor matrices
    (plain matrix products; no butterflies), one rounding to fp32."""
    C = np.asarray(C, np.float64)
    T, K = C.shape
    k, m = factor(K)
    A = 1 << k
    X = C.reshape(T, A, m)
    X = np.tensordot(X, small_factor(m).astype(np.float64), axes=([2], [0]))          # [T][A][m]
    X = np.tensordot(X, sylvester(k).astype(np.float64), axes=([1], [0]))             # [T][m][A]
    X = np.transpose(X, (0, 2, 1)).reshape(T, K)
    return (X / np.sqrt(np.float64(K))).astype(np.float32)
