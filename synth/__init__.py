"""Seeded synthetic inputs for the ResQ mixed-precision linear layer.

This module only draws random numbers and shapes them into the workloads
(activations with outlier channels, Gaussian weights, calibration batches).
It holds none of the method's arithmetic: no quantizer, no projection, no
GEMM.  Both the CPU oracle's tests and the CUDA path's tests/bench draw their
inputs from here so that the two sides always see identical bits.

The generator is counter based (splitmix64 finaliser over a 64-bit counter),
so a value depends only on (seed, stream, index) and not on numpy's or
torch's RNG implementation.

bf16 values are carried as numpy uint16 bit patterns (`*_bits`) or as float32
arrays whose values are exactly representable in bf16.
"""
from __future__ import annotations

import numpy as np

_GOLD = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)


def _mix(z: np.ndarray) -> np.ndarray:
    """splitmix64 output function on an array of uint64 counters."""
    with np.errstate(over="ignore"):
        z = (z ^ (z >> np.uint64(30))) * _M1
        z = (z ^ (z >> np.uint64(27))) * _M2
        z = z ^ (z >> np.uint64(31))
    return z


def _key(seed: int, stream: int) -> np.uint64:
    with np.errstate(over="ignore"):
        k = _mix(np.array([np.uint64(seed) * _GOLD + np.uint64(stream)], dtype=np.uint64))
        k = _mix(k + _GOLD)
    return k[0]


def uniform01(seed: int, stream: int, n: int, offset: int = 0) -> np.ndarray:
    """n doubles in the open interval (0, 1); element i depends only on (seed, stream, offset+i)."""
    idx = np.arange(offset, offset + n, dtype=np.uint64)
    with np.errstate(over="ignore"):
        bits = _mix(idx * _GOLD + _key(seed, stream))
    return ((bits >> np.uint64(11)).astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)


def normal(seed: int, stream: int, n: int, offset: int = 0) -> np.ndarray:
    """n iid N(0,1) doubles by Box-Muller on two counter streams."""
    u1 = uniform01(seed, 2 * stream, n, offset)
    u2 = uniform01(seed, 2 * stream + 1, n, offset)
    return np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)


def student_t4(seed: int, stream: int, n: int, offset: int = 0) -> np.ndarray:
    """n iid Student-t(nu=4) doubles: Z / sqrt(chi2_4 / 4) with chi2_4 a sum of four squared normals."""
    z = normal(seed, 8 * stream, n, offset)
    chi = np.zeros(n)
    for j in range(1, 5):
        g = normal(seed, 8 * stream + j, n, offset)
        chi += g * g
    return z / np.sqrt(chi / 4.0)


# ----------------------------------------------------------------------------
# bf16 carriers (format conversion only)
# ----------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (round to nearest, ties to even); returns uint16 bit patterns. Finite inputs."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = (u + np.uint32(0x7FFF) + lsb) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def to_bf16_values(x: np.ndarray) -> np.ndarray:
    """float32 array holding x rounded to bf16 (values exactly representable in bf16)."""
    return bf16_bits_to_f32(f32_to_bf16_bits(np.asarray(x, dtype=np.float32)))


# ----------------------------------------------------------------------------
# Workload pieces
# ----------------------------------------------------------------------------
SEED_ACT, SEED_CALIB, SEED_ROT, SEED_W, SEED_OUTLIER, SEED_P = 0, 1, 2, 3, 4, 5


def outlier_channels(K: int, count: int, seed: int = SEED_OUTLIER) -> np.ndarray:
    """`count` distinct channel indices in [0, K), seeded (argsort of a uniform stream)."""
    u = uniform01(seed, 0, K)
    return np.sort(np.argsort(u, kind="stable")[:count])


def n_outliers(K: int) -> int:
    """5 of 512 for the tiny layer, otherwise 1 % of the channels."""
    return 5 if K == 512 else int(0.01 * K)


def activations(T: int, K: int, dist: str = "t4", seed: int = SEED_ACT, stream: int = 0,
                scale: float = 20.0, row_offset: int = 0) -> np.ndarray:
    """bf16-valued float32 [T][K]: N(0,1) ("normal") or Student-t(4) ("t4") entries, iid per element,
    with n_outliers(K) seeded channels multiplied by `scale` (activation outliers about 20x larger
    than the rest, as the paper's introduction describes).  Row t is the same whatever T is, and
    `row_offset` shifts the window, so a row subset can be regenerated on its own."""
    n = T * K
    off = row_offset * K
    x = normal(seed, stream, n, off) if dist == "normal" else student_t4(seed, stream, n, off)
    x = x.reshape(T, K)
    ch = outlier_channels(K, n_outliers(K))
    x[:, ch] *= scale
    return to_bf16_values(x.astype(np.float32))


def weights(K: int, N: int, seed: int = SEED_W, stream: int = 0) -> np.ndarray:
    """bf16-valued float32 W [K][N] with iid N(0, 1/K) entries (input features along rows)."""
    w = normal(seed, stream, K * N).reshape(K, N) / np.sqrt(float(K))
    return to_bf16_values(w.astype(np.float32))


def projected_weights_direct(N: int, K: int, seed: int = SEED_W, stream: int = 0) -> np.ndarray:
    """float32 [N][K] with iid N(0, 1/K) entries, standing in for (P^T W)^T at sizes where the fp64
    product is too slow to form on the host: an orthogonal transform of iid Gaussian columns is again
    iid Gaussian with the same variance, so the distribution is the one the product would have."""
    chunk = 1 << 24
    out = np.empty(N * K, dtype=np.float32)
    inv = 1.0 / np.sqrt(float(K))
    for o in range(0, N * K, chunk):
        m = min(chunk, N * K - o)
        out[o:o + m] = (normal(seed, stream, m, o) * inv).astype(np.float32)
    return out.reshape(N, K)


def gaussian_matrix(n: int, seed: int = SEED_ROT, stream: int = 0) -> np.ndarray:
    """n x n iid N(0,1) doubles (raw material for a random rotation)."""
    return normal(seed, stream, n * n).reshape(n, n)


def kron_orthogonal_bf16(K: int, seed: int = SEED_P, inner: int = 128) -> np.ndarray:
    """A dense K x K matrix, orthogonal up to bf16 rounding, for sizes where PCA + QR on the host is
    too slow: the Kronecker product of two Haar-distributed factors (K/inner and inner wide), each
    the sign-fixed Q of a seeded Gaussian matrix.  Returned as bf16-valued float32.  This is input
    preparation only; the layer treats P as an opaque bf16 matrix."""
    assert K % inner == 0
    a = K // inner

    def haar(n, stream):
        q, rr = np.linalg.qr(gaussian_matrix(n, seed, stream))
        return q * np.sign(np.diag(rr))

    qa, qb = haar(a, 0), haar(inner, 1)
    out = np.empty((K, K), dtype=np.float32)
    for i in range(a):
        blk = np.kron(qa[i:i + 1, :], qb)  # inner x K
        out[i * inner:(i + 1) * inner, :] = to_bf16_values(blk.astype(np.float32))
    return out


SEED_ATTN = 7


def haar_orthogonal(n: int, seed: int = SEED_ATTN, stream: int = 0) -> np.ndarray:
    """n x n Haar-distributed orthogonal matrix (sign-fixed Q of a seeded Gaussian matrix), float64: a stand-in
    for a per-layer head basis such as U_C, which the method obtains from calibration data that is not here."""
    q, rr = np.linalg.qr(gaussian_matrix(n, seed, stream))
    return q * np.sign(np.diag(rr))


def head_vectors(T: int, H: int, d: int, seed: int = SEED_ATTN, stream: int = 1, lead: float = 4.0,
                 scale: float = 1.0, shift: float = 0.0) -> np.ndarray:
    """bf16-valued float32 [T][H][d] head vectors: iid N(0, 1) entries times `scale`, the first d/8 coefficients
    of every head `lead` times larger (a basis ordered by variance puts its high-variance coefficients
    first), plus `shift`."""
    x = normal(seed, stream, T * H * d).reshape(T, H, d) * scale
    x[:, :, : d // 8] *= lead
    return to_bf16_values((x + shift).astype(np.float32))


# ----------------------------------------------------------------------------
# The same counter-based streams on a torch device, for full-size workloads (hundreds of millions
# of draws).  The integer stream is identical to the numpy one; log/cos may differ in the last ulp.
# ----------------------------------------------------------------------------
def _s64(x: int) -> int:
    x &= (1 << 64) - 1
    return x - (1 << 64) if x >= (1 << 63) else x


def _t_lsr(z, k: int):
    return (z >> k) & ((1 << (64 - k)) - 1)


def _t_mix(z):
    z = (z ^ _t_lsr(z, 30)) * _s64(int(_M1))
    z = (z ^ _t_lsr(z, 27)) * _s64(int(_M2))
    return z ^ _t_lsr(z, 31)


def t_uniform01(seed: int, stream: int, n: int, offset: int, device):
    import torch
    idx = torch.arange(offset, offset + n, dtype=torch.int64, device=device)
    bits = _t_mix(idx * _s64(int(_GOLD)) + _s64(int(_key(seed, stream))))
    return (_t_lsr(bits, 11).to(torch.float64) + 0.5) * (1.0 / 9007199254740992.0)


def t_normal(seed: int, stream: int, n: int, offset: int, device):
    import torch
    u1 = t_uniform01(seed, 2 * stream, n, offset, device)
    u2 = t_uniform01(seed, 2 * stream + 1, n, offset, device)
    return torch.sqrt(-2.0 * torch.log(u1)) * torch.cos(2.0 * torch.pi * u2)


def t_student_t4(seed: int, stream: int, n: int, offset: int, device):
    import torch
    z = t_normal(seed, 8 * stream, n, offset, device)
    chi = torch.zeros(n, dtype=torch.float64, device=device)
    for j in range(1, 5):
        g = t_normal(seed, 8 * stream + j, n, offset, device)
        chi += g * g
    return z / torch.sqrt(chi / 4.0)


def t_activations(T: int, K: int, device, dist: str = "t4", seed: int = SEED_ACT, stream: int = 0,
                  scale: float = 20.0, row_offset: int = 0, rows_per_chunk: int = 512):
    """torch.bfloat16 [T][K] on `device`; same recipe as activations()."""
    import torch
    out = torch.empty((T, K), dtype=torch.bfloat16, device=device)
    ch = torch.from_numpy(outlier_channels(K, n_outliers(K))).to(device)
    gen = t_normal if dist == "normal" else t_student_t4
    for t0 in range(0, T, rows_per_chunk):
        rows = min(rows_per_chunk, T - t0)
        x = gen(seed, stream, rows * K, (row_offset + t0) * K, device).reshape(rows, K)
        x[:, ch] *= scale
        out[t0:t0 + rows] = x.to(torch.float32).to(torch.bfloat16)
    return out


def t_projected_weights_direct(N: int, K: int, device, seed: int = SEED_W, stream: int = 0,
                               rows_per_chunk: int = 1024):
    """torch.float32 [N][K] on `device`; same recipe as projected_weights_direct()."""
    import torch
    out = torch.empty((N, K), dtype=torch.float32, device=device)
    inv = 1.0 / float(np.sqrt(float(K)))
    for n0 in range(0, N, rows_per_chunk):
        rows = min(rows_per_chunk, N - n0)
        out[n0:n0 + rows] = (t_normal(seed, stream, rows * K, n0 * K, device) * inv).reshape(rows, K).to(torch.float32)
    return out


def t_kron_orthogonal_bf16(K: int, device, seed: int = SEED_P, inner: int = 128):
    """torch.bfloat16 [K][K] on `device`; same recipe as kron_orthogonal_bf16()."""
    import torch
    assert K % inner == 0
    a = K // inner

    def haar(n, stream):
        q, rr = np.linalg.qr(gaussian_matrix(n, seed, stream))
        return torch.from_numpy(q * np.sign(np.diag(rr))).to(device)

    qa, qb = haar(a, 0), haar(inner, 1)
    out = torch.empty((K, K), dtype=torch.bfloat16, device=device)
    for i in range(a):
        out[i * inner:(i + 1) * inner] = torch.kron(qa[i:i + 1, :], qb).to(torch.float32).to(torch.bfloat16)
    return out


def t_head_vectors(T: int, H: int, d: int, device, seed: int = SEED_ATTN, stream: int = 1, lead: float = 4.0,
                   scale: float = 1.0, shift: float = 0.0):
    """torch.bfloat16 [T][H][d] on `device`; same recipe as head_vectors()."""
    import torch
    x = t_normal(seed, stream, T * H * d, 0, device).reshape(T, H, d) * scale
    x[:, :, : d // 8] *= lead
    return (x + shift).to(torch.float32).to(torch.bfloat16)
