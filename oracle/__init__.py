"""CPU oracle for the ResQ mixed-precision linear layer -- TEST INFRASTRUCTURE ONLY.

Thin numpy wrappers around `resq_oracle.c` (plain C loops restating Eq. 1-4 of the paper) plus the
fp64 basis construction in `basis.py` (Eq. 5).  Only the tests, the smoke check and the benchmark's
CPU-baseline leg may import this package; the CUDA library never does, and shares no code with it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "resq_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")


def build(force: bool = False) -> str:
    """Compile resq_oracle.c with gcc (no fast-math, no FMA contraction, OpenMP over rows)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
                               "-fno-fast-math", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _c():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_quantize_vector.restype = ctypes.c_float
        _lib.oracle_int_gemm.restype = ctypes.c_long
        _lib.oracle_int_gemm_u8.restype = ctypes.c_long
        _lib.oracle_num_threads.restype = ctypes.c_int
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _chk(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def num_threads() -> int:
    return int(_c().oracle_num_threads())


# --------------------------------------------------------------------------- formats
def bf16_bits_to_f32(bits):
    bits = _chk(bits, np.uint16)
    out = np.empty(bits.shape, np.float32)
    _c().oracle_bf16_to_f32(_p(bits), ctypes.c_long(bits.size), _p(out))
    return out


def f32_to_bf16_bits(x):
    x = _chk(x, np.float32)
    out = np.empty(x.shape, np.uint16)
    _c().oracle_f32_to_bf16(_p(x), ctypes.c_long(x.size), _p(out))
    return out


# --------------------------------------------------------------------------- Eq. 1
def quantize_vector(x, bits: int, scale_fp16: bool = False):
    """Symmetric quantizer of Eq. 1 on one vector: returns (scale fp32, int8 codes)."""
    x = _chk(x, np.float32).ravel()
    code = np.empty(x.size, np.int8)
    s = _c().oracle_quantize_vector(_p(x), ctypes.c_long(x.size), int(bits), int(scale_fp16), _p(code))
    return np.float32(s), code


# --------------------------------------------------------------------------- Eq. 2 / Eq. 3
def split_quantize(C, r: int, scale_fp16: bool = False):
    """Rows of C [rows][K] fp32 -> (q8 [rows][r], q4 [rows][K-r] one code per byte, s8, s4)."""
    C = _chk(C, np.float32)
    rows, K = C.shape
    q8 = np.empty((rows, r), np.int8)
    q4 = np.empty((rows, K - r), np.int8)
    s8 = np.empty(rows, np.float32)
    s4 = np.empty(rows, np.float32)
    _c().oracle_split_quantize(_p(C), ctypes.c_long(rows), int(K), int(r), int(scale_fp16),
                               _p(q8), _p(q4), _p(s8), _p(s4))
    return q8, q4, s8, s4


def quantize_rows(X, bits: int):
    """Uniform-precision symmetric quantizer of Eq. 1 on each row of X [rows][n]: (codes int8, scales fp32 [rows])."""
    X = _chk(X, np.float32)
    rows, n = X.shape
    code = np.empty((rows, n), np.int8)
    s = np.empty(rows, np.float32)
    _c().oracle_quantize_rows(_p(X), ctypes.c_long(rows), int(n), int(bits), _p(code), _p(s))
    return code, s


def pack_nibbles(code):
    code = _chk(code, np.int8)
    assert code.shape[-1] % 2 == 0
    out = np.empty(code.shape[:-1] + (code.shape[-1] // 2,), np.uint8)
    _c().oracle_pack_nibbles(_p(code), ctypes.c_long(code.size), _p(out))
    return out


def unpack_nibbles(packed):
    packed = _chk(packed, np.uint8)
    out = np.empty(packed.shape[:-1] + (packed.shape[-1] * 2,), np.int8)
    _c().oracle_unpack_nibbles(_p(packed), ctypes.c_long(out.size), _p(out))
    return out


# --------------------------------------------------------------------------- projection
def project(X_bits, P_bits):
    """C = X·P with bf16 inputs (uint16 bit patterns), fp64 sums, one rounding to fp32."""
    X_bits = _chk(X_bits, np.uint16)
    P_bits = _chk(P_bits, np.uint16)
    T, K = X_bits.shape
    assert P_bits.shape == (K, K)
    C = np.empty((T, K), np.float32)
    _c().oracle_project(_p(X_bits), _p(P_bits), ctypes.c_long(T), int(K), _p(C))
    return C


# --------------------------------------------------------------------------- Eq. 4
def int_gemm(x, w):
    """acc[t][n] = sum_j x[t][j]·w[n][j] in int64, checked to fit int32."""
    x = _chk(x, np.int8)
    w = _chk(w, np.int8)
    T, Ks = x.shape
    N, Ks2 = w.shape
    assert Ks == Ks2
    acc = np.empty((T, N), np.int32)
    bad = _c().oracle_int_gemm(_p(x), _p(w), ctypes.c_long(T), ctypes.c_long(N), int(Ks), _p(acc))
    if bad:
        raise OverflowError(f"{bad} accumulators exceed int32")
    return acc


def epilogue(acc8, acc4, s_x8, s_x4, s_w8, s_w4):
    """(y32 fp32, ybf bf16 bits) = scaled sum of the two integer products."""
    acc8 = _chk(acc8, np.int32)
    acc4 = _chk(acc4, np.int32)
    T, N = acc8.shape
    s_x8, s_x4 = _chk(s_x8, np.float32), _chk(s_x4, np.float32)
    s_w8, s_w4 = _chk(s_w8, np.float32), _chk(s_w4, np.float32)
    assert s_x8.shape == (T,) and s_x4.shape == (T,) and s_w8.shape == (N,) and s_w4.shape == (N,)
    y32 = np.empty((T, N), np.float32)
    ybf = np.empty((T, N), np.uint16)
    _c().oracle_epilogue(_p(acc8), _p(acc4), _p(s_x8), _p(s_x4), _p(s_w8), _p(s_w4),
                         ctypes.c_long(T), ctypes.c_long(N), _p(y32), _p(ybf))
    return y32, ybf


# --------------------------------------------------------------------------- whole layer
@dataclass
class PackedWeights:
    """Quantized projected weights of one layer (Eq. 3), codes one per byte plus the canonical packing."""
    K: int
    N: int
    r: int
    q8: np.ndarray      # int8 [N][r]
    q4: np.ndarray      # int8 [N][K-r]
    w4_packed: np.ndarray  # uint8 [N][(K-r)/2]
    s8: np.ndarray      # fp32 [N] (fp16-representable when scale_fp16)
    s4: np.ndarray


def pack_weights(W_proj, r: int, scale_fp16: bool = False) -> PackedWeights:
    """W_proj = (U^T W)^T as fp32 [N][K]; per output channel and segment RTN of Eq. 3."""
    W_proj = _chk(W_proj, np.float32)
    N, K = W_proj.shape
    q8, q4, s8, s4 = split_quantize(W_proj, r, scale_fp16)
    return PackedWeights(K, N, r, q8, q4, pack_nibbles(q4), s8, s4)


@dataclass
class LayerResult:
    coeff: np.ndarray   # fp32 [T][K] pre-quantization coefficients
    x8: np.ndarray
    x4: np.ndarray      # int8 codes, one per byte
    x4_packed: np.ndarray
    s_x8: np.ndarray
    s_x4: np.ndarray
    acc8: np.ndarray
    acc4: np.ndarray
    y32: np.ndarray
    ybf: np.ndarray     # bf16 bits


def linear_from_coeff(C, pw: PackedWeights) -> LayerResult:
    """Eq. 2 on the rows of C followed by Eq. 4 and the dequantizing epilogue."""
    x8, x4, s_x8, s_x4 = split_quantize(C, pw.r)
    acc8 = int_gemm(x8, pw.q8)
    acc4 = int_gemm(x4, pw.q4)
    y32, ybf = epilogue(acc8, acc4, s_x8, s_x4, pw.s8, pw.s4)
    return LayerResult(np.asarray(C, np.float32), x8, x4, pack_nibbles(x4), s_x8, s_x4, acc8, acc4, y32, ybf)


def linear(X_bits, P_bits, pw: PackedWeights) -> LayerResult:
    """Whole layer.  P_bits None: the rows of X already are the coefficients (projection folded into
    the previous layer's weights, Section 4.3); otherwise C = X·P is formed online first."""
    C = bf16_bits_to_f32(X_bits) if P_bits is None else project(X_bits, P_bits)
    return linear_from_coeff(C, pw)


# --------------------------------------------------------------------------- asymmetric activations (Section 5.1)
def split_quantize_asym(C, r: int):
    """Rows of C [rows][K] fp32 -> (u8 [rows][r], u4 [rows][K-r] one code per byte, s8, s4, z8, z4):
    Eq. 1 in its asymmetric form per row and segment (z = min, s = (max - min) / (2^N - 1))."""
    C = _chk(C, np.float32)
    rows, K = C.shape
    u8 = np.empty((rows, r), np.uint8)
    u4 = np.empty((rows, K - r), np.uint8)
    s8, s4, z8, z4 = (np.empty(rows, np.float32) for _ in range(4))
    _c().oracle_split_quantize_asym(_p(C), ctypes.c_long(rows), int(K), int(r), _p(u8), _p(u4),
                                    _p(s8), _p(s4), _p(z8), _p(z4))
    return u8, u4, s8, s4, z8, z4


def int_gemm_u8(u, w):
    """acc[t][n] = sum_j u[t][j]·w[n][j], unsigned activation codes, int64 checked to fit int32."""
    u = _chk(u, np.uint8)
    w = _chk(w, np.int8)
    T, Ks = u.shape
    N, Ks2 = w.shape
    assert Ks == Ks2
    acc = np.empty((T, N), np.int32)
    bad = _c().oracle_int_gemm_u8(_p(u), _p(w), ctypes.c_long(T), ctypes.c_long(N), int(Ks), _p(acc))
    if bad:
        raise OverflowError(f"{bad} accumulators exceed int32")
    return acc


def weight_row_sums(w):
    w = _chk(w, np.int8)
    N, Ks = w.shape
    out = np.empty(N, np.int32)
    _c().oracle_weight_row_sums(_p(w), ctypes.c_long(N), int(Ks), _p(out))
    return out


def pack_nibbles_u(code):
    """Unsigned 4-bit codes (0..15), one per byte -> two per byte, code 2i in the low nibble."""
    code = _chk(code, np.uint8)
    return pack_nibbles(code.view(np.int8))


def epilogue_asym(acc8, acc4, s_x8, s_x4, z_x8, z_x4, s_w8, s_w4, wsum8, wsum4):
    acc8, acc4 = _chk(acc8, np.int32), _chk(acc4, np.int32)
    T, N = acc8.shape
    f = lambda a: _chk(a, np.float32)
    s_x8, s_x4, z_x8, z_x4, s_w8, s_w4 = f(s_x8), f(s_x4), f(z_x8), f(z_x4), f(s_w8), f(s_w4)
    wsum8, wsum4 = _chk(wsum8, np.int32), _chk(wsum4, np.int32)
    y32 = np.empty((T, N), np.float32)
    ybf = np.empty((T, N), np.uint16)
    _c().oracle_epilogue_asym(_p(acc8), _p(acc4), _p(s_x8), _p(s_x4), _p(z_x8), _p(z_x4), _p(s_w8), _p(s_w4),
                              _p(wsum8), _p(wsum4), ctypes.c_long(T), ctypes.c_long(N), _p(y32), _p(ybf))
    return y32, ybf


@dataclass
class AsymLayerResult:
    coeff: np.ndarray
    u8: np.ndarray          # uint8 codes [T][r]
    u4: np.ndarray          # uint8 codes 0..15, one per byte [T][K-r]
    u4_packed: np.ndarray
    s_x8: np.ndarray
    s_x4: np.ndarray
    z_x8: np.ndarray
    z_x4: np.ndarray
    acc8: np.ndarray
    acc4: np.ndarray
    wsum8: np.ndarray
    wsum4: np.ndarray
    y32: np.ndarray
    ybf: np.ndarray


def linear_asym_from_coeff(C, pw: PackedWeights) -> AsymLayerResult:
    u8, u4, s8, s4, z8, z4 = split_quantize_asym(C, pw.r)
    acc8, acc4 = int_gemm_u8(u8, pw.q8), int_gemm_u8(u4, pw.q4)
    ws8, ws4 = weight_row_sums(pw.q8), weight_row_sums(pw.q4)
    y32, ybf = epilogue_asym(acc8, acc4, s8, s4, z8, z4, pw.s8, pw.s4, ws8, ws4)
    return AsymLayerResult(np.asarray(C, np.float32), u8, u4, pack_nibbles_u(u4), s8, s4, z8, z4, acc8, acc4,
                           ws8, ws4, y32, ybf)


def linear_asym(X_bits, P_bits, pw: PackedWeights) -> AsymLayerResult:
    """Whole layer with asymmetric per-token activations and symmetric per-channel weights."""
    C = bf16_bits_to_f32(X_bits) if P_bits is None else project(X_bits, P_bits)
    return linear_asym_from_coeff(C, pw)
