"""GPU parity of the paper's own down_proj path (Section 4.3): Hadamard U_D fused with the quantizer, and the
uniform INT4 layer (r = 0) through every kernel.

The oracle sums the transform in fp64 and rounds once; the kernel adds in fp32 in butterfly order.  So, as for
the dense online projection: every code within +-1 of the oracle's, at most 0.1 % different, scales within a
few ulp; downstream everything is exact again given the kernel's own codes.  With r = 0 and the coefficients
given (folded path) codes, scales, accumulators are bit-exact.
"""
import numpy as np
import pytest
import torch

import oracle
import synth
from oracle import hadamard
from tests.gpu_util import bf16_bits_from_dev, bf16_to_dev, dev, host
from tests.test_gpu_parity import check_output

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def resq():
    import paper_2412_14363_b200 as m
    return m


def _ulp_diff(a, b):
    return np.abs(a.view(np.int32).astype(np.int64) - b.view(np.int32).astype(np.int64))


def _run(resq, X_bits, r):
    T, K = X_bits.shape
    K4 = K - r
    x8 = torch.empty((T, r), dtype=torch.int8, device="cuda") if r else None
    x4 = torch.empty((T, K4 // 2), dtype=torch.uint8, device="cuda")
    x4e = torch.empty((T, K4), dtype=torch.int8, device="cuda")
    s8 = torch.full((T,), float("nan"), dtype=torch.float32, device="cuda")
    s4 = torch.full((T,), float("nan"), dtype=torch.float32, device="cuda")
    resq.resq_hadamard_quantize(bf16_to_dev(X_bits), r, x8, x4, s8, s4, x4e)
    assert resq.resq_device_status() == resq.OK
    return x8, x4, x4e, s8, s4


@pytest.mark.parametrize("T,K,r", [(5, 64, 0), (16, 1024, 0), (33, 1024, 128), (7, 384, 0), (9, 896, 0), (20, 3072, 384),
                                   (300, 8192, 0), (130, 14336, 0), (3, 14336, 1792), (2, 28672, 0),
                                   (11, 1792, 0), (6, 3584, 448), (4, 7168, 0)])  # 28 * 2^6..8: register path with 1, 2, 4 warps
def test_hadamard_quantize_codes(resq, T, K, r):
    X = synth.activations(T, K, "t4", seed=600 + T)
    X_bits = synth.f32_to_bf16_bits(X)
    C = hadamard.transform(synth.bf16_bits_to_f32(X_bits))
    q8, q4, o8, o4 = oracle.split_quantize(C, r)
    x8, x4, x4e, s8, s4 = _run(resq, X_bits, r)
    g4 = host(x4e).astype(np.int32)
    assert (host(x4) == oracle.pack_nibbles(host(x4e))).all()
    assert np.abs(g4 - q4).max() <= 1
    diff = (g4 != q4).sum()
    if r:
        g8 = host(x8).astype(np.int32)
        assert np.abs(g8 - q8).max() <= 1
        diff += (g8 != q8).sum()
        assert _ulp_diff(host(s8), o8).max() <= 64
    else:
        assert (host(s8) == 0).all()
    assert diff / float(T * K) <= 1e-3
    assert _ulp_diff(host(s4), o4).max() <= 64     # fp32 butterflies: a few ulp of the largest coefficient


@pytest.mark.parametrize("T,K,N", [(150, 1024, 264), (16, 896, 72), (1, 3072, 1024), (40, 14336, 256)])
def test_uniform_int4_layer_exact_given_its_own_codes(resq, T, K, N):
    """Hadamard + uniform INT4 (r = 0) end to end: the kernel's codes and scales fed to the oracle's integer product
    and epilogue reproduce resq_mixed_gemm bit for bit (accumulators) / within tolerance (fp32 output)."""
    X_bits = synth.f32_to_bf16_bits(synth.activations(T, K, "t4", seed=650 + T))
    Wp = synth.projected_weights_direct(N, K, seed=660 + T)
    pw = oracle.pack_weights(Wp, 0)
    x8, x4, x4e, s8, s4 = _run(resq, X_bits, 0)
    g4, gs4 = host(x4e), host(s4)
    acc8, acc4 = np.zeros((T, N), np.int32), oracle.int_gemm(g4, pw.q4)
    y32, ybf = oracle.epilogue(acc8, acc4, np.zeros(T, np.float32), gs4, pw.s8, pw.s4)
    res = oracle.LayerResult(None, np.zeros((T, 0), np.int8), g4, oracle.pack_nibbles(g4), np.zeros(T, np.float32), gs4,
                             acc8, acc4, y32, ybf)
    desc = resq.layer_desc(K, N, 0)
    W = resq.resq_pack_weights(desc, dev(Wp))
    assert (host(W.w4) == pw.w4_packed).all() and (host(W.w4_i8) == pw.q4).all()
    assert (host(W.s_w4).view(np.uint32) == pw.s4.view(np.uint32)).all() and (host(W.s_w8) == 0).all()
    ws = resq.alloc_workspace(desc, T, False, True)
    yg = torch.full((T, N), float("nan"), dtype=torch.float32, device="cuda")
    a8 = torch.full((T, N), -1, dtype=torch.int32, device="cuda")
    a4 = torch.full((T, N), -1, dtype=torch.int32, device="cuda")
    resq.resq_mixed_gemm(W, None, x4, s8, s4, yg, ws, a8, a4, x4_i8=x4e)
    yb = torch.zeros((T, N), dtype=torch.bfloat16, device="cuda")
    resq.resq_mixed_gemm(W, None, x4, s8, s4, yb, ws, x4_i8=x4e)
    assert resq.resq_device_status() == resq.OK
    assert (host(a8) == 0).all() and (host(a4) == acc4).all()
    check_output(res, pw, host(yg), bf16_bits_from_dev(yb))


@pytest.mark.parametrize("T", [3, 64])
def test_uniform_int4_folded_bit_exact(resq, T):
    """r = 0 with the coefficients given: quantizer, packer, both GEMM kernels bit-exact against the oracle."""
    K, N = 2048, 512
    C_bits = synth.f32_to_bf16_bits(synth.activations(T, K, "t4", seed=690 + T))
    Wp = synth.projected_weights_direct(N, K, seed=691)
    pw = oracle.pack_weights(Wp, 0)
    res = oracle.linear(C_bits, None, pw)
    desc = resq.layer_desc(K, N, 0)
    W = resq.resq_pack_weights(desc, dev(Wp), with_w4_i8=T > 16)
    ws = resq.alloc_workspace(desc, T, False, T > 16)
    y32 = torch.empty((T, N), dtype=torch.float32, device="cuda")
    resq.resq_linear(W, bf16_to_dev(C_bits), None, y32, ws)
    ybf = torch.empty((T, N), dtype=torch.bfloat16, device="cuda")
    resq.resq_linear(W, bf16_to_dev(C_bits), None, ybf, ws)
    assert resq.resq_device_status() == resq.OK
    check_output(res, pw, host(y32), bf16_bits_from_dev(ybf))
