"""GPU parity of the asymmetric-activation path (Eq. 1, second form) through the C ABI against the CPU
oracle: unsigned codes, scales, zero-points, weight row sums and int32 accumulators bit for bit; the
fp32 epilogue within 1e-5 of the oracle's fp64-evaluated value relative to the sum of the magnitudes
of its four terms; the bf16 output the nearest-even rounding of the kernel's own fp32 value."""
import numpy as np
import pytest
import torch

import oracle
import synth
from tests.cases import synthetic_folded
from tests.gpu_util import bf16_bits_from_dev, bf16_to_dev, dev, host

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def resq():
    import paper_2412_14363_b200 as m
    return m


def _shifted(T, K, seed):
    """t4 coefficients with a per-token offset, so that the zero-points are far from zero."""
    C = synth.activations(T, K, "t4", seed=seed)
    C += np.linspace(-3.0, 5.0, T, dtype=np.float32)[:, None]
    return synth.f32_to_bf16_bits(C)


def _quantize(resq, C_bits, r):
    T, K = C_bits.shape
    K4 = K - r
    z = lambda *s, dt=torch.float32: torch.empty(s, dtype=dt, device="cuda")
    u8, u4, u4e = z(T, r, dt=torch.uint8), z(T, K4 // 2, dt=torch.uint8), z(T, K4, dt=torch.uint8)
    s8, s4, z8, z4 = z(T), z(T), z(T), z(T)
    resq.resq_project_quantize_asym(bf16_to_dev(C_bits), None, r, u8, u4, s8, s4, z8, z4, u4e)
    assert resq.resq_device_status() == resq.OK
    return u8, u4, u4e, s8, s4, z8, z4


@pytest.mark.parametrize("T,K,r", [(16, 512, 64), (1, 4096, 512), (17, 2048, 256), (129, 4096, 512),
                                   (5, 14336, 1792), (2, 64, 32), (7, 18464, 2304)])
def test_asym_quantize_bit_exact(resq, T, K, r):
    C_bits = _shifted(T, K, 800 + T)
    C = oracle.bf16_bits_to_f32(C_bits)
    C[0, :r] = C[0, 0]                       # a constant INT8 segment: s = 0, codes 0, z = the value
    C_bits = synth.f32_to_bf16_bits(C)
    u8, u4, u4e, s8, s4, z8, z4 = _quantize(resq, C_bits, r)
    o8, o4, os8, os4, oz8, oz4 = oracle.split_quantize_asym(oracle.bf16_bits_to_f32(C_bits), r)
    for g, o in ((s8, os8), (s4, os4), (z8, oz8), (z4, oz4)):
        assert (host(g).view(np.uint32) == o.view(np.uint32)).all()
    assert (host(u8) == o8).all()
    assert (host(u4e) == o4).all()
    assert (host(u4) == oracle.pack_nibbles_u(o4)).all()


def test_asym_quantize_ties(resq):
    """Rows with z = 0 and s = 1/4 exactly, full of .5 ties: both sides must round to even."""
    K, r = 1024, 512
    rng = np.random.default_rng(2)
    C = np.zeros((4, K), np.float32)
    for t in range(4):
        C[t, :r] = (rng.integers(0, 127, r) + 0.5) * 0.25   # (2k + 1) / 8 with 2k + 1 < 256: exact in bf16
        C[t, r:] = (rng.integers(0, 15, K - r) + 0.5) * 0.25
        C[t, 0], C[t, 1] = 0.0, 255 * 0.25
        C[t, r], C[t, r + 1] = 0.0, 15 * 0.25
    test_bits = synth.f32_to_bf16_bits(C)
    assert (synth.bf16_bits_to_f32(test_bits) == C).all()      # representable: the ties are real
    u8, u4, u4e, s8, s4, z8, z4 = _quantize(resq, test_bits, r)
    o8, o4, os8, os4, oz8, oz4 = oracle.split_quantize_asym(C, r)
    assert (os8 == 0.25).all() and (oz8 == 0).all()
    assert (host(u8) == o8).all() and (host(u4e) == o4).all()


def _check_output(res, pw, y32_gpu, ybf_bits=None):
    f = np.float64
    mag = (np.abs(res.acc8.astype(f) * res.s_x8[:, None] * pw.s8[None, :]) + np.abs(res.acc4.astype(f) * res.s_x4[:, None] * pw.s4[None, :])
           + np.abs(res.z_x8[:, None].astype(f) * pw.s8[None, :] * res.wsum8[None, :]) + np.abs(res.z_x4[:, None].astype(f) * pw.s4[None, :] * res.wsum4[None, :]))
    assert (np.abs(y32_gpu.astype(f) - res.y32) <= 1e-5 * mag + 1e-37).all()
    if ybf_bits is not None:
        assert (ybf_bits == synth.f32_to_bf16_bits(y32_gpu)).all()


@pytest.mark.parametrize("T,K,N,r,fp16,w4i8", [
    (16, 512, 512, 64, False, True),
    (17, 512, 264, 64, False, True),      # ragged rows and columns
    (300, 2048, 520, 256, True, False),   # two pair tiles of rows, partial column tile, kernel expands packed weights
    (2304, 1024, 2304, 128, False, True),  # 81 tiles on 74 CTA pairs: two rounds of the persistent grid
    (1, 4096, 1024, 512, True, True),     # a single token through the tile kernel
    (257, 1024, 768, 128, False, True),
])
def test_asym_mixed_gemm_bit_exact(resq, T, K, N, r, fp16, w4i8):
    C_bits = _shifted(T, K, 900 + T)
    _, Wp = synthetic_folded(2, K, N, r, seed_shift=T)
    pw = oracle.pack_weights(Wp, r, scale_fp16=fp16)
    res = oracle.linear_asym(C_bits, None, pw)
    desc = resq.layer_desc(K, N, r, resq.SCALE_FP16 if fp16 else resq.SCALE_FP32)
    sdt = torch.float16 if fp16 else torch.float32
    W = resq.Weights(desc, dev(pw.q8), dev(pw.w4_packed), dev(pw.s8).to(sdt), dev(pw.s4).to(sdt),
                     dev(pw.q4) if w4i8 else None)
    ws8, ws4 = resq.resq_weight_row_sums(W)
    assert (host(ws8) == res.wsum8).all() and (host(ws4) == res.wsum4).all()
    wsp = resq.alloc_workspace_asym(desc, T, False, w4i8)
    y32 = torch.full((T, N), float("nan"), dtype=torch.float32, device="cuda")
    a8 = torch.full((T, N), -1, dtype=torch.int32, device="cuda")
    a4 = torch.full((T, N), -1, dtype=torch.int32, device="cuda")
    # the ORACLE's codes in, packed INT4 activations (the kernel expands them)
    resq.resq_mixed_gemm_asym(W, ws8, ws4, dev(res.u8), dev(res.u4_packed), dev(res.s_x8), dev(res.s_x4),
                              dev(res.z_x8), dev(res.z_x4), y32, wsp, a8, a4)
    ybf = torch.zeros((T, N), dtype=torch.bfloat16, device="cuda")
    resq.resq_mixed_gemm_asym(W, ws8, ws4, dev(res.u8), None, dev(res.s_x8), dev(res.s_x4), dev(res.z_x8),
                              dev(res.z_x4), ybf, wsp, u4_u8=dev(res.u4))
    assert resq.resq_device_status() == resq.OK
    assert (host(a8) == res.acc8).all()
    assert (host(a4) == res.acc4).all()
    _check_output(res, pw, host(y32), bf16_bits_from_dev(ybf))


def test_asym_extreme_codes(resq):
    """All activation codes at 255 / 15 against weights at -128 / -8: largest accumulator magnitudes."""
    T, K, N, r = 130, 1024, 256, 128
    K4 = K - r
    q8, q4 = np.full((N, r), -128, np.int8), np.full((N, K4), -8, np.int8)
    pw = oracle.PackedWeights(K, N, r, q8, q4, oracle.pack_nibbles(q4), np.full(N, 0.01, np.float32), np.full(N, 0.1, np.float32))
    u8, u4 = np.full((T, r), 255, np.uint8), np.full((T, K4), 15, np.uint8)
    acc8, acc4 = oracle.int_gemm_u8(u8, q8), oracle.int_gemm_u8(u4, q4)
    ws8, ws4 = oracle.weight_row_sums(q8), oracle.weight_row_sums(q4)
    sx8, sx4, zx8, zx4 = (np.full(T, v, np.float32) for v in (0.5, 2.0, -1.25, 3.5))
    y32, ybf = oracle.epilogue_asym(acc8, acc4, sx8, sx4, zx8, zx4, pw.s8, pw.s4, ws8, ws4)
    desc = resq.layer_desc(K, N, r)
    W = resq.Weights(desc, dev(q8), dev(pw.w4_packed), dev(pw.s8), dev(pw.s4), dev(q4))
    g8, g4 = resq.resq_weight_row_sums(W)
    wsp = resq.alloc_workspace_asym(desc, T, False, True)
    y = torch.empty((T, N), dtype=torch.float32, device="cuda")
    a8 = torch.empty((T, N), dtype=torch.int32, device="cuda")
    a4 = torch.empty((T, N), dtype=torch.int32, device="cuda")
    resq.resq_mixed_gemm_asym(W, g8, g4, dev(u8), None, dev(sx8), dev(sx4), dev(zx8), dev(zx4), y, wsp, a8, a4, u4_u8=dev(u4))
    assert resq.resq_device_status() == resq.OK
    assert (host(a8) == acc8).all() and (host(a4) == acc4).all()
    mag = np.abs(y32.astype(np.float64)) + 1.0
    assert (np.abs(host(y).astype(np.float64) - y32) <= 1e-5 * (np.abs(acc8 * 0.5 * 0.01) + np.abs(acc4 * 2.0 * 0.1) + mag)).all()


@pytest.mark.parametrize("T,r", [(5, 256), (200, 256), (3, 0), (130, 0)])
def test_asym_linear_end_to_end(resq, T, r):
    """Whole layer; r = 0 is the uniform 4-bit layer (empty INT8 segment: s = 0, z = 0)."""
    K, N = 2048, 512
    C_bits = _shifted(T, K, 950 + T)
    _, Wp = synthetic_folded(2, K, N, r, seed_shift=3)
    pw = oracle.pack_weights(Wp, r)
    res = oracle.linear_asym(C_bits, None, pw)
    desc = resq.layer_desc(K, N, r)
    W = resq.resq_pack_weights(desc, dev(Wp))
    ws8, ws4 = resq.resq_weight_row_sums(W)
    wsp = resq.alloc_workspace_asym(desc, T, False, True)
    y32 = torch.empty((T, N), dtype=torch.float32, device="cuda")
    resq.resq_linear_asym(W, ws8, ws4, bf16_to_dev(C_bits), None, y32, wsp)
    ybf = torch.empty((T, N), dtype=torch.bfloat16, device="cuda")
    resq.resq_linear_asym(W, ws8, ws4, bf16_to_dev(C_bits), None, ybf, wsp)
    assert resq.resq_device_status() == resq.OK
    _check_output(res, pw, host(y32), bf16_bits_from_dev(ybf))


def test_asym_online_projection(resq):
    """Online projection + asymmetric quantization: codes within +-1 on <= 0.1 % (the coefficients come
    from another summation order), and exact again downstream given the kernel's own codes."""
    T, K, N, r = 150, 1024, 264, 128
    X_bits = synth.f32_to_bf16_bits(synth.activations(T, K, "t4", seed=77))
    P_bits = synth.f32_to_bf16_bits(synth.kron_orthogonal_bf16(K, inner=128))
    o8, o4, os8, os4, oz8, oz4 = oracle.split_quantize_asym(oracle.project(X_bits, P_bits), r)
    K4 = K - r
    desc = resq.layer_desc(K, N, r)
    wsp = resq.alloc_workspace_asym(desc, T, True, True)
    z = lambda *s, dt=torch.float32: torch.empty(s, dtype=dt, device="cuda")
    u8, u4e = z(T, r, dt=torch.uint8), z(T, K4, dt=torch.uint8)
    s8, s4, z8, z4 = z(T), z(T), z(T), z(T)
    resq.resq_project_quantize_asym(bf16_to_dev(X_bits), bf16_to_dev(P_bits), r, u8, None, s8, s4, z8, z4, u4e, wsp)
    assert resq.resq_device_status() == resq.OK
    g8, g4 = host(u8).astype(np.int32), host(u4e).astype(np.int32)
    assert np.abs(g8 - o8).max() <= 1 and np.abs(g4 - o4).max() <= 1
    assert ((g8 != o8).sum() + (g4 != o4).sum()) / float(T * K) <= 1e-3


@pytest.mark.parametrize("T,K,N,r,fp16", [
    (1, 4096, 4096, 512, True),      # o_proj shape, one token: streaming kernel, split staging
    (4, 4096, 1024, 512, True),
    (16, 4096, 6144, 512, True),     # packed staging (T > 8)
    (9, 2048, 264, 256, False),
    (3, 1056, 72, 96, False),        # segment lengths that are not multiples of a step
    (16, 14336, 256, 1792, True),    # down_proj reduction length
    (2, 4096, 8, 512, False),        # a single unit
    (16, 28672, 64, 3584, False),    # rows too wide to stage 9-16 tokens: two launches of 8 tokens
    (11, 28672, 72, 0, False),       # ... 8 + 3 tokens, uniform INT4, ragged channel block
])
def test_asym_decode_bit_exact(resq, T, K, N, r, fp16):
    """T <= 16 with packed codes: the weight-streaming kernel with unsigned activation codes."""
    C_bits = _shifted(T, K, 980 + T)
    _, Wp = synthetic_folded(2, K, N, r, seed_shift=40 + T)
    pw = oracle.pack_weights(Wp, r, scale_fp16=fp16)
    res = oracle.linear_asym(C_bits, None, pw)
    desc = resq.layer_desc(K, N, r, resq.SCALE_FP16 if fp16 else resq.SCALE_FP32)
    sdt = torch.float16 if fp16 else torch.float32
    W = resq.Weights(desc, dev(pw.q8), dev(pw.w4_packed), dev(pw.s8).to(sdt), dev(pw.s4).to(sdt), None)
    ws8, ws4 = resq.resq_weight_row_sums(W)
    wsp = resq.alloc_workspace_asym(desc, T, False, False)
    y32 = torch.full((T, N), float("nan"), dtype=torch.float32, device="cuda")
    a8 = torch.full((T, N), -1, dtype=torch.int32, device="cuda")
    a4 = torch.full((T, N), -1, dtype=torch.int32, device="cuda")
    resq.resq_mixed_gemm_asym(W, ws8, ws4, dev(res.u8), dev(res.u4_packed), dev(res.s_x8), dev(res.s_x4),
                              dev(res.z_x8), dev(res.z_x4), y32, wsp, a8, a4)
    ybf = torch.zeros((T, N), dtype=torch.bfloat16, device="cuda")
    resq.resq_mixed_gemm_asym(W, ws8, ws4, dev(res.u8), dev(res.u4_packed), dev(res.s_x8), dev(res.s_x4),
                              dev(res.z_x8), dev(res.z_x4), ybf, wsp)
    assert resq.resq_device_status() == resq.OK
    assert (host(a8) == res.acc8).all()
    assert (host(a4) == res.acc4).all()
    _check_output(res, pw, host(y32), bf16_bits_from_dev(ybf))
