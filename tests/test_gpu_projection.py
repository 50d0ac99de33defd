"""GPU parity of the online-projection path (C = X·P on the tensor cores, then split quantization).

The oracle sums each coefficient in fp64 and rounds once to fp32; the kernel accumulates bf16
products in fp32 in another order.  So: every code within +-1 of the oracle's, at most 0.1 % of the
codes different, scales within a few ulp.  Everything downstream is exact again: feeding the
kernel's own codes to the oracle's integer product and epilogue must reproduce resq_linear's output.
"""
import numpy as np
import pytest
import torch

import oracle
import synth
from tests.gpu_util import bf16_bits_from_dev, bf16_to_dev, dev, host
from tests.test_gpu_parity import check_output

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def resq():
    import paper_2412_14363_b200 as m
    return m


def _ulp_diff(a, b):
    return np.abs(a.view(np.int32).astype(np.int64) - b.view(np.int32).astype(np.int64))


@pytest.mark.parametrize("T,K,r,inner", [(16, 512, 64, 128), (200, 1024, 128, 128), (130, 1056, 128, 32),
                                         (300, 2048, 256, 128), (70, 4096, 512, 128), (4100, 512, 64, 128), (6, 14336, 1792, 128)])
def test_online_projection_codes(resq, T, K, r, inner):
    X_bits = synth.f32_to_bf16_bits(synth.activations(T, K, "t4", seed=400 + T))
    P_bits = synth.f32_to_bf16_bits(synth.kron_orthogonal_bf16(K, inner=inner))
    C = oracle.project(X_bits, P_bits)
    q8, q4, o8, o4 = oracle.split_quantize(C, r)

    K4 = K - r
    desc = resq.layer_desc(K, 8, r)
    ws = resq.alloc_workspace(desc, T, True, True)
    x8 = torch.empty((T, r), dtype=torch.int8, device="cuda")
    x4 = torch.empty((T, K4 // 2), dtype=torch.uint8, device="cuda")
    x4e = torch.empty((T, K4), dtype=torch.int8, device="cuda")
    s8 = torch.empty(T, dtype=torch.float32, device="cuda")
    s4 = torch.empty(T, dtype=torch.float32, device="cuda")
    resq.resq_project_quantize(bf16_to_dev(X_bits), bf16_to_dev(P_bits), r, x8, x4, s8, s4, x4e, ws)
    assert resq.resq_device_status() == resq.OK
    g8, g4 = host(x8).astype(np.int32), host(x4e).astype(np.int32)
    assert (host(x4) == oracle.pack_nibbles(host(x4e))).all()
    assert np.abs(g8 - q8).max() <= 1 and np.abs(g4 - q4).max() <= 1
    frac = ((g8 != q8).sum() + (g4 != q4).sum()) / float(T * K)
    assert frac <= 1e-3, frac
    # The tensor core adds each 16-term partial product into the fp32 accumulator with a truncating
    # add: at most one ulp per instruction, K/16 instructions per coefficient, plus the final roundings.
    tol = K // 16 + 4
    assert _ulp_diff(host(s8), o8).max() <= tol and _ulp_diff(host(s4), o4).max() <= tol


def test_linear_with_online_projection_is_exact_given_its_own_codes(resq):
    T, K, N, r = 150, 1024, 520, 128
    X_bits = synth.f32_to_bf16_bits(synth.activations(T, K, "t4", seed=77))
    P_bits = synth.f32_to_bf16_bits(synth.kron_orthogonal_bf16(K))
    Wp = synth.projected_weights_direct(N, K, seed=78)
    pw = oracle.pack_weights(Wp, r)
    desc = resq.layer_desc(K, N, r)
    W = resq.resq_pack_weights(desc, dev(Wp))
    ws = resq.alloc_workspace(desc, T, True, True)
    X, P = bf16_to_dev(X_bits), bf16_to_dev(P_bits)
    K4 = K - r
    x8 = torch.empty((T, r), dtype=torch.int8, device="cuda")
    x4e = torch.empty((T, K4), dtype=torch.int8, device="cuda")
    s8 = torch.empty(T, dtype=torch.float32, device="cuda")
    s4 = torch.empty(T, dtype=torch.float32, device="cuda")
    resq.resq_project_quantize(X, P, r, x8, None, s8, s4, x4e, ws)
    y32 = torch.empty((T, N), dtype=torch.float32, device="cuda")
    resq.resq_linear(W, X, P, y32, ws)
    ybf = torch.empty((T, N), dtype=torch.bfloat16, device="cuda")
    resq.resq_linear(W, X, P, ybf, ws)
    assert resq.resq_device_status() == resq.OK
    acc8, acc4 = oracle.int_gemm(host(x8), pw.q8), oracle.int_gemm(host(x4e), pw.q4)
    e32, ebf = oracle.epilogue(acc8, acc4, host(s8), host(s4), pw.s8, pw.s4)
    res = oracle.LayerResult(None, host(x8), host(x4e), None, host(s8), host(s4), acc8, acc4, e32, ebf)
    check_output(res, pw, host(y32), bf16_bits_from_dev(ybf))
    # and the layer approximates the unquantized product X·P·W_proj^T (this P is a plain rotation, not a
    # PCA basis, so the error is that of rotation-only 4-bit quantization: a sanity bound, not parity)
    ref = (synth.bf16_bits_to_f32(X_bits).astype(np.float64) @ synth.bf16_bits_to_f32(P_bits).astype(np.float64)) @ Wp.astype(np.float64).T
    assert np.linalg.norm(host(y32) - ref) / np.linalg.norm(ref) < 0.35


@pytest.mark.parametrize("T,K", [(1, 512), (130, 1056), (300, 2048), (520, 4096)])
def test_projection_alone_against_fp64_sums(resq, T, K):
    """resq_project: every fp32 coefficient within the accumulation error of the fp64-summed oracle value
    (one truncating fp32 add per 16-term block: K/16 + 4 ulp of the sum of the term magnitudes)."""
    X_bits = synth.f32_to_bf16_bits(synth.activations(T, K, "t4", seed=700 + T))
    P_bits = synth.f32_to_bf16_bits(synth.kron_orthogonal_bf16(K, inner=32 if K % 128 else 128))
    C_ref = oracle.project(X_bits, P_bits)
    C = torch.full((T, K), float("nan"), dtype=torch.float32, device="cuda")
    resq.resq_project(bf16_to_dev(X_bits), bf16_to_dev(P_bits), C)
    assert resq.resq_device_status() == resq.OK
    Xf = np.abs(synth.bf16_bits_to_f32(X_bits).astype(np.float64))
    Pf = np.abs(synth.bf16_bits_to_f32(P_bits).astype(np.float64))
    bound = (K // 16 + 4) * 2.0 ** -24 * (Xf @ Pf) + 1e-30
    assert (np.abs(host(C).astype(np.float64) - C_ref.astype(np.float64)) <= bound).all()


@pytest.mark.parametrize("T,K", [(4096, 1280), (2200, 2304)])
def test_projection_with_split_last_round(resq, T, K):
    """More 256 x 256 tiles than CTA pairs with a thin last round (80 and 81 tiles on 74 pairs): with the scratch
    workspace those tiles are cut along K and summed in slice order.  Same bound as above plus one rounding per
    slice; two calls give identical bits (fixed summation order); without the workspace the result obeys the same
    bound."""
    X_bits = synth.f32_to_bf16_bits(synth.activations(T, K, "t4", seed=900 + K))
    P_bits = synth.f32_to_bf16_bits(synth.kron_orthogonal_bf16(K, inner=128))
    C_ref = oracle.project(X_bits, P_bits).astype(np.float64)
    Xd, Pd = bf16_to_dev(X_bits), bf16_to_dev(P_bits)
    ws = torch.empty(resq.resq_project_workspace_bytes(), dtype=torch.uint8, device="cuda")
    ws.fill_(0xFF)
    outs = []
    for w in (ws, ws, None):
        C = torch.full((T, K), float("nan"), dtype=torch.float32, device="cuda")
        resq.resq_project(Xd, Pd, C, w)
        assert resq.resq_device_status() == resq.OK
        outs.append(host(C))
    Xf = np.abs(synth.bf16_bits_to_f32(X_bits).astype(np.float64))
    Pf = np.abs(synth.bf16_bits_to_f32(P_bits).astype(np.float64))
    bound = (K // 16 + 20) * 2.0 ** -24 * (Xf @ Pf) + 1e-30
    for C in outs:
        assert (np.abs(C.astype(np.float64) - C_ref) <= bound).all()
    assert (outs[0].view(np.uint32) == outs[1].view(np.uint32)).all()
    assert (outs[0] != outs[2]).any()          # the split really changed the summation order somewhere


@pytest.mark.parametrize("T,K", [(1, 512), (5, 1056), (16, 2048), (17, 4096), (33, 2304), (48, 1280), (64, 4096),
                                 (3, 14336), (16, 14336)])
def test_projection_few_token_rows(resq, T, K):
    """Up to 64 token rows take the kernel with the operand roles exchanged (columns of P on the MMA's rows, tokens on
    its columns, rounded up to 16), every tile cut along K when the scratch workspace is there.  Same bound as the
    tile kernel's; rows the call does not own stay untouched; repeated calls give identical bits."""
    X_bits = synth.f32_to_bf16_bits(synth.activations(T, K, "t4", seed=1100 + T))
    P_bits = synth.f32_to_bf16_bits(synth.kron_orthogonal_bf16(K, inner=32 if K % 128 else 128))
    C_ref = oracle.project(X_bits, P_bits).astype(np.float64)
    Xd, Pd = bf16_to_dev(X_bits), bf16_to_dev(P_bits)
    ws = torch.empty(resq.resq_project_workspace_bytes(), dtype=torch.uint8, device="cuda")
    ws.fill_(0xFF)
    Xf = np.abs(synth.bf16_bits_to_f32(X_bits).astype(np.float64))
    Pf = np.abs(synth.bf16_bits_to_f32(P_bits).astype(np.float64))
    bound = (K // 16 + 20) * 2.0 ** -24 * (Xf @ Pf) + 1e-30
    outs = []
    for w in (ws, ws, None):
        buf = torch.full((T + 2, K), float("nan"), dtype=torch.float32, device="cuda")
        resq.resq_project(Xd, Pd, buf[1:T + 1], w)
        assert resq.resq_device_status() == resq.OK
        got = host(buf)
        assert np.isnan(got[0]).all() and np.isnan(got[T + 1]).all()
        assert (np.abs(got[1:T + 1].astype(np.float64) - C_ref) <= bound).all()
        outs.append(got[1:T + 1])
    assert (outs[0].view(np.uint32) == outs[1].view(np.uint32)).all()


@pytest.mark.parametrize("N,K,r,fp16", [(64, 512, 64, False), (4104, 1024, 128, False), (264, 2048, 256, True)])
def test_pack_weights_projected(resq, N, K, r, fp16):
    """Weight projection at pack time (Section 4.3): W_raw·U on the tensor cores, then Eq. 3.  Against the oracle's
    fp64-summed projection: codes within +-1 on at most 0.1 %, scales within the same ulp bound as the online
    activation path; the one-code-per-byte copy and the packed nibbles agree with each other bit for bit."""
    W_bits = synth.f32_to_bf16_bits(synth.weights(K, N, seed=77).T.copy())          # [N][K]: rows = output channels
    U_bits = synth.f32_to_bf16_bits(synth.kron_orthogonal_bf16(K, inner=128))
    pw = oracle.pack_weights(oracle.project(W_bits, U_bits), r, scale_fp16=fp16)
    desc = resq.layer_desc(K, N, r, resq.SCALE_FP16 if fp16 else resq.SCALE_FP32)
    W = resq.resq_pack_weights_projected(desc, bf16_to_dev(W_bits), bf16_to_dev(U_bits))
    assert resq.resq_device_status() == resq.OK
    g8, g4 = host(W.w8).astype(np.int32), host(W.w4_i8).astype(np.int32)
    assert (host(W.w4) == oracle.pack_nibbles(host(W.w4_i8))).all()
    assert np.abs(g8 - pw.q8).max() <= 1 and np.abs(g4 - pw.q4).max() <= 1
    frac = ((g8 != pw.q8).sum() + (g4 != pw.q4).sum()) / float(N * K)
    assert frac <= 1e-3, frac
    if fp16:
        d8 = np.abs(host(W.s_w8).view(np.int16).astype(np.int32) - pw.s8.astype(np.float16).view(np.int16).astype(np.int32))
        d4 = np.abs(host(W.s_w4).view(np.int16).astype(np.int32) - pw.s4.astype(np.float16).view(np.int16).astype(np.int32))
        assert d8.max() <= 1 and d4.max() <= 1
    else:
        tol = K // 16 + 4
        assert _ulp_diff(host(W.s_w8), pw.s8).max() <= tol and _ulp_diff(host(W.s_w4), pw.s4).max() <= tol
