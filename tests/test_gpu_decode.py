"""GPU parity of the few-token (T <= 16) weight-streaming kernel: int32 accumulators bit-exact for every
K split, fp32 epilogue within tolerance, packed canonical weights with fp16 scales (the decode config)."""
import numpy as np
import pytest
import torch

import oracle
import synth
from tests.gpu_util import bf16_bits_from_dev, bf16_to_dev, dev, host
from tests.test_gpu_parity import check_output, oracle_case, run_mixed_gemm

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def resq():
    import paper_2412_14363_b200 as m
    return m


@pytest.mark.parametrize("T,K,N,r,fp16", [
    (1, 4096, 4096, 512, True),     # o_proj shape, one token (K split over a cluster of 8)
    (4, 4096, 1024, 512, True),
    (16, 4096, 4096, 512, True),
    (9, 2048, 264, 256, False),     # ragged channel block, second token tile partly filled
    (8, 512, 512, 64, False),       # r < one 64-byte step
    (16, 14336, 128, 1792, True),   # down_proj reduction length, few channels
    (3, 1056, 72, 96, False),       # segment lengths that are not multiples of a step
    (16, 4096, 28672, 512, True),   # gate|up: many units per CTA
    (16, 14336, 4096, 1792, True),  # down_proj: INT4 rows of 6272 bytes span four ring stages
    (16, 28672, 64, 3584, False),   # activations too large to stage whole: the cluster split-K kernel runs
    (5, 28672, 64, 3584, False),    # ... while 8 token rows of the same shape still fit
    (16, 28672, 64, 0, False),      # uniform INT4 at that width: no INT8 segment for the split-K kernel, two launches of 8 tokens
    (11, 28672, 72, 0, False),      # ... 8 + 3 tokens, ragged channel block
    (2, 4096, 8, 512, False),       # a single unit
])
def test_decode_bit_exact(resq, T, K, N, r, fp16):
    _, _, pw, res = oracle_case(T, K, N, r, fp16, seed_shift=50 + T)
    a8, a4, y32, ybf = run_mixed_gemm(resq, pw, res, fp16, with_w4_i8=False)
    assert (a8 == res.acc8).all()
    assert (a4 == res.acc4).all()
    check_output(res, pw, y32, ybf)


def test_decode_extreme_codes(resq):
    T, K, N, r = 16, 2048, 192, 256
    K4 = K - r
    x8 = np.full((T, r), -128, np.int8)
    x4 = np.full((T, K4), -8, np.int8)
    x4[:, 1::2] = 7
    q4 = np.full((N, K4), -8, np.int8)
    q4[::2, ::3] = 7
    pw = oracle.PackedWeights(K, N, r, np.full((N, r), -128, np.int8), q4, oracle.pack_nibbles(q4),
                              np.full(N, 0.01, np.float32), np.full(N, 0.1, np.float32))
    acc8, acc4 = oracle.int_gemm(x8, pw.q8), oracle.int_gemm(x4, pw.q4)
    sx8, sx4 = np.full(T, 0.5, np.float32), np.full(T, 2.0, np.float32)
    y32, ybf = oracle.epilogue(acc8, acc4, sx8, sx4, pw.s8, pw.s4)
    res = oracle.LayerResult(None, x8, x4, oracle.pack_nibbles(x4), sx8, sx4, acc8, acc4, y32, ybf)
    a8, a4, y, yb = run_mixed_gemm(resq, pw, res, with_w4_i8=False)
    assert (a8 == acc8).all() and (a4 == acc4).all()
    check_output(res, pw, y, yb)


@pytest.mark.parametrize("T", [1, 16])
def test_decode_linear_end_to_end(resq, T):
    """resq_linear for few tokens: quantize kernel + streaming kernel, packed weights only."""
    K, N, r = 4096, 1024, 512
    C_bits, Wp, _, _ = oracle_case(T, K, N, r, True, seed_shift=70 + T)
    pw = oracle.pack_weights(Wp, r, scale_fp16=True)
    res = oracle.linear(C_bits, None, pw)
    desc = resq.layer_desc(K, N, r, resq.SCALE_FP16)
    W = resq.resq_pack_weights(desc, dev(Wp), with_w4_i8=False)
    ws = resq.alloc_workspace(desc, T, False, False)
    y32 = torch.empty((T, N), dtype=torch.float32, device="cuda")
    resq.resq_linear(W, bf16_to_dev(C_bits), None, y32, ws)
    ybf = torch.empty((T, N), dtype=torch.bfloat16, device="cuda")
    resq.resq_linear(W, bf16_to_dev(C_bits), None, ybf, ws)
    assert resq.resq_device_status() == resq.OK
    check_output(res, pw, host(y32), bf16_bits_from_dev(ybf))


@pytest.mark.parametrize("T,K,N,r,fp16", [
    (1, 4096, 4096, 512, True), (4, 4096, 1024, 512, True), (16, 4096, 4096, 512, True),
    (9, 2048, 264, 256, False),     # second token tile partly filled
    (8, 512, 512, 64, False), (3, 1056, 72, 96, False),
    (16, 8192, 256, 1024, True),
    (5, 14336, 128, 1792, True), (16, 4096, 28672, 512, True),
    (7, 2048, 64, 0, False),        # uniform INT4: no INT8 segment
])
def test_decode_linear_shapes_and_zero_rows(resq, T, K, N, r, fp16):
    """resq_linear for up to 16 tokens without P (row quantizer, then the streaming kernel) over the shapes of the
    streaming kernel's own cases: the output bits of the oracle's layer; a zero row and a row whose INT8 segment is
    zero give scale 0 and codes 0; the split calls give the same bits."""
    C_bits, Wp, _, _ = oracle_case(T, K, N, r, fp16, seed_shift=170 + T)
    C_bits = C_bits.copy()
    if T >= 3:
        C_bits[1, :] = 0
        C_bits[2, :r] = 0
    pw = oracle.pack_weights(Wp, r, scale_fp16=fp16)
    res = oracle.linear(C_bits, None, pw)
    desc = resq.layer_desc(K, N, r, resq.SCALE_FP16 if fp16 else resq.SCALE_FP32)
    W = resq.resq_pack_weights(desc, dev(Wp), with_w4_i8=False)
    ws = resq.alloc_workspace(desc, T, False, False)
    y32 = torch.full((T, N), float("nan"), dtype=torch.float32, device="cuda")
    resq.resq_linear(W, bf16_to_dev(C_bits), None, y32, ws)
    ybf = torch.empty((T, N), dtype=torch.bfloat16, device="cuda")
    resq.resq_linear(W, bf16_to_dev(C_bits), None, ybf, ws)
    assert resq.resq_device_status() == resq.OK
    check_output(res, pw, host(y32), bf16_bits_from_dev(ybf))
    # the same through the split entry points
    K4 = K - r
    x8 = torch.empty((T, max(r, 1)), dtype=torch.int8, device="cuda")
    x4 = torch.empty((T, K4 // 2), dtype=torch.uint8, device="cuda")
    s8 = torch.empty(T, dtype=torch.float32, device="cuda")
    s4 = torch.empty(T, dtype=torch.float32, device="cuda")
    resq.resq_project_quantize(bf16_to_dev(C_bits), None, r, x8, x4, s8, s4, None, None)
    y2 = torch.empty((T, N), dtype=torch.float32, device="cuda")
    resq.resq_mixed_gemm(W, x8, x4, s8, s4, y2, ws)
    assert resq.resq_device_status() == resq.OK
    assert (host(y2).view(np.uint32) == host(y32).view(np.uint32)).all()


def test_decode_early_weights_back_to_back(resq):
    """With the early-weights option each launch may start while the previous one still runs and
    prefetches its weights before waiting for it; a chain of launches over different layers must give
    exactly what the same launches give one by one."""
    cases = [oracle_case(T, 4096, N, 512, True, seed_shift=90 + i) for i, (T, N) in enumerate([(16, 1024), (3, 2048), (16, 512)])]
    packs = []
    for _, _, pw, res in cases:
        desc = resq.layer_desc(pw.K, pw.N, pw.r, resq.SCALE_FP16)
        W = resq.Weights(desc, dev(pw.q8), dev(pw.w4_packed), dev(pw.s8).half(), dev(pw.s4).half(), None)
        T = res.x8.shape[0]
        packs.append((W, dev(res.x8), dev(res.x4_packed), dev(res.s_x8), dev(res.s_x4),
                      torch.zeros((T, pw.N), dtype=torch.float32, device="cuda"),
                      torch.full((T, pw.N), -1, dtype=torch.int32, device="cuda"),
                      torch.full((T, pw.N), -1, dtype=torch.int32, device="cuda"),
                      resq.alloc_workspace(desc, T, False, False)))
    torch.cuda.synchronize()
    resq.resq_set_option(resq.OPT_DECODE_EARLY_WEIGHTS, 1)
    try:
        for _ in range(3):
            for W, x8, x4, s8, s4, y, a8, a4, ws in packs:
                resq.resq_mixed_gemm(W, x8, x4, s8, s4, y, ws, a8, a4)
    finally:
        resq.resq_set_option(resq.OPT_DECODE_EARLY_WEIGHTS, 0)
    assert resq.resq_device_status() == resq.OK
    for (_, _, pw, res), (W, x8, x4, s8, s4, y, a8, a4, ws) in zip(cases, packs):
        assert (host(a8) == res.acc8).all() and (host(a4) == res.acc4).all()
        check_output(res, pw, host(y))


@pytest.mark.parametrize("T,K,N,r", [(1, 14336, 4096, 1792), (4, 14336, 4096, 1792), (16, 14336, 512, 1792),
                                     (16, 2304, 264, 288), (3, 2304, 72, 0)])
def test_decode_linear_with_online_projection(resq, T, K, N, r):
    """resq_linear with P given for up to 16 tokens -- the down_proj of a generation step through the public call:
    few-token projection kernel, slice reduction, row quantizer, streaming kernel.  The codes the path forms lie
    within +-1 of the oracle's (fp64-summed projection) on at most 0.1 % of the elements, the scales within the
    accumulation bound, and the layer output is exact given those codes."""
    X_bits = synth.f32_to_bf16_bits(synth.activations(T, K, "t4", seed=1300 + T))
    P_bits = synth.f32_to_bf16_bits(synth.kron_orthogonal_bf16(K, inner=128 if K % 128 == 0 else 32))
    Wp = synth.projected_weights_direct(N, K, seed=1301)
    pw = oracle.pack_weights(Wp, r, scale_fp16=True)
    desc = resq.layer_desc(K, N, r, resq.SCALE_FP16)
    W = resq.resq_pack_weights(desc, dev(Wp), with_w4_i8=False)
    ws = resq.alloc_workspace(desc, T, True, False)
    X, P = bf16_to_dev(X_bits), bf16_to_dev(P_bits)
    K4 = K - r
    x8 = torch.empty((T, r), dtype=torch.int8, device="cuda") if r else None
    x4 = torch.empty((T, K4 // 2), dtype=torch.uint8, device="cuda")
    s8 = torch.full((T,), -1.0, dtype=torch.float32, device="cuda")
    s4 = torch.full((T,), -1.0, dtype=torch.float32, device="cuda")
    resq.resq_project_quantize(X, P, r, x8, x4, s8, s4, None, ws)       # the codes the layer call forms inside
    y32 = torch.full((T, N), float("nan"), dtype=torch.float32, device="cuda")
    resq.resq_linear(W, X, P, y32, ws)
    ybf = torch.empty((T, N), dtype=torch.bfloat16, device="cuda")
    resq.resq_linear(W, X, P, ybf, ws)
    assert resq.resq_device_status() == resq.OK
    # against the oracle's projection + quantizer
    C = oracle.project(X_bits, P_bits)
    q8, q4, o8, o4 = oracle.split_quantize(C, r)
    g4 = oracle.unpack_nibbles(host(x4)).astype(np.int32)
    g8 = host(x8).astype(np.int32) if r else np.zeros((T, 0), np.int32)
    assert np.abs(g4 - q4).max() <= 1 and (r == 0 or np.abs(g8 - q8).max() <= 1)
    assert ((g8 != q8).sum() + (g4 != q4).sum()) / float(T * K) <= 1e-3
    ulp = lambda a, b: np.abs(a.view(np.int32).astype(np.int64) - b.view(np.int32).astype(np.int64))
    tol = K // 16 + 4
    assert ulp(host(s4), o4).max() <= tol and (r == 0 or ulp(host(s8), o8).max() <= tol)
    # exact given the path's own codes
    gs8, gs4 = host(s8), host(s4)
    acc8 = oracle.int_gemm(g8.astype(np.int8), pw.q8) if r else np.zeros((T, N), np.int32)
    acc4 = oracle.int_gemm(g4.astype(np.int8), pw.q4)
    e32, ebf = oracle.epilogue(acc8, acc4, gs8, gs4, pw.s8, pw.s4)
    res = oracle.LayerResult(None, g8.astype(np.int8), g4.astype(np.int8), None, gs8, gs4, acc8, acc4, e32, ebf)
    check_output(res, pw, host(y32), bf16_bits_from_dev(ybf))


def test_decode_layers_replay_from_a_cuda_graph(resq):
    """The library allocates nothing and never synchronises, so its calls can be recorded into a CUDA graph (the way a
    generation loop removes its launch overhead): two layers of a step -- one folded, one with the online projection --
    are captured once, the inputs are overwritten in place, and the replay gives, bit for bit, what direct calls give
    on the new inputs (and differs from the captured run's outputs)."""
    T, K, N, r = 4, 2304, 264, 288
    desc = resq.layer_desc(K, N, r, resq.SCALE_FP16)
    Wp = synth.projected_weights_direct(N, K, seed=1401)
    W = resq.resq_pack_weights(desc, dev(Wp), with_w4_i8=False)
    P = bf16_to_dev(synth.f32_to_bf16_bits(synth.kron_orthogonal_bf16(K, inner=32)))
    ws_f, ws_p = resq.alloc_workspace(desc, T, False, False), resq.alloc_workspace(desc, T, True, False)
    X = bf16_to_dev(synth.f32_to_bf16_bits(synth.activations(T, K, "t4", seed=1402)))
    X2 = bf16_to_dev(synth.f32_to_bf16_bits(synth.activations(T, K, "t4", seed=1403)))
    y_f = torch.zeros((T, N), dtype=torch.float32, device="cuda")
    y_p = torch.zeros((T, N), dtype=torch.float32, device="cuda")
    resq.resq_set_option(resq.OPT_DECODE_EARLY_WEIGHTS, 1)
    try:
        for _ in range(2):                       # first calls set function attributes: not inside a capture
            resq.resq_linear(W, X, None, y_f, ws_f)
            resq.resq_linear(W, X, P, y_p, ws_p)
        torch.cuda.synchronize()
        first = host(y_f).copy(), host(y_p).copy()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            resq.resq_linear(W, X, None, y_f, ws_f)
            resq.resq_linear(W, X, P, y_p, ws_p)
        X.copy_(X2)
        y_f.fill_(float("nan"))
        y_p.fill_(float("nan"))
        g.replay()
        torch.cuda.synchronize()
        got = host(y_f).copy(), host(y_p).copy()
        resq.resq_linear(W, X2, None, y_f, ws_f)
        resq.resq_linear(W, X2, P, y_p, ws_p)
        assert resq.resq_device_status() == resq.OK
        want = host(y_f), host(y_p)
    finally:
        resq.resq_set_option(resq.OPT_DECODE_EARLY_WEIGHTS, 0)
    for a, b, c in zip(got, want, first):
        assert np.isfinite(a).all() and (a.view(np.uint32) == b.view(np.uint32)).all()
        assert (a != c).any()
