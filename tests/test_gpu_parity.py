"""GPU parity: the CUDA path through the C ABI against the CPU oracle, element by element.

Integer work (codes, packed bytes, int32 accumulators) and fp32 scales must match bit for bit; the
fp32 epilogue within 1e-5 of the oracle's fp64-evaluated value, relative to the sum of the two
terms' magnitudes (the bare relative form is ill-posed when the terms cancel); the bf16 output must
be the nearest-even rounding of the kernel's own fp32 value and may differ from the oracle's bf16
only where the fp32 values straddle a rounding boundary.
"""
import numpy as np
import pytest
import torch

import oracle
import synth
from tests.cases import config1, config2_basis, synthetic_folded
from tests.gpu_util import bf16_bits_from_dev, bf16_to_dev, dev, host

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def resq():
    import paper_2412_14363_b200 as m
    return m


def _check_status(resq):
    st = resq.resq_device_status()
    assert st == resq.OK, resq.status_string(st)


def run_quantize(resq, C_bits, r, want_i8=True):
    T, K = C_bits.shape
    K4 = K - r
    X = bf16_to_dev(C_bits)
    x8 = torch.empty((T, r), dtype=torch.int8, device="cuda")
    x4 = torch.empty((T, K4 // 2), dtype=torch.uint8, device="cuda")
    x4e = torch.empty((T, K4), dtype=torch.int8, device="cuda") if want_i8 else None
    s8 = torch.empty(T, dtype=torch.float32, device="cuda")
    s4 = torch.empty(T, dtype=torch.float32, device="cuda")
    resq.resq_project_quantize(X, None, r, x8, x4, s8, s4, x4e)
    _check_status(resq)
    return x8, x4, s8, s4, x4e


def assert_quantize_matches(resq, C_bits, r):
    x8, x4, s8, s4, x4e = run_quantize(resq, C_bits, r)
    q8, q4, o8, o4 = oracle.split_quantize(oracle.bf16_bits_to_f32(C_bits), r)
    assert (host(s8).view(np.uint32) == o8.view(np.uint32)).all()
    assert (host(s4).view(np.uint32) == o4.view(np.uint32)).all()
    assert (host(x8) == q8).all()
    assert (host(x4) == oracle.pack_nibbles(q4)).all()
    assert (host(x4e) == q4).all()


@pytest.mark.parametrize("T,K,r", [(16, 512, 64), (1, 4096, 512), (17, 2048, 256), (129, 4096, 512),
                                   (5, 14336, 1792), (3, 28672, 3584), (2, 64, 32), (7, 18464, 2304)])
def test_split_quantize_bit_exact(resq, T, K, r):
    C = synth.activations(T, K, "t4", seed=100 + T)
    C[0, :r] = 0.0                      # a zero INT8 segment: scale 0, codes 0
    if T > 2:
        C[2, r:] = 0.0                  # a zero INT4 segment
    assert_quantize_matches(resq, synth.f32_to_bf16_bits(C), r)


def test_split_quantize_config1(resq):
    assert_quantize_matches(resq, config1().C_bits, 64)


def test_split_quantize_tie_rows(resq):
    """Rows whose scale is exactly 1 so that x/s hits .5 ties: both sides must round to even."""
    K, r = 64, 32
    C = np.zeros((2, K), np.float32)
    C[0, :r] = np.concatenate([[127.0], np.arange(0.5, 15.5, 1.0), np.zeros(r - 16)]).astype(np.float32)
    C[0, r:] = np.concatenate([[7.0, 0.5, 1.5, 2.5, 3.5, 4.5, 5.5, 6.5, -0.5, -1.5, -2.5, -6.5], np.zeros(K - r - 12)])
    C[1] = -C[0]
    assert_quantize_matches(resq, synth.f32_to_bf16_bits(C), r)


def test_split_quantize_power_of_two_scales(resq):
    """Rows whose absmax is 127 * 2^m / 7 * 2^m: the scales are powers of two, so bf16 inputs hit exact
    .5 ties by the thousand; a subnormal row and a huge row exercise the range ends of the reciprocal."""
    T, K, r = 40, 4096, 512
    rng = np.random.default_rng(5)
    C = synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(rng.uniform(-1, 1, (T, K)).astype(np.float32)))
    for t in range(T):
        m = float(2.0 ** (t % 9 - 4))
        half8 = (rng.integers(-126, 126, r) + 0.5) * m          # exact ties of the INT8 segment
        half4 = (rng.integers(-7, 7, K - r) + 0.5) * m
        C[t, :r] = np.where(rng.random(r) < 0.5, half8, C[t, :r] * 127 * m)
        C[t, r:] = np.where(rng.random(K - r) < 0.5, half4, C[t, r:] * 7 * m)
        C[t, 0], C[t, r] = 127 * m, -7 * m
    C[37] *= np.float32(2.0 ** -140)       # subnormal scales: 1/s overflows
    C[38] *= np.float32(2.0 ** 118)        # huge values
    C[39, r:] = 0.0
    bits = synth.f32_to_bf16_bits(C.astype(np.float32))
    assert_quantize_matches(resq, bits, r)


def test_pack_weights_near_ties(resq):
    """fp32 rows built so that x / s lands on, just below and just above k + 1/2 (a few ulp): the
    product-with-reciprocal shortcut must fall back to the division exactly where the two disagree."""
    N, K, r = 96, 2048, 256
    rng = np.random.default_rng(11)
    Wp = rng.standard_normal((N, K)).astype(np.float32)
    for n in range(N):
        for lo, hi, qmax in ((0, r, 127), (r, K, 7)):
            seg = Wp[n, lo:hi]
            a = np.float32(np.abs(seg).max() * (1.5 if n % 2 else 1.0))
            s = np.float32(a / np.float32(qmax))
            k = rng.integers(-qmax, qmax, seg.size).astype(np.float32) + np.float32(0.5)
            x = (k * s).astype(np.float32)
            ulps = rng.integers(-3, 4, seg.size).astype(np.int32)
            x = (x.view(np.int32) + ulps).view(np.float32)
            take = rng.random(seg.size) < 0.7
            seg[take] = x[take]
            seg[0] = a
    pw = oracle.pack_weights(Wp, r)
    desc = resq.layer_desc(K, N, r)
    W = resq.resq_pack_weights(desc, dev(Wp))
    _check_status(resq)
    assert (host(W.s_w8).view(np.uint32) == pw.s8.view(np.uint32)).all()
    assert (host(W.s_w4).view(np.uint32) == pw.s4.view(np.uint32)).all()
    assert (host(W.w8) == pw.q8).all()
    assert (host(W.w4_i8) == pw.q4).all()
    assert (host(W.w4) == pw.w4_packed).all()


@pytest.mark.parametrize("N,K,r,fp16", [(512, 512, 64, False), (512, 512, 64, True), (1024, 4096, 512, True),
                                        (264, 2048, 256, False), (64, 14336, 1792, True)])
def test_pack_weights_bit_exact(resq, N, K, r, fp16):
    Wp = synth.projected_weights_direct(N, K, seed=300 + N)
    Wp[1, :r] = 0.0
    pw = oracle.pack_weights(Wp, r, scale_fp16=fp16)
    desc = resq.layer_desc(K, N, r, resq.SCALE_FP16 if fp16 else resq.SCALE_FP32)
    W = resq.resq_pack_weights(desc, dev(Wp))
    _check_status(resq)
    assert (host(W.w8) == pw.q8).all()
    assert (host(W.w4) == pw.w4_packed).all()
    assert (host(W.w4_i8) == pw.q4).all()
    s8, s4 = host(W.s_w8.float()), host(W.s_w4.float())
    assert (s8.view(np.uint32) == pw.s8.view(np.uint32)).all()
    assert (s4.view(np.uint32) == pw.s4.view(np.uint32)).all()
    out = torch.empty((N, K - r), dtype=torch.int8, device="cuda")
    resq.resq_unpack_int4(W.w4, out)
    assert (host(out) == pw.q4).all()


def check_output(res, pw, y32_gpu, ybf_gpu_bits=None, y32_of_bf16_run=None):
    t8 = res.acc8.astype(np.float64) * res.s_x8[:, None].astype(np.float64) * pw.s8[None, :].astype(np.float64)
    t4 = res.acc4.astype(np.float64) * res.s_x4[:, None].astype(np.float64) * pw.s4[None, :].astype(np.float64)
    mag = np.abs(t8) + np.abs(t4)
    assert (np.abs(y32_gpu.astype(np.float64) - res.y32) <= 1e-5 * mag + 1e-37).all()
    if ybf_gpu_bits is not None:
        # bf16 mode rounds the kernel's own fp32 value to nearest even ...
        assert (ybf_gpu_bits == synth.f32_to_bf16_bits(y32_gpu)).all()
        # ... and equals the oracle's bf16 except where the two fp32 values straddle a boundary
        diff = ybf_gpu_bits != res.ybf
        if diff.any():
            a = synth.bf16_bits_to_f32(ybf_gpu_bits[diff]).astype(np.float64)
            b = synth.bf16_bits_to_f32(res.ybf[diff]).astype(np.float64)
            mid = 0.5 * (a + b)
            assert (np.abs(res.y32[diff] - mid) <= 1e-5 * mag[diff] + 1e-37).all()
            assert diff.mean() < 1e-3


def run_mixed_gemm(resq, pw, res, fp16=False, with_w4_i8=True, W=None):
    """Feeds the ORACLE's codes and scales to resq_mixed_gemm; returns (acc8, acc4, y32, ybf bits)."""
    T = res.x8.shape[0]
    desc = resq.layer_desc(pw.K, pw.N, pw.r, resq.SCALE_FP16 if fp16 else resq.SCALE_FP32)
    sdt = torch.float16 if fp16 else torch.float32
    W = resq.Weights(desc, dev(pw.q8), dev(pw.w4_packed), dev(pw.s8).to(sdt), dev(pw.s4).to(sdt),
                     dev(pw.q4) if with_w4_i8 else None)
    ws = resq.alloc_workspace(desc, T, False, with_w4_i8)
    x8, x4, s8, s4 = dev(res.x8), dev(res.x4_packed), dev(res.s_x8), dev(res.s_x4)
    y32 = torch.full((T, pw.N), float("nan"), dtype=torch.float32, device="cuda")
    a8 = torch.full((T, pw.N), -1, dtype=torch.int32, device="cuda")
    a4 = torch.full((T, pw.N), -1, dtype=torch.int32, device="cuda")
    resq.resq_mixed_gemm(W, x8, x4, s8, s4, y32, ws, a8, a4)  # packed activations in
    ybf = torch.zeros((T, pw.N), dtype=torch.bfloat16, device="cuda")
    resq.resq_mixed_gemm(W, x8, x4, s8, s4, ybf, ws)
    _check_status(resq)
    return host(a8), host(a4), host(y32), bf16_bits_from_dev(ybf)


def oracle_case(T, K, N, r, fp16=False, seed_shift=0):
    C_bits, Wp = synthetic_folded(T, K, N, r, seed_shift)
    pw = oracle.pack_weights(Wp, r, scale_fp16=fp16)
    return C_bits, Wp, pw, oracle.linear(C_bits, None, pw)


@pytest.mark.parametrize("T,K,N,r,fp16,w4i8", [
    (16, 512, 512, 64, False, True),      # tiny layer shape
    (17, 512, 264, 64, False, True),      # ragged rows and columns
    (129, 1024, 520, 128, True, True),    # several row tiles, partial column tile, fp16 weight scales
    (300, 2048, 512, 256, False, False),  # kernel expands the packed weights itself
    (128, 4096, 1024, 512, True, True),   # k/v projection shape of the 8B model
    (1, 512, 512, 64, False, True),
    (4, 4096, 256, 512, True, True),
    (2304, 1024, 2304, 128, False, True),   # 81 tiles on 74 CTA pairs: a second, thin round of the persistent grid
    (2200, 2048, 2560, 256, True, True),    # 90 tiles, ragged last row tile
    (2304, 1024, 2304, 0, False, True),     # the same with an empty INT8 segment
])
def test_mixed_gemm_bit_exact(resq, T, K, N, r, fp16, w4i8):
    _, _, pw, res = oracle_case(T, K, N, r, fp16, seed_shift=T)
    a8, a4, y32, ybf = run_mixed_gemm(resq, pw, res, fp16, w4i8)
    assert (a8 == res.acc8).all()
    assert (a4 == res.acc4).all()
    check_output(res, pw, y32, ybf)


def test_mixed_gemm_extreme_codes(resq):
    """All codes at the clip limits (-128 / -8): the accumulators reach their largest magnitudes."""
    T, K, N, r = 130, 1024, 256, 128
    K4 = K - r
    x8 = np.full((T, r), -128, np.int8)
    x4 = np.full((T, K4), -8, np.int8)
    x4[:, ::2] = 7
    pw = oracle.PackedWeights(K, N, r, np.full((N, r), -128, np.int8), np.full((N, K4), -8, np.int8), None,
                              np.full(N, 0.01, np.float32), np.full(N, 0.1, np.float32))
    pw.w4_packed = oracle.pack_nibbles(pw.q4)
    acc8, acc4 = oracle.int_gemm(x8, pw.q8), oracle.int_gemm(x4, pw.q4)
    sx8, sx4 = np.full(T, 0.5, np.float32), np.full(T, 2.0, np.float32)
    y32, ybf = oracle.epilogue(acc8, acc4, sx8, sx4, pw.s8, pw.s4)
    res = oracle.LayerResult(None, x8, x4, oracle.pack_nibbles(x4), sx8, sx4, acc8, acc4, y32, ybf)
    a8, a4, y, yb = run_mixed_gemm(resq, pw, res)
    assert (a8 == acc8).all() and (a4 == acc4).all()
    check_output(res, pw, y, yb)


def test_mixed_gemm_repeatable(resq):
    """Integer sums do not depend on order, so two runs must agree bit for bit (any difference is a race)."""
    _, _, pw, res = oracle_case(257, 1024, 768, 128, seed_shift=9)
    first = run_mixed_gemm(resq, pw, res)
    second = run_mixed_gemm(resq, pw, res)
    for a, b in zip(first, second):
        assert (a == b).all()


@pytest.mark.parametrize("T", [16, 200])
def test_linear_config1_end_to_end(resq, T):
    """Whole layer through resq_linear on the PCA + rotation case (folded projection)."""
    c = config1()
    C_bits = c.C_bits if T == 16 else synth.f32_to_bf16_bits(
        (synth.activations(T, c.K, "normal", seed=55).astype(np.float64) @ c.U).astype(np.float32))
    pw = oracle.pack_weights(c.W_proj, c.r)
    res = oracle.linear(C_bits, None, pw)
    desc = resq.layer_desc(c.K, c.N, c.r)
    W = resq.resq_pack_weights(desc, dev(c.W_proj))
    ws = resq.alloc_workspace(desc, T, False, True)
    y32 = torch.empty((T, c.N), dtype=torch.float32, device="cuda")
    resq.resq_linear(W, bf16_to_dev(C_bits), None, y32, ws)
    ybf = torch.empty((T, c.N), dtype=torch.bfloat16, device="cuda")
    resq.resq_linear(W, bf16_to_dev(C_bits), None, ybf, ws)
    _check_status(resq)
    check_output(res, pw, host(y32), bf16_bits_from_dev(ybf))


def test_linear_d2048_pca_basis_end_to_end(resq):
    """Whole layer on the PCA + rotation basis built at d = 2048 (the input width of the Llama-3.2-1B-shaped
    configuration): weights projected by the oracle's U, coefficients bf16(X·U) as a folded projection delivers them."""
    c = config2_basis()
    pw = oracle.pack_weights(c.W_proj, c.r)
    res = oracle.linear(c.C_bits, None, pw)
    desc = resq.layer_desc(c.K, c.N, c.r)
    W = resq.resq_pack_weights(desc, dev(c.W_proj))
    assert (host(W.w8) == pw.q8).all() and (host(W.w4) == pw.w4_packed).all()
    ws = resq.alloc_workspace(desc, c.T, False, True)
    y32 = torch.empty((c.T, c.N), dtype=torch.float32, device="cuda")
    resq.resq_linear(W, bf16_to_dev(c.C_bits), None, y32, ws)
    ybf = torch.empty((c.T, c.N), dtype=torch.bfloat16, device="cuda")
    resq.resq_linear(W, bf16_to_dev(c.C_bits), None, ybf, ws)
    _check_status(resq)
    check_output(res, pw, host(y32), bf16_bits_from_dev(ybf))
    # the quantized layer tracks the unquantized product (a sanity bound on the whole chain, not parity)
    ref = c.X.astype(np.float64) @ c.W.astype(np.float64)
    assert np.linalg.norm(host(y32) - ref) / np.linalg.norm(ref) < 0.25


@pytest.mark.parametrize("T,K,N,r,fp16", [
    (1280, 8192, 3840, 1024, False),   # 75 tiles on 74 CTA pairs: one tile in the last round
    (1250, 8192, 3832, 1024, True),    # the same with ragged rows and columns
    (1280, 8192, 3840, 6144, False),   # an INT8 segment three times as long as the INT4 one
    (1280, 8192, 3840, 0, False),      # uniform INT4 over 64 K blocks
    (2304, 8192, 2304, 1024, False),   # 81 tiles: seven in the last round
])
def test_mixed_gemm_long_reduction_thin_last_round(resq, T, K, N, r, fp16):
    """Reductions of 64 K blocks with a thin last round of the persistent grid (the accumulators reach their
    largest magnitudes of the parity suite, the ring wraps ten times per tile): both accumulators bit for bit on
    the rows of the last tiles and on sampled rows elsewhere; two runs agree bit for bit."""
    C_bits, Wp = synthetic_folded(T, K, N, r, seed_shift=300 + (r // 1024))
    pw = oracle.pack_weights(Wp, r, scale_fp16=fp16)
    q8, q4, s8, s4 = oracle.split_quantize(oracle.bf16_bits_to_f32(C_bits), r)
    desc = resq.layer_desc(K, N, r, resq.SCALE_FP16 if fp16 else resq.SCALE_FP32)
    sdt = torch.float16 if fp16 else torch.float32
    W = resq.Weights(desc, dev(pw.q8), dev(pw.w4_packed), dev(pw.s8).to(sdt), dev(pw.s4).to(sdt), dev(pw.q4))
    ws = resq.alloc_workspace(desc, T, False, True)
    ws.fill_(0x5A)
    x8, x4e, sx8, sx4 = dev(q8), dev(q4), dev(s8), dev(s4)
    outs = []
    for _ in range(2):
        y32 = torch.full((T, N), float("nan"), dtype=torch.float32, device="cuda")
        a8 = torch.full((T, N), -1, dtype=torch.int32, device="cuda")
        a4 = torch.full((T, N), -1, dtype=torch.int32, device="cuda")
        resq.resq_mixed_gemm(W, x8 if r else None, None, sx8, sx4, y32, ws, a8, a4, x4_i8=x4e)
        _check_status(resq)
        outs.append((host(a8), host(a4), host(y32)))
    for a, b in zip(outs[0], outs[1]):
        assert (a.view(np.uint32) == b.view(np.uint32)).all()
    rows = np.unique(np.concatenate([np.arange(max(0, T - 256), T), np.arange(0, T, 97), [255, 256, 1023, 1024]]))
    rows = rows[rows < T]
    acc8 = oracle.int_gemm(q8[rows], pw.q8) if r else np.zeros((rows.size, N), np.int32)
    acc4 = oracle.int_gemm(q4[rows], pw.q4)
    assert (outs[0][0][rows] == acc8).all()
    assert (outs[0][1][rows] == acc4).all()
    y_ref, ybf = oracle.epilogue(acc8, acc4, s8[rows], s4[rows], pw.s8, pw.s4)
    res = oracle.LayerResult(None, q8[rows], q4[rows], None, s8[rows], s4[rows], acc8, acc4, y_ref, ybf)
    check_output(res, pw, outs[0][2][rows])
