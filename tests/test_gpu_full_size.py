"""Parity at the full sizes of the Llama-3.2-1B, Llama-3-8B and Llama-3-70B prefill configurations, in the launch configuration
the benchmark times (all token rows, whole layers, the tile kernels), checked on sampled token rows that the
oracle can afford: for those rows everything the layer produces is compared -- codes, scales, the fp32 output
of every output channel."""
import numpy as np
import pytest
import torch

import oracle
import synth
from tests.gpu_util import host
from tests.test_gpu_parity import check_output

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def resq():
    import paper_2412_14363_b200 as m
    return m


def _bits(t):
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def _sample_rows(T):
    return np.unique(np.array([0, 1, 127, 128, 255, 256, T // 2 - 1, T // 2, T - 257, T - 129, T - 2, T - 1]))


@pytest.mark.parametrize("T,K,N", [
    (2048, 2048, 16384),    # Llama-3.2-1B gate|up
    (2048, 2048, 3072),     # Llama-3.2-1B q|k|v (2048 + 2 x 512 output channels)
    (2048, 2048, 2048),     # Llama-3.2-1B o
    (4096, 4096, 28672),    # 8B gate|up: the widest layer of the benchmark
    (4096, 4096, 6144),     # 8B q|k|v
    (8192, 8192, 10240),    # 70B q|k|v (8192 + 2 x 1024 output channels)
    (8192, 8192, 28672),    # 70B gate (one of the two halves; both together are the same kernel, twice the tiles)
])
def test_folded_layer_full_size_sampled_rows(resq, T, K, N):
    r = K // 8
    dev = torch.device("cuda")
    X = synth.t_activations(T, K, dev, "t4", seed=21)
    Wp = synth.t_projected_weights_direct(N, K, dev, seed=22)
    desc = resq.layer_desc(K, N, r)
    W = resq.resq_pack_weights(desc, Wp, with_w4_i8=True)
    pw = oracle.pack_weights(Wp.cpu().numpy(), r)
    del Wp
    assert (host(W.w8) == pw.q8).all() and (host(W.w4) == pw.w4_packed).all()
    assert (host(W.s_w8).view(np.uint32) == pw.s8.view(np.uint32)).all()
    ws = resq.alloc_workspace(desc, T, False, True)
    Y = torch.empty((T, N), dtype=torch.float32, device=dev)
    resq.resq_linear(W, X, None, Y, ws)
    assert resq.resq_device_status() == resq.OK
    rows = _sample_rows(T)
    res = oracle.linear(_bits(X[torch.from_numpy(rows).to(dev)]), None, pw)
    check_output(res, pw, host(Y[torch.from_numpy(rows).to(dev)]))


@pytest.mark.parametrize("T,K,N", [(2048, 8192, 2048), (4096, 14336, 4096), (8192, 28672, 8192)])
def test_down_proj_full_size_sampled_rows(resq, T, K, N):
    """down_proj with the online projection at full size: the kernel's codes on the sampled rows lie within +-1 of
    the oracle's on <= 0.1 %, and its output is exact given its own codes."""
    r = K // 8
    K4 = K - r
    dev = torch.device("cuda")
    X = synth.t_activations(T, K, dev, "t4", seed=31)
    P = synth.t_kron_orthogonal_bf16(K, dev)
    Wp = synth.t_projected_weights_direct(N, K, dev, seed=32)
    desc = resq.layer_desc(K, N, r)
    W = resq.resq_pack_weights(desc, Wp, with_w4_i8=True)
    pw = oracle.pack_weights(Wp.cpu().numpy(), r)
    del Wp
    ws = resq.alloc_workspace(desc, T, True, True)
    x8 = torch.empty((T, r), dtype=torch.int8, device=dev)
    x4e = torch.empty((T, K4), dtype=torch.int8, device=dev)
    s8 = torch.empty(T, dtype=torch.float32, device=dev)
    s4 = torch.empty(T, dtype=torch.float32, device=dev)
    resq.resq_project_quantize(X, P, r, x8, None, s8, s4, x4e, ws)
    Y = torch.empty((T, N), dtype=torch.float32, device=dev)
    resq.resq_mixed_gemm(W, x8, None, s8, s4, Y, ws, x4_i8=x4e)
    assert resq.resq_device_status() == resq.OK
    rows = _sample_rows(T)[::3]
    idx = torch.from_numpy(rows).to(dev)
    C = oracle.project(_bits(X[idx]), _bits(P))
    q8, q4, o8, o4 = oracle.split_quantize(C, r)
    g8, g4 = host(x8[idx]), host(x4e[idx])
    assert np.abs(g8.astype(np.int32) - q8).max() <= 1 and np.abs(g4.astype(np.int32) - q4).max() <= 1
    assert ((g8 != q8).sum() + (g4 != q4).sum()) / float(rows.size * K) <= 1e-3
    gs8, gs4 = host(s8[idx]), host(s4[idx])
    acc8, acc4 = oracle.int_gemm(g8, pw.q8), oracle.int_gemm(g4, pw.q4)
    y32, ybf = oracle.epilogue(acc8, acc4, gs8, gs4, pw.s8, pw.s4)
    res = oracle.LayerResult(None, g8, g4, oracle.pack_nibbles(g4), gs8, gs4, acc8, acc4, y32, ybf)
    check_output(res, pw, host(Y[idx]))


def test_attention_full_size_sampled_heads():
    """The attention-block path at the benchmark's size (Llama-3-8B geometry: 32 query / 8 KV heads, 16 sequences x
    8192 cached positions, 184.5 MB of cache), cache filled through resq_kv_append as the benchmark does.  For two
    sampled sequences the oracle recomputes every cache byte (bit for bit) and single-query attention of sampled
    query heads (within 1e-3 of the value magnitude, as in the small tests)."""
    import paper_2412_14363_b200 as resq
    from oracle import kv as okv
    from paper_2412_14363_b200 import kv
    from tests import kv_util
    from tests.gpu_util import dev as to_dev

    B, S, Hq, Hkv, D = 16, 8192, 32, 8, 128
    device = torch.device("cuda")
    W_C = np.ascontiguousarray(synth.haar_orthogonal(D).T.astype(np.float32))
    wq, s_u = kv.resq_uc_quantize(to_dev(W_C))
    cache = kv.KvCache(B, Hkv, S)
    cache.data.fill_(0xFF)
    pos = torch.arange(S, dtype=torch.int32, device=device)
    sampled = (3, 15)
    kept = {}
    for b in range(B):
        k = synth.t_head_vectors(S, Hkv, D, device, stream=1000 + b, lead=1.0, scale=1.5)
        v = synth.t_head_vectors(S, Hkv, D, device, stream=2000 + b, lead=4.0, shift=0.2)
        kv.resq_kv_append(cache, k, v, torch.full((S,), b, dtype=torch.int32, device=device), pos, wq, s_u)
        if b in sampled:
            kept[b] = (synth.bf16_bits_to_f32(_bits(k)), synth.bf16_bits_to_f32(_bits(v)))
    lens = np.full(B, S, np.int32)
    lens[3] = S - 45                                    # a ragged last block for one of the sampled sequences
    q = synth.t_head_vectors(B, Hq, D, device, stream=3000, lead=1.0, scale=1.5)
    q16 = torch.empty((B, Hq, D), dtype=torch.float16, device=device)
    kv.resq_query_project(q, wq, s_u, q16)
    out = torch.empty((B, Hq, D), dtype=torch.float32, device=device)
    kv.resq_attention_decode(cache, q16, to_dev(lens), out, kv.attention_workspace(cache, Hq))
    assert resq.resq_device_status() == resq.OK
    image = host(cache.data).reshape(B, Hkv, S // 32, kv_util.BLOCK_BYTES)
    out_h, q16_h = host(out), host(q16)
    # the projected queries of the sampled sequences, bit for bit
    Yq, _, _ = okv.project_int8(synth.bf16_bits_to_f32(_bits(q)).reshape(-1, D), *okv.quantize_uc(W_C))
    assert (q16_h.view(np.uint16) == okv.query_fp16(Yq).reshape(B, Hq, D).view(np.uint16)).all()
    for b in sampled:
        kf, vf = kept[b]
        Yk, _, _ = okv.project_int8(kf.reshape(-1, D), *okv.quantize_uc(W_C))
        hk, hv = okv.kv_quantize(Yk), okv.kv_quantize(vf.reshape(-1, D))
        for h in (0, 5):                                # every cache byte of two KV heads
            blocks = image[b, h]
            for which, rec, (o8, o4, om) in (("k", hk, kv_util.OFF["k"]), ("v", hv, kv_util.OFF["v"])):
                rows = np.arange(S) * Hkv + h
                assert (blocks[:, o8:o8 + 512].reshape(S, 16) == rec.c8[rows]).all(), (which, b, h)
                assert (blocks[:, o4:o4 + 1792].reshape(S, 56) == rec.c4[rows]).all(), (which, b, h)
                assert (np.ascontiguousarray(blocks[:, om:om + 512]).view(np.uint32).reshape(S, 4)
                        == rec.meta[rows].view(np.uint32)).all(), (which, b, h)
        dk, dv = okv.kv_dequantize(hk).reshape(S, Hkv, D), okv.kv_dequantize(hv).reshape(S, Hkv, D)
        n = int(lens[b])
        for hq in (0, 7, 22, 31):                       # sampled query heads: KV heads 0, 1, 5, 7
            hk_i = hq // (Hq // Hkv)
            ref = okv.attention_decode(q16_h[b:b + 1, hq:hq + 1], [[dk[:, hk_i]]], [[dv[:, hk_i]]], [n], 1, 1)[0, 0]
            vmax = np.abs(dv[:n, hk_i]).max()
            assert np.abs(out_h[b, hq] - ref).max() <= 1e-3 * vmax, (b, hq)


def test_prefill_attention_full_size_sampled_rows():
    """Causal attention of new tokens at the benchmark's size and launch shapes (Llama-3-8B geometry, one sequence of
    8192 positions): the whole sequence in one call (2048 tiles) and its last 1024 tokens (256 tiles).  Sampled
    (token, query head) rows -- first and last rows of tiles, rows on both sides of a 64-position step boundary, the
    very first and last tokens -- against the oracle's fp64 definition on the oracle's own codes, within 1e-3 of the
    value magnitude; the two calls agree on the rows they share to the same bound."""
    import paper_2412_14363_b200 as resq
    from oracle import kv as okv
    from paper_2412_14363_b200 import kv
    from tests.gpu_util import dev as to_dev

    S, Hq, Hkv, D, Tc = 8192, 32, 8, 128, 1024
    device = torch.device("cuda")
    W_C = np.ascontiguousarray(synth.haar_orthogonal(D).T.astype(np.float32))
    wq, s_u = kv.resq_uc_quantize(to_dev(W_C))
    cache = kv.KvCache(2, Hkv, S)
    cache.data.fill_(0xFF)
    k = synth.t_head_vectors(S, Hkv, D, device, stream=5000, lead=1.0, scale=1.5)
    v = synth.t_head_vectors(S, Hkv, D, device, stream=5001, lead=4.0, shift=0.2)
    kv.resq_kv_append(cache, k, v, torch.ones(S, dtype=torch.int32, device=device),
                      torch.arange(S, dtype=torch.int32, device=device), wq, s_u)
    q = synth.t_head_vectors(S, Hq, D, device, stream=5002, lead=1.0, scale=1.5)
    q16 = torch.empty((S, Hq, D), dtype=torch.float16, device=device)
    kv.resq_query_project(q, wq, s_u, q16)
    out = torch.full((S, Hq, D), float("nan"), dtype=torch.float32, device=device)
    kv.resq_attention_prefill(cache, q16, 1, 0, out)
    tail = torch.full((Tc, Hq, D), float("nan"), dtype=torch.float32, device=device)
    kv.resq_attention_prefill(cache, q16[S - Tc:].contiguous(), 1, S - Tc, tail)
    assert resq.resq_device_status() == resq.OK
    out_h, tail_h, q16_h = host(out), host(tail), host(q16)
    assert np.isfinite(out_h).all() and np.isfinite(tail_h).all()
    kf, vf = synth.bf16_bits_to_f32(_bits(k)), synth.bf16_bits_to_f32(_bits(v))
    Yk, _, _ = okv.project_int8(kf.reshape(-1, D), *okv.quantize_uc(W_C))
    dk = okv.kv_dequantize(okv.kv_quantize(Yk)).reshape(S, Hkv, D)
    dv = okv.kv_dequantize(okv.kv_quantize(vf.reshape(-1, D))).reshape(S, Hkv, D)
    g = Hq // Hkv
    tokens = [0, 1, 31, 32, 63, 64, 65, 4095, 4096, 7168, 7199, 7200, 8160, 8191]
    for t in tokens:
        for hq in (0, 7, 22, 31):
            h = hq // g
            ref = okv.attention_queries(q16_h[t:t + 1, hq:hq + 1], [[dk[:, h]]], [[dv[:, h]]], [0], [t + 1], 1, 1)[0, 0]
            vmax = np.abs(dv[:t + 1, h]).max()
            assert np.abs(out_h[t, hq] - ref).max() <= 1e-3 * vmax, (t, hq)
            if t >= S - Tc:
                assert np.abs(tail_h[t - (S - Tc), hq] - ref).max() <= 1e-3 * vmax, (t, hq)
    vall = np.abs(dv).max()
    assert np.abs(out_h[S - Tc:] - tail_h).max() <= 1e-3 * vall
