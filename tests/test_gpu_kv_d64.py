"""GPU parity of the attention-block path at d_head = 64 (the Llama-3.2-1B head width: 8 coefficients in 8 bits, 56
in 4; Section 4.3, Eq. 8; Section 5.1) through the C ABI against the CPU oracle: U_C codes, the projected
half-precision query and every cache byte bit for bit; attention (single-query, many-query and the causal run of new
tokens) within 1e-4 of the largest dequantized value magnitude -- at this width every step after the integer product
is fp32, so only summation order and the exponential's last bits separate the two sides."""
import numpy as np
import pytest
import torch

import synth
from oracle import kv as okv
from tests.gpu_util import bf16_to_dev, dev, host

pytestmark = pytest.mark.gpu
D, R8, B4 = 64, 8, 28
HALF, BLOCK_BYTES = 32 * (R8 + B4 + 16), 2 * 32 * (R8 + B4 + 16)


@pytest.fixture(scope="module")
def resq():
    import paper_2412_14363_b200 as m
    return m


@pytest.fixture(scope="module")
def kv():
    from paper_2412_14363_b200 import kv as m
    return m


@pytest.fixture(scope="module")
def uc(kv):
    W_C = np.ascontiguousarray(synth.haar_orthogonal(D).T.astype(np.float32))
    wq, s_u = kv.resq_uc_quantize(dev(W_C))
    return W_C, wq, s_u


def _record(image, which, b, h, pos):
    """(c8 [8], c4 [28], meta fp32 [4]) of one head vector from a cache image [n_seqs][H][blocks][BLOCK_BYTES]."""
    blk, p = image[b, h, pos // 32], pos % 32
    o = 0 if which == "k" else HALF
    return (blk[o + R8 * p: o + R8 * p + R8], blk[o + 32 * R8 + B4 * p: o + 32 * R8 + B4 * p + B4],
            blk[o + 32 * (R8 + B4) + 16 * p: o + 32 * (R8 + B4) + 16 * p + 16].copy().view(np.float32))


def _oracle_records(k, v, W_C):
    Yk, _, _ = okv.project_int8(k.reshape(-1, D), *okv.quantize_uc(W_C))
    return okv.kv_quantize(Yk), okv.kv_quantize(v.reshape(-1, D))


def test_uc_quantize_and_query_project_bit_exact(resq, kv, uc):
    W_C, wq, s_u = uc
    owq, os_u = okv.quantize_uc(W_C)
    assert (host(wq) == owq).all() and (host(s_u).view(np.uint32) == os_u.view(np.uint32)).all()
    T, H = 37, 32
    q = synth.head_vectors(T, H, D, stream=910, lead=1.0, scale=3.0)
    q[0, 0, :] = 0.0
    q_out = torch.empty((T, H, D), dtype=torch.float16, device="cuda")
    kv.resq_query_project(bf16_to_dev(synth.f32_to_bf16_bits(q)), wq, s_u, q_out)
    assert resq.resq_device_status() == resq.OK
    Y, _, _ = okv.project_int8(q.reshape(-1, D), owq, os_u)
    assert (host(q_out).view(np.uint16) == okv.query_fp16(Y).reshape(T, H, D).view(np.uint16)).all()


@pytest.mark.parametrize("T,H", [(70, 8), (5, 2)])
def test_kv_append_bit_exact(resq, kv, uc, T, H):
    W_C, wq, s_u = uc
    k = synth.head_vectors(T, H, D, stream=920 + T, lead=1.0, scale=2.0)
    v = synth.head_vectors(T, H, D, stream=940 + T, lead=4.0, shift=0.5)
    v[1, 0, :R8] = v[1, 0, 0]                  # a constant 8-bit segment: s = 0, codes 0
    cache = kv.KvCache(2, H, 128, d_head=D)
    assert cache.nbytes == 2 * H * 4 * BLOCK_BYTES
    cache.data.fill_(0xEE)
    seq_ids = np.ones(T, np.int32)
    positions = np.arange(3, 3 + T, dtype=np.int32)
    seq_ids[-1], positions[-1] = 5, 0          # out of range: skipped and reported
    kv.resq_kv_append(cache, bf16_to_dev(synth.f32_to_bf16_bits(k)), bf16_to_dev(synth.f32_to_bf16_bits(v)),
                      dev(seq_ids), dev(positions), wq, s_u)
    assert resq.resq_device_status() == kv.ERR_INDEX
    image = host(cache.data).reshape(2, H, 4, BLOCK_BYTES)
    hk, hv = _oracle_records(k, v, W_C)
    for t in range(T - 1):
        for h in range(H):
            row = t * H + h
            for which, rec in (("k", hk), ("v", hv)):
                c8, c4, meta = _record(image, which, 1, h, positions[t])
                assert (c8 == rec.c8[row]).all() and (c4 == rec.c4[row]).all(), (which, t, h)
                assert (meta.view(np.uint32) == rec.meta[row].view(np.uint32)).all(), (which, t, h)
    assert (image[0] == 0xEE).all()


def test_attention_three_forms_against_the_oracle(resq, kv, uc):
    """Llama-3.2-1B head geometry (32 query / 8 KV heads x 64): single-query over two sequences, many-query with
    scattered prefixes, and the causal run of new tokens, each against the oracle's fp64 definition; the fused
    project-and-append call fills one of the sequences."""
    W_C, wq, s_u = uc
    Hq, Hkv, S0, S1 = 32, 8, 150, 41
    cache = kv.KvCache(2, Hkv, 160, d_head=D)
    cache.data.fill_(0xFF)
    K_hat, V_hat = [None, None], [None, None]
    for b, n in ((0, S0), (1, S1)):
        k = synth.head_vectors(n, Hkv, D, stream=950 + b, lead=1.0, scale=1.5)
        v = synth.head_vectors(n, Hkv, D, stream=960 + b, lead=4.0, shift=0.3)
        args = (bf16_to_dev(synth.f32_to_bf16_bits(k)), bf16_to_dev(synth.f32_to_bf16_bits(v)), dev(np.full(n, b, np.int32)),
                dev(np.arange(n, dtype=np.int32)), wq, s_u)
        if b == 0:
            kv.resq_kv_append(cache, *args)
        else:
            qd = synth.head_vectors(n, Hq, D, stream=969, lead=1.0)
            qo = torch.empty((n, Hq, D), dtype=torch.float16, device="cuda")
            kv.resq_qkv_project_append(cache, bf16_to_dev(synth.f32_to_bf16_bits(qd)), qo, *args)
        hk, hv = _oracle_records(k, v, W_C)
        dk, dv = okv.kv_dequantize(hk).reshape(n, Hkv, D), okv.kv_dequantize(hv).reshape(n, Hkv, D)
        K_hat[b], V_hat[b] = [dk[:, h] for h in range(Hkv)], [dv[:, h] for h in range(Hkv)]
    vmax = max(np.abs(v).max() for b in range(2) for v in V_hat[b])
    T = 60
    q = synth.head_vectors(T, Hq, D, stream=970, lead=1.0, scale=1.5)
    q16 = torch.empty((T, Hq, D), dtype=torch.float16, device="cuda")
    kv.resq_query_project(bf16_to_dev(synth.f32_to_bf16_bits(q)), wq, s_u, q16)
    hq16 = host(q16)
    # causal run: the last T tokens of sequence 0
    out = torch.full((T, Hq, D), float("nan"), dtype=torch.float32, device="cuda")
    kv.resq_attention_prefill(cache, q16, 0, S0 - T, out)
    ref = okv.attention_queries(hq16, K_hat, V_hat, np.zeros(T, np.int32), np.arange(S0 - T + 1, S0 + 1), Hq, Hkv)
    assert np.abs(host(out) - ref).max() <= 1e-4 * vmax
    # many-query: scattered (sequence, prefix) pairs, one empty
    q_seq = (np.arange(T) % 2).astype(np.int32)
    q_len = np.where(q_seq == 0, (np.arange(T) * 7) % (S0 + 1), (np.arange(T) * 5) % (S1 + 1)).astype(np.int32)
    q_len[3] = 0
    kv.resq_attention_queries(cache, q16, dev(q_seq), dev(q_len), out)
    ref = okv.attention_queries(hq16, K_hat, V_hat, q_seq, q_len, Hq, Hkv)
    got = host(out)
    assert np.abs(got - ref).max() <= 1e-4 * vmax and (got[3] == 0).all()
    # single-query: one row per sequence
    one = torch.empty((2, Hq, D), dtype=torch.float32, device="cuda")
    kv.resq_attention_decode(cache, q16[:2].contiguous(), dev(np.array([S0, S1], np.int32)), one,
                             kv.attention_workspace(cache, Hq))
    ref = okv.attention_decode(hq16[:2], K_hat, V_hat, [S0, S1], Hq, Hkv)
    assert np.abs(host(one) - ref).max() <= 1e-4 * vmax
    assert resq.resq_device_status() == resq.OK
