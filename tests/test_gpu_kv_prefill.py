"""GPU parity of tile-wise causal attention over the quantized cache (resq_attention_prefill: Section 4.3, Eq. 8 with
the cache of Section 5.1) against the oracle's many-query definition in fp64 on the oracle's own codes.

Tolerance: 1e-3 of the largest dequantized value magnitude of the KV head, the single-query bound -- the only
roundings below fp32 are those of the softmax weights times the value scales to half (relative 2^-11 each, so the
weighted mean of the values moves by at most 2^-11 * max|v| ~ 4.9e-4 * max|v|); the integer codes are exact in half,
scores, softmax and accumulation are fp32."""
import numpy as np
import pytest
import torch

import synth
from oracle import kv as okv
from tests.gpu_util import bf16_to_dev, dev, host

pytestmark = pytest.mark.gpu
D = 128


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


def _fill(kv, uc, cache, b, n, Hkv, stream, v_scale=1.0, v_shift=0.3):
    """Appends n tokens to sequence b through the library and returns the oracle's dequantized keys / values."""
    W_C, wq, s_u = uc
    k = synth.head_vectors(n, Hkv, D, stream=stream, lead=1.0, scale=1.5)
    v = synth.to_bf16_values(synth.head_vectors(n, Hkv, D, stream=stream + 1, lead=4.0, shift=v_shift) * np.float32(v_scale))
    kv.resq_kv_append(cache, bf16_to_dev(synth.f32_to_bf16_bits(k)), bf16_to_dev(synth.f32_to_bf16_bits(v)),
                      dev(np.full(n, b, np.int32)), dev(np.arange(n, dtype=np.int32)), wq, s_u)
    Yk, _, _ = okv.project_int8(k.reshape(-1, D), *okv.quantize_uc(W_C))
    dk = okv.kv_dequantize(okv.kv_quantize(Yk)).reshape(n, Hkv, D)
    dv = okv.kv_dequantize(okv.kv_quantize(v.reshape(-1, D))).reshape(n, Hkv, D)
    return [dk[:, h] for h in range(Hkv)], [dv[:, h] for h in range(Hkv)]


@pytest.mark.parametrize("prefix,T,Hq,Hkv,v_scale", [
    (0, 37, 8, 2, 1.0),        # one ragged tile per KV head
    (20, 70, 4, 4, 1.0),       # group of 1; 90 positions in a 96-position cache: the last step has one block only
    (3, 200, 32, 8, 1.0),      # several tiles, tokens of a tile straddle a step boundary
    (100, 300, 12, 2, 1.0),    # group of 6: a tile's rows do not start on a token boundary
    (5, 90, 8, 8, 1e-4),       # value scales far below / above 1: the power-of-two normalisation
    (5, 90, 8, 8, 3e3),
    (260, 1, 8, 2, 1.0),       # a single new token (a generation step written as a prefill)
])
def test_attention_prefill_against_the_oracle(resq, kv, uc, prefix, T, Hq, Hkv, v_scale):
    S = prefix + T
    cap = ((S + 31) // 32) * 32
    cache = kv.KvCache(2, Hkv, cap)
    cache.data.fill_(0xFF)                      # unwritten positions hold NaN patterns
    _fill(kv, uc, cache, 0, min(S, 7), Hkv, 700)   # another sequence, never attended
    K_hat, V_hat = _fill(kv, uc, cache, 1, S, Hkv, 710, v_scale=v_scale)
    W_C, wq, s_u = uc
    q = synth.head_vectors(T, Hq, D, stream=720, lead=1.0, scale=1.5)
    q16 = torch.empty((T, Hq, D), dtype=torch.float16, device="cuda")
    kv.resq_query_project(bf16_to_dev(synth.f32_to_bf16_bits(q)), wq, s_u, q16)
    out = torch.full((T, Hq, D), float("nan"), dtype=torch.float32, device="cuda")
    kv.resq_attention_prefill(cache, q16, 1, prefix, out)
    torch.cuda.synchronize()
    assert resq.resq_device_status() == resq.OK
    ref = okv.attention_queries(host(q16), [None, K_hat], [None, V_hat], np.full(T, 1, np.int32),
                                np.arange(prefix + 1, S + 1, dtype=np.int32), Hq, Hkv)
    got = host(out)
    assert np.isfinite(got).all()
    g = Hq // Hkv
    for h in range(Hq):
        vmax = np.abs(V_hat[h // g]).max()
        err = np.abs(got[:, h] - ref[:, h]).max()
        assert err <= 1e-3 * vmax, (h, err, vmax)


def test_attention_prefill_agrees_with_the_many_query_call(resq, kv, uc):
    """The two evaluations of the same definition (tile-wise on tcgen05, row-wise on the single-query kernel) agree
    within the sum of their tolerances."""
    prefix, T, Hq, Hkv = 40, 150, 8, 2
    S = prefix + T
    cache = kv.KvCache(1, Hkv, 192)
    cache.data.fill_(0)
    _, V_hat = _fill(kv, uc, cache, 0, S, Hkv, 730)
    W_C, wq, s_u = uc
    q = synth.head_vectors(T, Hq, D, stream=740, lead=1.0, scale=1.5)
    q16 = torch.empty((T, Hq, D), dtype=torch.float16, device="cuda")
    kv.resq_query_project(bf16_to_dev(synth.f32_to_bf16_bits(q)), wq, s_u, q16)
    a = torch.empty((T, Hq, D), dtype=torch.float32, device="cuda")
    b = torch.empty_like(a)
    kv.resq_attention_prefill(cache, q16, 0, prefix, a)
    kv.resq_attention_queries(cache, q16, dev(np.zeros(T, np.int32)), dev(np.arange(prefix + 1, S + 1, dtype=np.int32)), b)
    assert resq.resq_device_status() == resq.OK
    vmax = max(np.abs(v).max() for v in V_hat)
    assert np.abs(host(a) - host(b)).max() <= 2e-3 * vmax


def test_attention_prefill_rejects_bad_ranges(resq, kv):
    cache = kv.KvCache(2, 2, 64)
    q16 = torch.zeros((8, 4, D), dtype=torch.float16, device="cuda")
    out = torch.empty((8, 4, D), dtype=torch.float32, device="cuda")
    for seq, pos0 in ((2, 0), (-1, 0), (0, -1), (0, 57)):
        with pytest.raises(resq.ResqError):
            kv.resq_attention_prefill(cache, q16, seq, pos0, out)
