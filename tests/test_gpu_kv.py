"""GPU parity of the attention-block path (Section 4.3, Eq. 8; Section 5.1) through the C ABI against the CPU
oracle: U_C codes, the projected half-precision query and every cache byte (codes, scales, zero-points) bit for
bit; single-query attention within 1e-3 of the largest dequantized value magnitude of the KV head (the softmax
weights times the value scales are rounded to half, relative 2^-11, before the second product; everything else
is fp32), against the oracle's fp64 attention on its own codes."""
import numpy as np
import pytest
import torch

import oracle
import synth
from oracle import kv as okv
from tests import kv_util
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
    """W_C = U_C^T and its codes on both sides (checked equal in test_uc_quantize)."""
    W_C = np.ascontiguousarray(synth.haar_orthogonal(D).T.astype(np.float32))
    wq, s_u = kv.resq_uc_quantize(dev(W_C))
    return W_C, wq, s_u


def test_uc_quantize(uc):
    W_C, wq, s_u = uc
    owq, os_u = okv.quantize_uc(W_C)
    assert (host(wq) == owq).all()
    assert (host(s_u).view(np.uint32) == os_u.view(np.uint32)).all()


@pytest.mark.parametrize("T,H", [(1, 32), (3, 5), (130, 32), (16, 1)])
def test_query_project_bit_exact(resq, kv, uc, T, H):
    W_C, wq, s_u = uc
    q = synth.head_vectors(T, H, D, stream=10 + T, lead=1.0, scale=3.0)
    q[0, 0, :] = 0.0                          # an all-zero head vector: scale 0, output 0
    q_out = torch.empty((T, H, D), dtype=torch.float16, device="cuda")
    kv.resq_query_project(bf16_to_dev(synth.f32_to_bf16_bits(q)), wq, s_u, q_out)
    assert resq.resq_device_status() == resq.OK
    Y, _, _ = okv.project_int8(q.reshape(-1, D), *okv.quantize_uc(W_C))
    ref = okv.query_fp16(Y).reshape(T, H, D)
    assert (host(q_out).view(np.uint16) == ref.view(np.uint16)).all()


def _oracle_records(k, v, W_C):
    """Oracle codes of key (through the 8-bit U_C projection) and value head vectors [T][H][128]."""
    Yk, _, _ = okv.project_int8(k.reshape(-1, D), *okv.quantize_uc(W_C))
    return okv.kv_quantize(Yk), okv.kv_quantize(v.reshape(-1, D))


def _check_cache(image, hk, hv, seq_ids, positions, H, skip=()):
    for t in range(len(seq_ids)):
        if t in skip:
            continue
        for h in range(H):
            row = t * H + h
            for which, rec in (("k", hk), ("v", hv)):
                c8, c4, meta = kv_util.get(image, which, seq_ids[t], h, positions[t])
                assert (c8 == rec.c8[row]).all(), (which, t, h)
                assert (c4 == rec.c4[row]).all(), (which, t, h)
                assert (meta.view(np.uint32) == rec.meta[row].view(np.uint32)).all(), (which, t, h)


@pytest.mark.parametrize("T,H", [(70, 8), (5, 2), (33, 3)])
def test_kv_append_prefill_bit_exact(resq, kv, uc, T, H):
    """One sequence, T consecutive positions starting at 3 (crosses cache blocks, ragged last warp tile)."""
    W_C, wq, s_u = uc
    k = synth.head_vectors(T, H, D, stream=20 + T, lead=1.0, scale=2.0)
    v = synth.head_vectors(T, H, D, stream=40 + T, lead=4.0, shift=0.5)
    v[1, 0, :16] = v[1, 0, 0]                 # a constant 8-bit segment: s = 0, codes 0
    cache = kv.KvCache(2, H, 128)
    cache.data.fill_(0xEE)
    seq_ids, positions = np.ones(T, np.int32), np.arange(3, 3 + T, dtype=np.int32)
    kv.resq_kv_append(cache, bf16_to_dev(synth.f32_to_bf16_bits(k)), bf16_to_dev(synth.f32_to_bf16_bits(v)),
                      dev(seq_ids), dev(positions), wq, s_u)
    assert resq.resq_device_status() == resq.OK
    image = host(cache.data).reshape(2, H, 128 // 32, kv_util.BLOCK_BYTES)
    hk, hv = _oracle_records(k, v, W_C)
    _check_cache(image, hk, hv, seq_ids, positions, H)
    assert (image[0] == 0xEE).all()           # the other sequence is untouched
    assert (kv_util.get(image, "k", 1, 0, 0)[0] == 0xEE).all() and (kv_util.get(image, "v", 1, H - 1, 3 + T)[1] == 0xEE).all()


def test_kv_append_decode_step_and_bad_index(resq, kv, uc):
    """One token for each of 6 sequences at scattered positions; one entry out of range is skipped and reported."""
    W_C, wq, s_u = uc
    B, H = 6, 8
    k = synth.head_vectors(B, H, D, stream=61, lead=1.0)
    v = synth.head_vectors(B, H, D, stream=62, scale=0.01)
    cache = kv.KvCache(B, H, 64)
    cache.data.zero_()
    seq_ids = np.arange(B, dtype=np.int32)[::-1].copy()
    positions = np.array([0, 31, 32, 63, 64, 17], np.int32)      # entry 4 is past the capacity
    kv.resq_kv_append(cache, bf16_to_dev(synth.f32_to_bf16_bits(k)), bf16_to_dev(synth.f32_to_bf16_bits(v)),
                      dev(seq_ids), dev(positions), wq, s_u)
    assert resq.resq_device_status() == kv.ERR_INDEX
    assert resq.resq_device_status() == resq.OK                   # reading clears it
    image = host(cache.data).reshape(B, H, 2, kv_util.BLOCK_BYTES)
    hk, hv = _oracle_records(k, v, W_C)
    _check_cache(image, hk, hv, seq_ids, positions, H, skip=(4,))
    assert (image[seq_ids[4]] == 0).all()


def test_fused_project_append_matches_the_two_calls(resq, kv, uc):
    """resq_qkv_project_append writes the same bytes as resq_query_project + resq_kv_append (a generation step:
    one token for each of 5 sequences, and a ragged prefill of 37 tokens)."""
    W_C, wq, s_u = uc
    for T, Hq, Hkv, seq, pos in ((5, 8, 2, np.arange(5), np.array([9, 0, 31, 32, 63])), (37, 4, 4, np.zeros(37), np.arange(20, 57))):
        q = bf16_to_dev(synth.f32_to_bf16_bits(synth.head_vectors(T, Hq, D, stream=700 + T, lead=1.0)))
        k = bf16_to_dev(synth.f32_to_bf16_bits(synth.head_vectors(T, Hkv, D, stream=710 + T, lead=1.0)))
        v = bf16_to_dev(synth.f32_to_bf16_bits(synth.head_vectors(T, Hkv, D, stream=720 + T)))
        seq_ids, positions = dev(seq.astype(np.int32)), dev(pos.astype(np.int32))
        ca, cb = kv.KvCache(5, Hkv, 64), kv.KvCache(5, Hkv, 64)
        ca.data.fill_(7)
        cb.data.fill_(7)
        qa = torch.empty((T, Hq, D), dtype=torch.float16, device="cuda")
        qb = torch.empty_like(qa)
        kv.resq_query_project(q, wq, s_u, qa)
        kv.resq_kv_append(ca, k, v, seq_ids, positions, wq, s_u)
        kv.resq_qkv_project_append(cb, q, qb, k, v, seq_ids, positions, wq, s_u)
        assert resq.resq_device_status() == resq.OK
        assert (host(qa).view(np.uint16) == host(qb).view(np.uint16)).all()
        assert (host(ca.data) == host(cb.data)).all()
        assert (host(ca.data) != 7).any()


def _attention_case(kv, seq_lens, Hq, Hkv, capacity, seed, v_scale=1.0, v_shift=0.3, fill=0xFF, device_consumer=False):
    """Cache image built on the CPU from the oracle's codes (no GPU kernel upstream), attention on both sides."""
    B = len(seq_lens)
    image = kv_util.empty_image(B, Hkv, capacity, fill)            # 0xFF: NaN scales in every unused slot
    K_hat = [[None] * Hkv for _ in range(B)]
    V_hat = [[None] * Hkv for _ in range(B)]
    vmax = np.zeros((B, Hkv))
    for b, S in enumerate(seq_lens):
        if S == 0:
            continue
        kf = synth.head_vectors(S, Hkv, D, seed=seed, stream=100 + b, lead=3.0, scale=0.7)
        vf = synth.head_vectors(S, Hkv, D, seed=seed, stream=200 + b, lead=4.0, scale=v_scale, shift=v_shift * v_scale)
        hk, hv = okv.kv_quantize(kf.reshape(-1, D)), okv.kv_quantize(vf.reshape(-1, D))
        dk, dv = okv.kv_dequantize(hk).reshape(S, Hkv, D), okv.kv_dequantize(hv).reshape(S, Hkv, D)
        for h in range(Hkv):
            K_hat[b][h], V_hat[b][h] = dk[:, h], dv[:, h]
            vmax[b, h] = np.abs(dv[:, h]).max()
            for pos in range(S):
                row = pos * Hkv + h
                kv_util.put(image, "k", b, h, pos, hk.c8[row], hk.c4[row], hk.meta[row])
                kv_util.put(image, "v", b, h, pos, hv.c8[row], hv.c4[row], hv.meta[row])
    q16 = synth.head_vectors(B, Hq, D, seed=seed, stream=300, lead=2.0, scale=0.5).astype(np.float16)
    ref = okv.attention_decode(q16, K_hat, V_hat, seq_lens, Hq, Hkv)
    cache = kv.KvCache(B, Hkv, capacity, data=dev(image.reshape(-1)))
    out = torch.full((B, Hq, D), float("nan"), dtype=torch.float32, device="cuda")
    ws = kv.attention_workspace(cache, Hq)
    ws.fill_(0xFF)
    q16_d, lens_d = dev(q16), dev(np.asarray(seq_lens, np.int32))
    if device_consumer:
        # A kernel enqueued right behind the call on the same stream, with no host synchronization in between,
        # must see the finished outputs: stream order is all a caller has between the attention and the o_proj
        # quantizer that follows it.
        spin = torch.empty(1 << 24, dtype=torch.float32, device="cuda")
        spin.fill_(1.0)                                    # keeps the GPU busy so that the three launches queue up
        kv.resq_attention_decode(cache, q16_d, lens_d, out, ws)
        seen = out.clone()
        return host(seen), ref, vmax
    kv.resq_attention_decode(cache, q16_d, lens_d, out, ws)
    return host(out), ref, vmax


def _assert_close(out, ref, vmax, Hq, Hkv, tol=1e-3):
    g = Hq // Hkv
    assert np.isfinite(out).all()
    for b in range(out.shape[0]):
        for h in range(Hq):
            err = np.abs(out[b, h] - ref[b, h]).max()
            assert err <= tol * max(vmax[b, h // g], 1e-30), (b, h, err, vmax[b, h // g])


@pytest.mark.parametrize("seq_lens,Hq,Hkv,capacity", [
    ([70, 0, 33, 1], 8, 2, 96),               # ragged tails, an empty sequence, a single position
    ([32, 64], 4, 4, 64),                      # one query head per KV head, full blocks
    ([45], 8, 1, 64),                          # eight query heads on one KV head
    ([2500, 1200], 32, 8, 2528),               # long: every (sequence, head) spread over several warps
])
def test_attention_decode(resq, kv, seq_lens, Hq, Hkv, capacity):
    out, ref, vmax = _attention_case(kv, seq_lens, Hq, Hkv, capacity, seed=11)
    assert resq.resq_device_status() == resq.OK
    _assert_close(out, ref, vmax, Hq, Hkv)
    for b, S in enumerate(seq_lens):
        if S == 0:
            assert (out[b] == 0).all()


def test_attention_many_short_sequences(resq, kv):
    """More (sequence, head) pairs than warps: several records per warp."""
    rng = np.random.default_rng(5)
    seq_lens = [int(x) for x in rng.integers(0, 65, 200)]
    out, ref, vmax = _attention_case(kv, seq_lens, 8, 8, 64, seed=12)
    assert resq.resq_device_status() == resq.OK
    _assert_close(out, ref, vmax, 8, 8)


def test_attention_outputs_are_complete_for_the_next_kernel_of_the_stream(resq, kv):
    """64 sequences x 8 KV heads of at most one cache block each: every (sequence, head) is seen by a single warp,
    so the merge kernel has nothing to add -- it must still hold the stream until the attention kernel has
    written every output, which a device-side copy enqueued straight after the call observes."""
    rng = np.random.default_rng(9)
    seq_lens = [int(x) for x in rng.integers(0, 33, 64)]
    for rep in range(3):
        out, ref, vmax = _attention_case(kv, seq_lens, 32, 8, 32, seed=14 + rep, device_consumer=True)
        assert resq.resq_device_status() == resq.OK
        _assert_close(out, ref, vmax, 32, 8)


@pytest.mark.parametrize("v_scale", [1e-7, 3e5])
def test_attention_value_magnitudes(resq, kv, v_scale):
    """Tiny and huge values: the half-precision weights are normalised by a power of two from the value scales."""
    out, ref, vmax = _attention_case(kv, [90, 40], 8, 2, 96, seed=13, v_scale=v_scale)
    assert resq.resq_device_status() == resq.OK
    _assert_close(out, ref, vmax, 8, 2)


def test_attention_bad_length_is_clamped_and_reported(resq, kv):
    cache = kv.KvCache(2, 2, 64)
    cache.data.zero_()
    out = torch.empty((2, 4, D), dtype=torch.float32, device="cuda")
    q16 = torch.zeros((2, 4, D), dtype=torch.float16, device="cuda")
    kv.resq_attention_decode(cache, q16, dev(np.array([65, -1], np.int32)), out, kv.attention_workspace(cache, 4))
    assert resq.resq_device_status() == kv.ERR_INDEX
    assert (host(out) == 0).all()             # all-zero cache: every value dequantizes to 0


def test_end_to_end_append_then_attend(resq, kv, uc):
    """The three calls chained on the GPU (project q, append k/v, attend) against the oracle chained on the CPU."""
    W_C, wq, s_u = uc
    B, Hq, Hkv, S = 2, 8, 2, 75
    cache = kv.KvCache(B, Hkv, 96)
    cache.data.fill_(0xFF)
    K_hat = [[None] * Hkv for _ in range(B)]
    V_hat = [[None] * Hkv for _ in range(B)]
    vmax = np.zeros((B, Hkv))
    for b in range(B):
        k = synth.head_vectors(S, Hkv, D, stream=400 + b, lead=1.0, scale=1.5)
        v = synth.head_vectors(S, Hkv, D, stream=500 + b, lead=4.0, shift=-0.2)
        kv.resq_kv_append(cache, bf16_to_dev(synth.f32_to_bf16_bits(k)), bf16_to_dev(synth.f32_to_bf16_bits(v)),
                          dev(np.full(S, b, np.int32)), dev(np.arange(S, dtype=np.int32)), wq, s_u)
        hk, hv = _oracle_records(k, v, W_C)
        dk, dv = okv.kv_dequantize(hk).reshape(S, Hkv, D), okv.kv_dequantize(hv).reshape(S, Hkv, D)
        for h in range(Hkv):
            K_hat[b][h], V_hat[b][h], vmax[b, h] = dk[:, h], dv[:, h], np.abs(dv[:, h]).max()
    q = synth.head_vectors(B, Hq, D, stream=600, lead=1.0, scale=1.5)
    q16 = torch.empty((B, Hq, D), dtype=torch.float16, device="cuda")
    kv.resq_query_project(bf16_to_dev(synth.f32_to_bf16_bits(q)), wq, s_u, q16)
    out = torch.empty((B, Hq, D), dtype=torch.float32, device="cuda")
    kv.resq_attention_decode(cache, q16, dev(np.full(B, S, np.int32)), out, kv.attention_workspace(cache, Hq))
    assert resq.resq_device_status() == resq.OK
    Yq, _, _ = okv.project_int8(q.reshape(-1, D), *okv.quantize_uc(W_C))
    ref = okv.attention_decode(okv.query_fp16(Yq).reshape(B, Hq, D), K_hat, V_hat, [S] * B, Hq, Hkv)
    _assert_close(host(out), ref, vmax, Hq, Hkv)


@pytest.mark.parametrize("prefix,Tq,Hq,Hkv", [(0, 37, 8, 2), (50, 70, 4, 4), (3, 200, 32, 8)])
def test_attention_many_queries_causal(resq, kv, uc, prefix, Tq, Hq, Hkv):
    """Prefill-shaped attention through the public calls: Tq new tokens of one sequence (after `prefix` cached ones)
    and a few of another are projected and appended, then every new token attends its own causal prefix of the
    quantized cache in ONE call.  Against the oracle's many-query definition on the oracle's own codes, within the
    single-query tolerance; rows with an empty prefix give 0; a bad sequence index is reported."""
    W_C, wq, s_u = uc
    S = prefix + Tq
    cap = ((S + 31) // 32) * 32
    cache = kv.KvCache(3, Hkv, cap)
    cache.data.fill_(0xFF)
    K_hat = [[None] * Hkv for _ in range(3)]
    V_hat = [[None] * Hkv for _ in range(3)]
    vmax = np.zeros((3, Hkv))
    for b, n in ((2, S), (0, 5)):
        k = synth.head_vectors(n, Hkv, D, stream=800 + b, lead=1.0, scale=1.5)
        v = synth.head_vectors(n, Hkv, D, stream=810 + b, lead=4.0, shift=0.3)
        kv.resq_kv_append(cache, bf16_to_dev(synth.f32_to_bf16_bits(k)), bf16_to_dev(synth.f32_to_bf16_bits(v)),
                          dev(np.full(n, b, np.int32)), dev(np.arange(n, dtype=np.int32)), wq, s_u)
        hk, hv = _oracle_records(k, v, W_C)
        dk, dv = okv.kv_dequantize(hk).reshape(n, Hkv, D), okv.kv_dequantize(hv).reshape(n, Hkv, D)
        for h in range(Hkv):
            K_hat[b][h], V_hat[b][h], vmax[b, h] = dk[:, h], dv[:, h], np.abs(dv[:, h]).max()
    # query rows: the Tq new tokens of sequence 2 (causal), three rows of sequence 0, one row with an empty prefix
    q_seq = np.r_[np.full(Tq, 2), [0, 0, 0], [2]].astype(np.int32)
    q_len = np.r_[np.arange(prefix + 1, S + 1), [1, 3, 5], [0]].astype(np.int32)
    n = q_seq.size
    q = synth.head_vectors(n, Hq, D, stream=820, lead=1.0, scale=1.5)
    q16 = torch.empty((n, Hq, D), dtype=torch.float16, device="cuda")
    kv.resq_query_project(bf16_to_dev(synth.f32_to_bf16_bits(q)), wq, s_u, q16)
    out = torch.full((n, Hq, D), float("nan"), dtype=torch.float32, device="cuda")
    kv.resq_attention_queries(cache, q16, dev(q_seq), dev(q_len), out)
    assert resq.resq_device_status() == resq.OK
    ref = okv.attention_queries(host(q16), K_hat, V_hat, q_seq, q_len, Hq, Hkv)
    got = host(out)
    assert np.isfinite(got).all() and (got[-1] == 0).all()
    g = Hq // Hkv
    for i in range(n):
        for h in range(Hq):
            assert np.abs(got[i, h] - ref[i, h]).max() <= 1e-3 * vmax[q_seq[i], h // g], (i, h)
    # the last causal row sees the whole sequence: the single-query call on that sequence agrees within tolerance
    one = torch.empty((3, Hq, D), dtype=torch.float32, device="cuda")
    q3 = torch.zeros((3, Hq, D), dtype=torch.float16, device="cuda")
    q3[2] = q16[Tq - 1]
    kv.resq_attention_decode(cache, q3, dev(np.array([0, 0, S], np.int32)), one, kv.attention_workspace(cache, Hq))
    assert np.abs(host(one)[2] - got[Tq - 1]).max() <= 2e-3 * vmax[2].max()
    # an out-of-range sequence index is reported
    bad = q_seq.copy()
    bad[0] = 3
    kv.resq_attention_queries(cache, q16, dev(bad), dev(q_len), out)
    assert resq.resq_device_status() == kv.ERR_INDEX
