"""resq_project_quantize_static: the online-projection quantizer for callers that cannot allocate.

Some users of the library have no workspace to offer: every byte of the GPU already belongs to their
own pool, or they sit in a loop where cudaMalloc (which synchronises the whole device) is off limits.
For them the fp32 staging panel is an 8 MiB array built into the library.  This file checks, through
the C ABI, that the variant gives exactly what the regular entry point gives -- it runs the same two
kernels, so codes and scales must be identical bit for bit -- on two calls in a row with different
inputs (the array keeps the first call's contents, which the second must not see).  For up to 64 token
rows -- a generation step, the likeliest use -- the regular call given its full workspace cuts the
projection along K and so adds in another order; there the variant is compared with the CPU oracle
under the online path's own criterion, bit for bit with the regular call given a panel-only workspace,
and within one code step of the regular call given its full workspace.

Collected last on purpose: a run that stops at the first failure has then already run everything else.
"""
import numpy as np
import pytest
import torch

import oracle
import synth
from tests.gpu_util import bf16_to_dev, host


def _outputs(T, K, r):
    K4 = K - r
    return (torch.full((T, r), 99, dtype=torch.int8, device="cuda"),
            torch.full((T, K4 // 2), 0x99, dtype=torch.uint8, device="cuda"),
            torch.full((T,), -1.0, dtype=torch.float32, device="cuda"),
            torch.full((T,), -1.0, dtype=torch.float32, device="cuda"),
            torch.full((T, K4), 99, dtype=torch.int8, device="cuda"))


@pytest.mark.gpu
def test_static_scratch_variant_matches_regular_entry_point_twice():
    import paper_2412_14363_b200 as resq
    K, r = 2048, 256
    P = bf16_to_dev(synth.f32_to_bf16_bits(synth.kron_orthogonal_bf16(K)))
    for call, T in enumerate((300, 130)):      # the second call is smaller: stale rows stay in the array
        X = bf16_to_dev(synth.f32_to_bf16_bits(synth.activations(T, K, "t4", seed=900 + call)))
        ref = _outputs(T, K, r)
        ws = resq.alloc_workspace(resq.layer_desc(K, 8, r), T, True, True)
        resq.resq_project_quantize(X, P, r, ref[0], ref[1], ref[2], ref[3], ref[4], ws)
        got = _outputs(T, K, r)
        resq.resq_project_quantize_static(X, P, r, got[0], got[1], got[2], got[3], got[4])
        assert resq.resq_device_status() == resq.OK
        for a, b in zip(got, ref):
            assert torch.equal(a, b)
        assert (host(got[2]) > 0).all() and (host(got[3]) > 0).all()
        assert np.abs(host(got[0])).max() == 127 and np.abs(host(got[4])).max() == 7


@pytest.mark.gpu
@pytest.mark.parametrize("T,K,r", [(1, 14336, 1792), (16, 14336, 1792), (64, 14336, 1792), (5, 8192, 0)])
def test_static_scratch_variant_few_rows_against_the_oracle(T, K, r):
    import paper_2412_14363_b200 as resq
    K4 = K - r
    X_bits = synth.f32_to_bf16_bits(synth.activations(T, K, "t4", seed=950 + T))
    P_bits = synth.f32_to_bf16_bits(synth.kron_orthogonal_bf16(K))
    X, P = bf16_to_dev(X_bits), bf16_to_dev(P_bits)
    q8, q4, o8, o4 = oracle.split_quantize(oracle.project(X_bits, P_bits), r)
    x8 = lambda t: t[0] if r else None                           # r = 0: no INT8 segment, NULL accepted

    def check_against_oracle(out):
        g8, g4 = host(out[0]).astype(np.int32), host(out[4]).astype(np.int32)
        assert (host(out[1]) == oracle.pack_nibbles(host(out[4]))).all()
        assert np.abs(g4 - q4).max() <= 1 and (r == 0 or np.abs(g8 - q8).max() <= 1)
        assert (((g8 != q8).sum() if r else 0) + (g4 != q4).sum()) / float(T * K) <= 1e-3
        ulp = lambda a, b: np.abs(a.view(np.int32).astype(np.int64) - b.view(np.int32).astype(np.int64))
        assert ulp(host(out[3]), o4).max() <= K // 16 + 4
        if r:
            assert ulp(host(out[2]), o8).max() <= K // 16 + 4
        else:
            assert (host(out[2]) == 0).all()                     # empty INT8 segment: scale 0

    for _ in range(2):                                           # two calls in a row
        got = _outputs(T, K, r)
        resq.resq_project_quantize_static(X, P, r, x8(got), got[1], got[2], got[3], got[4])
        assert resq.resq_device_status() == resq.OK
        check_against_oracle(got)
    # bit for bit what the regular call gives when its workspace holds the panel alone
    panel_only = torch.empty(((T * K * 4 + 255) // 256) * 256, dtype=torch.uint8, device="cuda")
    ref = _outputs(T, K, r)
    resq.resq_project_quantize(X, P, r, x8(ref), ref[1], ref[2], ref[3], ref[4], panel_only)
    for a, b in zip(got, ref):
        assert torch.equal(a, b)
    # the regular call with its full workspace adds the K slices in another order: one code step at most
    full = _outputs(T, K, r)
    resq.resq_project_quantize(X, P, r, x8(full), full[1], full[2], full[3], full[4],
                               resq.alloc_workspace(resq.layer_desc(K, 8, r), T, True, True))
    assert resq.resq_device_status() == resq.OK
    check_against_oracle(full)
    d4 = np.abs(host(full[4]).astype(np.int32) - host(got[4]).astype(np.int32))
    assert d4.max() <= 1 and (d4 != 0).mean() <= 2e-3


@pytest.mark.gpu
def test_static_scratch_variant_rejects_what_does_not_fit():
    import paper_2412_14363_b200 as resq
    K, r = 4096, 512
    T_max = resq.STATIC_SCRATCH_BYTES // (K * 4)
    X = torch.zeros((T_max + 1, K), dtype=torch.bfloat16, device="cuda")
    P = torch.zeros((K, K), dtype=torch.bfloat16, device="cuda")
    out = _outputs(T_max + 1, K, r)
    with pytest.raises(resq.ResqError) as e:
        resq.resq_project_quantize_static(X, P, r, out[0], out[1], out[2], out[3], out[4])
    assert e.value.status == resq.ERR_WORKSPACE
    with pytest.raises(resq.ResqError) as e:
        resq.resq_project_quantize_static(X[:4], None, r, out[0], out[1], out[2], out[3], out[4])
    assert e.value.status == resq.ERR_NULL
    # the largest size that fits goes through
    resq.resq_project_quantize_static(X[:T_max], P, r, out[0], out[1], out[2], out[3], out[4])
    assert resq.resq_device_status() == resq.OK
    assert not host(out[0][:T_max]).any()      # zero input: zero scales, zero codes
