"""GPU parity of GPTQ rounding at pack time (Section 5.1) through the C ABI: codes, packed bytes and scales bit for
bit against the oracle's fp64 sweep given the same inverse-Hessian factor, and the layer run on those weights."""
import numpy as np
import pytest
import torch

import oracle
import synth
from oracle import gptq
from tests.gpu_util import bf16_bits_from_dev, bf16_to_dev, dev, host
from tests.test_gpu_parity import check_output

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def resq():
    import paper_2412_14363_b200 as m
    return m


def _calibration(K, n, seed, dead_col=None):
    """Correlated calibration inputs with outlier channels: the Hessian is far from diagonal."""
    rng = np.random.default_rng(seed)
    X = synth.activations(n, K, "t4", seed=seed).astype(np.float64)
    X = X + 0.5 * np.roll(X, 1, axis=1) + 0.25 * (X @ (rng.standard_normal((K, 8)) / np.sqrt(K))) @ rng.standard_normal((8, K))
    if dead_col is not None:
        X[:, dead_col] = 0.0
    return X.astype(np.float32)


@pytest.mark.parametrize("N,K,r,fp16,dead_col", [(264, 512, 64, False, None), (72, 1024, 128, True, 17),
                                                 (40, 2048, 256, False, None), (16, 512, 0, False, 3)])
def test_pack_weights_gptq_bit_exact(resq, N, K, r, fp16, dead_col):
    Wp = synth.projected_weights_direct(N, K, seed=500 + N)
    H, dead = gptq.hessian(_calibration(K, 2 * K, 600 + N, dead_col))
    U = np.ascontiguousarray(gptq.inverse_factor(H).astype(np.float32))
    pw = gptq.pack_weights_gptq(Wp, r, U, dead, scale_fp16=fp16)
    desc = resq.layer_desc(K, N, r, resq.SCALE_FP16 if fp16 else resq.SCALE_FP32)
    W = resq.resq_pack_weights_gptq(desc, dev(Wp), dev(U), dev(dead.astype(np.uint8)) if dead.any() else None)
    assert resq.resq_device_status() == resq.OK
    assert (host(W.w8) == pw.q8).all()
    assert (host(W.w4_i8) == pw.q4).all()
    assert (host(W.w4) == pw.w4_packed).all()
    assert (host(W.s_w8.float()).view(np.uint32) == pw.s8.view(np.uint32)).all()
    assert (host(W.s_w4.float()).view(np.uint32) == pw.s4.view(np.uint32)).all()
    # the rounding differs from round-to-nearest and lowers the layer-output error on the calibration statistics
    rtn = oracle.pack_weights(Wp if not dead.any() else np.where(dead[None, :], 0, Wp).astype(np.float32), r, scale_fp16=fp16)
    assert (pw.q4 != rtn.q4).mean() > 0.05
    assert gptq.objective(Wp, pw, H).sum() < 0.9 * gptq.objective(Wp, rtn, H).sum()
    if dead_col is not None:
        assert not host(W.w4_i8 if dead_col >= r else W.w8)[:, dead_col - r if dead_col >= r else dead_col].any()


def test_layer_on_gptq_weights(resq):
    """resq_linear consumes the GPTQ-rounded weights like any packed weights: output exact against the oracle's layer."""
    T, K, N, r = 48, 1024, 264, 128
    C_bits = synth.f32_to_bf16_bits(synth.activations(T, K, "t4", seed=701))
    Wp = synth.projected_weights_direct(N, K, seed=702)
    H, dead = gptq.hessian(_calibration(K, 2 * K, 703))
    U = np.ascontiguousarray(gptq.inverse_factor(H).astype(np.float32))
    pw = gptq.pack_weights_gptq(Wp, r, U)
    res = oracle.linear(C_bits, None, pw)
    desc = resq.layer_desc(K, N, r)
    W = resq.resq_pack_weights_gptq(desc, dev(Wp), dev(U))
    ws = resq.alloc_workspace(desc, T, False, True)
    y32 = torch.empty((T, N), dtype=torch.float32, device="cuda")
    resq.resq_linear(W, bf16_to_dev(C_bits), None, y32, ws)
    ybf = torch.empty((T, N), dtype=torch.bfloat16, device="cuda")
    resq.resq_linear(W, bf16_to_dev(C_bits), None, ybf, ws)
    assert resq.resq_device_status() == resq.OK
    check_output(res, pw, host(y32), bf16_bits_from_dev(ybf))


def test_gptq_rejects_rows_too_wide_for_shared_memory(resq):
    K = 28672
    desc = resq.layer_desc(K, 8, K // 8)
    z = torch.zeros(16, dtype=torch.float32, device="cuda")
    st = resq.lib.resq_pack_weights_gptq(__import__("ctypes").byref(desc), z.data_ptr(), z.data_ptr(), None, z.data_ptr(), z.data_ptr(),
                                         z.data_ptr(), z.data_ptr(), None, None)
    assert st == resq.ERR_SHAPE
