"""Pins for the oracle's GPTQ rounding against what the algorithm's definition and the mathematics fix."""
import numpy as np

import oracle
import synth
from oracle import gptq


def _case(N=24, K=96, r=32, n=300, seed=0):
    rng = np.random.default_rng(seed)
    mix = rng.standard_normal((K, K)) * 0.3 + np.eye(K)                 # correlated input channels
    X = (rng.standard_normal((n, K)) @ mix).astype(np.float32)
    W = (rng.standard_normal((N, K)) / np.sqrt(K)).astype(np.float32)
    H, dead = gptq.hessian(X)
    U = gptq.inverse_factor(H).astype(np.float32)
    return X, W, H, dead, U


def test_inverse_factor_is_the_upper_cholesky_factor_of_the_inverse():
    _, _, H, _, _ = _case()
    U = gptq.inverse_factor(H)
    assert np.abs(np.tril(U, -1)).max() == 0 and (np.diag(U) > 0).all()
    assert np.abs(U.T @ U @ H - np.eye(H.shape[0])).max() < 1e-9


def test_identity_hessian_reduces_to_round_to_nearest():
    """With uncorrelated inputs of equal power nothing is fed back: the codes are those of Eq. 3's plain rounding."""
    rng = np.random.default_rng(1)
    W = (rng.standard_normal((16, 64)) / 8).astype(np.float32)
    U = np.eye(64, dtype=np.float32) * np.float32(0.7)
    pw = gptq.pack_weights_gptq(W, 32, U)
    rtn = oracle.pack_weights(W, 32)
    assert (pw.q8 == rtn.q8).all() and (pw.q4 == rtn.q4).all()
    assert (pw.s8.view(np.uint32) == rtn.s8.view(np.uint32)).all() and (pw.w4_packed == rtn.w4_packed).all()


def test_two_columns_by_hand():
    """Two coupled columns of the INT4 segment: the second weight receives -(w0 - q0) / U00 * U01 before it is
    rounded (the other columns are zero and uncoupled)."""
    W = np.array([[0.9, 0.35]], np.float32)
    U = np.array([[2.0, -0.5], [0.0, 1.0]], np.float32)
    Wp = np.zeros((1, 64), np.float32)
    Wp[0, 32:34] = W[0]
    Up = np.eye(64, dtype=np.float32)
    Up[32:34, 32:34] = U
    q8, q4, s8, s4 = gptq.gptq_codes(Wp, 32, Up)
    s = float(np.float32(np.float32(0.9) / np.float32(7.0)))
    w0 = float(np.float32(0.9))
    c0 = round(w0 / s)
    assert c0 == 7 and q4[0, 0] == 7
    e = (w0 - c0 * s) / 2.0
    w1 = float(np.float32(0.35)) - e * (-0.5)
    assert q4[0, 1] == int(np.clip(np.rint(w1 / s), -8, 7))


def test_feedback_lowers_the_layer_output_error_and_matches_the_activation_error():
    X, W, H, dead, U = _case()
    pw = gptq.pack_weights_gptq(W, 32, U, dead)
    rtn = oracle.pack_weights(W, 32)
    o_g, o_r = gptq.objective(W, pw, H), gptq.objective(W, rtn, H)
    assert o_g.sum() < 0.8 * o_r.sum()
    assert (o_g <= o_r * 1.05 + 1e-12).mean() > 0.9
    # the objective is the output error on the calibration inputs (plus the damping term): check it directly
    W_hat = np.concatenate([pw.q8 * pw.s8[:, None].astype(np.float64), pw.q4 * pw.s4[:, None].astype(np.float64)], axis=1)
    E = W.astype(np.float64) - W_hat
    direct = 2.0 / X.shape[0] * ((X.astype(np.float64) @ E.T) ** 2).sum(0)
    ridge = H[0, 0] - 2.0 / X.shape[0] * (X.astype(np.float64)[:, 0] ** 2).sum()      # the damping added to the diagonal
    assert ridge > 0
    assert np.allclose(o_g, direct + ridge * (E ** 2).sum(1), rtol=1e-9)


def test_dead_columns_are_zeroed_and_codes_stay_in_range():
    X, W, H, dead, U = _case(seed=3)
    X[:, 5] = 0.0
    H, dead = gptq.hessian(X)
    assert dead[5] and dead.sum() == 1
    U = gptq.inverse_factor(H).astype(np.float32)
    pw = gptq.pack_weights_gptq(W, 32, U, dead)
    assert (pw.q8[:, 5] == 0).all()
    assert pw.q8.min() >= -128 and pw.q8.max() <= 127 and pw.q4.min() >= -8 and pw.q4.max() <= 7
    # visiting the columns in blocks with the feedback applied lazily is the same computation: emulate two halves
    q8b, q4b, _, _ = gptq.gptq_codes(W, 32, U, dead)
    assert (q8b == pw.q8).all() and (q4b == pw.q4).all()


def test_row_independence_and_permutation():
    """Rows (output channels) never interact: quantizing a subset of rows gives the same codes for them."""
    _, W, H, dead, U = _case(seed=4)
    full = gptq.pack_weights_gptq(W, 32, U)
    part = gptq.pack_weights_gptq(W[[7, 3, 20]], 32, U)
    assert (part.q4 == full.q4[[7, 3, 20]]).all() and (part.q8 == full.q8[[7, 3, 20]]).all()
