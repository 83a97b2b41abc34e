"""Pins of the GPTQ oracle (residual-branch weight quantization, Sec. III-B) against what the algorithm's
definition fixes: special cases that reduce to round-to-nearest, a hand-computed two-channel case, the greedy
step's optimality property, invariances, and the reconstruction objective against round-to-nearest."""
import numpy as np
import torch

import oracle
from workloads import generator as gen


def rtn(R, group=64):
    q, s = gen._round_residual(torch.from_numpy(np.asarray(R, np.float64))) if group == 64 else (None, None)
    return q.numpy(), s.numpy()


def proxy_loss(R, q, s, H, group):
    D = R - q.astype(np.float64) * np.repeat(s.astype(np.float64), group, axis=0)
    return float(np.einsum("kn,kj,jn->", D, H, D))


def test_identity_hessian_reduces_to_round_to_nearest():
    # H = c I: H^-1 is diagonal, its Cholesky factor has no off-diagonal entries, no error is propagated.
    rng = np.random.default_rng(0)
    R = rng.normal(scale=0.02, size=(128, 24))
    R[64:128, 3] = 0.0
    for c in (1.0, 37.5):
        q, s = oracle.gptq_quantize(R, c * np.eye(128))
        q0, s0 = rtn(R)
        assert np.array_equal(q, q0) and np.array_equal(s, s0)


def test_two_channel_case_by_hand():
    # group = 2, one output channel, H = [[2, 1], [1, 2]] (no damping).  H^-1 = [[2, -1], [-1, 2]] / 3,
    # U = chol(H^-1, upper) = [[sqrt(2/3), -sqrt(1/6)], [0, sqrt(1/2)]].
    # w = (0.7, 0.38): scale = 0.1, q0 = 7, error 0; nothing to propagate -> q1 = round(3.8) = 4.
    q, s = oracle.gptq_quantize(np.array([[0.7], [0.38]]), np.array([[2.0, 1.0], [1.0, 2.0]]), group=2, percdamp=0.0)
    assert np.allclose(s, [[0.1]]) and q[:, 0].tolist() == [7, 4]
    # w = (0.33, 0.7): scale = 0.1, q0 = 3, error e = 0.03; the second weight becomes
    # 0.7 - e * U01 / U00 = 0.7 + 0.03 * 0.5 = 0.715 -> 7.15 -> 7 (and with e = 0.05 it would cross to 0.725 -> 7).
    q, s = oracle.gptq_quantize(np.array([[0.33], [0.7]]), np.array([[2.0, 1.0], [1.0, 2.0]]), group=2, percdamp=0.0)
    assert q[:, 0].tolist() == [3, 7]
    # w = (0.26, 0.64): q0 = round(0.26 / (0.64 / 7)) = round(2.84375) = 3 with scale 0.0914285..., error
    # 0.26 - 3 * 0.0914285 = -0.0142857; second weight 0.64 - 0.5 * 0.0142857 = 0.632857 -> 6.92 -> 7.
    q, s = oracle.gptq_quantize(np.array([[0.26], [0.64]]), np.array([[2.0, 1.0], [1.0, 2.0]]), group=2, percdamp=0.0)
    assert q[:, 0].tolist() == [3, 7]
    # A case where the compensation changes a code.  Three channels in one group; the first is uncorrelated with the
    # others and carries the group maximum 0.7 (scale 0.1, q = 7, no error).  For the other two H = [[2, -1], [-1, 2]]:
    # H^-1 = [[2, 1], [1, 2]] / 3, U01 / U00 = +0.5.  w1 = 0.33 -> q = 3, error 0.03; w2 = 0.665 - 0.03 * 0.5 = 0.65
    # -> 6.5 minus the FP32 rounding of the scale (0.1 is slightly above 0.1 in FP32) -> 6, where plain rounding of
    # 6.65 gives 7.
    H3 = np.array([[1.0, 0.0, 0.0], [0.0, 2.0, -1.0], [0.0, -1.0, 2.0]])
    q, s = oracle.gptq_quantize(np.array([[0.7], [0.33], [0.665]]), H3, group=3, percdamp=0.0)
    assert q[:, 0].tolist() == [7, 3, 6]
    q, s = oracle.gptq_quantize(np.array([[0.7], [0.33], [0.665]]), np.eye(3), group=3, percdamp=0.0)
    assert q[:, 0].tolist() == [7, 3, 7]


def test_update_minimises_the_remaining_objective():
    # After fixing the first input channel, the compensated remaining weights are the minimiser of the quadratic
    # objective over the still-free channels (the optimal-brain-surgeon step GPTQ is built on): with every later
    # channel left unquantized (a huge group so that nothing else is rounded) the loss must equal e0^2 / [H^-1]_00.
    rng = np.random.default_rng(2)
    K = 6
    X = rng.normal(size=(50, K))
    H = X.T @ X
    w = rng.normal(size=(K, 1))
    Hinv = np.linalg.inv(H)
    U = np.linalg.cholesky(Hinv).T
    e0 = 0.123
    w_rest = w[1:, 0] - e0 / U[0, 0] * U[0, 1:]                      # what the sweep leaves in the later channels
    d = np.concatenate([[e0], w[1:, 0] - w_rest])                    # w - w_hat
    loss = d @ H @ d
    assert np.isclose(loss, e0 ** 2 / Hinv[0, 0], rtol=1e-10)
    for _ in range(20):                                              # any other choice of the rest is worse
        alt = w_rest + rng.normal(scale=1e-2, size=K - 1)
        d2 = np.concatenate([[e0], w[1:, 0] - alt])
        assert d2 @ H @ d2 >= loss - 1e-12


def test_invariances():
    rng = np.random.default_rng(3)
    K, N = 128, 10
    X = rng.normal(size=(300, K)) * (1.0 + 5.0 * (rng.random(K) < 0.05))
    H = X.T @ X
    R = rng.normal(scale=0.02, size=(K, N))
    q, s = oracle.gptq_quantize(R, H)
    q2, s2 = oracle.gptq_quantize(R, 7.0 * H)                        # the objective's scale does not matter
    assert np.array_equal(q, q2) and np.array_equal(s, s2)
    perm = rng.permutation(N)                                        # output channels are independent
    q3, s3 = oracle.gptq_quantize(R[:, perm], H)
    assert np.array_equal(q3, q[:, perm]) and np.array_equal(s3, s[:, perm])
    q4, s4 = oracle.gptq_quantize(4.0 * R, H)                        # weights times a power of two: same codes
    assert np.array_equal(q4, q) and np.array_equal(s4, 4.0 * s)


def test_reconstruction_objective_beats_round_to_nearest():
    # tr((R - R_hat)^T H (R - R_hat)) = || X (R - R_hat) ||_F^2 on the calibration set: GPTQ's whole point.
    rng = np.random.default_rng(4)
    K, N = 256, 32
    base = rng.normal(size=(400, 16))
    X = base @ rng.normal(size=(16, K)) + 0.3 * rng.normal(size=(400, K))   # correlated input channels
    H = X.T @ X
    R = rng.normal(scale=0.02, size=(K, N))
    q, s = oracle.gptq_quantize(R, H)
    q0, s0 = rtn(R)
    assert q.min() >= -8 and q.max() <= 7
    assert proxy_loss(R, q, s, H, 64) < 0.8 * proxy_loss(R, q0, s0, H, 64)


def test_hessian_of_bf16_activations():
    x = gen.make_activations(40, 64, seed=1)
    H = oracle.gptq_hessian(gen.bf16_bits(x).numpy().view(np.uint16))
    xf = x.to(torch.float64).numpy()
    assert np.allclose(H, xf.T @ xf, rtol=1e-13) and np.allclose(H, H.T)


def test_equals_the_defining_recursion_with_explicit_inverse_downdates():
    # The algorithm's definition before its Cholesky reformulation (Frantar et al., 2023, Eq. 2-3 applied in a fixed
    # order): quantize the first free channel, move the free channels by
    #   delta = -(w_q - quant(w_q)) / [Hf^-1]_qq * (Hf^-1)[:, q],
    # then remove q from the inverse by one step of Gaussian elimination,
    #   Hf^-1 <- Hf^-1 - (Hf^-1)[:, q] (Hf^-1)[q, :] / [Hf^-1]_qq   (row and column q dropped).
    # Written here with no Cholesky factor at all; the oracle must produce the same codes and scales.
    rng = np.random.default_rng(5)
    K, N, group = 128, 6, 64
    X = rng.normal(size=(200, 8)) @ rng.normal(size=(8, K)) + 0.5 * rng.normal(size=(200, K))
    H = X.T @ X
    R = rng.normal(scale=0.02, size=(K, N))
    Hd = H + 0.01 * np.mean(np.diag(H)) * np.eye(K)
    Hinv = np.linalg.inv(Hd)
    W = R.copy()
    codes = np.zeros((K, N), np.int8)
    scales = np.zeros((K // group, N), np.float32)
    for k in range(K):
        if k % group == 0:
            scales[k // group] = (np.abs(W[k:k + group]).max(axis=0) / 7.0).astype(np.float32)
        s = scales[k // group].astype(np.float64)
        q = np.clip(np.rint(W[k] / s), -8, 7)
        codes[k] = q.astype(np.int8)
        err = W[k] - q * s
        # free channels are k..K-1; Hinv holds their inverse with index 0 = channel k
        W[k:] -= np.outer(Hinv[:, 0] / Hinv[0, 0], err)
        Hinv = (Hinv - np.outer(Hinv[:, 0], Hinv[0, :]) / Hinv[0, 0])[1:, 1:]
    q_o, s_o = oracle.gptq_quantize(R, H, group=group, percdamp=0.01)
    assert np.array_equal(s_o, scales)
    assert np.array_equal(q_o, codes)


# ---------------------------------------------------------------------------------------------------------------
# The same sweep on the MXFP4 grid (E2M1 elements, E8M0 exponent per 32 input channels)
# ---------------------------------------------------------------------------------------------------------------
E2M1 = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0])


def nearest_e2m1_by_search(v):
    # brute force over the eight magnitudes: smallest distance, and of two equally near ones the even index
    d = np.abs(v[..., None] - E2M1)
    best = d.min(axis=-1, keepdims=True)
    cand = np.where(d == best, np.arange(8), 99)
    lo = cand.min(axis=-1)
    hi = np.where(d == best, np.arange(8), -1).max(axis=-1)
    return np.where(lo == hi, lo, np.where(lo % 2 == 0, lo, hi))


def test_mx_identity_hessian_reduces_to_the_plain_mxfp4_conversion():
    rng = np.random.default_rng(6)
    R = rng.normal(scale=0.02, size=(128, 20))
    R[32:64, 3] = 0.0                                   # an all-zero block
    R[5, 7] = 0.0                                       # a zero element inside a block
    q0, e0 = gen._round_residual_mx(torch.from_numpy(R))
    for c in (1.0, 9.0):
        q, e = oracle.gptq_quantize_mx(R, c * np.eye(128))
        assert np.array_equal(q, q0.numpy()) and np.array_equal(e, e0.numpy())


def test_mx_hand_cases():
    # One block of 32 channels, one output channel, all weights zero except the first three.
    # w0 = 6.0 -> exponent floor(log2 6) - 2 = 0, scale 1, code 7 (value 6), no error.
    # H couples channels 1 and 2 as in the INT4 hand case ([[2, -1], [-1, 2]] -> U12 / U11 = +0.5).
    # w1 = 1.3 -> nearest 1.5 (index 3), error -0.2; w2 = 2.45 - (-0.2) * 0.5 = 2.55 -> nearest 3 (index 5), where
    # plain rounding of 2.45 gives 2 (index 4).
    K = 32
    H = np.eye(K)
    H[1:3, 1:3] = [[2.0, -1.0], [-1.0, 2.0]]
    w = np.zeros((K, 1))
    w[:3, 0] = [6.0, 1.3, 2.45]
    q, e = oracle.gptq_quantize_mx(w, H, percdamp=0.0)
    assert e[0, 0] == 127 and q[:3, 0].tolist() == [7, 3, 5]
    q, e = oracle.gptq_quantize_mx(w, np.eye(K), percdamp=0.0)
    assert q[:3, 0].tolist() == [7, 3, 4]
    # negative weights carry bit 3; the exponent follows the block's largest magnitude: 0.2 -> floor(log2 0.2) - 2 = -5
    w = np.zeros((K, 1))
    w[:2, 0] = [-0.2, 0.05]
    q, e = oracle.gptq_quantize_mx(w, np.eye(K), percdamp=0.0)
    assert e[0, 0] == 127 - 5 and q[:2, 0].tolist() == [8 + 7, 3]     # 0.2 * 32 = 6.4 -> 6 (saturates); 0.05 * 32 = 1.6 -> 1.5


def test_mx_equals_the_defining_recursion_with_explicit_inverse_downdates():
    rng = np.random.default_rng(7)
    K, N = 96, 5
    X = rng.normal(size=(150, 6)) @ rng.normal(size=(6, K)) + 0.5 * rng.normal(size=(150, K))
    H = X.T @ X
    R = rng.normal(scale=0.02, size=(K, N))
    Hinv = np.linalg.inv(H + 0.01 * np.mean(np.diag(H)) * np.eye(K))
    W = R.copy()
    codes = np.zeros((K, N), np.uint8)
    exps = np.zeros((K // 32, N), np.uint8)
    for k in range(K):
        if k % 32 == 0:
            ex = np.floor(np.log2(np.abs(W[k:k + 32]).max(axis=0))) - 2
            exps[k // 32] = (ex + 127).astype(np.uint8)
        scale = 2.0 ** ex
        idx = nearest_e2m1_by_search(np.minimum(np.abs(W[k]) / scale, 6.0))
        codes[k] = idx + 8 * (W[k] < 0)
        err = W[k] - np.sign(W[k]) * E2M1[idx] * scale
        W[k:] -= np.outer(Hinv[:, 0] / Hinv[0, 0], err)
        Hinv = (Hinv - np.outer(Hinv[:, 0], Hinv[0, :]) / Hinv[0, 0])[1:, 1:]
    q_o, e_o = oracle.gptq_quantize_mx(R, H, percdamp=0.01)
    assert np.array_equal(e_o, exps) and np.array_equal(q_o, codes)


def test_mx_objective_beats_the_plain_conversion():
    rng = np.random.default_rng(8)
    K, N = 256, 24
    X = rng.normal(size=(400, 16)) @ rng.normal(size=(16, K)) + 0.3 * rng.normal(size=(400, K))
    H = X.T @ X
    R = rng.normal(scale=0.02, size=(K, N))
    q, e = oracle.gptq_quantize_mx(R, H)
    q0, e0 = gen._round_residual_mx(torch.from_numpy(R))
    deq = lambda c, x: gen.mx_dequantize(torch.from_numpy(np.asarray(c)), torch.from_numpy(np.asarray(x))).numpy()
    loss = lambda D: float(np.einsum("kn,kj,jn->", D, H, D))
    assert loss(R - deq(q, e)) < 0.8 * loss(R - deq(q0.numpy(), e0.numpy()))
