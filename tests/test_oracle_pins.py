"""Pins of the CPU oracle against things that are not the oracle.

Every check here compares the oracle with something fixed by the paper's equations or by plain
mathematics: hand-derived quantizer cases (Eq. 3-4, 8-9), exact round trips of on-grid values, the
nearest-integer property of rounding, brute-force integer dot products, the r = 0 reduction to a
plain W4A4 product (Eq. 2), the "quantization disabled" identity X-hat (L1 L2 + R) = X W (Eq. 5-6),
and a fully exactly-representable layer whose output is the FP64 matrix product of its raw inputs.
"""
import os

import numpy as np
import pytest
import torch

import oracle
from workloads import generator as gen

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
G = 64


def bits(t):
    """torch bfloat16 tensor -> numpy uint16 bit patterns."""
    return gen.bf16_bits(t).numpy().view(np.uint16)


def bf16_bits_of(values):
    return bits(torch.tensor(np.asarray(values, dtype=np.float32)).to(torch.bfloat16))


# ----------------------------------------------------------------------------- BF16 conversion
def test_bf16_rounding_matches_independent_implementation():
    rng = np.random.default_rng(0)
    vals = np.concatenate([
        rng.standard_normal(2000).astype(np.float32) * 10.0 ** rng.integers(-6, 6, 2000),
        # exact ties between two BF16 neighbours, both parities of the kept LSB
        np.array([1.00390625, 1.01171875, -1.00390625, 3.0078125, 3.0234375, 0.0, -0.0,
                  65280.0, 3.3895313892515355e38], dtype=np.float32),
    ])
    want = bits(torch.from_numpy(vals).to(torch.bfloat16))
    got = np.array([oracle.f32_to_bf16(float(v)) for v in vals], dtype=np.uint16)
    assert np.array_equal(got, want)
    assert oracle.f32_to_bf16(1.00390625) == 0x3F80  # tie -> even (down)
    assert oracle.f32_to_bf16(1.01171875) == 0x3F82  # tie -> even (up)


# ----------------------------------------------------------------------------- quantizer, golden cases
def _golden_cases():
    cases = []
    with open(os.path.join(GOLDEN, "quantizer_cases.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            name, rho, xs, scale, codes = [p.strip() for p in line.split("|")]
            cases.append((name, float(rho), [float(v) for v in xs.split()], float(scale),
                          [int(v) for v in codes.split()]))
    return cases


@pytest.mark.parametrize("case", _golden_cases(), ids=lambda c: c[0])
def test_quantizer_hand_derived_cases(case):
    name, rho, xs, scale, codes = case
    # Put the case in the second of three groups, at shuffled positions, to catch group/index slips.
    K = 3 * G
    pos = np.random.default_rng(len(name)).permutation(G)[: len(xs)]
    x = np.zeros((1, K), np.float32)
    x[0, G + pos] = xs
    x[0, 0] = 100.0  # a loud neighbour group must not leak into this group's range
    x[0, 2 * G + 5] = -0.001
    q, s = oracle.quantize(bf16_bits_of(x), np.ones(K, np.float32), rho)
    assert s[0, 1] == np.float32(scale)
    assert q[0, G + pos].tolist() == codes
    others = np.setdiff1d(np.arange(G), pos)
    assert not q[0, G + others].any()
    assert q[0, 0] == 7 or rho < 1.0


def test_on_grid_round_trip_is_exact():
    # x = c * 2^e with c in -7..7 and a +-7 in every group, lambda a power of two, rho = 1:
    # s = 2^e' exactly, q = c, s * q = xhat exactly.
    rng = np.random.default_rng(1)
    M, K = 9, 4 * G
    c = rng.integers(-7, 8, size=(M, K))
    e = rng.integers(-6, 5, size=(M, K // G))
    for m in range(M):
        for g in range(K // G):
            c[m, g * G + rng.integers(0, G)] = 7 if (m + g) % 2 else -7
    lam_exp = rng.integers(-3, 4, size=K)
    lam = (2.0 ** lam_exp).astype(np.float32)
    xhat = c * 2.0 ** np.repeat(e, G, axis=1)
    x = (xhat * lam[None, :]).astype(np.float32)
    q, s, xh = oracle.quantize(bf16_bits_of(x), lam, 1.0, want_xhat=True)
    assert np.array_equal(xh, xhat.astype(np.float32))
    assert np.array_equal(s, (2.0 ** e).astype(np.float32))
    assert np.array_equal(q, c.astype(np.int8))
    assert np.array_equal(np.repeat(s, G, axis=1) * q, xhat.astype(np.float32))


def test_zero_groups_and_rows():
    K = 2 * G
    x = np.zeros((3, K), np.float32)
    x[1, G + 3] = 2.0
    q, s = oracle.quantize(bf16_bits_of(x), np.full(K, 0.5, np.float32), 0.8)
    assert not q[0].any() and not s[0].any() and not q[2].any()
    assert s[1, 0] == 0 and not q[1, :G].any()
    assert s[1, 1] == np.float32(np.float32(0.8) * np.float32(4.0)) / np.float32(7.0)
    assert q[1, G + 3] == 7  # rint(4 / s) = rint(8.75) = 9 -> clipped to 7


def test_nearest_integer_property_and_range():
    # For every element the code is a nearest integer of xhat / s (exact arithmetic), or the clip.
    rng = np.random.default_rng(2)
    M, K = 64, 8 * G
    x = rng.standard_normal((M, K)).astype(np.float32)
    x[:, 17] *= 40
    lam = np.exp(rng.standard_normal(K) * 0.5).astype(np.float32)
    for rho in (1.0, 0.9, 0.6):
        q, s, xh = oracle.quantize(bf16_bits_of(x), lam, rho, want_xhat=True)
        # xhat itself: the FP32 product of the BF16 value with the FP32 reciprocal, within half an ulp of x / lam
        xb = gen.bf16_to_f32(torch.from_numpy(x).to(torch.bfloat16)).numpy().astype(np.float64)
        assert np.allclose(xh, xb / lam.astype(np.float64), rtol=2.0 ** -22, atol=0)
        z = xh.astype(np.float64) / np.repeat(s, G, axis=1).astype(np.float64)
        zc = np.clip(z, -8.0, 7.0)
        assert np.all(np.abs(zc - q) <= 0.5 + 1e-5)
        assert q.min() >= -8 and q.max() <= 7
        a = np.abs(xh).reshape(M, K // G, G).max(axis=2)
        assert np.allclose(s, rho * a / 7.0, rtol=3 * 2.0 ** -24, atol=0)
        if rho == 1.0:
            # the group's extreme element always lands on +-7, and -8 is unreachable
            assert np.all(np.abs(q).reshape(M, K // G, G).max(axis=2) == 7)
            assert q.min() >= -7
        else:
            assert np.all(np.abs(q).reshape(M, K // G, G).max(axis=2) >= 7)
    # scale is monotone in rho
    s_lo = oracle.quantize(bf16_bits_of(x), lam, 0.6)[1]
    s_hi = oracle.quantize(bf16_bits_of(x), lam, 0.9)[1]
    assert np.all(s_lo < s_hi)


# ----------------------------------------------------------------------------- integer partial sums
def test_partials_brute_force_tiny():
    rng = np.random.default_rng(3)
    M, K, N = 3, 2 * G, 5
    q = rng.integers(-8, 8, size=(M, K)).astype(np.int8)
    qw = rng.integers(-8, 8, size=(K, N)).astype(np.int8)
    P = oracle.partials(q, qw)
    for m in range(M):
        for g in range(K // G):
            for n in range(N):
                acc = 0
                for k in range(g * G, (g + 1) * G):
                    acc += int(q[m, k]) * int(qw[k, n])
                assert P[m, g, n] == acc


def test_partials_sum_to_ungrouped_product_and_bound():
    rng = np.random.default_rng(4)
    M, K, N = 17, 5 * G, 96
    q = rng.integers(-8, 8, size=(M, K)).astype(np.int8)
    qw = rng.integers(-8, 8, size=(K, N)).astype(np.int8)
    q[0, :G] = -8
    qw[:G, 0] = -8
    P = oracle.partials(q, qw)
    assert np.array_equal(P.sum(axis=1), q.astype(np.int64) @ qw.astype(np.int64))
    assert np.abs(P).max() <= 64 * 64 and P[0, 0, 0] == 4096
    for g in range(K // G):
        sl = slice(g * G, (g + 1) * G)
        assert np.array_equal(P[:, g, :], q[:, sl].astype(np.int64) @ qw[sl].astype(np.int64))


# ----------------------------------------------------------------------------- low-rank down projection
def test_lowrank_down_against_fp64_matmul():
    rng = np.random.default_rng(5)
    M, K, r = 11, 3 * G, 16
    x = torch.from_numpy(rng.standard_normal((M, K)).astype(np.float32)).to(torch.bfloat16)
    lam = np.exp(rng.standard_normal(K) * 0.3).astype(np.float32)
    L1 = torch.from_numpy(rng.standard_normal((K, r)).astype(np.float32) * 0.1).to(torch.bfloat16)
    T = oracle.lowrank_down(bits(x), lam, bits(L1))
    rl = (np.float32(1.0) / lam).astype(np.float32)
    xh = x.to(torch.float32).numpy() * rl[None, :]  # FP32 product, rounded once
    xb = torch.from_numpy(xh).to(torch.bfloat16).to(torch.float64).numpy()
    want = xb @ L1.to(torch.float64).numpy()
    assert np.allclose(T, want, rtol=2.0 ** -23, atol=1e-30)
    # with small-integer inputs everything is exact
    xi = torch.from_numpy(rng.integers(-4, 5, (M, K)).astype(np.float32)).to(torch.bfloat16)
    Li = torch.from_numpy(rng.integers(-3, 4, (K, r)).astype(np.float32)).to(torch.bfloat16)
    Ti = oracle.lowrank_down(bits(xi), np.ones(K, np.float32), bits(Li))
    assert np.array_equal(Ti, (xi.to(torch.float64) @ Li.to(torch.float64)).numpy().astype(np.float32))


# ----------------------------------------------------------------------------- assembly
def _dequant_matmul(q, s, qw, sw):
    a = q.astype(np.float64) * np.repeat(s.astype(np.float64), G, axis=1)
    b = qw.astype(np.float64) * np.repeat(sw.astype(np.float64), G, axis=0)
    return a @ b


def test_r0_reduces_to_plain_w4a4_product():
    # Eq. 2: with no low-rank branch the layer is Q_A(X) Q_W(W) -- dequantize both, multiply in FP64.
    rng = np.random.default_rng(6)
    M, K, N = 13, 4 * G, 40
    x = rng.standard_normal((M, K)).astype(np.float32)
    lam = np.exp(rng.standard_normal(K) * 0.3).astype(np.float32)
    qw = rng.integers(-8, 8, size=(K, N)).astype(np.int8)
    sw = np.exp(rng.standard_normal((K // G, N))).astype(np.float32) * 0.01
    bias = rng.standard_normal(N).astype(np.float32)
    rows = np.arange(M, dtype=np.int32)
    out = oracle.forward_rows(bf16_bits_of(x), rows, lam, 0.85, None, None, qw, sw, bias)
    want = _dequant_matmul(out["q"], out["s"], qw, sw) + bias.astype(np.float64)[None, :]
    assert np.allclose(out["Y64"], want, rtol=1e-12, atol=1e-12)
    # and without a bias the bias term is really absent
    out0 = oracle.forward_rows(bf16_bits_of(x), rows, lam, 0.85, None, None, qw, sw, None)
    assert np.allclose(out0["Y64"], want - bias.astype(np.float64)[None, :], rtol=1e-12, atol=1e-12)


def test_exactly_representable_layer_equals_fp64_product_of_raw_inputs():
    # On-grid activations (lossless 4-bit), power-of-two smoothing, small-integer low-rank factors:
    # nothing is rounded anywhere, so Y must equal  (X / lam) (L1 L2 + R_deq) + b  computed directly
    # from the raw inputs in FP64 -- no quantizer, no grouping, no intermediate T on this side.
    rng = np.random.default_rng(7)
    M, K, N, r = 10, 3 * G, 24, 4
    c = rng.integers(-7, 8, size=(M, K))
    e = rng.integers(-3, 3, size=(M, K // G))
    for m in range(M):
        for g in range(K // G):
            c[m, g * G + rng.integers(0, G)] = 7
    lam = (2.0 ** rng.integers(-2, 3, size=K)).astype(np.float32)
    xhat = c * 2.0 ** np.repeat(e, G, axis=1)
    x = (xhat * lam[None, :]).astype(np.float32)
    qw = rng.integers(-8, 8, size=(K, N)).astype(np.int8)
    sw = (2.0 ** rng.integers(-6, -1, size=(K // G, N))).astype(np.float32)
    L1 = rng.integers(-2, 3, size=(K, r)).astype(np.float32)
    L2 = rng.integers(-2, 3, size=(r, N)).astype(np.float32) * 0.25
    bias = rng.integers(-4, 5, size=N).astype(np.float32) * 0.125
    rows = np.arange(M, dtype=np.int32)
    out = oracle.forward_rows(bf16_bits_of(x), rows, lam, 1.0, bf16_bits_of(L1), bf16_bits_of(L2), qw, sw, bias,
                              want_partials=True)
    R_deq = qw.astype(np.float64) * np.repeat(sw.astype(np.float64), G, axis=0)
    want = (x.astype(np.float64) / lam[None, :]) @ (L1.astype(np.float64) @ L2.astype(np.float64) + R_deq) + bias
    assert np.array_equal(out["Y64"], want)
    # the BF16 output is the round-to-nearest-even of that
    wantb = bits(torch.from_numpy(want.astype(np.float32)).to(torch.bfloat16))
    assert np.array_equal(out["Ybf16"], wantb)
    # stepwise entry points agree with the fused one
    q, s = oracle.quantize(bf16_bits_of(x), lam, 1.0)
    T = oracle.lowrank_down(bf16_bits_of(x), lam, bf16_bits_of(L1))
    P = oracle.partials(q, qw)
    Y, Yb = oracle.assemble(P, s, sw, T, bf16_bits_of(L2), bias)
    assert np.array_equal(q, out["q"]) and np.array_equal(s, out["s"]) and np.array_equal(T, out["T"])
    assert np.array_equal(P, out["P"]) and np.array_equal(Y, out["Y64"]) and np.array_equal(Yb, out["Ybf16"])


def test_general_layer_against_independent_assembly():
    # Random (inexact) case with K != N and r > 0: Y64 = dequant product + T L2 + b, each piece
    # recomputed with numpy from the oracle's integer/scale outputs.
    rng = np.random.default_rng(8)
    M, K, N, r = 12, 2 * G, 3 * G + 8, 16
    x = rng.standard_normal((M, K)).astype(np.float32)
    x[:, 5] *= 30
    lam = np.exp(rng.standard_normal(K) * 0.3).astype(np.float32)
    qw = rng.integers(-8, 8, size=(K, N)).astype(np.int8)
    sw = np.exp(rng.standard_normal((K // G, N))).astype(np.float32) * 0.01
    L1 = torch.from_numpy(rng.standard_normal((K, r)).astype(np.float32) * 0.1).to(torch.bfloat16)
    L2 = torch.from_numpy(rng.standard_normal((r, N)).astype(np.float32) * 0.1).to(torch.bfloat16)
    bias = rng.standard_normal(N).astype(np.float32) * 0.1
    rows = np.array([11, 0, 5, 5, 3], dtype=np.int32)
    out = oracle.forward_rows(bf16_bits_of(x), rows, lam, 0.7, bits(L1), bits(L2), qw, sw, bias)
    q_all, s_all = oracle.quantize(bf16_bits_of(x), lam, 0.7)
    assert np.array_equal(out["q"], q_all[rows]) and np.array_equal(out["s"], s_all[rows])
    want = (_dequant_matmul(out["q"], out["s"], qw, sw)
            + out["T"].astype(np.float64) @ L2.to(torch.float64).numpy() + bias.astype(np.float64)[None, :])
    assert np.allclose(out["Y64"], want, rtol=1e-12, atol=1e-12)
    assert np.array_equal(out["Y64"][2], out["Y64"][3])  # same row twice -> same result


# ----------------------------------------------------------------------------- Eq. 5-6 identities with the generator
def test_quantization_disabled_reproduces_xw():
    x = gen.make_activations(32, 256, outlier_idx=gen.outlier_channels(256, 0, 0, count=3), outlier_gain=40, seed=0)
    layer = gen.make_layer_svd(256, 192, 16, x, seed=1, bias_std=0.01)
    X64 = x.to(torch.float64).numpy()
    Y = oracle.forward_noquant(X64, layer.lam.to(torch.float64).numpy(), layer.L1.to(torch.float64).numpy(),
                               layer.L2.to(torch.float64).numpy(), layer.R.numpy(),
                               layer.bias.to(torch.float64).numpy())
    want = X64 @ layer.W.numpy() + layer.bias.to(torch.float64).numpy()[None, :]
    assert np.allclose(Y, want, rtol=1e-10, atol=1e-10 * np.abs(want).max())


def _rel_err(layer, x, rho):
    rows = np.arange(x.shape[0], dtype=np.int32)
    out = oracle.forward_rows(bits(x), rows, layer.lam.numpy(), rho,
                              None if layer.L1 is None else bits(layer.L1),
                              None if layer.L2 is None else bits(layer.L2),
                              layer.qweight.numpy(), layer.wscale.numpy(), None)
    want = x.to(torch.float64).numpy() @ layer.W.numpy()
    return float(np.linalg.norm(out["Y64"] - want) / np.linalg.norm(want))


def test_quantized_layer_approximates_xw_and_rank_helps():
    K, N = 512, 256
    idx = gen.outlier_channels(K, 0, 3, count=4)
    x = gen.make_activations(48, K, outlier_idx=idx, outlier_gain=40, seed=2)
    errs = [_rel_err(gen.make_layer_svd(K, N, r, x, seed=3), x, 1.0) for r in (0, 16, 64)]
    assert errs[0] < 0.35, errs
    assert errs[2] < errs[1] < errs[0], errs
    # A far too small clip ratio over-clips and is clearly worse than a moderate one (Sec. III-A).
    layer = gen.make_layer_svd(K, N, 16, x, seed=3)
    assert _rel_err(layer, x, 0.2) > 1.5 * _rel_err(layer, x, 0.9)


def test_generator_residual_rounding_is_on_grid():
    x = gen.make_activations(16, 128, seed=4)
    layer = gen.make_layer_svd(128, 64, 8, x, seed=5)
    q = layer.qweight.numpy()
    assert q.min() >= -8 and q.max() <= 7
    deq = q.astype(np.float64) * np.repeat(layer.wscale.numpy().astype(np.float64), G, axis=0)
    step = np.repeat(layer.wscale.numpy().astype(np.float64), G, axis=0)
    assert np.all(np.abs(deq - layer.R.numpy()) <= 0.5 * step * (1 + 1e-6) + 1e-12)


def test_power_of_two_scaling_and_row_independence():
    # Multiplying the activations by 2^k is exact in BF16 and FP32, so the quantizer must return the same codes with
    # scales multiplied by 2^k (Eq. 3-5 are homogeneous); rows are quantized independently of one another (Eq. 4's
    # maximum runs over one token's group only), so any subset or permutation of rows gives the same per-row result.
    rng = np.random.default_rng(21)
    M, K = 12, 3 * G
    x = rng.normal(size=(M, K)).astype(np.float32)
    x[:, 5] *= 30.0
    lam = (0.5 + rng.random(K)).astype(np.float32)
    xb = bf16_bits_of(x)
    q0, s0 = oracle.quantize(xb, lam, 0.85)
    for k in (-5, 3):
        xk = bf16_bits_of(oracle.bf16_bits_to_f64(xb).astype(np.float32) * np.float32(2.0 ** k))
        qk, sk = oracle.quantize(xk, lam, 0.85)
        assert np.array_equal(qk, q0)
        assert np.array_equal(sk, s0 * np.float32(2.0 ** k))
    perm = rng.permutation(M)
    qp, sp = oracle.quantize(xb[perm], lam, 0.85)
    assert np.array_equal(qp, q0[perm]) and np.array_equal(sp, s0[perm])
    q1, s1 = oracle.quantize(xb[3:4], lam, 0.85)
    assert np.array_equal(q1, q0[3:4]) and np.array_equal(s1, s0[3:4])


def test_smaller_clip_ratio_never_shrinks_a_code():
    # Eq. 8-9: a smaller rho shrinks the scale, so |x / s| grows: magnitudes of the codes are non-decreasing as rho
    # falls (until they saturate at 7), and the scale is proportional to rho up to FP32 rounding.
    rng = np.random.default_rng(22)
    x = rng.normal(size=(6, 2 * G)).astype(np.float32)
    lam = np.ones(2 * G, np.float32)
    xb = bf16_bits_of(x)
    prev_q, prev_s = None, None
    for rho in (1.0, 0.9, 0.75, 0.6, 0.5):
        q, s = oracle.quantize(xb, lam, rho)
        assert q.min() >= -8 and q.max() <= 7
        if prev_q is not None:
            assert np.all(np.abs(q.astype(np.int32)) >= np.abs(prev_q.astype(np.int32))), "a code shrank when rho fell"
            assert np.all(s <= prev_s)
        np.testing.assert_allclose(s, oracle.quantize(xb, lam, 1.0)[1] * rho, rtol=3e-7)
        prev_q, prev_s = q, s
