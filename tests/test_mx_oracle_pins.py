"""Pins of the MXFP4 half of the CPU oracle against things that are not the oracle: hand-derived E2M1 rounding
cases, exact round trips of on-grid blocks, the shared-exponent rule on hand-computed blocks (with and without
the clip ratio of Eq. 8), an independent dequantize-then-FP64-matmul, a scalar-loop brute force, and a fully
exactly-representable layer equal to the FP64 product of its raw inputs."""
import os

import numpy as np
import torch

import oracle
from workloads import generator as gen

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
GRID = [0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0]


def bits(t):
    return gen.bf16_bits(t).numpy().view(np.uint16)


def test_e2m1_rounding_golden_cases():
    n = 0
    with open(os.path.join(GOLDEN, "e2m1_cases.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            v, want = [float(p) for p in line.split("|")]
            got = float(oracle.e2m1_values(np.array([oracle.e2m1_rne_sat(float(np.float32(v)))], np.uint8))[0])
            assert got == want, (v, got, want)
            n += 1
    assert n >= 25


def test_e2m1_rounding_is_nearest_on_a_dense_sweep():
    # Property: the chosen grid value is a nearest one (independent of how ties are broken).
    for v in np.linspace(-7.0, 7.0, 2801).astype(np.float32):
        got = float(oracle.e2m1_values(np.array([oracle.e2m1_rne_sat(float(v))], np.uint8))[0])
        best = min(abs(abs(float(v)) - g) for g in GRID)
        assert abs(abs(float(v)) - abs(got)) <= best + 1e-12 and (got == 0.0 or np.sign(got) == np.sign(v))


def _x_row(values):
    return torch.tensor(np.asarray(values, np.float32)).to(torch.bfloat16).reshape(1, -1)


def test_shared_exponent_and_round_trip_on_grid_blocks():
    lam = np.ones(64, np.float32)
    # block 0: max 6 * 2^-3 -> floor(log2(0.75)) = -1, shared exponent -3; block 1: max 4 * 2^5 = 128 -> 7 - 2 = 5
    b0 = [g * 2.0 ** -3 for g in GRID] * 4
    b1 = [(-1) ** i * g * 2.0 ** 5 for i, g in enumerate([4.0, 3.0, 2.0, 1.5, 1.0, 0.5, 0.0, 4.0] * 4)]
    x = _x_row(b0 + b1)
    codes, exps = oracle.mx_quantize(bits(x), lam, 1.0)
    assert list(exps[0]) == [127 - 3, 127 + 5]
    got = oracle.e2m1_values(codes[0]) * np.repeat(2.0 ** (exps[0].astype(np.float64) - 127), 32)
    assert np.array_equal(got, x.to(torch.float64).numpy()[0])


def test_clip_ratio_moves_the_shared_exponent_and_saturates():
    lam = np.ones(32, np.float32)
    x = _x_row([4.0, 3.0, 1.0, -4.0] + [0.5] * 28)
    # rho = 1: max 4 -> exponent 2 - 2 = 0: values as they are.
    c1, e1 = oracle.mx_quantize(bits(x), lam, 1.0)
    assert e1[0, 0] == 127 and list(oracle.e2m1_values(c1[0])[:4]) == [4.0, 3.0, 1.0, -4.0]
    # rho = 0.5: threshold 2 -> exponent 1 - 2 = -1: values double, 8 and 6 both land on 6 (clipping), 0.5 -> 1.
    c2, e2 = oracle.mx_quantize(bits(x), lam, 0.5)
    assert e2[0, 0] == 126 and list(oracle.e2m1_values(c2[0])[:5]) == [6.0, 6.0, 2.0, -6.0, 1.0]
    # a block maximum of 7.5 exceeds the largest element 6 * 2^0 even at rho = 1 (MX conversion saturates)
    c3, e3 = oracle.mx_quantize(bits(_x_row([7.5] + [1.0] * 31)), lam, 1.0)
    assert e3[0, 0] == 127 and oracle.e2m1_values(c3[0])[0] == 6.0
    # zero block
    c4, e4 = oracle.mx_quantize(bits(_x_row([0.0] * 32)), lam, 0.7)
    assert e4[0, 0] == 0 and not c4.any()


def test_forward_equals_dequantize_then_fp64_matmul():
    rng = np.random.default_rng(5)
    M, K, N = 6, 128, 24
    x = torch.tensor(rng.standard_normal((M, K)) * np.where(rng.random(K) < 0.05, 30.0, 1.0), dtype=torch.float32).to(torch.bfloat16)
    lam = np.exp(rng.standard_normal(K) * 0.3).astype(np.float32)
    layer = gen.make_layer_mx_direct(K, N, 0, seed=9, with_bias=True)
    out = oracle.mx_forward_rows(bits(x), np.arange(M), lam, 0.8, None, None, layer.wcodes.numpy(), layer.wexps.numpy(),
                                 layer.bias.numpy())
    a = oracle.e2m1_values(out["codes"]) * np.repeat(2.0 ** (out["exps"].astype(np.float64) - 127), 32, axis=1)
    w = gen.mx_dequantize(layer.wcodes, layer.wexps).numpy()
    want = a @ w + layer.bias.numpy().astype(np.float64)
    assert np.allclose(out["Y64"], want, rtol=1e-13, atol=1e-300)


def test_whole_chain_against_scalar_brute_force():
    f32 = np.float32
    rng = np.random.default_rng(21)
    M, K, N = 2, 64, 3
    xv = (rng.standard_normal((M, K)) * 3.0).astype(np.float32)
    x = torch.tensor(xv).to(torch.bfloat16)
    xf = x.to(torch.float32).numpy()
    lam = np.exp(rng.standard_normal(K) * 0.3).astype(np.float32)
    layer = gen.make_layer_mx_direct(K, N, 0, seed=4, with_bias=False)
    wc, we = layer.wcodes.numpy(), layer.wexps.numpy()
    rho = f32(0.9)
    want = np.zeros((M, N))
    for m in range(M):
        for b in range(K // 32):
            xh = [f32(f32(xf[m, k]) * f32(f32(1.0) / lam[k])) for k in range(32 * b, 32 * b + 32)]
            u = f32(rho * max(abs(v) for v in xh))
            e = int(np.floor(np.log2(float(u)))) - 2          # u is a normal number here
            vals = []
            for v in xh:
                t = float(v) / 2.0 ** e
                cands = sorted(GRID, key=lambda g: (abs(abs(t) - g), GRID.index(g) % 2))  # nearest, even code on ties
                vals.append(np.sign(t) * min(cands[0], 6.0))
            for n in range(N):
                dot = sum(vals[j] * float(oracle.e2m1_values(np.array([wc[32 * b + j, n]], np.uint8))[0]) for j in range(32))
                want[m, n] += dot * 2.0 ** e * 2.0 ** (int(we[b, n]) - 127)
    out = oracle.mx_forward_rows(bits(x), np.arange(M), lam, float(rho), None, None, wc, we, None)
    assert np.allclose(out["Y64"], want, rtol=1e-13, atol=0.0)


def test_exactly_representable_layer_equals_product_of_raw_inputs():
    # Activations and weights that MXFP4 represents exactly (rho = 1, lambda = 1), BF16 low-rank factors and T
    # exact as well: the layer must return the FP64 product of its raw inputs, computed here without any quantizer.
    rng = np.random.default_rng(2)
    M, K, N, r = 4, 96, 8, 4
    xa = rng.choice(GRID, size=(M, K)) * rng.choice([-1.0, 1.0], size=(M, K))
    xa[:, ::32] = 6.0
    xa = xa * np.repeat(2.0 ** rng.integers(-3, 3, size=(M, K // 32)), 32, axis=1)
    x = torch.tensor(xa, dtype=torch.float32).to(torch.bfloat16)
    assert np.array_equal(x.to(torch.float64).numpy(), xa)
    wcodes = rng.integers(0, 16, size=(K, N)).astype(np.uint8)
    wexps = rng.integers(120, 126, size=(K // 32, N)).astype(np.uint8)
    W = gen.mx_dequantize(torch.tensor(wcodes), torch.tensor(wexps)).numpy()
    L1 = torch.tensor(rng.integers(-2, 3, size=(K, r)) * 0.25, dtype=torch.float32).to(torch.bfloat16)
    L2 = torch.tensor(rng.integers(-2, 3, size=(r, N)) * 0.5, dtype=torch.float32).to(torch.bfloat16)
    bias = (rng.integers(-4, 5, size=N) * 0.125).astype(np.float32)
    want = xa @ W + (xa @ L1.to(torch.float64).numpy()) @ L2.to(torch.float64).numpy() + bias
    out = oracle.mx_forward_rows(bits(x), np.arange(M), np.ones(K, np.float32), 1.0, bits(L1), bits(L2), wcodes, wexps, bias)
    assert np.array_equal(out["Y64"], want)


def test_generator_weight_rounding_agrees_with_the_element_rule():
    # The generator's MXFP4 rounding of weights (tooling) and the oracle's element conversion are written
    # independently; on the same scaled values they must choose the same grid points.
    rng = np.random.default_rng(8)
    R = torch.tensor(rng.standard_normal((64, 5)) * 0.02, dtype=torch.float64)
    codes, exps = gen._round_residual_mx(R)
    scaled = (R.reshape(2, 32, 5) / torch.pow(torch.tensor(2.0, dtype=torch.float64), exps.to(torch.float64) - 127.0)[:, None, :]).reshape(64, 5)
    for k in range(64):
        for n in range(5):
            v = float(np.float32(scaled[k, n].item()))
            if float(scaled[k, n]) == v:  # exactly representable in FP32: same input on both sides
                assert (oracle.e2m1_rne_sat(v) & 7) == (int(codes[k, n]) & 7)


def test_power_of_two_scaling_shifts_exponents_and_blocks_are_independent():
    # The MX conversion is homogeneous under powers of two: x * 2^k keeps every element code and adds k to every
    # shared exponent; a block's result depends on that block's 32 values only, so replacing another block of the
    # row (or another row) changes nothing in it.
    rng = np.random.default_rng(31)
    M, K = 5, 128
    x = torch.tensor(rng.normal(size=(M, K)).astype(np.float32)).to(torch.bfloat16)
    x[:, 7] *= 25.0
    lam = (2.0 ** rng.integers(-2, 3, size=K)).astype(np.float32)
    codes, exps = oracle.mx_quantize(bits(x), lam, 0.9)
    for k in (-4, 6):
        ck, ek = oracle.mx_quantize(bits((x.to(torch.float32) * 2.0 ** k).to(torch.bfloat16)), lam, 0.9)
        assert np.array_equal(oracle.e2m1_values(ck), oracle.e2m1_values(codes))
        nz = exps > 0
        assert np.array_equal(ek[nz].astype(np.int32), exps[nz].astype(np.int32) + k)
    y = x.clone()
    y[:, 32:64] = torch.tensor(rng.normal(size=(M, 32)).astype(np.float32)).to(torch.bfloat16) * 1000.0
    y[1:] = y[1:] * 3.0
    cy, ey = oracle.mx_quantize(bits(y), lam, 0.9)
    keep = np.r_[0:32, 64:128]
    assert np.array_equal(cy[0, keep], codes[0, keep]) and np.array_equal(ey[0, [0, 2, 3]], exps[0, [0, 2, 3]])
