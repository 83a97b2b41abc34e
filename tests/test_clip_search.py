"""Clipping-ratio search (Sec. III-C, Eq. 8-10): pins of the oracle's search (CPU) and parity of the CUDA search
against it (GPU, through the C ABI)."""
import math

import numpy as np
import pytest
import torch

import oracle
from workloads import generator as gen

G = 64


def bits(t):
    return gen.bf16_bits(t).numpy().view(np.uint16)


# ----------------------------------------------------------------------------- oracle pins (no GPU)
def _on_grid_layer(M=8, K=128, N=16, seed=3):
    """Everything exactly representable: activations k * 2^-3 with k in [-7, 7] and |k| = 7 present in every group,
    lambda = 1, weight codes times power-of-two scales, no low-rank branch, no bias.  With rho = 1 the
    quantizer reproduces the activations exactly, so the quantized layer equals the plain product."""
    rng = np.random.default_rng(seed)
    k = rng.integers(-7, 8, size=(M, K))
    k[:, ::G] = 7  # the group maximum is exactly 7 steps
    x = torch.tensor(k * 0.125, dtype=torch.float32).to(torch.bfloat16)
    qw = rng.integers(-8, 8, size=(K, N)).astype(np.int8)
    sw = (2.0 ** rng.integers(-6, -2, size=(K // G, N))).astype(np.float32)
    lam = np.ones(K, np.float32)
    return x, lam, qw, sw


def test_search_picks_the_exact_ratio_on_grid_data():
    # Closed form: Y_ref is the FP64 product of the raw inputs (no quantizer on this side); rho = 1 reproduces it
    # bit for bit (objective 0), every smaller ratio clips or re-grids at least the group maxima (objective > 0).
    x, lam, qw, sw = _on_grid_layer()
    W = qw.astype(np.float64).reshape(-1, G, qw.shape[1]) * sw.astype(np.float64)[:, None, :]
    y = x.to(torch.float64).numpy() @ W.reshape(qw.shape)
    yref = bits(torch.tensor(y, dtype=torch.float64).to(torch.bfloat16))
    cands = [0.5, 0.75, 0.9, 1.0]
    best, errs = oracle.clip_search([bits(x)], [yref], lam, cands, None, None, qw, sw, None)
    assert best == 3 and errs[3] == 0.0
    assert all(e > 0.0 for e in errs[:3])
    # Order of the candidates must not matter for the winner; samples add up.
    best2, errs2 = oracle.clip_search([bits(x), bits(x)], [yref, yref], lam, cands[::-1], None, None, qw, sw, None)
    assert best2 == 0 and errs2 == [2.0 * e for e in errs[::-1]]


def _brute_force_objective(x_rows, yref_rows, lam, rho, qw, sw, bias):
    """Eq. 3-5, 8-11 written out with scalar loops for a tiny layer without low-rank branch."""
    f32 = np.float32
    total = 0.0
    K, N = qw.shape
    for xr, yr in zip(x_rows, yref_rows):
        acc = np.zeros(N, np.float64)
        for g in range(K // G):
            xh = [f32(f32(xr[k]) * f32(f32(1.0) / f32(lam[k]))) for k in range(g * G, (g + 1) * G)]
            a = max(abs(v) for v in xh)
            if a == 0.0:
                continue
            s = f32(f32(f32(rho) * a) / f32(7.0))
            inv = f32(f32(1.0) / s)
            q = [int(min(7, max(-8, np.rint(f32(v * inv))))) for v in xh]
            for n in range(N):
                p = sum(q[j] * int(qw[g * G + j, n]) for j in range(G))
                acc[n] += float(p) * float(s) * float(sw[g, n])
        if bias is not None:
            acc += bias.astype(np.float64)
        yhat = torch.tensor(acc, dtype=torch.float64).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
        total += float(np.sum((yr - yhat) ** 2))
    return total


def test_search_objective_against_brute_force_on_a_tiny_layer():
    rng = np.random.default_rng(11)
    M, K, N = 3, 128, 4
    x = torch.tensor(rng.standard_normal((M, K)) * np.where(rng.random(K) < 0.05, 20.0, 1.0), dtype=torch.float32).to(torch.bfloat16)
    lam = np.exp(rng.standard_normal(K) * 0.3).astype(np.float32)
    qw = rng.integers(-8, 8, size=(K, N)).astype(np.int8)
    sw = np.exp(rng.uniform(math.log(2e-3), math.log(2e-2), size=(K // G, N))).astype(np.float32)
    bias = (rng.standard_normal(N) * 0.01).astype(np.float32)
    W = qw.astype(np.float64).reshape(-1, G, N) * sw.astype(np.float64)[:, None, :]
    yref_t = torch.tensor((x.to(torch.float64).numpy() / lam.astype(np.float64)) @ W.reshape(K, N) + bias, dtype=torch.float64).to(torch.bfloat16)
    cands = [0.55, 0.7, 0.85, 1.0]
    best, errs = oracle.clip_search([bits(x)], [bits(yref_t)], lam, cands, None, None, qw, sw, bias)
    xf, yf = x.to(torch.float32).numpy(), yref_t.to(torch.float64).numpy()
    want = [_brute_force_objective(xf, yf, lam, c, qw, sw, bias) for c in cands]
    assert np.allclose(errs, want, rtol=1e-12, atol=0.0)
    assert best == int(np.argmin(want))


# ----------------------------------------------------------------------------- CUDA parity
def _gpu_modules():
    import paper_2605_27003_b200 as w4
    return w4


def _search_case(M, K, N, r, n_samples, cands, seed, bias):
    w4 = _gpu_modules()
    dev = "cuda:0"
    idx = gen.outlier_channels(K, 0, seed, count=max(2, K // 128))
    xs = [gen.make_activations(M, K, outlier_idx=idx, outlier_gain=40.0, seed=seed + 10 * s) for s in range(n_samples)]
    layer = gen.make_layer_svd(K, N, r, xs[0], seed=seed + 1, bias_std=0.01 if bias else None)
    yrefs = [gen.reference_output(x, layer) for x in xs]
    want_best, want_errs = oracle.clip_search([bits(x) for x in xs], [bits(y) for y in yrefs], layer.lam.numpy(), cands,
                                              None if r == 0 else bits(layer.L1), None if r == 0 else bits(layer.L2),
                                              layer.qweight.numpy(), layer.wscale.numpy(),
                                              None if layer.bias is None else layer.bias.numpy())
    ctx = w4.Context(0, M, K, r)
    L = w4.Layer(ctx, [layer], num_bins=3, layer_id=1, num_layers=2)
    table = torch.full((1, 2, 3), 0.123, dtype=torch.float32, device=dev)
    xd = [x.to(dev) for x in xs]
    yd = [y.to(dev) for y in yrefs]
    best, errs = w4.w4a4_clip_search(L.ptr, xd, yd, M, 0, 2, cands, table)
    ctx.check()
    # The objective: every term differs from the oracle's only where FP32 accumulation moved a BF16 rounding.
    assert np.allclose(errs, want_errs, rtol=2e-3, atol=0.0), (errs, want_errs)
    # The winner is unique unless two objectives are closer than that tolerance; then either is valid.
    order = np.argsort(want_errs)
    if want_errs[order[1]] > want_errs[order[0]] * (1.0 + 5e-3):
        assert best == want_best
    else:
        assert errs[best] <= min(errs) * (1.0 + 1e-12)
    t = table.cpu()
    assert t[0, 1, 2].item() == np.float32(cands[best])
    t[0, 1, 2] = 0.123
    assert torch.all(t == 0.123), "only the searched entry may change"
    # The forward with the table's new entry is the forward with that ratio.
    Y1 = L.forward(xd[0], 0, 2, table)
    table2 = torch.full((1, 2, 3), float(np.float32(cands[best])), dtype=torch.float32, device=dev)
    Y2 = L.forward(xd[0], 0, 0, table2)
    torch.cuda.synchronize()
    assert torch.equal(Y1, Y2)
    L.close()
    ctx.close()


@pytest.mark.gpu
def test_clip_search_tiny_config():
    _search_case(256, 512, 512, 16, 2, [0.5, 0.6, 0.7, 0.8, 0.9, 1.0], seed=0, bias=False)


@pytest.mark.gpu
def test_clip_search_ragged_no_lowrank_with_bias():
    _search_case(200, 704, 384, 0, 1, [1.0, 0.65, 0.8], seed=5, bias=True)


@pytest.mark.gpu
def test_clip_search_rejects_bad_arguments():
    w4 = _gpu_modules()
    dev = "cuda:0"
    x = gen.make_activations(64, 128, seed=1)
    layer = gen.make_layer_svd(128, 128, 0, x, seed=2)
    ctx = w4.Context(0, 64, 128, 0)
    L = w4.Layer(ctx, [layer], num_bins=1)
    table = torch.ones((1, 1, 1), dtype=torch.float32, device=dev)
    xd, yd = x.to(dev), gen.reference_output(x, layer).to(dev)
    for cands in ([], [1.5], [0.0], [float("nan")]):
        with pytest.raises(w4.W4A4Error):
            w4.w4a4_clip_search(L.ptr, [xd], [yd], 64, 0, 0, cands, table)
    with pytest.raises(w4.W4A4Error):
        w4.w4a4_clip_search(L.ptr, [xd], [yd], 64, 0, 5, [1.0], table)   # bin out of range
    with pytest.raises(w4.W4A4Error):
        w4.w4a4_clip_search(L.ptr, [xd], [yd], 65, 0, 0, [1.0], table)   # M beyond the context
    assert table.item() == 1.0
    L.close()
    ctx.close()


# ----------------------------------------------------------------------------- MXFP4 variant
def test_mx_search_picks_the_exact_ratio_on_grid_data():
    # Activations that MXFP4 represents exactly at rho = 1 (block maximum 6 * 2^k), exact weights: Y_ref is the FP64
    # product of the raw inputs; rho = 1 reproduces it bit for bit, rho <= 0.5 lowers every shared exponent by one
    # and clips the block maxima (6 -> 12 saturates).
    rng = np.random.default_rng(4)
    M, K, N = 6, 128, 8
    grid = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0])
    xa = rng.choice(grid, size=(M, K)) * rng.choice([-1.0, 1.0], size=(M, K))
    xa[:, ::32] = 6.0
    x = torch.tensor(xa, dtype=torch.float32).to(torch.bfloat16)
    wcodes = rng.integers(0, 16, size=(K, N)).astype(np.uint8)
    wexps = rng.integers(122, 126, size=(K // 32, N)).astype(np.uint8)
    W = gen.mx_dequantize(torch.tensor(wcodes), torch.tensor(wexps)).numpy()
    yref = bits(torch.tensor(xa @ W, dtype=torch.float64).to(torch.bfloat16))
    cands = [0.4, 0.5, 0.8, 1.0]
    best, errs = oracle.mx_clip_search([bits(x)], [yref], np.ones(K, np.float32), cands, None, None, wcodes, wexps, None)
    assert errs[3] == 0.0 and errs[2] == 0.0        # 0.8 * 6 = 4.8 stays in the binade of 4: same exponent, same result
    assert errs[0] > 0.0 and errs[1] > 0.0           # 0.5 * 6 = 3 and 0.4 * 6 = 2.4 drop a binade: the 6s saturate
    assert best == 2                                 # the first of the tied minima


@pytest.mark.gpu
def test_mx_clip_search_parity():
    w4 = _gpu_modules()
    dev = "cuda:0"
    M, K, N, r = 200, 512, 384, 16
    cands = [0.45, 0.55, 0.7, 0.85, 1.0]
    idx = gen.outlier_channels(K, 0, 3, count=6)
    xs = [gen.make_activations(M, K, outlier_idx=idx, outlier_gain=40.0, seed=30 + s) for s in range(2)]
    layer = gen.make_layer_mx_svd(K, N, r, xs[0], seed=31, bias_std=0.01)
    yrefs = [gen.reference_output(x, layer) for x in xs]
    want_best, want_errs = oracle.mx_clip_search([bits(x) for x in xs], [bits(y) for y in yrefs], layer.lam.numpy(), cands,
                                                 bits(layer.L1), bits(layer.L2), layer.wcodes.numpy(), layer.wexps.numpy(),
                                                 layer.bias.numpy())
    ctx = w4.Context(0, M, K, r)
    L = w4.MxLayer(ctx, [layer.to(dev)], num_bins=2)
    table = torch.full((1, 1, 2), 0.123, dtype=torch.float32, device=dev)
    best, errs = w4.w4a4_mx_clip_search(L.ptr, [x.to(dev) for x in xs], [y.to(dev) for y in yrefs], M, 0, 1, cands, table)
    ctx.check()
    assert np.allclose(errs, want_errs, rtol=2e-3, atol=0.0), (errs, want_errs)
    order = np.argsort(want_errs)
    if want_errs[order[1]] > want_errs[order[0]] * (1.0 + 5e-3):
        assert best == want_best
    t = table.cpu()
    assert t[0, 0, 1].item() == np.float32(cands[best]) and t[0, 0, 0].item() == np.float32(0.123)
    L.close()
    ctx.close()
