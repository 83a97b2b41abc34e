"""Parity of the CUDA path (through the C ABI) with the CPU oracle, element by element.

Bars: integer codes, group scales and per-group int32 partial sums bit-exact; the BF16 output within
|Y_gpu - Y_oracle| <= 2^-7 |Y_oracle| + 1e-3 rms(Y_oracle) (rms over the compared rows); the low-rank
intermediate T (FP32 accumulation on the GPU, FP64 in the oracle) within 1e-4 relative to the row's
largest |T|.
"""
import os

import numpy as np
import pytest
import torch

import oracle
import paper_2605_27003_b200 as w4
from paper_2605_27003_b200 import build as pkg_build
from workloads import generator as gen

pytestmark = pytest.mark.gpu
G = 64
DEV = "cuda:0"


@pytest.fixture(scope="module", autouse=True)
def _built():
    pkg_build.build()
    w4.load_library()


def bits(t):
    return gen.bf16_bits(t.cpu()).numpy().view(np.uint16)


def y_within_tolerance(y_gpu_bf16: torch.Tensor, y64: np.ndarray):
    got = y_gpu_bf16.to(torch.float64).cpu().numpy()
    rms = float(np.sqrt(np.mean(y64 ** 2)))
    bound = 2.0 ** -7 * np.abs(y64) + 1e-3 * rms
    err = np.abs(got - y64)
    worst = float((err / bound).max()) if err.size else 0.0
    return worst, rms


def oracle_rows(x_rows: torch.Tensor, layer, rho: float, want_partials=False):
    rows = np.arange(x_rows.shape[0], dtype=np.int32)
    return oracle.forward_rows(
        bits(x_rows), rows, layer.lam.cpu().numpy(), rho,
        None if layer.L1 is None else bits(layer.L1), None if layer.L2 is None else bits(layer.L2),
        layer.qweight.cpu().numpy(), layer.wscale.cpu().numpy(),
        None if layer.bias is None else layer.bias.cpu().numpy(), want_partials=want_partials)


GUARD = 3   # sentinel rows in front of and behind every output buffer of run_case


def guarded(shape, dtype, sentinel):
    """A tensor of `shape` cut out of a larger allocation whose GUARD leading and trailing rows hold `sentinel`."""
    rows = shape[0]
    buf = torch.full((rows + 2 * GUARD,) + tuple(shape[1:]), sentinel, dtype=dtype, device=DEV)
    return buf, buf[GUARD:GUARD + rows]


def guards_intact(buf, sentinel):
    ref = torch.full_like(buf[:GUARD], sentinel)
    return torch.equal(buf[:GUARD], ref) and torch.equal(buf[buf.shape[0] - GUARD:], ref)


def run_case(x: torch.Tensor, experts, clip: torch.Tensor, expert_id: int, bin_id: int, rows=None,
             check_partials_tiles=(), layer_id=0, num_layers=1, max_M=None):
    """Runs quantize tap + forward (+ partial taps) on the GPU and compares with the oracle on `rows`.  Every output
    buffer sits between sentinel guard rows that must come back untouched."""
    M, K = x.shape
    lay = experts[expert_id]
    N, r = lay.N, lay.r
    ctx = w4.Context(0, max_M or max(M, 1), K, r)
    L = w4.Layer(ctx, [e.to(DEV) for e in experts], num_bins=clip.shape[2], num_layers=num_layers, layer_id=layer_id)
    clip_d = clip.to(DEV)
    rho = float(clip[expert_id, layer_id, bin_id])
    xd = x.to(DEV)
    codes_buf, codes = guarded((M, K), torch.int8, 99)
    scales_buf, scales = guarded((M, K // G), torch.float32, -1.0)
    t_buf, T = guarded((M, max(r, 1)), torch.float32, -7.0)
    y_buf, Y = guarded((M, N), torch.bfloat16, 1234.0)
    w4.w4a4_debug_quantize(L.ptr, xd, M, expert_id, bin_id, clip_d, codes, scales, T if r > 0 else None)
    w4.w4a4_linear_forward(L.ptr, xd, M, expert_id, bin_id, clip_d, Y)
    torch.cuda.synchronize()
    ctx.check()
    assert guards_intact(codes_buf, 99) and guards_intact(scales_buf, -1.0) and guards_intact(t_buf, -7.0), \
        "the quantize tap wrote outside its buffers"
    assert guards_intact(y_buf, 1234.0), "the forward wrote outside Y"
    if rows is None:
        rows = np.arange(M)
    rows = np.asarray(rows)
    ref = oracle_rows(x[rows], lay, rho)
    rt = torch.from_numpy(rows).to(DEV)
    assert np.array_equal(codes[rt].cpu().numpy(), ref["q"]), "activation codes differ"
    assert np.array_equal(scales[rt].cpu().numpy().view(np.uint32), ref["s"].view(np.uint32)), "scales differ"
    if r > 0:
        t_gpu = T[rt].cpu().numpy().astype(np.float64)
        t_ref = ref["T"].astype(np.float64)
        tol = 1e-4 * np.abs(t_ref).max(axis=1, keepdims=True) + 1e-30
        assert np.all(np.abs(t_gpu - t_ref) <= tol), "low-rank intermediate differs"
    worst, rms = y_within_tolerance(Y[rt], ref["Y64"])
    assert worst <= 1.0, f"output outside tolerance: worst err/bound = {worst:.3f} (rms {rms:.4g})"
    bm, bn = w4.w4a4_tile_shape()
    for (m0, n0) in check_partials_tiles:
        p_buf, P = guarded((bm, K // G, bn), torch.int32, -5)
        y2_buf, Y2 = guarded((M, N), torch.bfloat16, 1234.0)
        w4.w4a4_debug_partials(L.ptr, xd, M, expert_id, bin_id, clip_d, Y2, m0, n0, P)
        torch.cuda.synchronize()
        ctx.check()
        assert guards_intact(p_buf, -5) and guards_intact(y2_buf, 1234.0), "the partial-sum tap wrote outside its buffers"
        assert torch.equal(Y2, Y), "the debug-tap forward must give the same output"
        # The oracle's partial sums of the compared rows that fall into the tile (at most 12 of them: the array
        # is [rows, G, N] int32).
        sel = [int(rw) for rw in rows if m0 <= rw < min(m0 + bm, M)][:12]
        assert sel, "no compared row falls into the requested tile"
        pref = oracle_rows(x[np.array(sel)], lay, rho, want_partials=True)["P"]
        Pg = P.cpu().numpy()
        for i, rw in enumerate(sel):
            assert np.array_equal(Pg[rw - m0], pref[i][:, n0:n0 + bn]), f"partials differ at row {rw}"
    L.close()
    ctx.close()
    return worst


def tiny_inputs(M=256, K=512, N=512, r=16, seed=0, bias=False):
    idx = gen.outlier_channels(K, 0, seed, count=4)
    x = gen.make_activations(M, K, outlier_idx=idx, outlier_gain=40.0, seed=seed)
    layer = gen.make_layer_svd(K, N, r, x, seed=seed + 1, bias_std=0.01 if bias else None)
    return x, layer


@pytest.mark.parametrize("sc", [1, 2, 3, 5])
def test_tile_order_in_super_columns_gives_the_same_result(sc):
    # The GEMM walks its output tiles in super-columns (all row blocks of `sc` column tiles before the next `sc`), sized
    # for the L2 at full scale.  Forced here on a layer of 3 row blocks x 5 column tiles: widths that divide the
    # column count, that leave a narrower last super-column, and the plain order; every tile's output against the
    # oracle and the partial sums of the first and last tile.
    M, K, N, r = 300, 256, 640, 16
    x, layer = tiny_inputs(M, K, N, r, seed=21, bias=True)
    clip = torch.full((1, 1, 1), 0.8, dtype=torch.float32)
    ctx = w4.Context(0, M, K, r)
    w4.w4a4_debug_set_tile_order(ctx.ptr, sc)
    L = w4.Layer(ctx, [layer.to(DEV)], num_bins=1)
    y = L.forward(x.to(DEV), 0, 0, clip.to(DEV))
    bm, bn = w4.w4a4_tile_shape()
    P = torch.full((bm, K // G, bn), -5, dtype=torch.int32, device=DEV)
    y2 = torch.empty_like(y)
    w4.w4a4_debug_partials(L.ptr, x.to(DEV), M, 0, 0, clip.to(DEV), y2, 256, 512, P)
    torch.cuda.synchronize()
    ctx.check()
    ref = oracle_rows(x, layer, 0.8, want_partials=True)
    worst, _ = y_within_tolerance(y, ref["Y64"])
    assert worst <= 1.0 and torch.equal(y, y2)
    Pg = P.cpu().numpy()
    for row in range(256, M):
        assert np.array_equal(Pg[row - 256], ref["P"][row][:, 512:640])
    L.close()
    ctx.close()


def test_tiny_config_full_parity():
    # M=256, K=N=512, r=16, one bin with rho=0.9, no bias; every row, every tile's partial sums.
    x, layer = tiny_inputs()
    clip = torch.full((1, 1, 1), 0.9, dtype=torch.float32)
    tiles = [(m0, n0) for m0 in (0, 128) for n0 in (0, 128, 256, 384)]
    run_case(x, [layer], clip, 0, 0, check_partials_tiles=tiles)


@pytest.mark.parametrize("M,K,N,r,bias", [
    (333, 640, 256, 32, True),    # ragged M, G=10 (not a multiple of 4)
    (200, 704, 128, 64, True),    # G=11: odd group count -> half-filled last stage; r=64 -> two low-rank stages
    (129, 512, 384, 0, True),     # no low-rank branch
    (1, 128, 128, 16, False),     # a single token, a single stage
    (127, 1024, 256, 32, False),
])
def test_ragged_shapes_and_ranks(M, K, N, r, bias):
    x, layer = tiny_inputs(M, K, N, r, seed=10 + r + M, bias=bias)
    clip = gen.make_clip_table(1, 3, 4, [(0.6, 1.0)], seed=M)
    last_tile_m0 = ((M - 1) // 128) * 128
    run_case(x, [layer], clip, 0, 2, check_partials_tiles=[(0, 0), (last_tile_m0, N - 128)], layer_id=1, num_layers=3,
             max_M=M + 77)


def test_two_experts_and_bins_select_their_own_constants():
    M, K, N, r = 160, 512, 256, 16
    x, e0 = tiny_inputs(M, K, N, r, seed=3, bias=True)
    e1 = gen.make_layer_direct(K, N, r, seed=4)
    clip = gen.make_clip_table(2, 2, 8, [(0.6, 1.0), (0.8, 1.0)], seed=5)
    for expert, b in ((0, 0), (1, 7), (1, 3)):
        run_case(x, [e0, e1], clip, expert, b, layer_id=1, num_layers=2)


def test_degenerate_inputs_zero_rows_and_exact_grid():
    M, K, N, r = 140, 256, 128, 16
    x, layer = tiny_inputs(M, K, N, r, seed=6)
    x = x.clone()
    x[5] = 0          # an all-zero token
    x[7, 64:128] = 0  # an all-zero group
    xi = torch.randint(-7, 8, (K,), generator=torch.Generator().manual_seed(1)).to(torch.float32)
    xi[::64] = 7.0
    x[9] = (xi * layer.lam * 0.25).to(torch.bfloat16)  # roughly on-grid row
    clip = torch.tensor([[[1.0, 0.5]]], dtype=torch.float32)
    run_case(x, [layer], clip, 0, 0, check_partials_tiles=[(0, 0)])
    run_case(x, [layer], clip, 0, 1, check_partials_tiles=[(128, 0)])


def test_empty_batch_and_argument_errors():
    x, layer = tiny_inputs(64, 128, 128, 16, seed=8)
    ctx = w4.Context(0, 64, 128, 16)
    L = w4.Layer(ctx, [layer.to(DEV)], num_bins=2)
    clip = torch.ones(1, 1, 2, device=DEV)
    Y = torch.empty(64, 128, dtype=torch.bfloat16, device=DEV)
    w4.w4a4_linear_forward(L.ptr, x.to(DEV), 0, 0, 0, clip, Y)  # M = 0: nothing launched, no error
    for kwargs, status in ((dict(M=65), 2), (dict(expert=1), 1), (dict(bin=2), 1)):
        with pytest.raises(w4.W4A4Error) as ei:
            w4.w4a4_linear_forward(L.ptr, x.to(DEV), kwargs.get("M", 64), kwargs.get("expert", 0),
                                   kwargs.get("bin", 0), clip, Y)
        assert ei.value.status == status
    bad = gen.make_layer_direct(128, 128, 16, seed=1)
    bad.qweight[3, 5] = 9
    with pytest.raises(w4.W4A4Error) as ei:
        w4.Layer(ctx, [bad.to(DEV)], num_bins=2)
    assert ei.value.status == 1
    with pytest.raises(w4.W4A4Error) as ei:
        w4.Layer(ctx, [gen.make_layer_direct(256, 128, 16, seed=1).to(DEV)], num_bins=2)  # K beyond the context
    assert ei.value.status == 2
    torch.cuda.synchronize()
    ctx.check()
    L.close()
    ctx.close()


# ----------------------------------------------------------------------------- full-size workloads, sampled rows
def sampled_rows(M, n_random, seed):
    """The tile-boundary rows (first and last row, both sides of the first tile boundary and of the last one) plus
    n_random seeded rows: rows are independent, so the oracle on a row subset is exact for those rows."""
    fixed = [0, 127, 128, M - 1, (M - 1) // 128 * 128, (M - 1) // 128 * 128 - 1]
    rng = np.random.default_rng(seed)
    rnd = rng.choice(M, size=n_random, replace=False).tolist()
    return np.array(sorted(set(r for r in fixed + rnd if 0 <= r < M)))


def big_layer(K, N, r, x_calib, seed):
    return gen.make_layer_svd(K, N, r, x_calib, seed=seed, bias_std=0.01, device=DEV, exact_svd=False,
                              keep_float64=False).to("cpu")


def test_attention_projection_full_size_sampled_rows():
    # M = 32760 (21 x 30 x 52 latent grid), K = N = 5120, r = 32; sigma decays over 8 bins; 1% outlier channels x50.
    M, K, N, r = 32760, 5120, 5120, 32
    idx = gen.outlier_channels(K, 0.01, 2)
    clip = gen.make_clip_table(1, 1, 8, [(0.6, 1.0)], seed=2)
    calib = gen.make_activations(1024, K, sigma=gen.sigma_for_bin(0), outlier_idx=idx, outlier_gain=50.0, seed=2000,
                                 device=DEV)
    layer = big_layer(K, N, r, calib, 2001)
    for b in (0, 5):
        x = gen.make_activations(M, K, sigma=gen.sigma_for_bin(b), outlier_idx=idx, outlier_gain=50.0, seed=2002 + b,
                                 device=DEV).cpu()
        rows = sampled_rows(M, 256, b)
        last = (M - 1) // 128 * 128
        run_case(x, [layer], clip, 0, b, rows=rows, check_partials_tiles=[(0, 0), (last, N - 128)])


def test_packed_qkv_full_size_sampled_rows():
    # The self-attention q, k and v of the DiT workload as one layer: M = 32760, K = 5120, N = 3 x 5120, joint rank 96
    # (three rank-32 projections; L2 block-diagonal), direct-recipe constants.  At this size the activation kernel runs
    # its widest instantiation, the GEMM three low-rank stages per tile and two super-columns of 60 column tiles.
    M, K, N1, r = 32760, 5120, 5120, 32
    lay = gen.make_layer_direct(K, 3 * N1, 3 * r, seed=4400, device=DEV)
    for i in range(3):
        for j in range(3):
            if i != j:
                lay.L2[r * i:r * (i + 1), N1 * j:N1 * (j + 1)] = 0
    lay = lay.to("cpu")
    clip = gen.make_clip_table(1, 1, 8, [(0.6, 1.0)], seed=5)
    x = gen.make_activations(M, K, sigma=gen.sigma_for_bin(2), outlier_idx=gen.outlier_channels(K, 0.01, 44), outlier_gain=50.0,
                             seed=4401, device=DEV).cpu()
    rows = sampled_rows(M, 64, 9)
    last = (M - 1) // 128 * 128
    run_case(x, [lay], clip, 0, 2, rows=rows, check_partials_tiles=[(0, 0), (last, 3 * N1 - 128)])


def test_ffn_pair_full_size_sampled_rows():
    # up 5120 -> 13824 and down 13824 -> 5120 at M = 32760; the down input is GELU of a Gaussian with
    # 1% outlier channels x80; two experts with their own clip tables.
    M, r = 32760, 32
    clip = gen.make_clip_table(2, 1, 8, [(0.6, 1.0), (0.8, 1.0)], seed=3)
    # up projection
    K, N = 5120, 13824
    idx = gen.outlier_channels(K, 0.01, 3)
    calib = gen.make_activations(1024, K, sigma=1.0, outlier_idx=idx, outlier_gain=50.0, seed=3000, device=DEV)
    up = big_layer(K, N, r, calib, 3001)
    x = gen.make_activations(M, K, sigma=1.0, outlier_idx=idx, outlier_gain=50.0, seed=3002, device=DEV).cpu()
    rows = sampled_rows(M, 256, 31)
    run_case(x, [up, up], clip, 1, 4, rows=rows, check_partials_tiles=[((M - 1) // 128 * 128, 0)])
    del x, up
    # down projection
    K, N = 13824, 5120
    idx = gen.outlier_channels(K, 0.01, 4)
    calib = gen.make_activations(1024, K, dist="gelu", outlier_idx=idx, outlier_gain=80.0, seed=3003, device=DEV)
    down = big_layer(K, N, r, calib, 3004)
    x = gen.make_activations(M, K, dist="gelu", outlier_idx=idx, outlier_gain=80.0, seed=3005, device=DEV).cpu()
    run_case(x, [down, down], clip, 0, 1, rows=rows, check_partials_tiles=[(0, N - 128)])


def test_dit_step_layers_both_experts_sampled_rows():
    # Layers of one denoising step (direct-recipe constants, two resident experts, 8 bins, several layers in
    # the clip table): the step index picks expert (s >= 20) and bin s // 5; parity per distinct shape.
    M, r = 32760, 32
    clip = gen.make_clip_table(2, 4, 8, [(0.6, 1.0), (0.8, 1.0)], seed=4)
    rows = sampled_rows(M, 24, 41)
    for layer_id, (K, N, step) in enumerate(((5120, 5120, 3), (5120, 13824, 22), (13824, 5120, 39))):
        expert, b = (1 if step >= 20 else 0), step // 5
        experts = [gen.make_layer_direct(K, N, r, seed=4000 + 2 * layer_id + e, device=DEV).to("cpu") for e in range(2)]
        dist = "gelu" if K == 13824 else "normal"
        x = gen.make_activations(M, K, dist=dist, outlier_idx=gen.outlier_channels(K, 0.01, 40 + K), outlier_gain=50.0,
                                 seed=4100 + layer_id, device=DEV).cpu()
        run_case(x, experts, clip, expert, b, rows=rows, layer_id=layer_id, num_layers=4,
                 check_partials_tiles=[((M - 1) // 128 * 128, N - 128)])
        del x, experts


SWEEP_POINTS = [(1560, K, N, r, frac, alpha)            # one latent frame: every (K, N, r) of the sweep
                for (K, N) in ((5120, 5120), (5120, 13824), (13824, 5120))
                for (r, frac, alpha) in ((0, 0.0, 0.7), (16, 0.01, 1.0), (32, 0.05, 0.7), (64, 0.01, 1.0))] + [
    (32760, 5120, 5120, 64, 0.05, 1.0),    # the widest rank at the main token count
    (75600, 5120, 13824, 16, 0.01, 0.7),   # the largest token count (21 x 45 x 80 grid)
    (75600, 13824, 5120, 0, 0.0, 1.0),
]


@pytest.mark.parametrize("M,K,N,r,frac,alpha", SWEEP_POINTS)
def test_sweep_points_sampled_rows(M, K, N, r, frac, alpha):
    layer = gen.make_layer_direct(K, N, r, seed=5000 + r + K // 64, device=DEV).to("cpu")
    x = gen.make_activations(M, K, outlier_idx=gen.outlier_channels(K, frac, 50), outlier_gain=50.0, seed=5100,
                             device=DEV).cpu()
    clip = torch.tensor([[[alpha]]], dtype=torch.float32)
    run_case(x, [layer], clip, 0, 0, rows=sampled_rows(M, 18, 51), check_partials_tiles=[(0, 0)])


def test_host_buffer_forward_equals_device_forward():
    # X and Y in pinned host memory, M split into chunks with a ragged last chunk: rows are independent, so
    # the chunked three-stream pipeline must reproduce the device-resident forward bit for bit.
    M, K, N, r = 1000, 512, 256, 16
    x, layer = tiny_inputs(M, K, N, r, seed=12, bias=True)
    ctx = w4.Context(0, M, K, r)
    L = w4.Layer(ctx, [layer.to(DEV)], num_bins=2)
    clip = torch.tensor([[[0.9, 0.7]]], dtype=torch.float32, device=DEV)
    y_dev = L.forward(x.to(DEV), 0, 1, clip)
    with pytest.raises(w4.W4A4Error):  # host I/O has to be enabled first
        w4.w4a4_linear_forward_host(L.ptr, x.pin_memory(), M, 0, 1, clip, torch.empty(M, N, dtype=torch.bfloat16).pin_memory())
    w4.w4a4_ctx_enable_host_io(ctx.ptr, 384, N)
    xh = x.pin_memory()
    for _ in range(2):
        yh = torch.zeros(M, N, dtype=torch.bfloat16).pin_memory()
        w4.w4a4_linear_forward_host(L.ptr, xh, M, 0, 1, clip, yh)
        torch.cuda.synchronize()
        assert torch.equal(yh, y_dev.cpu())
    ctx.check()
    L.close()
    ctx.close()


@pytest.mark.parametrize("M,K,N,r", [(300, 512, 256, 16), (391, 1024, 384, 32)])
def test_qkv_packed_as_one_layer_shares_one_activation_pass(M, K, N, r):
    # q, k and v read the same input with the same smoothing vector and the same clipping-ratio entry, so their
    # activation quantization and low-rank down-projection can be done once: pack the three projections as ONE layer
    # along N (codes, scales and bias side by side; L1 side by side, L2 block-diagonal; joint rank 3 r, padded to 64
    # at r = 16 and 96 at the rank the DiT workload uses).  The packed layer must give what the three layers give
    # (same codes and scales by construction; the output within the layer's tolerance, because the low-rank sum now
    # runs over 3 r terms, two thirds of them exact zeros), and what the oracle gives for the packed constants.
    R = 64 if r == 16 else 3 * r
    idx = gen.outlier_channels(K, 0, 5, count=4)
    x = gen.make_activations(M, K, outlier_idx=idx, outlier_gain=40.0, seed=5)
    parts = [gen.make_layer_svd(K, N, r, x, seed=50 + i, bias_std=0.01) for i in range(3)]
    lam = parts[0].lam
    for p_ in parts:                               # one smoothing vector for the three projections
        p_.lam = lam
    L1 = torch.zeros((K, R), dtype=torch.bfloat16)
    L2 = torch.zeros((R, 3 * N), dtype=torch.bfloat16)
    for i, p_ in enumerate(parts):
        L1[:, r * i:r * (i + 1)] = p_.L1
        L2[r * i:r * (i + 1), N * i:N * (i + 1)] = p_.L2
    packed = gen.LayerInputs(K, 3 * N, R, lam, L1, L2, torch.cat([p_.qweight for p_ in parts], dim=1),
                             torch.cat([p_.wscale for p_ in parts], dim=1), torch.cat([p_.bias for p_ in parts]))
    clip = torch.full((1, 1, 2), 0.85)
    ctx = w4.Context(0, M, K, R)
    clip_d, xd = clip.to(DEV), x.to(DEV)
    Lp = w4.Layer(ctx, [packed.to(DEV)], num_bins=2)
    Yp = Lp.forward(xd, 0, 1, clip_d).float().cpu().numpy()
    ctx.check()
    # the joint down-projection against the oracle's, column block by column block
    codes = torch.empty((M, K), dtype=torch.int8, device=DEV)
    scales = torch.empty((M, K // G), dtype=torch.float32, device=DEV)
    T = torch.empty((M, R), dtype=torch.float32, device=DEV)
    w4.w4a4_debug_quantize(Lp.ptr, xd, M, 0, 1, clip_d, codes, scales, T)
    torch.cuda.synchronize()
    Lp.close()
    ys = []
    for p_ in parts:
        Li = w4.Layer(ctx, [p_.to(DEV)], num_bins=2)
        ys.append(Li.forward(xd, 0, 1, clip_d).float().cpu().numpy())
        ctx.check()
        Li.close()
    ctx.close()
    Ys = np.concatenate(ys, axis=1)
    ref = oracle_rows(x, packed, 0.85)
    assert np.array_equal(codes.cpu().numpy(), ref["q"]) and \
        np.array_equal(scales.cpu().numpy().view(np.uint32), ref["s"].view(np.uint32))
    t_ref = ref["T"].astype(np.float64)
    assert np.all(np.abs(T.cpu().numpy() - t_ref) <= 1e-4 * np.abs(t_ref).max(axis=1, keepdims=True) + 1e-30)
    Y64 = ref["Y64"]
    bound = 2.0 ** -7 * np.abs(Y64) + 1e-3 * np.sqrt(np.mean(Y64 ** 2))
    assert np.all(np.abs(Yp - Y64) <= bound) and np.all(np.abs(Ys - Y64) <= bound)
    assert np.mean(Yp == Ys) > 0.9                 # nearly always the same BF16 value
