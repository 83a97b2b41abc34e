"""Parity of the MXFP4 variant's CUDA path against the oracle, through the C ABI (GPU only)."""
import numpy as np
import pytest
import torch

import oracle
from workloads import generator as gen

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def bits(t):
    return gen.bf16_bits(t.cpu()).numpy().view(np.uint16)


def y_within_tolerance(y_gpu_bf16, y64):
    """Output tolerance of the layer: |Y_gpu - Y64| <= 2^-7 |Y64| + 1e-3 rms(Y64), rms over the compared outputs."""
    yg = y_gpu_bf16.to(torch.float64).cpu().numpy()
    rms = float(np.sqrt(np.mean(y64 ** 2)))
    bound = 2.0 ** -7 * np.abs(y64) + 1e-3 * rms
    return float(np.max(np.abs(yg - y64) / bound)), rms


def run_mx_case(x, experts, clip, expert_id, bin_id, rows=None, layer_id=0, num_layers=1, max_M=None):
    import paper_2605_27003_b200 as w4
    lay = experts[expert_id]
    M, K, N, r = x.shape[0], lay.K, lay.N, lay.r
    ctx = w4.Context(0, max_M or M, K, r)
    L = w4.MxLayer(ctx, [e.to(DEV) for e in experts], num_bins=clip.shape[2], layer_id=layer_id, num_layers=num_layers)
    clip_d = clip.to(DEV)
    rho = float(clip[expert_id, layer_id, bin_id])
    xd = x.to(DEV)
    codes = torch.full((M, K), 99, dtype=torch.uint8, device=DEV)
    exps = torch.full((M, K // 32), 77, dtype=torch.uint8, device=DEV)
    T = torch.zeros((M, max(r, 1)), dtype=torch.float32, device=DEV)
    w4.w4a4_mx_debug_quantize(L.ptr, xd, M, expert_id, bin_id, clip_d, codes, exps, T if r > 0 else None)
    Y = L.forward(xd, expert_id, bin_id, clip_d)
    torch.cuda.synchronize()
    ctx.check()
    rows = np.arange(M) if rows is None else np.asarray(rows)
    ref = oracle.mx_forward_rows(bits(x), rows.astype(np.int32), lay.lam.numpy(), rho,
                                 None if r == 0 else bits(lay.L1), None if r == 0 else bits(lay.L2),
                                 lay.wcodes.numpy(), lay.wexps.numpy(), None if lay.bias is None else lay.bias.numpy())
    rt = torch.as_tensor(rows, device=DEV)
    # element values (a negative zero and a positive zero are the same element) and scale bytes: exact
    assert np.array_equal(oracle.e2m1_values(codes[rt].cpu().numpy()), oracle.e2m1_values(ref["codes"])), "elements differ"
    assert np.array_equal(exps[rt].cpu().numpy(), ref["exps"]), "scale exponents differ"
    if r > 0:
        t_gpu, t_ref = T[rt].cpu().numpy().astype(np.float64), ref["T"].astype(np.float64)
        assert np.all(np.abs(t_gpu - t_ref) <= 1e-4 * np.abs(t_ref).max(axis=1, keepdims=True) + 1e-30)
    worst, _ = y_within_tolerance(Y[rt], ref["Y64"])
    assert worst <= 1.0, f"output outside tolerance: worst err/bound = {worst:.3f}"
    L.close()
    ctx.close()
    return worst


def mx_inputs(M, K, N, r, seed=0, bias=False):
    idx = gen.outlier_channels(K, 0, seed, count=max(2, K // 128))
    x = gen.make_activations(M, K, outlier_idx=idx, outlier_gain=40.0, seed=seed)
    return x, gen.make_layer_mx_svd(K, N, r, x, seed=seed + 1, bias_std=0.01 if bias else None)


def test_mx_tiny_config_full_parity():
    x, layer = mx_inputs(256, 512, 512, 16)
    run_mx_case(x, [layer], torch.full((1, 1, 1), 0.9), 0, 0)


@pytest.mark.parametrize("M,K,N,r,bias,rho", [
    (333, 768, 256, 32, True, 0.8),     # ragged M, three K stages
    (129, 256, 384, 0, True, 1.0),      # no low-rank branch, one K stage
    (200, 1024, 128, 64, False, 0.65),  # r = 64: two low-rank stages
    (1, 256, 128, 16, True, 0.9),       # a single token
])
def test_mx_ragged_shapes(M, K, N, r, bias, rho):
    x, layer = mx_inputs(M, K, N, r, seed=3 + M, bias=bias)
    clip = torch.full((1, 3, 4), 0.5)
    clip[0, 1, 2] = rho
    run_mx_case(x, [layer], clip, 0, 2, layer_id=1, num_layers=3, max_M=M + 77)


def test_mx_two_experts_direct_recipe():
    M, K, N, r = 300, 512, 256, 32
    x = gen.make_activations(M, K, outlier_idx=gen.outlier_channels(K, 0.02, 4), outlier_gain=50.0, seed=9)
    experts = [gen.make_layer_mx_direct(K, N, r, seed=20), gen.make_layer_mx_direct(K, N, r, seed=21)]
    clip = gen.make_clip_table(2, 1, 4, [(0.6, 1.0), (0.8, 1.0)], seed=5)
    run_mx_case(x, experts, clip, 1, 3)
    run_mx_case(x, experts, clip, 0, 1)


def test_mx_degenerate_inputs():
    # all-zero activations, a zero block inside a row, values that saturate
    K, N = 256, 128
    layer = gen.make_layer_mx_direct(K, N, 16, seed=2)
    x = torch.zeros(64, K, dtype=torch.bfloat16)
    run_mx_case(x, [layer], torch.ones(1, 1, 1), 0, 0)
    x = gen.make_activations(64, K, seed=3)
    x[:, 32:64] = 0
    x[5, 100] = 3.0e4
    run_mx_case(x, [layer], torch.full((1, 1, 1), 0.3), 0, 0)


def test_mx_argument_errors():
    import paper_2605_27003_b200 as w4
    ctx = w4.Context(0, 64, 512, 16)
    with pytest.raises(w4.W4A4Error):
        w4.MxLayer(ctx, [gen.make_layer_mx_direct(320, 128, 16, seed=1).to(DEV)], num_bins=1)   # K not a multiple of 256
    bad = gen.make_layer_mx_direct(256, 128, 0, seed=1)
    bad.wexps[0, 0] = 255
    with pytest.raises(w4.W4A4Error):
        w4.MxLayer(ctx, [bad.to(DEV)], num_bins=1)                                             # NaN scale byte
    L = w4.MxLayer(ctx, [gen.make_layer_mx_direct(256, 128, 0, seed=1).to(DEV)], num_bins=2)
    x = gen.make_activations(64, 256, seed=1).to(DEV)
    clip = torch.ones(1, 1, 2, device=DEV)
    with pytest.raises(w4.W4A4Error):
        L.forward(x, 0, 2, clip)
    with pytest.raises(w4.W4A4Error):
        L.forward(x, 1, 0, clip)
    Y = L.forward(x[:0], 0, 0, clip)
    assert Y.shape == (0, 128)
    L.close()
    ctx.close()


@pytest.mark.parametrize("name", ["attn_proj", "ffn_up", "ffn_down"])
def test_mx_full_size_sampled_rows(name):
    # The three layer shapes of the DiT at M = 32760: tile-boundary rows (the pair kernel's 256-row tiles included)
    # plus 256 seeded random rows, all output columns.
    shape = gen.CONFIG_SHAPES[name]
    M, K, N, r = shape["M"], shape["K"], shape["N"], shape["r"]
    dist = "gelu" if name == "ffn_down" else "normal"
    x = gen.make_activations(M, K, sigma=1.0 if dist == "gelu" else gen.sigma_for_bin(2), dist=dist,
                             outlier_idx=gen.outlier_channels(K, 0.01, 7), outlier_gain=80.0 if dist == "gelu" else 50.0,
                             seed=31, device=DEV).cpu()
    layer = gen.make_layer_mx_direct(K, N, r, seed=32)
    rng = np.random.default_rng(1)
    last = (M - 1) // 128 * 128
    rows = sorted({0, 127, 128, 255, 256, last - 1, last, M - 1, *rng.choice(M, 256, replace=False).tolist()})
    clip = gen.make_clip_table(1, 1, 8, [(0.6, 1.0)], seed=6)
    run_mx_case(x, [layer], clip, 0, 2, rows=rows)
