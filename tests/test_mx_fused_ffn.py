"""Fused pair of MXFP4 layers (the FFN: up-projection whose GEMM epilogue quantizes for the down-projection):
parity against the oracle through the C ABI (GPU only).

The fused epilogue must produce for the second layer exactly what that layer's own activation kernel would produce
from the first layer's stored BF16 output.  The first layer's output (checked against the oracle in its own tests)
is taken from the unfused path, which computes it with the same arithmetic; the oracle then quantizes it and runs
the second layer in FP64."""
import numpy as np
import pytest
import torch

import oracle
from workloads import generator as gen

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def bits(t):
    return gen.bf16_bits(t.cpu()).numpy().view(np.uint16)


def run_fused_case(M, K, H, N2, r1, r2, act, rho1, rho2, bias, seed=0):
    import paper_2605_27003_b200 as w4
    idx = gen.outlier_channels(K, 0, seed, count=max(2, K // 128))
    x = gen.make_activations(M, K, outlier_idx=idx, outlier_gain=40.0, seed=seed)
    up = gen.make_layer_mx_svd(K, H, r1, x, seed=seed + 1, bias_std=0.01 if bias else None)
    hid = gen.make_activations(M, H, outlier_idx=gen.outlier_channels(H, 0, seed + 2, count=max(2, H // 128)),
                               outlier_gain=20.0, seed=seed + 2)
    down = gen.make_layer_mx_svd(H, N2, r2, hid, seed=seed + 3, bias_std=0.01 if bias else None)
    ctx = w4.Context(0, M + 5, max(K, H), max(r1, r2))
    clip = torch.full((1, 2, 3), 0.5)
    clip[0, 0, 1], clip[0, 1, 1] = rho1, rho2
    clip_d = clip.to(DEV)
    Lup = w4.MxLayer(ctx, [up.to(DEV)], num_bins=3, num_layers=2, layer_id=0, output_activation=act)
    Ldn = w4.MxLayer(ctx, [down.to(DEV)], num_bins=3, num_layers=2, layer_id=1)
    xd = x.to(DEV)
    # unfused path: the first layer's BF16 output, and the two-call result for comparison
    y1 = Lup.forward(xd, 0, 1, clip_d)
    y2_two_calls = Ldn.forward(y1, 0, 1, clip_d)
    # fused path
    y2 = torch.empty(M, N2, dtype=torch.bfloat16, device=DEV)
    w4.w4a4_mx_ffn_forward(Lup.ptr, Ldn.ptr, xd, M, 0, 1, clip_d, y2)
    codes = torch.full((M, H), 99, dtype=torch.uint8, device=DEV)
    exps = torch.full((M, H // 32), 77, dtype=torch.uint8, device=DEV)
    T = torch.zeros((M, max(r2, 1)), dtype=torch.float32, device=DEV)
    w4.w4a4_mx_debug_fused_input(Ldn.ptr, M, codes, exps, T if r2 > 0 else None)
    torch.cuda.synchronize()
    ctx.check()
    rows = np.arange(M).astype(np.int32)
    # The oracle's second layer is fed the GPU's own first-layer output y1 here (itself checked against the oracle in
    # test_mx_gpu_parity.py): codes and exponents are compared bit for bit, and a first-layer output that differs
    # from the oracle's by one BF16 ulp -- which the layer's tolerance allows -- legitimately changes them.  The
    # chain with no GPU intermediate is test_fused_ffn_against_the_oracle_only_chain below.
    ref = oracle.mx_forward_rows(bits(y1), rows, down.lam.numpy(), float(rho2),
                                 None if r2 == 0 else bits(down.L1), None if r2 == 0 else bits(down.L2),
                                 down.wcodes.numpy(), down.wexps.numpy(), None if down.bias is None else down.bias.numpy())
    assert np.array_equal(oracle.e2m1_values(codes.cpu().numpy()), oracle.e2m1_values(ref["codes"])), "elements differ"
    assert np.array_equal(exps.cpu().numpy(), ref["exps"]), "scale exponents differ"
    if r2 > 0:
        t_gpu, t_ref = T.cpu().numpy().astype(np.float64), ref["T"].astype(np.float64)
        assert np.all(np.abs(t_gpu - t_ref) <= 1e-4 * np.abs(t_ref).max(axis=1, keepdims=True) + 1e-30), "T differs"
    y64 = ref["Y64"]
    rms = float(np.sqrt(np.mean(y64 ** 2)))
    bound = 2.0 ** -7 * np.abs(y64) + 1e-3 * rms
    worst = float(np.max(np.abs(y2.to(torch.float64).cpu().numpy() - y64) / bound))
    assert worst <= 1.0, f"fused output outside tolerance: worst err/bound = {worst:.3f}"
    # The two paths feed the second GEMM the same codes and exponents; T may differ in its last bit.
    d = (y2.to(torch.float32) - y2_two_calls.to(torch.float32)).abs().max().item()
    assert d <= 2.0 ** -6 * max(1.0, y2_two_calls.abs().max().item()), f"fused and two-call results differ by {d}"
    Lup.close()
    Ldn.close()
    ctx.close()


@pytest.mark.parametrize("M,K,H,N2,r1,r2,act,bias", [
    (333, 512, 768, 256, 16, 32, 1, True),     # ragged M (three row tiles: the last pair has one), GELU, three column tiles
    (256, 256, 512, 128, 0, 16, 1, False),     # no low-rank branch upstream, r' = 16
    (300, 512, 768, 512, 32, 64, 0, True),     # r' = 64 (two T buffers of 64 columns), no activation
    (517, 256, 1024, 256, 32, 0, 1, True),     # next layer without a low-rank branch
    (129, 256, 256, 128, 64, 16, 1, False),    # one row past the first tile, a single column tile, r = 64 upstream
    (1025, 512, 1536, 384, 16, 32, 1, True),   # nine row tiles (an odd count), six column tiles = one full run
    (640, 256, 1792, 128, 0, 32, 0, False),    # seven column tiles: a run of six and a run of one
])
def test_fused_ffn_matches_oracle(M, K, H, N2, r1, r2, act, bias):
    run_fused_case(M, K, H, N2, r1, r2, act, 0.9, 0.8, bias, seed=11 + M)


def test_fused_ffn_against_the_oracle_only_chain():
    """Oracle layer 1 -> GELU -> BF16 -> oracle layer 2, no GPU value anywhere in the expected result.  The GPU's
    hidden activation may differ from the oracle's by a BF16 ulp where the layer tolerance allows it, and the second
    layer's quantizer is not continuous, so the bound has two parts: the layer tolerance around the oracle-only
    result, plus D = |oracle layer 2 on the GPU's hidden - oracle layer 2 on the oracle's hidden|, the oracle's own
    sensitivity to that difference (both terms of D are CPU results; the GPU only supplies an input of one of them)."""
    import paper_2605_27003_b200 as w4
    M, K, H, N2, r1, r2, rho1, rho2 = 333, 512, 768, 256, 16, 32, 0.9, 0.8
    idx = gen.outlier_channels(K, 0, 3, count=4)
    x = gen.make_activations(M, K, outlier_idx=idx, outlier_gain=40.0, seed=3)
    up = gen.make_layer_mx_svd(K, H, r1, x, seed=4, bias_std=0.01)
    hid = gen.make_activations(M, H, outlier_idx=gen.outlier_channels(H, 0, 5, count=6), outlier_gain=20.0, seed=5)
    down = gen.make_layer_mx_svd(H, N2, r2, hid, seed=6, bias_std=0.01)
    rows = np.arange(M).astype(np.int32)

    def second_layer(h_bits):
        return oracle.mx_forward_rows(h_bits, rows, down.lam.numpy(), rho2, bits(down.L1), bits(down.L2), down.wcodes.numpy(),
                                      down.wexps.numpy(), down.bias.numpy())["Y64"]

    r1o = oracle.mx_forward_rows(bits(x), rows, up.lam.numpy(), rho1, bits(up.L1), bits(up.L2), up.wcodes.numpy(),
                                 up.wexps.numpy(), up.bias.numpy())
    h_or = torch.from_numpy(oracle.gelu_tanh(r1o["Y64"]).astype(np.float32)).to(torch.bfloat16)
    y64_chain = second_layer(bits(h_or))

    ctx = w4.Context(0, M, max(K, H), max(r1, r2))
    clip = torch.full((1, 2, 1), rho1)
    clip[0, 1, 0] = rho2
    clip_d = clip.to(DEV)
    Lup = w4.MxLayer(ctx, [up.to(DEV)], num_bins=1, num_layers=2, layer_id=0, output_activation=1)
    Ldn = w4.MxLayer(ctx, [down.to(DEV)], num_bins=1, num_layers=2, layer_id=1)
    xd = x.to(DEV)
    h_gpu = Lup.forward(xd, 0, 0, clip_d)
    y2 = torch.empty(M, N2, dtype=torch.bfloat16, device=DEV)
    w4.w4a4_mx_ffn_forward(Lup.ptr, Ldn.ptr, xd, M, 0, 0, clip_d, y2)
    torch.cuda.synchronize()
    ctx.check()
    # the hidden activations: equal on nearly every element, within the first layer's tolerance everywhere
    g64 = oracle.gelu_tanh(r1o["Y64"])
    tol1 = 1.13 * (2.0 ** -7 * np.abs(r1o["Y64"]) + 1e-3 * float(np.sqrt(np.mean(r1o["Y64"] ** 2)))) + 2.0 ** -8 * np.abs(g64)
    assert np.all(np.abs(h_gpu.to(torch.float64).cpu().numpy() - g64) <= tol1)
    assert (h_gpu.cpu() == h_or).float().mean().item() > 0.99
    sens = np.abs(second_layer(bits(h_gpu)) - y64_chain)
    rms = float(np.sqrt(np.mean(y64_chain ** 2)))
    bound = 2.0 ** -7 * np.abs(y64_chain) + 1e-3 * rms + sens
    worst = float(np.max(np.abs(y2.to(torch.float64).cpu().numpy() - y64_chain) / bound))
    assert worst <= 1.0, f"fused output outside tolerance of the oracle-only chain: worst err/bound = {worst:.3f}"
    assert float(np.sqrt(np.mean(sens ** 2))) < 0.02 * rms   # the sensitivity term stays a small correction
    Lup.close()
    Ldn.close()
    ctx.close()


def test_fused_ffn_many_tiles():
    # Enough items that clusters walk several column tiles of one row pair and several row pairs.
    run_fused_case(2048 + 77, 512, 2048, 512, 32, 32, 1, 0.85, 0.9, True, seed=5)


def test_fused_ffn_full_size_sampled_rows():
    """The bench's configuration (M = 32760, 5120 -> 13824 -> 5120, r = 32, GELU): sampled token rows of the second
    layer's input and output against the oracle."""
    import paper_2605_27003_b200 as w4
    up_s, dn_s = gen.CONFIG_SHAPES["ffn_up"], gen.CONFIG_SHAPES["ffn_down"]
    M, K, H, N, r = up_s["M"], up_s["K"], up_s["N"], dn_s["N"], up_s["r"]
    x = gen.make_activations(M, K, sigma=gen.sigma_for_bin(2), outlier_idx=gen.outlier_channels(K, 0.01, 7),
                             outlier_gain=50.0, seed=41, device=DEV)
    up = gen.make_layer_mx_direct(K, H, r, seed=42)
    down = gen.make_layer_mx_direct(H, N, r, seed=43)
    clip = gen.make_clip_table(1, 2, 8, [(0.6, 1.0)], seed=6)
    clip_d = clip.to(DEV)
    ctx = w4.Context(0, M, max(K, H), r)
    Lup = w4.MxLayer(ctx, [up.to(DEV)], num_bins=8, num_layers=2, layer_id=0, output_activation=1)
    Ldn = w4.MxLayer(ctx, [down.to(DEV)], num_bins=8, num_layers=2, layer_id=1)
    y1 = Lup.forward(x, 0, 2, clip_d)
    y2 = torch.empty(M, N, dtype=torch.bfloat16, device=DEV)
    w4.w4a4_mx_ffn_forward(Lup.ptr, Ldn.ptr, x, M, 0, 2, clip_d, y2)
    codes = torch.empty((M, H), dtype=torch.uint8, device=DEV)
    exps = torch.empty((M, H // 32), dtype=torch.uint8, device=DEV)
    T = torch.empty((M, r), dtype=torch.float32, device=DEV)
    w4.w4a4_mx_debug_fused_input(Ldn.ptr, M, codes, exps, T)
    torch.cuda.synchronize()
    ctx.check()
    rng = np.random.default_rng(2)
    rows = np.array(sorted({0, 127, 128, 255, 256, M - 1, (M - 1) // 256 * 256, *rng.integers(0, M, 3).tolist()}), dtype=np.int32)
    rt = torch.as_tensor(rows.astype(np.int64), device=DEV)
    ref = oracle.mx_forward_rows(bits(y1[rt]), np.arange(len(rows), dtype=np.int32), down.lam.numpy(), float(clip[0, 1, 2]),
                                 bits(down.L1), bits(down.L2), down.wcodes.numpy(), down.wexps.numpy(), None)
    assert np.array_equal(oracle.e2m1_values(codes[rt].cpu().numpy()), oracle.e2m1_values(ref["codes"])), "elements differ"
    assert np.array_equal(exps[rt].cpu().numpy(), ref["exps"]), "scale exponents differ"
    t_gpu, t_ref = T[rt].cpu().numpy().astype(np.float64), ref["T"].astype(np.float64)
    assert np.all(np.abs(t_gpu - t_ref) <= 1e-4 * np.abs(t_ref).max(axis=1, keepdims=True) + 1e-30), "T differs"
    y64 = ref["Y64"]
    rms = float(np.sqrt(np.mean(y64 ** 2)))
    bound = 2.0 ** -7 * np.abs(y64) + 1e-3 * rms
    worst = float(np.max(np.abs(y2[rt].to(torch.float64).cpu().numpy() - y64) / bound))
    assert worst <= 1.0, f"fused output outside tolerance: worst err/bound = {worst:.3f}"
    Lup.close()
    Ldn.close()
    ctx.close()


def test_fused_ffn_rejects_small_m():
    import paper_2605_27003_b200 as w4
    x = gen.make_activations(64, 256, outlier_idx=gen.outlier_channels(256, 0, 0, count=2), outlier_gain=10.0, seed=0)
    up = gen.make_layer_mx_svd(256, 256, 16, x, seed=1)
    down = gen.make_layer_mx_svd(256, 128, 16, x, seed=2)
    ctx = w4.Context(0, 64, 256, 16)
    Lup = w4.MxLayer(ctx, [up.to(DEV)], num_bins=1, num_layers=2, layer_id=0)
    Ldn = w4.MxLayer(ctx, [down.to(DEV)], num_bins=1, num_layers=2, layer_id=1)
    clip = torch.full((1, 2, 1), 0.9, device=DEV)
    y = torch.empty(64, 128, dtype=torch.bfloat16, device=DEV)
    with pytest.raises(w4.W4A4Error):
        w4.w4a4_mx_ffn_forward(Lup.ptr, Ldn.ptr, x.to(DEV), 64, 0, 0, clip, y)
    Lup.close()
    Ldn.close()
    ctx.close()
