"""The fused output activation (GELU, tanh form): pin of the oracle's formula and parity of both CUDA variants."""
import numpy as np
import pytest
import torch

import oracle
from workloads import generator as gen

DEV = "cuda:0"


def bits(t):
    return gen.bf16_bits(t.cpu()).numpy().view(np.uint16)


def test_oracle_gelu_against_library_routine():
    y = np.concatenate([np.linspace(-12.0, 12.0, 4001), np.array([0.0, -0.0, 1e-8, -1e-8, 30.0, -30.0])])
    want = torch.nn.functional.gelu(torch.tensor(y, dtype=torch.float64), approximate="tanh").numpy()
    assert np.allclose(oracle.gelu_tanh(y), want, rtol=1e-12, atol=1e-14)  # the far negative tail cancels to ~1e-16
    assert oracle.gelu_tanh(np.array([0.0]))[0] == 0.0 and abs(oracle.gelu_tanh(np.array([30.0]))[0] - 30.0) < 1e-12


def _bound(y64):
    # The pre-activation tolerance of the layer, carried through a function whose slope is at most 1.13.
    return 1.13 * (2.0 ** -7 * np.abs(y64) + 1e-3 * float(np.sqrt(np.mean(y64 ** 2))))


@pytest.mark.gpu
def test_int4_layer_with_fused_gelu():
    import paper_2605_27003_b200 as w4
    M, K, N, r = 300, 512, 384, 16
    idx = gen.outlier_channels(K, 0, 1, count=4)
    x = gen.make_activations(M, K, outlier_idx=idx, outlier_gain=40.0, seed=4)
    layer = gen.make_layer_svd(K, N, r, x, seed=5, bias_std=0.5)
    ctx = w4.Context(0, M, K, r)
    clip = torch.full((1, 1, 1), 0.85, device=DEV)
    plain = w4.Layer(ctx, [layer.to(DEV)], num_bins=1)
    fused = w4.Layer(ctx, [layer.to(DEV)], num_bins=1, output_activation=w4.binding.ACT_GELU_TANH)
    y_plain = plain.forward(x.to(DEV), 0, 0, clip)
    y_fused = fused.forward(x.to(DEV), 0, 0, clip)
    torch.cuda.synchronize()
    ctx.check()
    ref = oracle.forward_rows(bits(x), np.arange(M, dtype=np.int32), layer.lam.numpy(), 0.85, bits(layer.L1), bits(layer.L2),
                              layer.qweight.numpy(), layer.wscale.numpy(), layer.bias.numpy())
    err = np.abs(y_fused.to(torch.float64).cpu().numpy() - oracle.gelu_tanh(ref["Y64"]))
    assert np.all(err <= _bound(ref["Y64"]))
    assert not torch.equal(y_plain, y_fused)          # the flag does something: negative outputs are squashed
    assert (y_fused.float().min() > -0.2).item() and (y_plain.float().min() < -0.5).item()
    with pytest.raises(w4.W4A4Error):
        w4.Layer(ctx, [layer.to(DEV)], num_bins=1, output_activation=7)
    plain.close()
    fused.close()
    ctx.close()


@pytest.mark.gpu
def test_mxfp4_layer_with_fused_gelu():
    import paper_2605_27003_b200 as w4
    M, K, N, r = 200, 512, 256, 32
    x = gen.make_activations(M, K, outlier_idx=gen.outlier_channels(K, 0.02, 3), outlier_gain=30.0, seed=6)
    layer = gen.make_layer_mx_svd(K, N, r, x, seed=7, bias_std=0.5)
    ctx = w4.Context(0, M, K, r)
    clip = torch.full((1, 1, 1), 1.0, device=DEV)
    fused = w4.MxLayer(ctx, [layer.to(DEV)], num_bins=1, output_activation=w4.binding.ACT_GELU_TANH)
    y = fused.forward(x.to(DEV), 0, 0, clip)
    torch.cuda.synchronize()
    ctx.check()
    ref = oracle.mx_forward_rows(bits(x), np.arange(M, dtype=np.int32), layer.lam.numpy(), 1.0, bits(layer.L1), bits(layer.L2),
                                 layer.wcodes.numpy(), layer.wexps.numpy(), layer.bias.numpy())
    err = np.abs(y.to(torch.float64).cpu().numpy() - oracle.gelu_tanh(ref["Y64"]))
    assert np.all(err <= _bound(ref["Y64"]))
    fused.close()
    ctx.close()
