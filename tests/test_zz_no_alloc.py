"""The allocation-free activation-quantization entry point, against the oracle and against the regular path.

Callers that may not allocate device memory (host callbacks, latency-critical paths, runtimes that own all
device memory through their own pool) use w4a4_quantize_noalloc, whose scratch is a fixed array inside the library.  Here
it is called through the C ABI twice in a row per case, on different inputs, and each result must equal (a) what the
CPU oracle's quantizer gives for the same input and (b) what the context-based tap (w4a4_debug_quantize) returns:
integer codes and FP32 scales bit for bit, the bar the other parity tests use for these quantities.  The cases cover a
token count that is a multiple of neither 4 nor 16 (padded scratch pitch, half-filled last warp) and the largest
size the built-in scratch admits.  The file name keeps this test last in collection order.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2605_27003_b200 as w4
from paper_2605_27003_b200 import build as pkg_build
from workloads import generator as gen

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def bits(t):
    return gen.bf16_bits(t.cpu()).numpy().view(np.uint16)


@pytest.mark.parametrize("M,K", [(200, 1024), (203, 1024), (256, 16384)])
def test_noalloc_quantize_matches_oracle_and_context_path_on_two_calls_in_a_row(M, K):
    pkg_build.build()
    w4.load_library()
    N = 128
    layer = gen.make_layer_direct(K, N, 0, seed=11).to(DEV)
    ctx = w4.Context(0, M, K, 0)
    L = w4.Layer(ctx, [layer], num_bins=4)
    rhos = [1.0, 0.9, 0.75, 0.6]
    clip = torch.tensor([[rhos]], dtype=torch.float32, device=DEV)
    idx = gen.outlier_channels(K, 0.01, 5)
    for call, (seed, b) in enumerate(((21, 2), (22, 0))):
        x = gen.make_activations(M, K, sigma=1.5, outlier_idx=idx, outlier_gain=30.0, seed=seed, device=DEV)
        if call == 1:
            x[3] = 0  # an all-zero token: scales 0, codes 0
        codes_ref = torch.full((M, K), 99, dtype=torch.int8, device=DEV)
        scales_ref = torch.full((M, K // 64), -1.0, dtype=torch.float32, device=DEV)
        w4.w4a4_debug_quantize(L.ptr, x, M, 0, b, clip, codes_ref, scales_ref, None)
        codes = torch.full((M, K), 77, dtype=torch.int8, device=DEV)
        scales = torch.full((M, K // 64), -2.0, dtype=torch.float32, device=DEV)
        w4.w4a4_quantize_noalloc(x, M, K, layer.lam, clip, b, codes, scales)
        torch.cuda.synchronize()
        q_or, s_or = oracle.quantize(bits(x), layer.lam.cpu().numpy(), rhos[b])
        assert np.array_equal(codes.cpu().numpy(), q_or), f"call {call}: codes differ from the oracle"
        assert np.array_equal(scales.cpu().numpy().view(np.uint32), s_or.view(np.uint32)), \
            f"call {call}: scales differ from the oracle"
        assert torch.equal(codes, codes_ref), f"call {call}: codes differ from the context path"
        assert np.array_equal(scales.cpu().numpy().view(np.uint32), scales_ref.cpu().numpy().view(np.uint32)), \
            f"call {call}: scales differ from the context path"
    ctx.check()
    L.close()
    ctx.close()


def test_noalloc_quantize_refuses_sizes_beyond_its_scratch():
    pkg_build.build()
    w4.load_library()
    lam = torch.ones(32768, dtype=torch.float32, device=DEV)
    clip = torch.ones(1, dtype=torch.float32, device=DEV)
    x = torch.empty(1, dtype=torch.bfloat16, device=DEV)
    codes = torch.empty(1, dtype=torch.int8, device=DEV)
    scales = torch.empty(1, dtype=torch.float32, device=DEV)
    # sizes beyond the built-in scratch are refused with a clear status, nothing is launched
    with pytest.raises(w4.W4A4Error) as ei:
        w4.w4a4_quantize_noalloc(x, 8192, 1024, lam, clip, 0, codes, scales)  # M * K > 4 Mi
    assert ei.value.status == 2
    with pytest.raises(w4.W4A4Error) as ei:
        w4.w4a4_quantize_noalloc(x, 1, 32768, lam, clip, 0, codes, scales)  # K > 16384
    assert ei.value.status == 2
    torch.cuda.synchronize()
