"""The two failure paths no healthy run reaches, exercised without hanging or faulting the GPU.

1. Bounded waits.  Every mbarrier wait of the library's kernels goes through one helper that gives up after a time
   limit, records a code in the context's device error word and lets the kernel return normally.  The probe launches
   a one-warp kernel that waits, through that helper, for a barrier phase nobody completes (no copy, no tensor-core
   operation, no tensor memory), with a limit of a millisecond or less.  What is checked is the contract the header
   states: the next status query reports W4A4_ERR_TIMEOUT once, the one after it W4A4_OK, and the context still
   computes correct results afterwards.
   The same is then done to the real GEMM: `w4a4_debug_stalled_gemm` withholds one operand stage from every CTA, so
   that the producer, both MMA-issuing warps and the epilogue warps all run into a 1 ms limit and leave through the
   kernel's common tail (drain of copies in flight, release of tensor memory).
2. Allocation failures.  A countdown hook makes the n-th device allocation fail as a refused cudaMalloc would.  Walking
   n over every allocation of w4a4_ctx_create and w4a4_pack_weights checks that each partial construction returns
   W4A4_ERR_ALLOC, leaks nothing (device memory in use returns to where it was) and leaves the library usable.
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
ERR_ALLOC, ERR_TIMEOUT = 3, 6


def bits(t):
    return gen.bf16_bits(t.cpu()).numpy().view(np.uint16)


def forward_matches_oracle(ctx, L, layer, M, seed):
    x = gen.make_activations(M, layer.K, seed=seed)
    clip = torch.ones((1, 1, 1), dtype=torch.float32, device=DEV)
    y = torch.empty((M, layer.N), dtype=torch.bfloat16, device=DEV)
    w4.w4a4_linear_forward(L.ptr, x.to(DEV), M, 0, 0, clip, y)
    torch.cuda.synchronize()
    ref = oracle.forward_rows(bits(x), np.arange(M, dtype=np.int32), layer.lam.cpu().numpy(), 1.0, bits(layer.L1),
                              bits(layer.L2), layer.qweight.cpu().numpy(), layer.wscale.cpu().numpy(),
                              None if layer.bias is None else layer.bias.cpu().numpy())["Y64"]
    got = y.to(torch.float64).cpu().numpy()
    bound = 2.0 ** -7 * np.abs(ref) + 1e-3 * float(np.sqrt(np.mean(ref ** 2)))
    return bool(np.all(np.abs(got - ref) <= bound))


@pytest.mark.parametrize("limit_ns", [1_000_000, 20_000])
def test_a_wait_that_nobody_answers_gives_up_and_is_reported_once(limit_ns):
    pkg_build.build()
    w4.load_library()
    ctx = w4.Context(0, 256, 512, 16)
    assert w4.w4a4_query_status(ctx.ptr) == 0
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    w4.w4a4_debug_wait_probe(ctx.ptr, limit_ns)
    ev1.record()
    torch.cuda.synchronize()
    assert ev0.elapsed_time(ev1) < 500.0, "the probe must end by itself shortly after its limit"
    assert w4.w4a4_query_status(ctx.ptr) == ERR_TIMEOUT
    assert w4.w4a4_query_status(ctx.ptr) == 0, "the flag is cleared by the query that reported it"
    ctx.close()


def test_the_context_computes_correctly_after_a_reported_timeout():
    pkg_build.build()
    w4.load_library()
    M, K, N, r = 200, 512, 256, 16
    layer = gen.make_layer_direct(K, N, r, seed=3).to(DEV)
    ctx = w4.Context(0, M, K, r)
    L = w4.Layer(ctx, [layer], num_bins=1)
    w4.w4a4_debug_wait_probe(ctx.ptr, 50_000)
    with pytest.raises(w4.W4A4Error) as ei:
        ctx.check()
    assert ei.value.status == ERR_TIMEOUT
    assert forward_matches_oracle(ctx, L, layer, M, seed=8)
    ctx.check()
    L.close()
    ctx.close()


def test_a_stalled_gemm_pipeline_gives_up_cleans_up_and_the_context_recovers():
    # The real GEMM (TMA producer, two MMA-issuing warps, sixteen epilogue warps, TMEM) with one operand stage
    # withheld and a 1 ms wait limit: every role's wait runs out, the CTAs leave through the common tail (error
    # word, drain, TMEM release) and the kernel ends by itself.  Then: TIMEOUT once, OK after, and a forward on
    # the same context (which needs all 512 TMEM columns of every SM again) matches the oracle.
    pkg_build.build()
    w4.load_library()
    M, K, N, r = 700, 1024, 512, 32
    layer = gen.make_layer_direct(K, N, r, seed=6).to(DEV)
    ctx = w4.Context(0, M, K, r)
    L = w4.Layer(ctx, [layer], num_bins=1)
    x = gen.make_activations(M, K, seed=12).to(DEV)
    clip = torch.ones((1, 1, 1), dtype=torch.float32, device=DEV)
    y = torch.zeros((M, N), dtype=torch.bfloat16, device=DEV)
    w4.w4a4_quantize_activations(L.ptr, x, M, 0, 0, clip)
    torch.cuda.synchronize()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    w4.w4a4_debug_stalled_gemm(L.ptr, M, 0, y, 3, 1_000_000)
    ev1.record()
    torch.cuda.synchronize()
    assert ev0.elapsed_time(ev1) < 500.0, "the stalled kernel must end by itself shortly after its limit"
    assert w4.w4a4_query_status(ctx.ptr) == ERR_TIMEOUT
    assert w4.w4a4_query_status(ctx.ptr) == 0
    assert forward_matches_oracle(ctx, L, layer, M, seed=13)
    ctx.check()
    L.close()
    ctx.close()


def test_the_probe_rejects_limits_it_would_not_honour_quickly():
    pkg_build.build()
    w4.load_library()
    ctx = w4.Context(0, 128, 512, 0)
    for bad in (0, 100_000_001):
        with pytest.raises(w4.W4A4Error) as ei:
            w4.w4a4_debug_wait_probe(ctx.ptr, bad)
        assert ei.value.status == 1
    assert w4.w4a4_query_status(ctx.ptr) == 0
    ctx.close()


def used_bytes():
    torch.cuda.synchronize()
    free, total = torch.cuda.mem_get_info(0)
    return total - free


def test_every_allocation_of_context_and_handle_construction_fails_cleanly():
    pkg_build.build()
    w4.load_library()
    M, K, N, r = 200, 512, 256, 16
    layer = gen.make_layer_direct(K, N, r, seed=4).to(DEV)
    try:
        # the context: walk the failing allocation forward until construction succeeds
        base = used_bytes()
        ctx = None
        ctx_allocs = 0
        for n in range(64):
            w4.w4a4_debug_fail_allocation_after(n)
            try:
                ctx = w4.Context(0, M, K, r)
            except w4.W4A4Error as e:
                assert e.status == ERR_ALLOC, f"allocation {n} of the context: {e}"
                assert used_bytes() == base, f"allocation {n} of the context: device memory was not given back"
                continue
            ctx_allocs = n
            break
        w4.w4a4_debug_fail_allocation_after(-1)
        assert ctx is not None and ctx_allocs >= 5, "the hook must have reached every allocation of the context"

        # the handle
        warm = w4.Layer(ctx, [layer], num_bins=1)   # grows the context's shared weight image once, outside the walk
        warm.close()
        base = used_bytes()
        L = None
        handle_allocs = 0
        for n in range(64):
            w4.w4a4_debug_fail_allocation_after(n)
            try:
                L = w4.Layer(ctx, [layer], num_bins=1)
            except w4.W4A4Error as e:
                assert e.status == ERR_ALLOC, f"allocation {n} of the handle: {e}"
                assert used_bytes() == base, f"allocation {n} of the handle: device memory was not given back"
                continue
            handle_allocs = n
            break
        w4.w4a4_debug_fail_allocation_after(-1)
        assert L is not None and handle_allocs >= 6, "the hook must have reached every allocation of the handle"

        # and the survivors work
        assert forward_matches_oracle(ctx, L, layer, M, seed=9)
        ctx.check()
        L.close()
        ctx.close()
    finally:
        w4.w4a4_debug_fail_allocation_after(-1)
