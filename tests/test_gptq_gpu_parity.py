"""GPTQ on the residual branch (Sec. III-B) on the GPU against the FP64 oracle, through the C ABI (GPU only).

Both sides work in FP64 but reach U = chol(H^-1, upper) by different routes (the oracle inverts H and factors the
inverse; the library factors H from the last channel to the first and inverts the triangular factor), so their
error-compensated weights differ by rounding noise, about 1e-10 relative.  A weight that sits that close to a
rounding boundary may take the neighbouring code on one side, and every later input channel of that OUTPUT channel
then follows a different but equally valid trajectory; output channels do not interact.  The tests therefore demand
bit-equal codes and scales on all but a handful of output channels and, on those, an objective value as good as the
oracle's."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from workloads import generator as gen

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def bits(t):
    return gen.bf16_bits(t.cpu()).numpy().view(np.uint16)


def gpu_gptq(R, xhat=None, H=None, percdamp=0.01, own_workspace=False):
    import paper_2605_27003_b200 as w4
    K, N = R.shape
    ws = None
    if own_workspace:
        ws = torch.empty(w4.w4a4_gptq_workspace_bytes(K, N, 0 if xhat is None else xhat.shape[0]), dtype=torch.uint8,
                         device=DEV)
    codes = torch.full((K, N), 99, dtype=torch.int8, device=DEV)
    scales = torch.full((K // 64, N), -1.0, dtype=torch.float32, device=DEV)
    w4.w4a4_gptq_quantize(R.to(DEV), codes, scales, Xhat=None if xhat is None else xhat.to(DEV),
                          H=None if H is None else torch.from_numpy(H).to(DEV), percdamp=percdamp, workspace=ws)
    return codes.cpu().numpy(), scales.cpu().numpy()


def objective(R, q, s, H):
    D = R - q.astype(np.float64) * np.repeat(s.astype(np.float64), 64, axis=0)
    return np.einsum("kn,kj,jn->n", D, H, D)


def compare(R64, H, q_gpu, s_gpu, q_ref, s_ref, max_bad_columns):
    bad = np.flatnonzero((q_gpu != q_ref).any(axis=0) | (s_gpu != s_ref).any(axis=0))
    assert bad.size <= max_bad_columns, f"{bad.size} output channels differ"
    if bad.size:
        o_gpu = objective(R64[:, bad], q_gpu[:, bad], s_gpu[:, bad], H)
        o_ref = objective(R64[:, bad], q_ref[:, bad], s_ref[:, bad], H)
        assert np.all(o_gpu <= o_ref * 1.05), (o_gpu, o_ref)
    assert q_gpu.min() >= -8 and q_gpu.max() <= 7


def test_identity_statistic_is_round_to_nearest():
    # H = c I: nothing is propagated, so the result is the plain group quantizer's, bit for bit.
    R, _ = gen.make_gptq_inputs(256, 200, 8, seed=1)
    R[64:128, 5] = 0.0
    q0, s0 = gen._round_residual(R.double())
    for c in (1.0, 12.5):
        q, s = gpu_gptq(R, H=c * np.eye(256))
        assert np.array_equal(q, q0.numpy()) and np.array_equal(s, s0.numpy())


@pytest.mark.parametrize("K,N,M_cal,dead,percdamp", [
    (64, 40, 96, (), 0.01),                # a single group: no update between groups
    (256, 96, 300, (), 0.01),
    (512, 130, 384, (3, 200), 0.01),       # ragged N, dead input channels
    (320, 257, 100, (), 0.05),             # fewer calibration tokens than channels: H is singular before damping
    (1024, 512, 1500, (1023,), 0.002),
])
def test_matches_oracle(K, N, M_cal, dead, percdamp):
    R, xhat = gen.make_gptq_inputs(K, N, M_cal, seed=K + N, dead=dead)
    R64 = R.double().numpy()
    H = oracle.gptq_hessian(bits(xhat))
    q_ref, s_ref = oracle.gptq_quantize(R64, H, percdamp=percdamp)
    q, s = gpu_gptq(R, xhat=xhat, percdamp=percdamp)
    compare(R64, H, q, s, q_ref, s_ref, max_bad_columns=max(1, N // 200))
    # the compensation must have mattered: the plain quantizer gives different codes and a worse objective
    q0, s0 = gen._round_residual(R.double())
    assert (q != q0.numpy()).mean() > 0.05
    Rz = R64.copy()
    Rz[list(dead), :] = 0.0
    assert objective(Rz, q, s, H).sum() < 0.9 * objective(Rz, q0.numpy(), s0.numpy(), H).sum()
    # and the statistic handed over directly gives the same result as the activations
    q2, s2 = gpu_gptq(R, H=H, percdamp=percdamp)
    compare(R64, H, q2, s2, q_ref, s_ref, max_bad_columns=max(1, N // 200))
    # a caller-owned workspace changes nothing, bit for bit
    q3, s3 = gpu_gptq(R, xhat=xhat, percdamp=percdamp, own_workspace=True)
    assert np.array_equal(q3, q) and np.array_equal(s3, s)


@pytest.mark.parametrize("K,N,n_cols", [(5120, 5120, 40), (13824, 5120, 8)])
def test_full_size_layer_on_sampled_output_channels(K, N, n_cols):
    # The sizes the bench times (attention projection and FFN down-projection, 2048 calibration tokens).  Output
    # channels are independent, so the oracle runs on a sample of them with the full statistic.
    M_cal = 2048
    R, xhat = gen.make_gptq_inputs(K, N, M_cal, seed=7)
    q, s = gpu_gptq(R, xhat=xhat)
    cols = np.sort(np.random.default_rng(3).choice(N, n_cols, replace=False))
    R64 = R[:, cols].double().numpy()
    H = oracle.gptq_hessian(bits(xhat))
    q_ref, s_ref = oracle.gptq_quantize(R64, H)
    compare(R64, H, q[:, cols], s[:, cols], q_ref, s_ref, max_bad_columns=2)


def test_argument_errors():
    import paper_2605_27003_b200 as w4
    lib = w4.load_library()
    R = torch.zeros(64, 8, device=DEV)
    codes = torch.zeros(64, 8, dtype=torch.int8, device=DEV)
    scales = torch.zeros(1, 8, device=DEV)
    H = torch.eye(64, dtype=torch.float64, device=DEV)
    x = torch.zeros(4, 64, dtype=torch.bfloat16, device=DEV)
    p = lambda t: ctypes.c_void_p(t.data_ptr())
    call = lambda *a: lib.w4a4_gptq_quantize(*a, None, 0, None)
    assert call(0, p(R), None, 0, None, 64, 8, 0.01, p(codes), p(scales)) == 1        # no statistic
    assert call(0, p(R), p(x), 4, p(H), 64, 8, 0.01, p(codes), p(scales)) == 1        # two statistics
    assert call(0, None, None, 0, p(H), 64, 8, 0.01, p(codes), p(scales)) == 1
    assert call(0, p(R), None, 0, p(H), 96, 8, 0.01, p(codes), p(scales)) == 2        # K not a multiple of 64
    assert call(0, p(R), p(x), 0, None, 64, 8, 0.01, p(codes), p(scales)) == 2        # no calibration tokens
    assert call(0, p(R), None, 0, p(H), 64, 8, -1.0, p(codes), p(scales)) == 1
    need = w4.w4a4_gptq_workspace_bytes(64, 8, 0)
    assert need > 0 and w4.w4a4_gptq_workspace_bytes(96, 8, 0) == 0
    small = torch.empty(need - 256, dtype=torch.uint8, device=DEV)
    assert lib.w4a4_gptq_quantize(0, p(R), None, 0, p(H), 64, 8, 0.01, p(codes), p(scales), p(small), need - 256,
                                  None) == 1                                              # workspace too small
    # not positive definite (and no damping): reported, not a fault
    Hbad = -torch.eye(64, dtype=torch.float64, device=DEV)
    assert call(0, p(R), None, 0, p(Hbad), 64, 8, 0.0, p(codes), p(scales)) == 1
    torch.cuda.synchronize()


def test_gptq_codes_lower_the_layer_error_on_held_out_tokens():
    # The point of the step (Sec. III-B): with the statistic of calibration tokens, the residual's quantization error
    # as seen through fresh tokens of the same distribution is far below round-to-nearest's -- for the weights alone
    # (FP64 check of the codes the GPU produced) and through the real W4A4 forward, where the 4-bit activations add
    # the same noise to both.
    import paper_2605_27003_b200 as w4
    K, N, M_cal, M_eval = 512, 256, 1024, 512
    R, x = gen.make_gptq_inputs(K, N, M_cal + M_eval, seed=11)
    cal, ev = x[:M_cal].contiguous(), x[M_cal:].contiguous()
    q, s = gpu_gptq(R, xhat=cal)
    q0, s0 = gen._round_residual(R.double())
    q0, s0 = q0.numpy(), s0.numpy()
    deq = lambda c, sc: c.astype(np.float64) * np.repeat(sc.astype(np.float64), 64, axis=0)
    Xe, R64 = ev.double().numpy(), R.double().numpy()
    target = Xe @ R64
    err_w = lambda c, sc: float(((Xe @ deq(c, sc) - target) ** 2).sum())
    assert err_w(q, s) < 0.5 * err_w(q0, s0)

    ctx = w4.Context(0, M_eval, K, 0)
    clip = torch.ones((1, 1, 1), dtype=torch.float32, device=DEV)
    errs = []
    for codes, scales in ((q, s), (q0, s0)):
        lay = gen.LayerInputs(K, N, 0, torch.ones(K), None, None, torch.from_numpy(codes), torch.from_numpy(scales), None)
        L = w4.Layer(ctx, [lay.to(DEV)], num_bins=1)
        Y = L.forward(ev.to(DEV), 0, 0, clip).double().cpu().numpy()
        ctx.check()
        L.close()
        errs.append(float(((Y - target) ** 2).sum()))
    ctx.close()
    assert errs[0] < 0.9 * errs[1], errs


# ---------------------------------------------------------------------------------------------------------------
# The same step on the MXFP4 grid (w4a4_mx_gptq_quantize)
# ---------------------------------------------------------------------------------------------------------------
def gpu_gptq_mx(R, xhat=None, H=None, percdamp=0.01):
    import paper_2605_27003_b200 as w4
    K, N = R.shape
    codes = torch.full((K, N), 99, dtype=torch.uint8, device=DEV)
    exps = torch.full((K // 32, N), 77, dtype=torch.uint8, device=DEV)
    w4.w4a4_mx_gptq_quantize(R.to(DEV), codes, exps, Xhat=None if xhat is None else xhat.to(DEV),
                             H=None if H is None else torch.from_numpy(H).to(DEV), percdamp=percdamp)
    return codes.cpu().numpy(), exps.cpu().numpy()


def mx_deq(c, e):
    return gen.mx_dequantize(torch.from_numpy(c), torch.from_numpy(e)).numpy()


def test_mx_identity_statistic_is_the_plain_conversion():
    R, _ = gen.make_gptq_inputs(256, 150, 8, seed=2)
    R[32:64, 5] = 0.0
    R[7, 9] = 0.0
    q0, e0 = gen._round_residual_mx(R.double())
    q, e = gpu_gptq_mx(R, H=3.0 * np.eye(256))
    assert np.array_equal(q, q0.numpy()) and np.array_equal(e, e0.numpy())


@pytest.mark.parametrize("K,N,M_cal,dead,percdamp", [
    (64, 33, 96, (), 0.01),
    (512, 130, 384, (3, 200), 0.01),
    (1024, 300, 1500, (1023,), 0.002),
])
def test_mx_matches_oracle(K, N, M_cal, dead, percdamp):
    R, xhat = gen.make_gptq_inputs(K, N, M_cal, seed=K + N + 1, dead=dead)
    R64 = R.double().numpy()
    H = oracle.gptq_hessian(bits(xhat))
    q_ref, e_ref = oracle.gptq_quantize_mx(R64, H, percdamp=percdamp)
    q, e = gpu_gptq_mx(R, xhat=xhat, percdamp=percdamp)
    bad = np.flatnonzero((q != q_ref).any(axis=0) | (e != e_ref).any(axis=0))
    assert bad.size <= max(1, N // 200), f"{bad.size} output channels differ"
    obj = lambda c, x, cols: np.einsum("kn,kj,jn->n", R64[:, cols] - mx_deq(c, x)[:, cols], H, R64[:, cols] - mx_deq(c, x)[:, cols])
    if bad.size:
        assert np.all(obj(q, e, bad) <= 1.05 * obj(q_ref, e_ref, bad))
    q0, e0 = gen._round_residual_mx(R.double())
    Rz = R64.copy()
    Rz[list(dead), :] = 0.0
    D, D0 = Rz - mx_deq(q, e), Rz - mx_deq(q0.numpy(), e0.numpy())
    assert np.einsum("kn,kj,jn->", D, H, D) < 0.9 * np.einsum("kn,kj,jn->", D0, H, D0)
    assert q.max() <= 15


def test_mx_gptq_codes_lower_the_layer_error_on_held_out_tokens():
    import paper_2605_27003_b200 as w4
    K, N, M_cal, M_eval = 512, 256, 1024, 512
    R, x = gen.make_gptq_inputs(K, N, M_cal + M_eval, seed=12)
    cal, ev = x[:M_cal].contiguous(), x[M_cal:].contiguous()
    q, e = gpu_gptq_mx(R, xhat=cal)
    q0, e0 = gen._round_residual_mx(R.double())
    q0, e0 = q0.numpy(), e0.numpy()
    Xe, R64 = ev.double().numpy(), R.double().numpy()
    target = Xe @ R64
    err_w = lambda c, x_: float(((Xe @ mx_deq(c, x_) - target) ** 2).sum())
    assert err_w(q, e) < 0.6 * err_w(q0, e0)
    ctx = w4.Context(0, M_eval, K, 0)
    clip = torch.ones((1, 1, 1), dtype=torch.float32, device=DEV)
    errs = []
    for codes, exps in ((q, e), (q0, e0)):
        lay = gen.MxLayerInputs(K, N, 0, torch.ones(K), None, None, torch.from_numpy(codes), torch.from_numpy(exps), None)
        L = w4.MxLayer(ctx, [lay.to(DEV)], num_bins=1)
        Y = L.forward(ev.to(DEV), 0, 0, clip).double().cpu().numpy()
        ctx.check()
        L.close()
        errs.append(float(((Y - target) ** 2).sum()))
    ctx.close()
    assert errs[0] < 0.95 * errs[1], errs


def test_mx_full_size_layer_on_sampled_output_channels():
    K, N, M_cal = 5120, 5120, 2048
    R, xhat = gen.make_gptq_inputs(K, N, M_cal, seed=8)
    q, e = gpu_gptq_mx(R, xhat=xhat)
    cols = np.sort(np.random.default_rng(4).choice(N, 24, replace=False))
    H = oracle.gptq_hessian(bits(xhat))
    q_ref, e_ref = oracle.gptq_quantize_mx(R[:, cols].double().numpy(), H)
    bad = np.flatnonzero((q[:, cols] != q_ref).any(axis=0) | (e[:, cols] != e_ref).any(axis=0))
    assert bad.size <= 1, f"{bad.size} of the sampled output channels differ"


def test_statistic_accumulated_over_batches():
    # Calibration tokens arrive in batches: H += Xhat^T Xhat per batch, then the sweep on the accumulated statistic.
    import paper_2605_27003_b200 as w4
    K, N = 320, 150
    sizes = (100, 4096 + 37, 300)                  # the middle batch is longer than the library's conversion chunk
    R, x = gen.make_gptq_inputs(K, N, sum(sizes), seed=21)
    H = torch.zeros((K, K), dtype=torch.float64, device=DEV)
    m0 = 0
    for m in sizes:
        w4.w4a4_gptq_accumulate(x[m0:m0 + m].contiguous().to(DEV), H)
        m0 += m
    H_ref = oracle.gptq_hessian(bits(x))
    Hg = H.cpu().numpy()
    iu = np.triu_indices(K)
    assert np.allclose(Hg[iu], H_ref[iu], rtol=1e-12, atol=1e-9 * np.abs(H_ref).max())
    # the sweep reads only the upper triangle: garbage below the diagonal must not matter
    Hd = H.clone()
    Hd[np.tril_indices(K, -1)] = float("nan")
    codes = torch.empty((K, N), dtype=torch.int8, device=DEV)
    scales = torch.empty((K // 64, N), dtype=torch.float32, device=DEV)
    w4.w4a4_gptq_quantize(R.to(DEV), codes, scales, H=Hd)
    R64 = R.double().numpy()
    q_ref, s_ref = oracle.gptq_quantize(R64, H_ref)
    compare(R64, H_ref, codes.cpu().numpy(), scales.cpu().numpy(), q_ref, s_ref, max_bad_columns=1)
