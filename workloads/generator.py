"""Seeded synthetic inputs shaped like a video DiT's quantized linears.

Everything here is *input preparation*: drawing activations with sparse
large-magnitude channels, choosing the diagonal smoothing matrix (Eq. 5),
splitting the smoothed weight into a low-rank pair plus a residual (Eq. 6) and
rounding that residual to 4-bit codes with per-group scales.  Those are the
offline steps whose results the inference-time layer consumes as constants; the
inference-time arithmetic itself (activation quantization, integer GEMM,
rescale, low-rank branch) lives elsewhere and is never imported from here.

All tensors are torch tensors so the same recipe runs on CPU (small cases,
oracle tests) or on a CUDA device (full-size cases, where the result is copied
to the host for the oracle).  A given (seed, device type) pair is reproducible.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Optional, Sequence

import torch

GROUP = 64

# (M, K, N, r) of the workloads named by the benchmark contract.
CONFIG_SHAPES = {
    "tiny": dict(M=256, K=512, N=512, r=16),
    "attn_proj": dict(M=32760, K=5120, N=5120, r=32),
    "ffn_up": dict(M=32760, K=5120, N=13824, r=32),
    "ffn_down": dict(M=32760, K=13824, N=5120, r=32),
}


def bf16_bits(t: torch.Tensor) -> torch.Tensor:
    """View a bfloat16 tensor as its raw 16-bit patterns (int16 storage)."""
    assert t.dtype == torch.bfloat16
    return t.contiguous().view(torch.int16)


def bf16_to_f32(t: torch.Tensor) -> torch.Tensor:
    assert t.dtype == torch.bfloat16
    return t.to(torch.float32)


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


@dataclass
class LayerInputs:
    """Constants of one quantized linear for one expert (what calibration would hand over)."""

    K: int
    N: int
    r: int
    lam: torch.Tensor  # [K] float32, > 0          (diagonal of D_l, Eq. 5)
    L1: Optional[torch.Tensor]  # [K, r] bfloat16   (Eq. 6)
    L2: Optional[torch.Tensor]  # [r, N] bfloat16
    qweight: torch.Tensor  # [K, N] int8 in [-8, 7] (4-bit residual codes)
    wscale: torch.Tensor  # [K/64, N] float32       (one scale per 64-row group and column)
    bias: Optional[torch.Tensor]  # [N] float32
    # Only filled by the SVD recipe (float64): the unquantized pieces, for identity checks.
    W: Optional[torch.Tensor] = None  # [K, N]  original weight
    R: Optional[torch.Tensor] = None  # [K, N]  residual before rounding, diag(lam) W - L1 L2
    extra: dict = field(default_factory=dict)

    def to(self, device) -> "LayerInputs":
        def mv(x):
            return None if x is None else x.to(device)

        return LayerInputs(self.K, self.N, self.r, mv(self.lam), mv(self.L1), mv(self.L2), mv(self.qweight),
                           mv(self.wscale), mv(self.bias), mv(self.W), mv(self.R), dict(self.extra))


def outlier_channels(K: int, fraction: float, seed: int, count: Optional[int] = None) -> torch.Tensor:
    """Seeded set of distinct channel indices that carry large magnitudes."""
    n = count if count is not None else int(round(K * fraction))
    if n <= 0:
        return torch.empty(0, dtype=torch.long)
    g = _gen(seed * 7919 + 13, "cpu")
    return torch.randperm(K, generator=g)[:n].sort().values


def make_activations(M: int, K: int, *, sigma: float = 1.0, outlier_idx: Optional[torch.Tensor] = None,
                     outlier_gain: float = 1.0, dist: str = "normal", seed: int = 0,
                     device="cpu") -> torch.Tensor:
    """BF16 activations [M, K]: Gaussian (or GELU of a Gaussian), a few channels scaled up.

    dist="normal": N(0, sigma).  dist="gelu": sigma * GELU(N(0,1)) -- heavy right tail,
    small negative lobe, like the input of an FFN down-projection.
    """
    g = _gen(seed, device)
    x = torch.randn(M, K, generator=g, device=device, dtype=torch.float32)
    if dist == "gelu":
        x = torch.nn.functional.gelu(x)
    elif dist != "normal":
        raise ValueError(dist)
    x = x * float(sigma)
    if outlier_idx is not None and outlier_idx.numel() > 0 and outlier_gain != 1.0:
        x[:, outlier_idx.to(x.device)] *= float(outlier_gain)
    return x.to(torch.bfloat16)


def make_gptq_inputs(K: int, N: int, M_cal: int, *, seed: int = 0, shared: int = 8, dead: Sequence[int] = (),
                     w_std: float = 0.02):
    """Inputs of the residual-branch weight quantization: residual weights R [K, N] (FP32 values) and smoothed
    calibration activations [M_cal, K] in BF16 whose channels are correlated (a few shared directions on top of
    independent noise, a few channels scaled up), so that the second-order statistic is far from diagonal.  Channels
    listed in `dead` are zero in every calibration token."""
    g = _gen(seed * 15485863 + 3, "cpu")
    R = (torch.randn(K, N, generator=g, dtype=torch.float32) * w_std)
    z = torch.randn(M_cal, K, generator=g, dtype=torch.float32)
    mix = torch.randn(shared, K, generator=g, dtype=torch.float32)
    x = z + 0.8 * torch.randn(M_cal, shared, generator=g, dtype=torch.float32) @ mix
    idx = outlier_channels(K, 0, seed, count=max(2, K // 128))
    x[:, idx] *= 6.0
    for k in dead:
        x[:, k] = 0.0
    return R, x.to(torch.bfloat16)


def make_clip_table(num_experts: int, num_layers: int, num_bins: int,
                    ranges: Sequence[Sequence[float]], seed: int = 0) -> torch.Tensor:
    """FP32 clip ratios [E, L, B]; expert e draws uniformly from ranges[e] = (lo, hi)."""
    g = _gen(seed * 104729 + 7, "cpu")
    t = torch.empty(num_experts, num_layers, num_bins, dtype=torch.float32)
    for e in range(num_experts):
        lo, hi = ranges[e]
        t[e] = lo + (hi - lo) * torch.rand(num_layers, num_bins, generator=g, dtype=torch.float32)
    return t


def _round_residual(R: torch.Tensor):
    """Residual [K, N] float64 -> int8 codes in [-8, 7] and FP32 group scales [K/64, N].

    Per (64-row group, column): scale = absmax / 7 (FP32), code = round-half-even(R / scale)
    clamped to [-8, 7]; an all-zero group gets scale 0 and codes 0.
    """
    K, N = R.shape
    G = K // GROUP
    Rg = R.reshape(G, GROUP, N)
    amax = Rg.abs().amax(dim=1)  # [G, N]
    scale = (amax / 7.0).to(torch.float32)
    safe = torch.where(scale > 0, scale, torch.ones_like(scale)).to(torch.float64)
    q = torch.round(Rg / safe[:, None, :]).clamp_(-8, 7)
    q = torch.where(scale[:, None, :] > 0, q, torch.zeros_like(q))
    return q.reshape(K, N).to(torch.int8), scale


def make_layer_svd(K: int, N: int, r: int, x_calib: torch.Tensor, *, w_std: float = 0.02,
                   bias_std: Optional[float] = None, seed: int = 0, device="cpu",
                   exact_svd: Optional[bool] = None, keep_float64: bool = True) -> LayerInputs:
    """Smoothing + truncated-SVD split + round-to-nearest residual, from a random weight.

    W ~ N(0, w_std) rounded to BF16;  lam_k = sqrt(max_m |X_mk| / max_n |W_kn|) on the
    calibration activations;  What = diag(lam) W;  L1, L2 = rank-r truncated SVD of What with
    sqrt(singular value) on each side, rounded to BF16;  R = What - L1 L2 (with the rounded
    factors, so that L1 L2 + R == What to FP64 round-off);  codes/scales from _round_residual.
    """
    assert K % GROUP == 0
    g = _gen(seed, device)
    W = (torch.randn(K, N, generator=g, device=device, dtype=torch.float32) * w_std).to(torch.bfloat16)
    W64 = W.to(torch.float64)
    xmax = x_calib.to(device).to(torch.float32).abs().amax(dim=0)  # [K]
    wmax = W64.abs().amax(dim=1).to(torch.float32)  # [K]
    lam = torch.sqrt(torch.clamp(xmax, min=1e-6) / torch.clamp(wmax, min=1e-6)).to(torch.float32)
    What = lam.to(torch.float64)[:, None] * W64
    L1b = L2b = None
    if r > 0:
        if exact_svd is None:
            exact_svd = max(K, N) <= 2048
        if exact_svd:
            U, S, Vh = torch.linalg.svd(What, full_matrices=False)
            U, S, Vh = U[:, :r], S[:r], Vh[:r]
        else:
            U, S, V = torch.svd_lowrank(What.to(torch.float32), q=r + 8, niter=4)
            U, S, Vh = U[:, :r].to(torch.float64), S[:r].to(torch.float64), V[:, :r].T.to(torch.float64)
        rootS = torch.sqrt(S)
        L1b = (U * rootS[None, :]).to(torch.float32).to(torch.bfloat16)
        L2b = (rootS[:, None] * Vh).to(torch.float32).to(torch.bfloat16)
        R = What - L1b.to(torch.float64) @ L2b.to(torch.float64)
    else:
        R = What
    q, scale = _round_residual(R)
    bias = None
    if bias_std is not None:
        bias = torch.randn(N, generator=g, device=device, dtype=torch.float32) * bias_std
    return LayerInputs(K, N, r, lam, L1b, L2b, q, scale, bias,
                       W=W64 if keep_float64 else None, R=R if keep_float64 else None)


def make_layer_direct(K: int, N: int, r: int, *, seed: int = 0, device="cpu", with_bias: bool = True) -> LayerInputs:
    """Constants drawn directly (no SVD): for sweeps and for the many layers of a whole denoising step.

    codes = clamp(round(N(0, 2.5)), -8, 7); scales log-uniform in [2e-3, 2e-2];
    lam log-normal(0, 0.5); L1 ~ N(0, 0.05), L2 ~ N(0, 0.05); bias ~ N(0, 0.01).
    """
    assert K % GROUP == 0
    g = _gen(seed, device)
    q = torch.round(torch.randn(K, N, generator=g, device=device, dtype=torch.float32) * 2.5).clamp_(-8, 7)
    q = q.to(torch.int8)
    u = torch.rand(K // GROUP, N, generator=g, device=device, dtype=torch.float32)
    scale = (2e-3 * torch.exp(u * math.log(10.0))).to(torch.float32)
    lam = torch.exp(0.5 * torch.randn(K, generator=g, device=device, dtype=torch.float32))
    L1 = L2 = None
    if r > 0:
        L1 = (0.05 * torch.randn(K, r, generator=g, device=device, dtype=torch.float32)).to(torch.bfloat16)
        L2 = (0.05 * torch.randn(r, N, generator=g, device=device, dtype=torch.float32)).to(torch.bfloat16)
    bias = None
    if with_bias:
        bias = 0.01 * torch.randn(N, generator=g, device=device, dtype=torch.float32)
    return LayerInputs(K, N, r, lam, L1, L2, q, scale, bias)


# ----------------------------------------------------------------------------- MXFP4 variant of the layer constants
MX_BLOCK = 32
_E2M1_GRID = (0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0)


@dataclass
class MxLayerInputs:
    """Constants of one MXFP4-quantized linear (OCP MX v1.0: E2M1 elements, one E8M0 scale per 32 input channels)."""

    K: int
    N: int
    r: int
    lam: torch.Tensor  # [K] float32
    L1: Optional[torch.Tensor]  # [K, r] bfloat16
    L2: Optional[torch.Tensor]  # [r, N] bfloat16
    wcodes: torch.Tensor  # [K, N] uint8: E2M1 code (bit 3 sign, bits 0-2 magnitude index)
    wexps: torch.Tensor  # [K/32, N] uint8: E8M0 exponent, scale = 2^(e - 127)
    bias: Optional[torch.Tensor]  # [N] float32
    W: Optional[torch.Tensor] = None  # [K, N] float64 original weight (SVD recipe only)

    def to(self, device) -> "MxLayerInputs":
        def mv(x):
            return None if x is None else x.to(device)

        return MxLayerInputs(self.K, self.N, self.r, mv(self.lam), mv(self.L1), mv(self.L2), mv(self.wcodes),
                             mv(self.wexps), mv(self.bias), mv(self.W))


def mx_dequantize(codes: torch.Tensor, exps: torch.Tensor) -> torch.Tensor:
    """[K, N] E2M1 codes + [K/32, N] E8M0 exponents -> float64 values."""
    grid = torch.tensor(_E2M1_GRID, dtype=torch.float64, device=codes.device)
    v = grid[(codes & 7).long()]
    v = torch.where((codes & 8) != 0, -v, v)
    K, N = codes.shape
    scale = torch.pow(torch.tensor(2.0, dtype=torch.float64, device=codes.device), exps.to(torch.float64) - 127.0)
    return (v.view(K // MX_BLOCK, MX_BLOCK, N) * scale[:, None, :]).view(K, N)


def _round_residual_mx(R: torch.Tensor):
    """Residual [K, N] float64 -> MXFP4 per (32-row block, column), the MX specification's conversion:
    shared exponent floor(log2(block max)) - 2, elements rounded to the nearest E2M1 value (ties to the even
    code), saturating at 6."""
    K, N = R.shape
    B = K // MX_BLOCK
    Rb = R.reshape(B, MX_BLOCK, N)
    amax = Rb.abs().amax(dim=1)
    e = torch.floor(torch.log2(torch.clamp(amax, min=2.0 ** -120))) - 2.0
    e = torch.where(amax > 0, e, torch.full_like(e, -127.0)).clamp_(-127.0, 125.0)
    v = (Rb / torch.pow(torch.tensor(2.0, dtype=torch.float64, device=R.device), e)[:, None, :]).abs().clamp_(max=6.0)
    grid = torch.tensor(_E2M1_GRID, dtype=torch.float64, device=R.device)
    idx = torch.zeros_like(v, dtype=torch.int64)
    for i in range(7):
        lo, hi = _E2M1_GRID[i], _E2M1_GRID[i + 1]
        mid = 0.5 * (lo + hi)
        up = (v > mid) | ((v == mid) & (i % 2 == 1))  # ties go to the even code
        idx = torch.where((v >= lo) & (v < hi) & up, torch.full_like(idx, i + 1), idx)
        idx = torch.where((v >= lo) & (v < hi) & ~up, torch.full_like(idx, i), idx)
    idx = torch.where(v >= 6.0, torch.full_like(idx, 7), idx)
    codes = (idx + 8 * (Rb < 0).long()).to(torch.uint8).reshape(K, N)
    del grid
    return codes, (e + 127.0).to(torch.uint8)


def make_layer_mx_svd(K: int, N: int, r: int, x_calib: torch.Tensor, *, seed: int = 0, bias_std: Optional[float] = None,
                      device="cpu") -> MxLayerInputs:
    """The SVD recipe of make_layer_svd with the residual rounded to MXFP4 instead of INT4."""
    base = make_layer_svd(K, N, r, x_calib, seed=seed, bias_std=bias_std, device=device)
    codes, exps = _round_residual_mx(base.R)
    return MxLayerInputs(K, N, r, base.lam, base.L1, base.L2, codes, exps, base.bias, W=base.W)


def make_layer_mx_direct(K: int, N: int, r: int, *, seed: int = 0, device="cpu", with_bias: bool = True) -> MxLayerInputs:
    """MXFP4 constants drawn directly: codes uniform over the 16 E2M1 patterns, exponents uniform in [-9, -6] + 127;
    lam, L1, L2, bias as in make_layer_direct."""
    g = _gen(seed, device)
    codes = torch.randint(0, 16, (K, N), generator=g, device=device, dtype=torch.uint8)
    exps = torch.randint(118, 122, (K // MX_BLOCK, N), generator=g, device=device, dtype=torch.uint8)
    lam = torch.exp(0.5 * torch.randn(K, generator=g, device=device, dtype=torch.float32))
    L1 = L2 = None
    if r > 0:
        L1 = (0.05 * torch.randn(K, r, generator=g, device=device, dtype=torch.float32)).to(torch.bfloat16)
        L2 = (0.05 * torch.randn(r, N, generator=g, device=device, dtype=torch.float32)).to(torch.bfloat16)
    bias = 0.01 * torch.randn(N, generator=g, device=device, dtype=torch.float32) if with_bias else None
    return MxLayerInputs(K, N, r, lam, L1, L2, codes, exps, bias)


def reference_output(x: torch.Tensor, layer: LayerInputs) -> torch.Tensor:
    """The full-precision layer output Y = X W + b that a calibration run would record (Eq. 10's target), BF16.

    W is the layer's original weight when the recipe kept it, else the weight its quantized pieces stand for,
    diag(1/lam) (L1 L2 + codes * scale).  FP64 on the CPU, FP32 on a GPU (tooling, not part of the method)."""
    dev = x.device
    wide = torch.float64 if dev.type == "cpu" else torch.float32
    if layer.W is not None:
        W = layer.W.to(dev, wide)
    else:
        G = layer.K // 64
        deq = layer.qweight.to(dev, wide).view(G, 64, layer.N) * layer.wscale.to(dev, wide).view(G, 1, layer.N)
        W = deq.view(layer.K, layer.N)
        if layer.r > 0:
            W = W + layer.L1.to(dev, wide) @ layer.L2.to(dev, wide)
        W = W / layer.lam.to(dev, wide).view(-1, 1)
    y = x.to(wide) @ W
    if layer.bias is not None:
        y = y + layer.bias.to(dev, wide)
    return y.to(torch.bfloat16)


def sigma_for_bin(bin_index: int, sigma0: float = 2.0, decay: float = 0.8) -> float:
    """Activation spread per timestep bin: large at early (high-noise) bins, shrinking later."""
    return sigma0 * (decay ** bin_index)
