"""ctypes front end of the CPU oracle (TEST INFRASTRUCTURE ONLY).

Only the tests, the smoke check and the benchmark's CPU-baseline / reference leg may import this
package.  It compiles ``w4a4_oracle.cpp`` with gcc (single thread, ``-O2 -ffp-contract=off``) into a
shared library next to the source and marshals numpy arrays into it.  Nothing here touches CUDA and
nothing in the CUDA package imports it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "w4a4_oracle.cpp")
_LIB = os.path.join(_HERE, "libw4a4_oracle.so")
CXXFLAGS = ["-O2", "-std=c++17", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared"]
GROUP = 64

_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle if the shared library is missing or older than its source."""
    with _lock:
        if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
            tmp = _LIB + ".tmp%d" % os.getpid()
            subprocess.run(["g++", *CXXFLAGS, "-o", tmp, _SRC], check=True)
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        _lib.oracle_f32_to_bf16.restype = ctypes.c_uint16
        _lib.oracle_f32_to_bf16.argtypes = [ctypes.c_float]
    return _lib


def _p(a, dtype):
    """Pointer to a C-contiguous numpy array of the given dtype (None -> NULL)."""
    if a is None:
        return None
    assert isinstance(a, np.ndarray) and a.dtype == dtype and a.flags["C_CONTIGUOUS"], (a.dtype, dtype)
    return a.ctypes.data_as(ctypes.c_void_p)


def _as(a, dtype):
    return None if a is None else np.ascontiguousarray(a, dtype=dtype)


def f32_to_bf16(x: float) -> int:
    return int(_load().oracle_f32_to_bf16(ctypes.c_float(x)))


def quantize(X_bits, lam, rho, want_xhat=False):
    """Eq. 3-5, 8-9 on every row.  X_bits: [M, K] uint16 BF16 patterns.  -> codes int8 [M,K], scales f32 [M,G]."""
    X_bits = _as(X_bits, np.uint16)
    lam = _as(lam, np.float32)
    M, K = X_bits.shape
    q = np.empty((M, K), np.int8)
    s = np.empty((M, K // GROUP), np.float32)
    xh = np.empty((M, K), np.float32) if want_xhat else None
    rc = _load().oracle_quantize(_p(X_bits, np.uint16), _p(lam, np.float32), ctypes.c_float(rho), M, K,
                                 _p(q, np.int8), _p(s, np.float32), _p(xh, np.float32))
    assert rc == 0
    return (q, s, xh) if want_xhat else (q, s)


def lowrank_down(X_bits, lam, L1_bits):
    """T = X-hat L1 (Eq. 7), FP64 accumulation, returned as FP32 [M, r]."""
    X_bits = _as(X_bits, np.uint16)
    lam = _as(lam, np.float32)
    L1_bits = _as(L1_bits, np.uint16)
    M, K = X_bits.shape
    r = L1_bits.shape[1]
    T = np.empty((M, r), np.float32)
    rc = _load().oracle_lowrank_down(_p(X_bits, np.uint16), _p(lam, np.float32), _p(L1_bits, np.uint16), M, K, r,
                                     _p(T, np.float32))
    assert rc == 0
    return T


def partials(q, qw):
    """Per-group integer partial sums P[m, g, n] (Eq. 7, 4-bit branch before rescaling)."""
    q = _as(q, np.int8)
    qw = _as(qw, np.int8)
    M, K = q.shape
    N = qw.shape[1]
    P = np.empty((M, K // GROUP, N), np.int32)
    rc = _load().oracle_partials(_p(q, np.int8), _p(qw, np.int8), M, K, N, _p(P, np.int32))
    assert rc == 0
    return P


def assemble(P, s, sw, T, L2_bits, bias):
    """Eq. 7/11: Y64 [M,N] and its BF16 rounding from partials, scales, low-rank pieces and bias."""
    P = _as(P, np.int32)
    s = _as(s, np.float32)
    sw = _as(sw, np.float32)
    M, G, N = P.shape
    K = G * GROUP
    r = 0 if T is None else T.shape[1]
    T = _as(T, np.float32)
    L2_bits = _as(L2_bits, np.uint16)
    bias = _as(bias, np.float32)
    Y = np.empty((M, N), np.float64)
    Yb = np.empty((M, N), np.uint16)
    rc = _load().oracle_assemble(_p(P, np.int32), _p(s, np.float32), _p(sw, np.float32), _p(T, np.float32),
                                 _p(L2_bits, np.uint16), _p(bias, np.float32), M, K, N, r, _p(Y, np.float64),
                                 _p(Yb, np.uint16))
    assert rc == 0
    return Y, Yb


def forward_rows(X_bits, rows, lam, rho, L1_bits, L2_bits, qw, sw, bias, want_partials=False):
    """Whole layer on the chosen rows of X.  Returns a dict with q, s, T, (P), Y64, Ybf16 indexed by position in rows."""
    X_bits = _as(X_bits, np.uint16)
    rows = _as(rows, np.int32)
    lam = _as(lam, np.float32)
    qw = _as(qw, np.int8)
    sw = _as(sw, np.float32)
    bias = _as(bias, np.float32)
    M, K = X_bits.shape
    N = qw.shape[1]
    G = K // GROUP
    r = 0 if L1_bits is None else L1_bits.shape[1]
    L1_bits = _as(L1_bits, np.uint16)
    L2_bits = _as(L2_bits, np.uint16)
    n = rows.shape[0]
    assert rows.min(initial=0) >= 0 and rows.max(initial=0) < max(M, 1)
    out = dict(q=np.empty((n, K), np.int8), s=np.empty((n, G), np.float32),
               T=np.empty((n, r), np.float32) if r > 0 else None,
               P=np.empty((n, G, N), np.int32) if want_partials else None,
               Y64=np.empty((n, N), np.float64), Ybf16=np.empty((n, N), np.uint16))
    rc = _load().oracle_forward_rows(_p(X_bits, np.uint16), _p(rows, np.int32), n, K, N, r, _p(lam, np.float32),
                                     ctypes.c_float(rho), _p(L1_bits, np.uint16), _p(L2_bits, np.uint16),
                                     _p(qw, np.int8), _p(sw, np.float32), _p(bias, np.float32),
                                     _p(out["q"], np.int8), _p(out["s"], np.float32), _p(out["T"], np.float32),
                                     _p(out["P"], np.int32), _p(out["Y64"], np.float64), _p(out["Ybf16"], np.uint16))
    assert rc == 0
    return out


def forward_noquant(X, lam, L1, L2, R, bias):
    """Eq. 5-7 with both quantizers off, FP64 throughout: (X/lam) L1 L2 + (X/lam) R + b."""
    X = _as(X, np.float64)
    lam = _as(lam, np.float64)
    R = _as(R, np.float64)
    M, K = X.shape
    N = R.shape[1]
    r = 0 if L1 is None else L1.shape[1]
    L1 = _as(L1, np.float64)
    L2 = _as(L2, np.float64)
    bias = _as(bias, np.float64)
    Y = np.empty((M, N), np.float64)
    rc = _load().oracle_forward_noquant(_p(X, np.float64), _p(lam, np.float64), _p(L1, np.float64), _p(L2, np.float64),
                                        _p(R, np.float64), _p(bias, np.float64), M, K, N, r, _p(Y, np.float64))
    assert rc == 0
    return Y


def bf16_bits_to_f64(bits):
    """BF16 bit patterns -> the values they denote, as FP64 (exact)."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def clip_search(X_samples_bits, Yref_samples_bits, lam, candidates, L1_bits, L2_bits, qw, sw, bias):
    """Timestep-wise clipping-ratio search for one (layer, bin), Sec. III-C, Eq. 10.

    For every candidate ratio rho the objective is the sum, over the calibration samples of the bin, of the
    squared Euclidean distance between the full-precision layer output Y (given, BF16) and the output of the
    quantized layer with that ratio (Eq. 11, rounded to BF16 as the layer stores it), accumulated in FP64.
    Returns (index of the smallest objective -- the first one on ties --, list of objectives).
    """
    errs = []
    for rho in candidates:
        e = 0.0
        for Xb, Yb in zip(X_samples_bits, Yref_samples_bits):
            Xb = _as(Xb, np.uint16)
            out = forward_rows(Xb, np.arange(Xb.shape[0], dtype=np.int32), lam, float(np.float32(rho)), L1_bits, L2_bits,
                               qw, sw, bias)
            d = bf16_bits_to_f64(Yb) - bf16_bits_to_f64(out["Ybf16"])
            e += float(np.sum(d * d))
        errs.append(e)
    best = 0
    for i in range(1, len(errs)):
        if errs[i] < errs[best]:
            best = i
    return best, errs


# ----------------------------------------------------------------------------- MXFP4 variant
MX_BLOCK = 32
E2M1_VALUES = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0])


def e2m1_values(codes):
    """E2M1 codes (bit 3 = sign, bits 0-2 = magnitude index) -> the values they denote."""
    codes = np.asarray(codes, dtype=np.uint8)
    v = E2M1_VALUES[codes & 7]
    return np.where(codes & 8, -v, v)


def e2m1_rne_sat(v: float) -> int:
    lib = _load()
    lib.oracle_e2m1_rne_sat.restype = ctypes.c_uint8
    lib.oracle_e2m1_rne_sat.argtypes = [ctypes.c_float]
    return int(lib.oracle_e2m1_rne_sat(ctypes.c_float(v)))


def mx_quantize(X_bits, lam, rho):
    """MXFP4 activation quantization (OCP MX v1.0 conversion with the clip threshold of Eq. 8 as block maximum).
    -> codes uint8 [M, K] (E2M1), exps uint8 [M, K/32] (E8M0)."""
    X_bits = _as(X_bits, np.uint16)
    lam = _as(lam, np.float32)
    M, K = X_bits.shape
    codes = np.empty((M, K), np.uint8)
    exps = np.empty((M, K // MX_BLOCK), np.uint8)
    rc = _load().oracle_mx_quantize(_p(X_bits, np.uint16), _p(lam, np.float32), ctypes.c_float(rho), M, K,
                                    _p(codes, np.uint8), _p(exps, np.uint8))
    assert rc == 0
    return codes, exps


def mx_forward_rows(X_bits, rows, lam, rho, L1_bits, L2_bits, wcodes, wexps, bias):
    """Whole MXFP4 layer on the chosen rows.  Returns dict(codes, exps, T, Y64, Ybf16) indexed by position in rows."""
    X_bits = _as(X_bits, np.uint16)
    rows = _as(rows, np.int32)
    lam = _as(lam, np.float32)
    wcodes = _as(wcodes, np.uint8)
    wexps = _as(wexps, np.uint8)
    bias = _as(bias, np.float32)
    M, K = X_bits.shape
    N = wcodes.shape[1]
    r = 0 if L1_bits is None else L1_bits.shape[1]
    L1_bits = _as(L1_bits, np.uint16)
    L2_bits = _as(L2_bits, np.uint16)
    n = rows.shape[0]
    out = dict(codes=np.empty((n, K), np.uint8), exps=np.empty((n, K // MX_BLOCK), np.uint8),
               T=np.empty((n, r), np.float32) if r > 0 else None,
               Y64=np.empty((n, N), np.float64), Ybf16=np.empty((n, N), np.uint16))
    rc = _load().oracle_mx_forward_rows(_p(X_bits, np.uint16), _p(rows, np.int32), n, K, N, r, _p(lam, np.float32),
                                        ctypes.c_float(rho), _p(L1_bits, np.uint16), _p(L2_bits, np.uint16),
                                        _p(wcodes, np.uint8), _p(wexps, np.uint8), _p(bias, np.float32),
                                        _p(out["codes"], np.uint8), _p(out["exps"], np.uint8), _p(out["T"], np.float32),
                                        _p(out["Y64"], np.float64), _p(out["Ybf16"], np.uint16))
    assert rc == 0
    return out


def mx_clip_search(X_samples_bits, Yref_samples_bits, lam, candidates, L1_bits, L2_bits, wcodes, wexps, bias):
    """Eq. 10 for the MXFP4 variant: as clip_search, with mx_forward_rows as the quantized layer."""
    errs = []
    for rho in candidates:
        e = 0.0
        for Xb, Yb in zip(X_samples_bits, Yref_samples_bits):
            Xb = _as(Xb, np.uint16)
            out = mx_forward_rows(Xb, np.arange(Xb.shape[0], dtype=np.int32), lam, float(np.float32(rho)), L1_bits,
                                  L2_bits, wcodes, wexps, bias)
            d = bf16_bits_to_f64(Yb) - bf16_bits_to_f64(out["Ybf16"])
            e += float(np.sum(d * d))
        errs.append(e)
    best = 0
    for i in range(1, len(errs)):
        if errs[i] < errs[best]:
            best = i
    return best, errs


def gelu_tanh(y):
    """GELU in its tanh form, 0.5 y (1 + tanh(sqrt(2/pi) (y + 0.044715 y^3))), on FP64 values: the output
    activation a layer can be asked to fuse (the FFN's nonlinearity; not part of the paper's equations)."""
    y = np.asarray(y, dtype=np.float64)
    return 0.5 * y * (1.0 + np.tanh(np.sqrt(2.0 / np.pi) * (y + 0.044715 * y ** 3)))


def gptq_hessian(Xhat_bits):
    """Layer-wise second-order statistic of GPTQ (Frantar et al., 2023, Sec. 3: H = 2 X X^T for the layer's inputs;
    the factor 2 cancels in every quantity derived from it) for smoothed calibration activations X_hat [M, K] given
    as BF16 bit patterns: H = X_hat^T X_hat in FP64."""
    X = bf16_bits_to_f64(Xhat_bits)
    return X.T @ X


def gptq_quantize(R, H, group=64, percdamp=0.01):
    """GPTQ (Frantar et al., 2023, Algorithm 1 with the Cholesky reformulation of Sec. 4, step 3) on the residual
    branch (Sec. III-B: "we further apply GPTQ to the residual branch instead of simple round-to-nearest").

    R [K, N] FP64: residual weights, input channels along rows.  H [K, K] FP64: X_hat^T X_hat of the calibration
    activations.  Input channels are quantized in order; after each one its quantization error, scaled by the
    matching entry of U = chol(H^-1, upper), is spread over the input channels still to come.  Readings where the
    papers leave a choice: INT4 grid and group scale exactly as the round-to-nearest quantizer (scale = FP32(max
    |w| / 7) over the group's 64 input channels, code = round-half-even(w / scale) clamped to [-8, 7], zero group ->
    scale 0, codes 0), the scale being taken from the error-compensated weights when the sweep enters the group (not
    fixed from the original weights beforehand), input channels in natural order (no activation ordering); dead input channels (H_kk = 0) get H_kk = 1 and zero weights; damping percdamp *
    mean(diag H) on the diagonal; the lazy-batch block equals the group (pure bookkeeping: the result does not depend
    on it).  -> codes int8 [K, N], scales FP32 [K / group, N]."""
    W = np.array(R, dtype=np.float64, copy=True)
    H = np.array(H, dtype=np.float64, copy=True)
    K, N = W.shape
    assert H.shape == (K, K) and K % group == 0
    dead = np.diag(H) == 0
    H[dead, dead] = 1.0
    W[dead, :] = 0.0
    H[np.diag_indices(K)] += percdamp * np.mean(np.diag(H))
    Hinv = np.linalg.inv(H)
    U = np.linalg.cholesky((Hinv + Hinv.T) / 2).T          # upper, H^-1 = U^T U
    codes = np.zeros((K, N), np.int8)
    scales = np.zeros((K // group, N), np.float32)
    for k in range(K):
        g = k // group
        if k % group == 0:
            scales[g] = (np.abs(W[k:k + group]).max(axis=0) / 7.0).astype(np.float32)
        s = scales[g].astype(np.float64)
        safe = np.where(s > 0, s, 1.0)
        q = np.where(s > 0, np.clip(np.rint(W[k] / safe), -8, 7), 0.0)
        codes[k] = q.astype(np.int8)
        err = (W[k] - q * s) / U[k, k]
        W[k + 1:] -= np.outer(U[k, k + 1:], err)
    return codes, scales


def _mx_block_exponent(amax):
    """Shared exponent of an MXFP4 block (OCP MX v1.0, Sec. 6.3): floor(log2(largest magnitude)) minus the largest
    E2M1 exponent (2), kept within E8M0's range; an all-zero block gets the smallest exponent.  amax FP64 array."""
    m, ex = np.frexp(amax)                                 # amax = m * 2^ex, 0.5 <= m < 1  ->  floor(log2) = ex - 1
    e = np.where(amax > 0, ex - 1 - 2, -127)
    return np.clip(e, -127, 125).astype(np.int64)


def _e2m1_round_index(v):
    """Nearest E2M1 magnitude index for v >= 0 (saturating at 6), ties to the even index: one comparison per
    midpoint, strict where the lower neighbour is the even one."""
    idx = np.zeros(v.shape, np.int64)
    for i in range(7):
        mid = 0.5 * (E2M1_VALUES[i] + E2M1_VALUES[i + 1])
        idx += ((v > mid) | ((v == mid) & (i % 2 == 1))).astype(np.int64)
    return idx


def gptq_quantize_mx(R, H, percdamp=0.01):
    """GPTQ (as gptq_quantize: Frantar et al., 2023, Algorithm 1 with the Cholesky reformulation) on the residual
    branch with the MXFP4 grid of the MX variant instead of INT4: per 32 input channels and output channel one E8M0
    exponent, taken from the error-compensated weights when the sweep enters the block (floor(log2 max|w|) - 2), and
    E2M1 elements, nearest with ties to the even code, saturating at 6, sign bit from the compensated weight.  Dead
    channels, damping and the order of the sweep as in gptq_quantize.
    -> codes uint8 [K, N] (bit 3 sign, bits 0-2 magnitude index), exps uint8 [K / 32, N] (exponent + 127)."""
    W = np.array(R, dtype=np.float64, copy=True)
    H = np.array(H, dtype=np.float64, copy=True)
    K, N = W.shape
    assert H.shape == (K, K) and K % 32 == 0
    dead = np.diag(H) == 0
    H[dead, dead] = 1.0
    W[dead, :] = 0.0
    H[np.diag_indices(K)] += percdamp * np.mean(np.diag(H))
    Hinv = np.linalg.inv(H)
    U = np.linalg.cholesky((Hinv + Hinv.T) / 2).T          # upper, H^-1 = U^T U
    codes = np.zeros((K, N), np.uint8)
    exps = np.zeros((K // 32, N), np.uint8)
    e = np.zeros(N, np.int64)
    for k in range(K):
        if k % 32 == 0:
            e = _mx_block_exponent(np.abs(W[k:k + 32]).max(axis=0))
            exps[k // 32] = (e + 127).astype(np.uint8)
        scale = np.ldexp(1.0, e)
        idx = _e2m1_round_index(np.minimum(np.abs(W[k]) / scale, 6.0))
        codes[k] = (idx + 8 * (W[k] < 0)).astype(np.uint8)
        deq = np.where(W[k] < 0, -1.0, 1.0) * E2M1_VALUES[idx] * scale
        err = (W[k] - deq) / U[k, k]
        W[k + 1:] -= np.outer(U[k, k + 1:], err)
    return codes, exps

