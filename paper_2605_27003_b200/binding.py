"""ctypes binding of libw4a4: argument marshalling only, same names as the C entry points.

Every step of the layer runs inside the library's CUDA kernels.  PyTorch appears here solely as the
owner of device memory (``tensor.data_ptr()``) and of the CUDA stream.  Importing this module fails
loudly if the shared library has not been built; there is no fallback of any kind.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libw4a4.so")

ACT_NONE, ACT_GELU_TANH = 0, 1
W4A4_OK = 0
STATUS_NAMES = {0: "OK", 1: "ERR_INVALID_ARG", 2: "ERR_SHAPE", 3: "ERR_ALLOC", 4: "ERR_CUDA", 5: "ERR_ARCH",
                6: "ERR_TIMEOUT"}

# Every symbol include/w4a4.h declares.
EXPORTED_SYMBOLS = (
    "w4a4_ctx_create", "w4a4_ctx_destroy", "w4a4_pack_weights", "w4a4_destroy", "w4a4_linear_forward",
    "w4a4_ctx_enable_host_io", "w4a4_linear_forward_host", "w4a4_quantize_activations", "w4a4_gemm_from_workspace", "w4a4_debug_quantize", "w4a4_debug_partials",
    "w4a4_tile_shape", "w4a4_quantize_noalloc", "w4a4_clip_search",
    "w4a4_mx_pack_weights", "w4a4_mx_destroy", "w4a4_mx_handle_bytes", "w4a4_mx_linear_forward",
    "w4a4_mx_quantize_activations", "w4a4_mx_gemm_from_workspace", "w4a4_mx_debug_quantize", "w4a4_mx_clip_search",
    "w4a4_mx_ffn_forward", "w4a4_mx_debug_fused_input", "w4a4_gptq_quantize", "w4a4_mx_gptq_quantize", "w4a4_gptq_accumulate", "w4a4_gptq_workspace_bytes", "w4a4_query_status", "w4a4_debug_wait_probe", "w4a4_debug_stalled_gemm", "w4a4_debug_set_tile_order",
    "w4a4_debug_fail_allocation_after", "w4a4_handle_bytes", "w4a4_ctx_bytes", "w4a4_status_string",
)


class W4A4Error(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)} ({_lib().w4a4_status_string(status).decode()})")


class WeightDesc(ctypes.Structure):
    _fields_ = [
        ("K", ctypes.c_int), ("N", ctypes.c_int), ("r", ctypes.c_int), ("group", ctypes.c_int),
        ("num_experts", ctypes.c_int), ("num_bins", ctypes.c_int), ("num_layers", ctypes.c_int),
        ("layer_id", ctypes.c_int), ("pointers_on_device", ctypes.c_int), ("output_activation", ctypes.c_int),
        ("qweight", ctypes.POINTER(ctypes.c_void_p)), ("wscale", ctypes.POINTER(ctypes.c_void_p)),
        ("lambda_", ctypes.POINTER(ctypes.c_void_p)), ("L1", ctypes.POINTER(ctypes.c_void_p)),
        ("L2", ctypes.POINTER(ctypes.c_void_p)), ("bias", ctypes.POINTER(ctypes.c_void_p)),
    ]


class MxWeightDesc(ctypes.Structure):
    _fields_ = [
        ("K", ctypes.c_int), ("N", ctypes.c_int), ("r", ctypes.c_int),
        ("num_experts", ctypes.c_int), ("num_bins", ctypes.c_int), ("num_layers", ctypes.c_int),
        ("layer_id", ctypes.c_int), ("pointers_on_device", ctypes.c_int), ("output_activation", ctypes.c_int),
        ("wcodes", ctypes.POINTER(ctypes.c_void_p)), ("wexps", ctypes.POINTER(ctypes.c_void_p)),
        ("lambda_", ctypes.POINTER(ctypes.c_void_p)), ("L1", ctypes.POINTER(ctypes.c_void_p)),
        ("L2", ctypes.POINTER(ctypes.c_void_p)), ("bias", ctypes.POINTER(ctypes.c_void_p)),
    ]


_LIB = None


def _lib():
    global _LIB
    if _LIB is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2605_27003_b200.build` "
                              "(nvcc, sm_100a). There is no fallback path.")
        lib = ctypes.CDLL(LIB_PATH)
        vp, ci = ctypes.c_void_p, ctypes.c_int
        lib.w4a4_status_string.restype = ctypes.c_char_p
        lib.w4a4_status_string.argtypes = [ci]
        lib.w4a4_ctx_create.argtypes = [ci, ci, ci, ci, ctypes.POINTER(vp)]
        lib.w4a4_ctx_destroy.argtypes = [vp]
        lib.w4a4_ctx_destroy.restype = None
        lib.w4a4_pack_weights.argtypes = [vp, ctypes.POINTER(WeightDesc), ctypes.POINTER(vp)]
        lib.w4a4_destroy.argtypes = [vp]
        lib.w4a4_destroy.restype = None
        lib.w4a4_linear_forward.argtypes = [vp, vp, ci, ci, ci, vp, vp, vp]
        lib.w4a4_ctx_enable_host_io.argtypes = [vp, ci, ci]
        lib.w4a4_linear_forward_host.argtypes = [vp, vp, ci, ci, ci, vp, vp, vp]
        lib.w4a4_quantize_activations.argtypes = [vp, vp, ci, ci, ci, vp, vp]
        lib.w4a4_gemm_from_workspace.argtypes = [vp, ci, ci, vp, vp]
        lib.w4a4_debug_quantize.argtypes = [vp, vp, ci, ci, ci, vp, vp, vp, vp, vp]
        lib.w4a4_debug_partials.argtypes = [vp, vp, ci, ci, ci, vp, vp, ci, ci, vp, vp]
        lib.w4a4_quantize_noalloc.argtypes = [vp, ci, ci, vp, vp, ci, vp, vp, vp]
        lib.w4a4_clip_search.argtypes = [vp, ctypes.POINTER(vp), ctypes.POINTER(vp), ci, ci, ci, ci,
                                         ctypes.POINTER(ctypes.c_float), ci, vp, ctypes.POINTER(ctypes.c_double),
                                         ctypes.POINTER(ci), vp]
        lib.w4a4_mx_pack_weights.argtypes = [vp, ctypes.POINTER(MxWeightDesc), ctypes.POINTER(vp)]
        lib.w4a4_mx_destroy.argtypes = [vp]
        lib.w4a4_mx_destroy.restype = None
        lib.w4a4_mx_handle_bytes.argtypes = [vp]
        lib.w4a4_mx_handle_bytes.restype = ctypes.c_size_t
        lib.w4a4_mx_linear_forward.argtypes = [vp, vp, ci, ci, ci, vp, vp, vp]
        lib.w4a4_mx_quantize_activations.argtypes = [vp, vp, ci, ci, ci, vp, vp]
        lib.w4a4_mx_gemm_from_workspace.argtypes = [vp, ci, ci, vp, vp]
        lib.w4a4_mx_debug_quantize.argtypes = [vp, vp, ci, ci, ci, vp, vp, vp, vp, vp]
        lib.w4a4_mx_ffn_forward.argtypes = [vp, vp, vp, ci, ci, ci, vp, vp, vp]
        lib.w4a4_mx_debug_fused_input.argtypes = [vp, ci, vp, vp, vp, vp]
        lib.w4a4_mx_clip_search.argtypes = lib.w4a4_clip_search.argtypes
        lib.w4a4_gptq_quantize.argtypes = [ci, vp, vp, ci, vp, ci, ci, ctypes.c_double, vp, vp, vp, ctypes.c_size_t, vp]
        lib.w4a4_mx_gptq_quantize.argtypes = lib.w4a4_gptq_quantize.argtypes
        lib.w4a4_gptq_accumulate.argtypes = [ci, vp, ci, ci, vp, vp]
        lib.w4a4_gptq_workspace_bytes.argtypes = [ci, ci, ci]
        lib.w4a4_gptq_workspace_bytes.restype = ctypes.c_size_t
        lib.w4a4_tile_shape.argtypes = [ctypes.POINTER(ci), ctypes.POINTER(ci)]
        lib.w4a4_tile_shape.restype = None
        lib.w4a4_query_status.argtypes = [vp]
        lib.w4a4_debug_wait_probe.argtypes = [vp, ctypes.c_uint64, vp]
        lib.w4a4_debug_stalled_gemm.argtypes = [vp, ci, ci, vp, ci, ctypes.c_uint64, vp]
        lib.w4a4_debug_fail_allocation_after.argtypes = [ci]
        lib.w4a4_debug_set_tile_order.argtypes = [vp, ci]
        lib.w4a4_debug_fail_allocation_after.restype = None
        lib.w4a4_handle_bytes.argtypes = [vp]
        lib.w4a4_handle_bytes.restype = ctypes.c_size_t
        lib.w4a4_ctx_bytes.argtypes = [vp]
        lib.w4a4_ctx_bytes.restype = ctypes.c_size_t
        _LIB = lib
    return _LIB


def load_library():
    """Loads libw4a4.so (raises ImportError if it has not been built)."""
    return _lib()


def _check(status: int, where: str):
    if status != W4A4_OK:
        raise W4A4Error(status, where)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream) -> ctypes.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


# ----------------------------------------------------------------------------- C entry points, same names
def w4a4_status_string(status: int) -> str:
    return _lib().w4a4_status_string(status).decode()


def w4a4_tile_shape():
    m, n = ctypes.c_int(0), ctypes.c_int(0)
    _lib().w4a4_tile_shape(ctypes.byref(m), ctypes.byref(n))
    return m.value, n.value


def w4a4_ctx_create(device: int, max_M: int, max_K: int, max_r: int) -> ctypes.c_void_p:
    out = ctypes.c_void_p()
    _check(_lib().w4a4_ctx_create(device, max_M, max_K, max_r, ctypes.byref(out)), "w4a4_ctx_create")
    return out


def w4a4_ctx_destroy(ctx):
    _lib().w4a4_ctx_destroy(ctx)


def w4a4_pack_weights(ctx, *, K: int, N: int, r: int, num_bins: int, num_layers: int, layer_id: int,
                      qweight: Sequence[torch.Tensor], wscale: Sequence[torch.Tensor],
                      lam: Sequence[torch.Tensor], L1: Optional[Sequence[torch.Tensor]],
                      L2: Optional[Sequence[torch.Tensor]], bias: Optional[Sequence[Optional[torch.Tensor]]],
                      group: int = 64, output_activation: int = 0) -> ctypes.c_void_p:
    """One tensor per expert in every list; all on the host or all on one CUDA device, contiguous."""
    E = len(qweight)
    on_dev = qweight[0].is_cuda
    keep = []

    def arr(ts, dtype, shape):
        if ts is None:
            return None
        a = (ctypes.c_void_p * E)()
        for i, t in enumerate(ts):
            if t is None:
                a[i] = None
                continue
            assert t.dtype == dtype and tuple(t.shape) == shape and t.is_contiguous() and t.is_cuda == on_dev, \
                (t.dtype, tuple(t.shape), shape)
            keep.append(t)
            a[i] = t.data_ptr()
        return a

    G = K // group
    d = WeightDesc(K=K, N=N, r=r, group=group, num_experts=E, num_bins=num_bins, num_layers=num_layers,
                   layer_id=layer_id, pointers_on_device=int(on_dev), output_activation=output_activation)
    d.qweight = arr(qweight, torch.int8, (K, N))
    d.wscale = arr(wscale, torch.float32, (G, N))
    d.lambda_ = arr(lam, torch.float32, (K,))
    d.L1 = arr(L1, torch.bfloat16, (K, r)) if r > 0 else None
    d.L2 = arr(L2, torch.bfloat16, (r, N)) if r > 0 else None
    d.bias = arr(bias, torch.float32, (N,)) if bias is not None else None
    out = ctypes.c_void_p()
    _check(_lib().w4a4_pack_weights(ctx, ctypes.byref(d), ctypes.byref(out)), "w4a4_pack_weights")
    return out


def w4a4_destroy(handle):
    _lib().w4a4_destroy(handle)


def w4a4_linear_forward(handle, X: torch.Tensor, M: int, expert_id: int, timestep_bin: int,
                        clip_table: torch.Tensor, Y: torch.Tensor, stream=None):
    _check(_lib().w4a4_linear_forward(handle, _ptr(X), M, expert_id, timestep_bin, _ptr(clip_table), _ptr(Y),
                                      _stream(stream)), "w4a4_linear_forward")


def w4a4_ctx_enable_host_io(ctx, chunk_rows: int, max_N: int):
    _check(_lib().w4a4_ctx_enable_host_io(ctx, chunk_rows, max_N), "w4a4_ctx_enable_host_io")


def w4a4_linear_forward_host(handle, X_host: torch.Tensor, M: int, expert_id: int, timestep_bin: int,
                             clip_table: torch.Tensor, Y_host: torch.Tensor, stream=None):
    """X_host / Y_host are CPU tensors (pinned for overlap); clip_table is a CUDA tensor."""
    assert not X_host.is_cuda and not Y_host.is_cuda and clip_table.is_cuda
    _check(_lib().w4a4_linear_forward_host(handle, _ptr(X_host), M, expert_id, timestep_bin, _ptr(clip_table),
                                           _ptr(Y_host), _stream(stream)), "w4a4_linear_forward_host")


def w4a4_quantize_activations(handle, X, M, expert_id, timestep_bin, clip_table, stream=None):
    _check(_lib().w4a4_quantize_activations(handle, _ptr(X), M, expert_id, timestep_bin, _ptr(clip_table),
                                            _stream(stream)), "w4a4_quantize_activations")


def w4a4_gemm_from_workspace(handle, M, expert_id, Y, stream=None):
    _check(_lib().w4a4_gemm_from_workspace(handle, M, expert_id, _ptr(Y), _stream(stream)), "w4a4_gemm_from_workspace")


def w4a4_debug_quantize(handle, X, M, expert_id, timestep_bin, clip_table, codes, scales, T, stream=None):
    _check(_lib().w4a4_debug_quantize(handle, _ptr(X), M, expert_id, timestep_bin, _ptr(clip_table), _ptr(codes),
                                      _ptr(scales), _ptr(T), _stream(stream)), "w4a4_debug_quantize")


def w4a4_debug_partials(handle, X, M, expert_id, timestep_bin, clip_table, Y, m0, n0, P, stream=None):
    _check(_lib().w4a4_debug_partials(handle, _ptr(X), M, expert_id, timestep_bin, _ptr(clip_table), _ptr(Y), m0, n0,
                                      _ptr(P), _stream(stream)), "w4a4_debug_partials")


def w4a4_quantize_noalloc(X, M, K, lam, clip_table, clip_index, codes, scales, stream=None):
    """Context-free activation quantization into caller buffers; the library's built-in scratch is used."""
    _check(_lib().w4a4_quantize_noalloc(_ptr(X), M, K, _ptr(lam), _ptr(clip_table), clip_index, _ptr(codes),
                                        _ptr(scales), _stream(stream)), "w4a4_quantize_noalloc")


def w4a4_clip_search(handle, X_samples, Yref_samples, M, expert_id, timestep_bin, candidates, clip_table, stream=None,
                     *, mx: bool = False):
    """Eq. 10 on the device: returns (index of the best candidate, list of the candidates' squared errors) and
    writes the winning ratio into the clip table entry of (expert, layer, bin).  mx=True: MXFP4 handle."""
    n_s, n_c = len(X_samples), len(candidates)
    xs = (ctypes.c_void_p * n_s)(*[_ptr(x) for x in X_samples])
    ys = (ctypes.c_void_p * n_s)(*[_ptr(y) for y in Yref_samples])
    cand = (ctypes.c_float * n_c)(*[float(c) for c in candidates])
    errs = (ctypes.c_double * n_c)()
    best = ctypes.c_int(-1)
    fn, name = (_lib().w4a4_mx_clip_search, "w4a4_mx_clip_search") if mx else (_lib().w4a4_clip_search, "w4a4_clip_search")
    _check(fn(handle, xs, ys, n_s, M, expert_id, timestep_bin, cand, n_c, _ptr(clip_table), errs, ctypes.byref(best),
              _stream(stream)), name)
    return int(best.value), [float(e) for e in errs]


def w4a4_mx_clip_search(handle, X_samples, Yref_samples, M, expert_id, timestep_bin, candidates, clip_table, stream=None):
    return w4a4_clip_search(handle, X_samples, Yref_samples, M, expert_id, timestep_bin, candidates, clip_table, stream,
                            mx=True)


# ----------------------------------------------------------------------------- MXFP4 variant
def w4a4_mx_pack_weights(ctx, *, K: int, N: int, r: int, num_bins: int, num_layers: int, layer_id: int,
                         wcodes: Sequence[torch.Tensor], wexps: Sequence[torch.Tensor], lam: Sequence[torch.Tensor],
                         L1: Optional[Sequence[torch.Tensor]], L2: Optional[Sequence[torch.Tensor]],
                         bias: Optional[Sequence[Optional[torch.Tensor]]], output_activation: int = 0) -> ctypes.c_void_p:
    """One tensor per expert in every list; all on the host or all on one CUDA device, contiguous."""
    E = len(wcodes)
    on_dev = wcodes[0].is_cuda
    keep = []

    def arr(ts, dtype, shape):
        if ts is None:
            return None
        a = (ctypes.c_void_p * E)()
        for i, t in enumerate(ts):
            if t is None:
                a[i] = None
                continue
            assert t.dtype == dtype and tuple(t.shape) == shape and t.is_contiguous() and t.is_cuda == on_dev, \
                (t.dtype, tuple(t.shape), shape)
            keep.append(t)
            a[i] = t.data_ptr()
        return a

    d = MxWeightDesc(K=K, N=N, r=r, num_experts=E, num_bins=num_bins, num_layers=num_layers, layer_id=layer_id,
                     pointers_on_device=int(on_dev), output_activation=output_activation)
    d.wcodes = arr(wcodes, torch.uint8, (K, N))
    d.wexps = arr(wexps, torch.uint8, (K // 32, N))
    d.lambda_ = arr(lam, torch.float32, (K,))
    d.L1 = arr(L1, torch.bfloat16, (K, r)) if r > 0 else None
    d.L2 = arr(L2, torch.bfloat16, (r, N)) if r > 0 else None
    d.bias = arr(bias, torch.float32, (N,)) if bias is not None else None
    out = ctypes.c_void_p()
    _check(_lib().w4a4_mx_pack_weights(ctx, ctypes.byref(d), ctypes.byref(out)), "w4a4_mx_pack_weights")
    return out


def w4a4_mx_destroy(handle):
    _lib().w4a4_mx_destroy(handle)


def w4a4_mx_handle_bytes(handle) -> int:
    return int(_lib().w4a4_mx_handle_bytes(handle))


def w4a4_mx_linear_forward(handle, X, M, expert_id, timestep_bin, clip_table, Y, stream=None):
    _check(_lib().w4a4_mx_linear_forward(handle, _ptr(X), M, expert_id, timestep_bin, _ptr(clip_table), _ptr(Y),
                                         _stream(stream)), "w4a4_mx_linear_forward")


def w4a4_mx_quantize_activations(handle, X, M, expert_id, timestep_bin, clip_table, stream=None):
    _check(_lib().w4a4_mx_quantize_activations(handle, _ptr(X), M, expert_id, timestep_bin, _ptr(clip_table),
                                               _stream(stream)), "w4a4_mx_quantize_activations")


def w4a4_mx_gemm_from_workspace(handle, M, expert_id, Y, stream=None):
    _check(_lib().w4a4_mx_gemm_from_workspace(handle, M, expert_id, _ptr(Y), _stream(stream)),
           "w4a4_mx_gemm_from_workspace")


def w4a4_mx_debug_quantize(handle, X, M, expert_id, timestep_bin, clip_table, codes, exps, T=None, stream=None):
    _check(_lib().w4a4_mx_debug_quantize(handle, _ptr(X), M, expert_id, timestep_bin, _ptr(clip_table), _ptr(codes),
                                         _ptr(exps), _ptr(T), _stream(stream)), "w4a4_mx_debug_quantize")


def w4a4_mx_ffn_forward(up, down, X, M, expert_id, timestep_bin, clip_table, Y, stream=None):
    _check(_lib().w4a4_mx_ffn_forward(up, down, _ptr(X), M, expert_id, timestep_bin, _ptr(clip_table), _ptr(Y),
                                      _stream(stream)), "w4a4_mx_ffn_forward")


def w4a4_mx_debug_fused_input(down, M, codes, exps, T=None, stream=None):
    _check(_lib().w4a4_mx_debug_fused_input(down, M, _ptr(codes), _ptr(exps), _ptr(T), _stream(stream)),
           "w4a4_mx_debug_fused_input")


def w4a4_gptq_workspace_bytes(K: int, N: int, M_cal: int) -> int:
    return int(_lib().w4a4_gptq_workspace_bytes(K, N, M_cal))


def w4a4_gptq_quantize(R, codes, scales, Xhat=None, H=None, percdamp=0.01, workspace=None, stream=None):
    """GPTQ on the residual branch (Sec. III-B).  R device FP32 [K, N]; Xhat device BF16 [M_cal, K] or H device FP64
    [K, K] (exactly one); codes device int8 [K, N] and scales device FP32 [K/64, N] are written.  workspace: a device
    byte tensor of at least w4a4_gptq_workspace_bytes bytes, or None (the library allocates for the call)."""
    K, N = R.shape
    M_cal = Xhat.shape[0] if Xhat is not None else 0
    ws_bytes = workspace.numel() * workspace.element_size() if workspace is not None else 0
    _check(_lib().w4a4_gptq_quantize(R.device.index or 0, _ptr(R), _ptr(Xhat), M_cal, _ptr(H), K, N, float(percdamp),
                                     _ptr(codes), _ptr(scales), _ptr(workspace), ws_bytes, _stream(stream)),
           "w4a4_gptq_quantize")


def w4a4_gptq_accumulate(Xhat, H, stream=None):
    """H (device FP64 [K, K], upper triangle) += Xhat^T Xhat for one batch of calibration tokens (device BF16 [M, K])."""
    M_cal, K = Xhat.shape
    _check(_lib().w4a4_gptq_accumulate(Xhat.device.index or 0, _ptr(Xhat), M_cal, K, _ptr(H), _stream(stream)),
           "w4a4_gptq_accumulate")


def w4a4_mx_gptq_quantize(R, codes, exps, Xhat=None, H=None, percdamp=0.01, workspace=None, stream=None):
    """GPTQ on the residual branch on the MXFP4 grid.  As w4a4_gptq_quantize, with codes device uint8 [K, N] (E2M1) and
    exps device uint8 [K/32, N] (E8M0) written."""
    K, N = R.shape
    M_cal = Xhat.shape[0] if Xhat is not None else 0
    ws_bytes = workspace.numel() * workspace.element_size() if workspace is not None else 0
    _check(_lib().w4a4_mx_gptq_quantize(R.device.index or 0, _ptr(R), _ptr(Xhat), M_cal, _ptr(H), K, N,
                                        float(percdamp), _ptr(codes), _ptr(exps), _ptr(workspace), ws_bytes,
                                        _stream(stream)), "w4a4_mx_gptq_quantize")


def w4a4_query_status(ctx) -> int:
    return int(_lib().w4a4_query_status(ctx))


def w4a4_debug_wait_probe(ctx, limit_ns: int, stream=None):
    """Test hook: enqueues a one-warp kernel whose bounded wait gives up after limit_ns (sets the context's error word)."""
    _check(_lib().w4a4_debug_wait_probe(ctx, int(limit_ns), _stream(stream)), "w4a4_debug_wait_probe")


def w4a4_debug_stalled_gemm(handle, M: int, expert_id: int, Y, stall_stage: int, limit_ns: int, stream=None):
    """Test hook: the GEMM on the current workspace with one operand stage withheld and a short wait limit."""
    _check(_lib().w4a4_debug_stalled_gemm(handle, M, expert_id, _ptr(Y), int(stall_stage), int(limit_ns),
                                          _stream(stream)), "w4a4_debug_stalled_gemm")


def w4a4_debug_set_tile_order(ctx, super_column_tiles: int):
    """Test hook: forces the super-column width of the INT4 GEMM's tile order (0: automatic)."""
    _check(_lib().w4a4_debug_set_tile_order(ctx, int(super_column_tiles)), "w4a4_debug_set_tile_order")


def w4a4_debug_fail_allocation_after(n: int):
    """Test hook: the (n + 1)-th device allocation the library attempts from now on fails once; n < 0 disarms."""
    _lib().w4a4_debug_fail_allocation_after(int(n))


def w4a4_handle_bytes(handle) -> int:
    return int(_lib().w4a4_handle_bytes(handle))


def w4a4_ctx_bytes(ctx) -> int:
    return int(_lib().w4a4_ctx_bytes(ctx))


# ----------------------------------------------------------------------------- small conveniences
class Context:
    """Owns a w4a4_ctx_t (per-stream workspace)."""

    def __init__(self, device: int, max_M: int, max_K: int, max_r: int):
        self.device, self.max_M, self.max_K, self.max_r = device, max_M, max_K, max_r
        self.ptr = w4a4_ctx_create(device, max_M, max_K, max_r)

    def check(self):
        st = w4a4_query_status(self.ptr)
        _check(st, "w4a4_query_status")

    def close(self):
        if self.ptr is not None:
            w4a4_ctx_destroy(self.ptr)
            self.ptr = None

    def __del__(self):  # pragma: no cover
        try:
            self.close()
        except Exception:
            pass


class Layer:
    """Owns a w4a4_handle_t built from one LayerInputs-like object per expert."""

    def __init__(self, ctx: Context, experts, *, num_bins: int, num_layers: int = 1, layer_id: int = 0,
                 output_activation: int = 0):
        e0 = experts[0]
        self.ctx, self.K, self.N, self.r, self.E = ctx, e0.K, e0.N, e0.r, len(experts)
        has_bias = any(e.bias is not None for e in experts)
        self.ptr = w4a4_pack_weights(
            ctx.ptr, K=e0.K, N=e0.N, r=e0.r, num_bins=num_bins, num_layers=num_layers, layer_id=layer_id,
            qweight=[e.qweight.contiguous() for e in experts], wscale=[e.wscale.contiguous() for e in experts],
            lam=[e.lam.contiguous() for e in experts],
            L1=[e.L1.contiguous() for e in experts] if e0.r > 0 else None,
            L2=[e.L2.contiguous() for e in experts] if e0.r > 0 else None,
            bias=[None if e.bias is None else e.bias.contiguous() for e in experts] if has_bias else None,
            output_activation=output_activation)

    def forward(self, X: torch.Tensor, expert_id: int, timestep_bin: int, clip_table: torch.Tensor,
                Y: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        assert X.dtype == torch.bfloat16 and X.is_cuda and X.is_contiguous() and X.shape[1] == self.K
        M = X.shape[0]
        if Y is None:
            Y = torch.empty(M, self.N, dtype=torch.bfloat16, device=X.device)
        w4a4_linear_forward(self.ptr, X, M, expert_id, timestep_bin, clip_table, Y, stream)
        return Y

    def close(self):
        if self.ptr is not None:
            w4a4_destroy(self.ptr)
            self.ptr = None

    def __del__(self):  # pragma: no cover
        try:
            self.close()
        except Exception:
            pass


class MxLayer:
    """Owns a w4a4_mx_handle_t built from one MxLayerInputs-like object per expert."""

    def __init__(self, ctx: Context, experts, *, num_bins: int, num_layers: int = 1, layer_id: int = 0,
                 output_activation: int = 0):
        e0 = experts[0]
        self.ctx, self.K, self.N, self.r, self.E = ctx, e0.K, e0.N, e0.r, len(experts)
        has_bias = any(e.bias is not None for e in experts)
        self.ptr = w4a4_mx_pack_weights(
            ctx.ptr, K=e0.K, N=e0.N, r=e0.r, num_bins=num_bins, num_layers=num_layers, layer_id=layer_id,
            wcodes=[e.wcodes.contiguous() for e in experts], wexps=[e.wexps.contiguous() for e in experts],
            lam=[e.lam.contiguous() for e in experts],
            L1=[e.L1.contiguous() for e in experts] if e0.r > 0 else None,
            L2=[e.L2.contiguous() for e in experts] if e0.r > 0 else None,
            bias=[None if e.bias is None else e.bias.contiguous() for e in experts] if has_bias else None,
            output_activation=output_activation)

    def forward(self, X: torch.Tensor, expert_id: int, timestep_bin: int, clip_table: torch.Tensor,
                Y: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        assert X.dtype == torch.bfloat16 and X.is_cuda and X.is_contiguous() and X.shape[1] == self.K
        M = X.shape[0]
        if Y is None:
            Y = torch.empty(M, self.N, dtype=torch.bfloat16, device=X.device)
        w4a4_mx_linear_forward(self.ptr, X, M, expert_id, timestep_bin, clip_table, Y, stream)
        return Y

    def close(self):
        if self.ptr is not None:
            w4a4_mx_destroy(self.ptr)
            self.ptr = None

    def __del__(self):  # pragma: no cover
        try:
            self.close()
        except Exception:
            pass
