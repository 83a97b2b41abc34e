// Host-side pieces shared by the translation units of libw4a4: the context object, small CUDA helpers.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "../../include/w4a4.h"

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct w4a4_ctx {
  int device = 0;
  int max_M = 0, max_K = 0, max_r = 0;
  uint8_t* codes = nullptr;   // [max_M, K] activation codes, one E4M3 byte each (pitch K of the running layer)
  float* scales = nullptr;    // [K/64, scales_ld] group-major activation scales
  uint8_t* a_sop = nullptr;   // token-side scale operands of the GEMM's scale MMA: [ceil(max_M/128)][ceil(G/2)][2048]
  int scales_ld = 0;          // max_M rounded up to a multiple of 4 (16-byte rows for TMA)
  uint16_t* t_hilo = nullptr; // [max_M, 2r] BF16 high | low parts of Xh L1
  uint8_t* b8 = nullptr;      // [N, K] E4M3 image of the running layer's weight codes (rewritten by every forward)
  size_t b8_bytes = 0;        // grows to the largest N x K packed on this context
  float* t_partial = nullptr; // [kMaxKSplits, min(max_M, kKSplitMaxRows), max_r] FP32 partial sums of T when kernel 1 splits K
  uint8_t* mx_sfa = nullptr;  // MXFP4 variant: activation scale atoms [ceil(max_M/128)][max_K/128][512] (allocated on first use)
  // MXFP4 variant, fused FFN (allocated with mx_sfa): the second workspace a producing GEMM's epilogue quantizes
  // the next layer's input into, while the first still holds its own operands.
  uint8_t* mx_codes2 = nullptr;   // [max_M, max_K / 2]
  uint8_t* mx_sfa2 = nullptr;     // scale atoms, as mx_sfa
  float* mx_t32 = nullptr;        // [max_M, max_r] FP32 accumulators of the next layer's T
  uint16_t* t_hilo2 = nullptr;    // [max_M, 2 max_r] BF16 high | low of the same
  int* d_err = nullptr;       // device error word
  size_t bytes = 0;
  int num_sms = 0;
  size_t l2_bytes = 0;        // size of the device's L2 (sizes the GEMM's tile order)
  int debug_sc_tiles = 0;     // test hook: forced super-column width of the GEMM's tile order (0: automatic)
  EncodeTiledFn encode = nullptr;
  // Host-buffer forward (w4a4_linear_forward_host): staging buffers, copy streams and events.
  int host_chunk_rows = 0, host_max_N = 0;
  uint16_t* hx[2] = {nullptr, nullptr};  // device staging of an activation chunk (double buffered)
  uint16_t* hy[2] = {nullptr, nullptr};  // device staging of an output chunk
  cudaStream_t s_h2d = nullptr, s_compute = nullptr, s_d2h = nullptr;
  cudaEvent_t ev_in[2] = {nullptr, nullptr}, ev_done[2] = {nullptr, nullptr}, ev_out[2] = {nullptr, nullptr};
  cudaEvent_t ev_begin = nullptr, ev_end = nullptr;
};

// Test hook for the allocation-failure paths (w4a4_debug_fail_allocation_after): a countdown over the device
// allocations of the whole library, -1 when idle.  The allocation that finds it at 0 fails once, exactly as a refused
// cudaMalloc would, and the hook disarms itself.  One definition, in w4a4_api.cu.
extern std::atomic<int> g_w4a4_alloc_countdown;

inline bool alloc_failure_injected() {
  int c = g_w4a4_alloc_countdown.load(std::memory_order_relaxed);
  while (c >= 0) {
    if (g_w4a4_alloc_countdown.compare_exchange_weak(c, c - 1, std::memory_order_relaxed)) return c == 0;
  }
  return false;
}

namespace {

struct DeviceGuard {
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) ok = false;
    if (ok && prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
  }
  ~DeviceGuard() {
    int cur = -1;
    if (prev >= 0 && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
  }
};

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

template <typename T>
w4a4_status_t dev_alloc(T** p, size_t count, size_t* tally) {
  *p = nullptr;
  if (count == 0) return W4A4_OK;
  void* q = nullptr;
  if (alloc_failure_injected() || cudaMalloc(&q, count * sizeof(T)) != cudaSuccess) {
    cudaGetLastError();
    return W4A4_ERR_ALLOC;
  }
  *p = static_cast<T*>(q);
  if (tally) *tally += count * sizeof(T);
  return W4A4_OK;
}

inline bool encode_2d(EncodeTiledFn fn, CUtensorMap* tm, CUtensorMapDataType dt, size_t elem, void* base, uint64_t inner,
               uint64_t outer, uint64_t pitch_bytes, uint32_t box_inner, uint32_t box_outer, CUtensorMapSwizzle sw) {
  const cuuint64_t dims[2] = {inner, outer};
  const cuuint64_t strides[1] = {pitch_bytes};
  const cuuint32_t box[2] = {box_inner, box_outer};
  const cuuint32_t es[2] = {1, 1};
  (void)elem;
  return fn(tm, dt, 2, base, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
            CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Brings `count` elements at `src` (host or device) into a fresh device staging buffer when needed.
template <typename T>
w4a4_status_t stage_in(const T* src, size_t count, bool on_device, const T** dev, T** owned) {
  *owned = nullptr;
  if (on_device) {
    *dev = src;
    return W4A4_OK;
  }
  w4a4_status_t st = dev_alloc(owned, count, nullptr);
  if (st != W4A4_OK) return st;
  if (cudaMemcpy(*owned, src, count * sizeof(T), cudaMemcpyHostToDevice) != cudaSuccess) return W4A4_ERR_CUDA;
  *dev = *owned;
  return W4A4_OK;
}

}  // namespace
