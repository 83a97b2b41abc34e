// w4a4_quantize_noalloc: the activation-quantization step for callers that must not allocate.
//
// Some users of this library run where device allocation is off the table: inside a host callback, on
// a latency-critical path where a hidden cudaMalloc (which synchronises the device) is unacceptable, or
// inside a runtime that owns every byte of device memory through its own pool.  For them this one
// entry point runs the activation kernel without a context or a handle: its scratch (reciprocal smoothing vector, nibble-packed codes,
// group-major scales) lives in a fixed array that is part of the library image, and the caller
// supplies every input and output buffer.
#include "../../include/w4a4.h"

#include <cuda_runtime.h>

#include <mutex>

#include "quantize_kernel.cuh"

namespace {

constexpr int kNoAllocMaxK = 16384;                        // input channels
constexpr long long kNoAllocMaxElems = 4ll * 1024 * 1024;  // M * K
constexpr size_t kRlamBytes = static_cast<size_t>(kNoAllocMaxK) * sizeof(float);         // 64 KiB
constexpr size_t kScaleBytes = static_cast<size_t>(kNoAllocMaxElems / 64 + 4 * (kNoAllocMaxK / 64)) * sizeof(float);
constexpr size_t kCodeBytes = static_cast<size_t>(kNoAllocMaxElems / 2);                  // 2 MiB
constexpr size_t kRlamOff = 0;
constexpr size_t kScaleOff = kRlamOff + kRlamBytes;
constexpr size_t kCodeOff = (kScaleOff + kScaleBytes + 255) & ~static_cast<size_t>(255);
constexpr size_t kScratchBytes = kCodeOff + kCodeBytes;

// The scratch itself: about 2.3 MiB of device memory on every GPU that loads the library, held until
// the process exits.  In host code this name is only a stand-in; the device address is obtained once
// per device with cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
unsigned char* g_scratch_ptr[kMaxDevices] = {nullptr};

// Returns the device address of the scratch array on the current device (looked up once per device).
w4a4_status_t scratch_for_current_device(unsigned char** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return W4A4_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (g_scratch_ptr[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || p == nullptr) {
      cudaGetLastError();
      return W4A4_ERR_CUDA;
    }
    g_scratch_ptr[dev] = static_cast<unsigned char*>(p);
  }
  *out = g_scratch_ptr[dev];
  return W4A4_OK;
}

__global__ void noalloc_reciprocal_kernel(const float* __restrict__ lam, float* __restrict__ out, int K) {
  const int k = blockIdx.x * blockDim.x + threadIdx.x;
  if (k < K) out[k] = __fdiv_rn(1.0f, lam[k]);
}

// Packed, K-interleaved nibbles -> one code per byte, row-major [M, K].
__global__ void noalloc_decode_codes_kernel(const uint8_t* __restrict__ packed, int8_t* __restrict__ codes, int M, int K) {
  const size_t idx = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (idx >= static_cast<size_t>(M) * K) return;
  const int k = idx % K;
  const size_t m = idx / K;
  const int c = k >> 5, o = k & 31;
  const uint8_t b = packed[m * (K >> 1) + 16 * c + 4 * ((o & 15) >> 2) + (o & 3)];
  const int nib = (o >> 4) ? (b >> 4) : (b & 0xF);
  codes[idx] = static_cast<int8_t>((nib ^ 8) - 8);
}

// Group-major scratch scales -> [M, G].
__global__ void noalloc_decode_scales_kernel(const float* __restrict__ ws, int ld, float* __restrict__ out, int M, int G) {
  const size_t idx = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (idx >= static_cast<size_t>(M) * G) return;
  const int g = idx % G;
  const size_t m = idx / G;
  out[idx] = ws[static_cast<size_t>(g) * ld + m];
}

}  // namespace

extern "C" w4a4_status_t w4a4_quantize_noalloc(const void* X, int M, int K, const float* lambda,
                                               const float* clip_table, int clip_index, int8_t* codes,
                                               float* scales, void* stream) {
  if (M < 0 || clip_index < 0) return W4A4_ERR_INVALID_ARG;
  if (K <= 0 || K % 64 != 0 || K > kNoAllocMaxK) return W4A4_ERR_SHAPE;
  if (static_cast<long long>(M) * K > kNoAllocMaxElems) return W4A4_ERR_SHAPE;  // beyond the built-in scratch
  if (M == 0) return W4A4_OK;
  if (!X || !lambda || !clip_table || !codes || !scales) return W4A4_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(X) & 15u) != 0) return W4A4_ERR_INVALID_ARG;

  unsigned char* scratch = nullptr;
  const w4a4_status_t st = scratch_for_current_device(&scratch);
  if (st != W4A4_OK) return st;
  float* rlam = reinterpret_cast<float*>(scratch + kRlamOff);
  float* ws_scales = reinterpret_cast<float*>(scratch + kScaleOff);
  uint8_t* ws_codes = scratch + kCodeOff;
  const int G = K / 64;
  const int ld = (M + 3) & ~3;
  cudaStream_t s = static_cast<cudaStream_t>(stream);

  // Every scratch byte that is read below is written first by this same call: nothing has to start at zero.
  noalloc_reciprocal_kernel<<<(K + 255) / 256, 256, 0, s>>>(lambda, rlam, K);
  constexpr int kWarps = w4a4::quantize_warps(0);
  w4a4::quantize_kernel<0, kWarps, w4a4::kCodesPacked><<<(M + w4a4::kQuantRows * kWarps - 1) / (w4a4::kQuantRows * kWarps), 32 * kWarps,
                                     w4a4::quantize_smem_bytes(0), s>>>(
      static_cast<const uint16_t*>(X), M, K, rlam, clip_table, clip_index, nullptr, ws_codes, ws_scales, ld, nullptr, nullptr, nullptr);
  const size_t nc = static_cast<size_t>(M) * K, ns = static_cast<size_t>(M) * G;
  noalloc_decode_codes_kernel<<<static_cast<unsigned>((nc + 255) / 256), 256, 0, s>>>(ws_codes, codes, M, K);
  noalloc_decode_scales_kernel<<<static_cast<unsigned>((ns + 255) / 256), 256, 0, s>>>(ws_scales, ld, scales, M, G);
  return cudaGetLastError() == cudaSuccess ? W4A4_OK : W4A4_ERR_CUDA;
}
