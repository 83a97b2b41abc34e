// C-ABI entry points of libw4a4: context / handle management, weight repacking and the launches of the
// forward kernels (activation quantization, weight expansion, GEMM) and of the clipping-ratio search; the MXFP4
// variant's entry points are in w4a4_mx_api.cuh, included at the end.  Host code only does argument checks,
// descriptor set-up and launches.
#include "../../include/w4a4.h"

#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "gemm_w4a4_kernel.cuh"
#include "host_common.h"
#include "quantize_kernel.cuh"

namespace w4a4 {

// ------------------------------------------------------------------------------------ setup kernels
// lambda -> 1/lambda (Eq. 5), IEEE FP32 division, once.
__global__ void reciprocal_kernel(const float* __restrict__ lam, float* __restrict__ out, int K) {
  const int k = blockIdx.x * blockDim.x + threadIdx.x;
  if (k < K) out[k] = __fdiv_rn(1.0f, lam[k]);
}

// Residual codes [K, N] (one per byte) -> [N, K/2] nibble-packed as code + 8 (the weights' format at rest);
// byte j of a row holds K offsets 2 j (low nibble) and 2 j + 1 (high nibble).  One thread builds one
// 16-byte chunk (32 consecutive K of one output channel).
__global__ void pack_weight_kernel(const int8_t* __restrict__ q, uint8_t* __restrict__ out, int K, int N,
                                   int* __restrict__ bad) {
  const int n = blockIdx.x * blockDim.x + threadIdx.x;  // output channel = packed row
  const int c = blockIdx.y;
  if (n >= N) return;
  const int ch = n;
  uint32_t w[4] = {0, 0, 0, 0};
  bool oob = false;
  for (int o = 0; o < 32; ++o) {
    const int v = q[static_cast<size_t>(32 * c + o) * N + ch];
    oob |= (v < -8 || v > 7);
    const uint32_t nib = static_cast<uint32_t>(v + 8) & 0xFu;
    w[o >> 3] |= nib << (4 * (o & 7));
  }
  if (oob) atomicOr(bad, 1);
  *reinterpret_cast<uint4*>(out + static_cast<size_t>(n) * (K >> 1) + 16 * c) = make_uint4(w[0], w[1], w[2], w[3]);
}

// L1 [K, r] BF16 -> B fragments of mma.sync m16n8k16 in the K order the activation kernel uses,
// stored [group][i][n-tile pair][lane][n-tile of the pair] so that one 16-byte load feeds two MMAs.
__global__ void l1_fragment_kernel(const uint16_t* __restrict__ L1, uint2* __restrict__ out, int K, int r) {
  const int NT = r / 8;
  const size_t total = static_cast<size_t>(K / 64) * 4 * NT * 32;
  const size_t idx = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  const int sub = idx & 1;             // n-tile inside the pair
  const int lane = (idx >> 1) & 31;
  const int np = (idx >> 6) % (NT / 2);
  const int i = ((idx >> 6) / (NT / 2)) & 3;
  const int g = (idx >> 6) / (NT / 2) / 4;
  const int nt = 2 * np + sub;
  const int j = lane & 3, n = 8 * nt + (lane >> 2);
  uint16_t v[4];
  for (int e = 0; e < 4; ++e) {
    const int ch = 64 * g + l1_fragment_channel(j, 4 * i + e);
    v[e] = L1[static_cast<size_t>(ch) * r + n];
  }
  out[idx] = make_uint2(static_cast<uint32_t>(v[0]) | (static_cast<uint32_t>(v[1]) << 16),
                        static_cast<uint32_t>(v[2]) | (static_cast<uint32_t>(v[3]) << 16));
}

// L2 [r, N] BF16 -> [N, 2r]: the transposed factor twice, matching the [T_hi | T_lo] split of T.
__global__ void l2_dup_kernel(const uint16_t* __restrict__ L2, uint16_t* __restrict__ out, int r, int N) {
  const size_t idx = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (idx >= static_cast<size_t>(N) * 2 * r) return;
  const int c = idx % (2 * r);
  const int n = idx / (2 * r);
  const int ch = n;
  out[idx] = L2[static_cast<size_t>(c % r) * N + ch];
}

// Eq. 10: index of the smallest accumulated error (the first one on ties); the winning ratio goes into the
// clip table entry of (expert, layer, bin).
__global__ void clip_argmin_kernel(const double* __restrict__ err, const float* __restrict__ cand, int n,
                                   float* __restrict__ table_entry, int* __restrict__ best) {
  if (blockIdx.x != 0 || threadIdx.x != 0) return;
  int b = 0;
  for (int i = 1; i < n; ++i) {
    if (err[i] < err[b]) b = i;
  }
  *table_entry = cand[b];
  *best = b;
}

// Test-only decoders of the activation kernel's outputs.
__global__ void decode_codes_kernel(const uint8_t* __restrict__ e4m3, int8_t* __restrict__ codes, int M, int K) {
  const size_t idx = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (idx >= static_cast<size_t>(M) * K) return;
  codes[idx] = static_cast<int8_t>(e4m3_integer_value(e4m3[idx]));
}
// Group-major workspace scales -> [M, G].
__global__ void decode_scales_kernel(const float* __restrict__ ws, int ld, float* __restrict__ out, int M, int G) {
  const size_t idx = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (idx >= static_cast<size_t>(M) * G) return;
  const int g = idx % G;
  const size_t m = idx / G;
  out[idx] = ws[static_cast<size_t>(g) * ld + m];
}
__global__ void decode_t_kernel(const uint16_t* __restrict__ thl, float* __restrict__ T, int M, int r) {
  const size_t idx = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (idx >= static_cast<size_t>(M) * r) return;
  const int c = idx % r;
  const size_t m = idx / r;
  const float hi = __uint_as_float(static_cast<uint32_t>(thl[m * 2 * r + c]) << 16);
  const float lo = __uint_as_float(static_cast<uint32_t>(thl[m * 2 * r + r + c]) << 16);
  T[idx] = hi + lo;
}

}  // namespace w4a4

using namespace w4a4;

// ------------------------------------------------------------------------------------ host objects
struct ExpertData {
  uint8_t* bpacked = nullptr;  // [N, K/2]
  float* wscale = nullptr;     // [G, N]
  uint8_t* b_sop = nullptr;    // weight scale operands of the scale MMA: [N/128][ceil(G/2)][4096]
  float* rlam = nullptr;       // [K]
  uint2* l1frag = nullptr;
  uint16_t* l2dup = nullptr;   // [N, 2r]
  float* bias = nullptr;       // [N] or null
  CUtensorMap tmL2, tmSopB;
};

struct w4a4_layer {
  w4a4_ctx* ctx = nullptr;
  int K = 0, N = 0, r = 0, E = 0, B = 0, L = 0, layer_id = 0, act = 0;
  std::vector<ExpertData> experts;
  CUtensorMap tmA, tmSopA, tmT, tmB;
  const uint8_t* tmB_base = nullptr;  // the context's weight-byte scratch this handle's tmB was encoded for
  size_t bytes = 0;
};

namespace {

void free_expert(ExpertData& e) {
  cudaFree(e.bpacked);
  cudaFree(e.wscale);
  cudaFree(e.b_sop);
  cudaFree(e.rlam);
  cudaFree(e.l1frag);
  cudaFree(e.l2dup);
  cudaFree(e.bias);
  e = ExpertData();
}


w4a4_status_t check_forward_args(w4a4_handle_t h, const void* X, int M, int expert_id, int bin,
                                 const float* clip_table, bool need_x) {
  if (!h || !h->ctx) return W4A4_ERR_INVALID_ARG;
  if (M < 0) return W4A4_ERR_INVALID_ARG;
  if (M > h->ctx->max_M) return W4A4_ERR_SHAPE;
  if (expert_id < 0 || expert_id >= h->E) return W4A4_ERR_INVALID_ARG;
  if (need_x) {
    if (bin < 0 || bin >= h->B) return W4A4_ERR_INVALID_ARG;
    if (M > 0 && (!X || !aligned16(X))) return W4A4_ERR_INVALID_ARG;
    if (!clip_table) return W4A4_ERR_INVALID_ARG;
  }
  return W4A4_OK;
}

// Index of (expert, this layer, bin) in a clip table (Sec. III-C: one ratio per expert, layer and timestep bin).
int clip_table_index(const w4a4_layer* h, int expert_id, int bin) { return (expert_id * h->L + h->layer_id) * h->B + bin; }

// Kernel 1 with the ratio read from clip_table[clip_index].
w4a4_status_t launch_quantize_at(w4a4_handle_t h, const void* X, int M, int expert_id, const float* clip_table,
                                 int clip_index, cudaStream_t stream) {
  if (M == 0) return W4A4_OK;
  w4a4_ctx* ctx = h->ctx;
  const ExpertData& e = h->experts[expert_id];
  const int rows_per_cta = kQuantRows * quantize_warps(h->r);
  const int row_ctas = (M + rows_per_cta - 1) / rows_per_cta;
  const int splits = quantize_k_splits(row_ctas, h->K / 64, M, ctx->num_sms);
  const dim3 grid(row_ctas, splits), block(32 * quantize_warps(h->r));
  const uint16_t* x = static_cast<const uint16_t*>(X);
#define W4A4_LAUNCH_Q(R)                                                                                         \
  quantize_kernel<R, quantize_warps(R), kCodesE4M3><<<grid, block, quantize_smem_bytes(R), stream>>>(x, M, h->K, e.rlam, clip_table, clip_index, e.l1frag, ctx->codes, \
                                                 ctx->scales, ctx->scales_ld, ctx->t_hilo, ctx->t_partial,     \
                                                 reinterpret_cast<uint2*>(ctx->a_sop))
  switch (h->r) {
    case 0: W4A4_LAUNCH_Q(0); break;
    case 16: W4A4_LAUNCH_Q(16); break;
    case 32: W4A4_LAUNCH_Q(32); break;
    case 64: W4A4_LAUNCH_Q(64); break;
    case 96: W4A4_LAUNCH_Q(96); break;
    default: return W4A4_ERR_SHAPE;
  }
#undef W4A4_LAUNCH_Q
  if (splits > 1 && h->r > 0) {
    const size_t nt = static_cast<size_t>(M) * h->r;
    t_reduce_kernel<<<static_cast<unsigned>((nt + 255) / 256), 256, 0, stream>>>(ctx->t_partial, splits, M, h->r, ctx->t_hilo);
  }
  return cudaGetLastError() == cudaSuccess ? W4A4_OK : W4A4_ERR_CUDA;
}

w4a4_status_t launch_quantize(w4a4_handle_t h, const void* X, int M, int expert_id, int bin, const float* clip_table,
                              cudaStream_t stream) {
  return launch_quantize_at(h, X, M, expert_id, clip_table, clip_table_index(h, expert_id, bin), stream);
}

// Kernel 2 (preceded by the expansion of the expert's 4-bit weights unless `expand` is false, i.e. the
// context's byte image already holds them).  With yref set, the squared distance to yref is accumulated into
// *sq_err instead of storing Y.
w4a4_status_t launch_gemm(w4a4_handle_t h, int M, int expert_id, void* Y, cudaStream_t stream, int32_t* dbg_P,
                          int dbg_m0, int dbg_n0, const void* yref = nullptr, double* sq_err = nullptr,
                          bool expand = true, int stall_stage = -1, uint64_t wait_limit_ns = kWaitLimitNs) {
  if (M == 0) return W4A4_OK;
  w4a4_ctx* ctx = h->ctx;
  const ExpertData& e = h->experts[expert_id];
  GemmParams p;
  p.bias = e.bias;
  p.Y = static_cast<uint16_t*>(Y);
  p.M = M;
  p.N = h->N;
  p.K = h->K;
  p.r = h->r;
  p.tiles_m = (M + kBM - 1) / kBM;
  p.tiles_n = h->N / kBN;
  // Tile order: super-columns whose weight bytes (kBN x K per column tile) take about two ninths of L2 (28 MB of
  // 126), of equal width; a weight image that fits such a budget as a whole keeps the plain row-major order.
  {
    const size_t budget = ctx->l2_bytes * 2 / 9;
    int sc = static_cast<int>(budget / (static_cast<size_t>(kBN) * h->K));
    if (sc < 1) sc = 1;
    if (sc >= p.tiles_n) {
      sc = p.tiles_n;
    } else {
      const int ns = (p.tiles_n + sc - 1) / sc;
      sc = (p.tiles_n + ns - 1) / ns;
    }
    if (ctx->debug_sc_tiles > 0) sc = ctx->debug_sc_tiles < p.tiles_n ? ctx->debug_sc_tiles : p.tiles_n;
    p.sc_tiles = sc;
  }
  p.err = ctx->d_err;
  p.wait_limit_ns = wait_limit_ns;
  p.dbg_stall_stage = stall_stage;
  p.dbg_P = dbg_P;
  p.dbg_m0 = dbg_m0;
  p.dbg_n0 = dbg_n0;
  p.yref = static_cast<const uint16_t*>(yref);
  p.sq_err = sq_err;
  p.act = h->act;
  // The context's weight-byte scratch may have been reallocated (a larger layer packed since): re-aim the map.
  if (h->tmB_base != ctx->b8) {
    if (!encode_2d(ctx->encode, &h->tmB, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, ctx->b8, h->K, h->N, h->K, kBK, kBN,
                   CU_TENSOR_MAP_SWIZZLE_128B))
      return W4A4_ERR_CUDA;
    h->tmB_base = ctx->b8;
  }
  if (expand) {
    const size_t chunks = static_cast<size_t>(h->N) * h->K / 32;
    expand_weight_kernel<<<static_cast<unsigned>((chunks + 255) / 256), 256, 0, stream>>>(
        reinterpret_cast<const uint4*>(e.bpacked), reinterpret_cast<uint4*>(ctx->b8), chunks);
  }
  // Persistent: one CTA per SM walks the 128 x 128 tiles.
  const int num_tiles = p.tiles_m * p.tiles_n;
  const dim3 grid(num_tiles < ctx->num_sms ? num_tiles : ctx->num_sms), block(kGemmThreads);
  const CUtensorMap& tmT = h->r > 0 ? h->tmT : h->tmA;   // unused when r == 0
  const CUtensorMap& tmL2 = h->r > 0 ? e.tmL2 : h->tmB;
  if (dbg_P || stall_stage >= 0) {
    gemm_w4a4_kernel<true><<<grid, block, kGemmSmemBytes, stream>>>(h->tmA, h->tmB, tmT, tmL2, h->tmSopA, e.tmSopB, p);
  } else {
    gemm_w4a4_kernel<false><<<grid, block, kGemmSmemBytes, stream>>>(h->tmA, h->tmB, tmT, tmL2, h->tmSopA, e.tmSopB, p);
  }
  const cudaError_t le = cudaGetLastError();
  return le == cudaSuccess ? W4A4_OK : W4A4_ERR_CUDA;
}

}  // namespace

// ------------------------------------------------------------------------------------ C ABI
std::atomic<int> g_w4a4_alloc_countdown{-1};

extern "C" {

const char* w4a4_status_string(w4a4_status_t s) {
  switch (s) {
    case W4A4_OK: return "ok";
    case W4A4_ERR_INVALID_ARG: return "invalid argument";
    case W4A4_ERR_SHAPE: return "unsupported shape";
    case W4A4_ERR_ALLOC: return "allocation failed";
    case W4A4_ERR_CUDA: return "CUDA error";
    case W4A4_ERR_ARCH: return "device is not compute capability 10.x";
    case W4A4_ERR_TIMEOUT: return "a kernel gave up on a bounded wait";
  }
  return "unknown status";
}

void w4a4_tile_shape(int* tile_m, int* tile_n) {
  if (tile_m) *tile_m = kBM;
  if (tile_n) *tile_n = kBN;
}

w4a4_status_t w4a4_ctx_create(int device, int max_M, int max_K, int max_r, w4a4_ctx_t* out) {
  if (!out) return W4A4_ERR_INVALID_ARG;
  *out = nullptr;
  if (max_M <= 0 || max_K <= 0 || max_K % 64 != 0 || max_r < 0 || max_r > 96) return W4A4_ERR_SHAPE;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess) {
    cudaGetLastError();
    return W4A4_ERR_CUDA;
  }
  if (device < 0 || device >= ndev) return W4A4_ERR_INVALID_ARG;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return W4A4_ERR_CUDA;
  if (prop.major != 10) return W4A4_ERR_ARCH;
  DeviceGuard guard(device);
  if (!guard.ok) return W4A4_ERR_CUDA;

  w4a4_ctx* ctx = new (std::nothrow) w4a4_ctx();
  if (!ctx) return W4A4_ERR_ALLOC;
  ctx->device = device;
  ctx->max_M = max_M;
  ctx->max_K = max_K;
  ctx->max_r = max_r;
  ctx->num_sms = prop.multiProcessorCount;
  ctx->l2_bytes = static_cast<size_t>(prop.l2CacheSize);
  ctx->scales_ld = (max_M + 3) & ~3;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
      qres != cudaDriverEntryPointSuccess) {
    delete ctx;
    return W4A4_ERR_CUDA;
  }
  ctx->encode = reinterpret_cast<EncodeTiledFn>(fn);
  w4a4_status_t st = dev_alloc(&ctx->codes, static_cast<size_t>(max_M) * max_K, &ctx->bytes);
  if (st == W4A4_OK) st = dev_alloc(&ctx->scales, static_cast<size_t>(ctx->scales_ld) * (max_K / 64), &ctx->bytes);
  if (st == W4A4_OK && cudaMemset(ctx->scales, 0, sizeof(float) * ctx->scales_ld * (max_K / 64)) != cudaSuccess) st = W4A4_ERR_CUDA;
  const size_t a_sop_bytes = static_cast<size_t>((max_M + 127) / 128) * ((max_K / 64 + 1) / 2) * kSopATile;
  if (st == W4A4_OK) st = dev_alloc(&ctx->a_sop, a_sop_bytes, &ctx->bytes);
  // Rows past M and the unused half of an odd last stage are multiplied by zeros: they only have to be finite.
  if (st == W4A4_OK && cudaMemset(ctx->a_sop, 0, a_sop_bytes) != cudaSuccess) st = W4A4_ERR_CUDA;
  if (st == W4A4_OK) st = dev_alloc(&ctx->t_hilo, static_cast<size_t>(max_M) * 2 * (max_r > 0 ? max_r : 8), &ctx->bytes);
  if (st == W4A4_OK && max_r > 0)
    st = dev_alloc(&ctx->t_partial,
                   static_cast<size_t>(kMaxKSplits) * (max_M < kKSplitMaxRows ? max_M : kKSplitMaxRows) * max_r, &ctx->bytes);
  if (st == W4A4_OK) st = dev_alloc(&ctx->d_err, 1, &ctx->bytes);
  if (st == W4A4_OK && cudaMemset(ctx->d_err, 0, sizeof(int)) != cudaSuccess) st = W4A4_ERR_CUDA;
  // The workspace is read by TMA for rows up to max_M even when fewer are valid: start it defined.
  if (st == W4A4_OK && cudaMemset(ctx->codes, 0, static_cast<size_t>(max_M) * max_K) != cudaSuccess) st = W4A4_ERR_CUDA;
  if (st == W4A4_OK &&
      cudaMemset(ctx->t_hilo, 0, static_cast<size_t>(max_M) * 2 * (max_r > 0 ? max_r : 8) * sizeof(uint16_t)) != cudaSuccess)
    st = W4A4_ERR_CUDA;
  if (st == W4A4_OK) {
    cudaFuncSetAttribute(quantize_kernel<64, quantize_warps(64), kCodesE4M3>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                         static_cast<int>(quantize_smem_bytes(64)));
    cudaFuncSetAttribute(quantize_kernel<96, quantize_warps(96), kCodesE4M3>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                         static_cast<int>(quantize_smem_bytes(96)));
    const cudaError_t e1 = cudaFuncSetAttribute(gemm_w4a4_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kGemmSmemBytes);
    const cudaError_t e2 = cudaFuncSetAttribute(gemm_w4a4_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kGemmSmemBytes);
    if (e1 != cudaSuccess || e2 != cudaSuccess) {
      cudaGetLastError();
      st = W4A4_ERR_CUDA;
    }
  }
  if (st != W4A4_OK) {
    w4a4_ctx_destroy(ctx);
    return st;
  }
  *out = ctx;
  return W4A4_OK;
}

void w4a4_ctx_destroy(w4a4_ctx_t ctx) {
  if (!ctx) return;
  DeviceGuard guard(ctx->device);
  cudaFree(ctx->codes);
  cudaFree(ctx->b8);
  cudaFree(ctx->mx_sfa);
  cudaFree(ctx->mx_codes2);
  cudaFree(ctx->mx_sfa2);
  cudaFree(ctx->mx_t32);
  cudaFree(ctx->t_hilo2);
  cudaFree(ctx->t_partial);
  cudaFree(ctx->scales);
  cudaFree(ctx->a_sop);
  cudaFree(ctx->t_hilo);
  cudaFree(ctx->d_err);
  for (int i = 0; i < 2; ++i) {
    cudaFree(ctx->hx[i]);
    cudaFree(ctx->hy[i]);
    if (ctx->ev_in[i]) cudaEventDestroy(ctx->ev_in[i]);
    if (ctx->ev_done[i]) cudaEventDestroy(ctx->ev_done[i]);
    if (ctx->ev_out[i]) cudaEventDestroy(ctx->ev_out[i]);
  }
  if (ctx->ev_begin) cudaEventDestroy(ctx->ev_begin);
  if (ctx->ev_end) cudaEventDestroy(ctx->ev_end);
  if (ctx->s_h2d) cudaStreamDestroy(ctx->s_h2d);
  if (ctx->s_compute) cudaStreamDestroy(ctx->s_compute);
  if (ctx->s_d2h) cudaStreamDestroy(ctx->s_d2h);
  delete ctx;
}

size_t w4a4_ctx_bytes(w4a4_ctx_t ctx) { return ctx ? ctx->bytes : 0; }
size_t w4a4_handle_bytes(w4a4_handle_t h) { return h ? h->bytes : 0; }

void w4a4_destroy(w4a4_handle_t h) {
  if (!h) return;
  if (h->ctx) {
    DeviceGuard guard(h->ctx->device);
    for (auto& e : h->experts) free_expert(e);
  }
  delete h;
}

w4a4_status_t w4a4_pack_weights(w4a4_ctx_t ctx, const w4a4_weight_desc_t* d, w4a4_handle_t* out) {
  if (!out) return W4A4_ERR_INVALID_ARG;
  *out = nullptr;
  if (!ctx || !d) return W4A4_ERR_INVALID_ARG;
  if (d->group != 64 || d->K <= 0 || d->K % 64 != 0 || d->N <= 0 || d->N % kBN != 0) return W4A4_ERR_SHAPE;
  if (!(d->r == 0 || d->r == 16 || d->r == 32 || d->r == 64 || d->r == 96)) return W4A4_ERR_SHAPE;
  if (d->K > ctx->max_K || d->r > ctx->max_r) return W4A4_ERR_SHAPE;
  if (d->num_experts < 1 || d->num_bins < 1 || d->num_layers < 1 || d->layer_id < 0 || d->layer_id >= d->num_layers)
    return W4A4_ERR_INVALID_ARG;
  if (!d->qweight || !d->wscale || !d->lambda || (d->r > 0 && (!d->L1 || !d->L2))) return W4A4_ERR_INVALID_ARG;
  if (d->output_activation != W4A4_ACT_NONE && d->output_activation != W4A4_ACT_GELU_TANH) return W4A4_ERR_INVALID_ARG;
  for (int e = 0; e < d->num_experts; ++e) {
    if (!d->qweight[e] || !d->wscale[e] || !d->lambda[e] || (d->r > 0 && (!d->L1[e] || !d->L2[e])))
      return W4A4_ERR_INVALID_ARG;
  }
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return W4A4_ERR_CUDA;

  w4a4_layer* h = new (std::nothrow) w4a4_layer();
  if (!h) return W4A4_ERR_ALLOC;
  h->ctx = ctx;
  h->K = d->K;
  h->N = d->N;
  h->r = d->r;
  h->E = d->num_experts;
  h->B = d->num_bins;
  h->L = d->num_layers;
  h->layer_id = d->layer_id;
  h->act = d->output_activation;
  h->experts.resize(d->num_experts);
  const int K = d->K, N = d->N, r = d->r, G = K / 64;
  const bool dev = d->pointers_on_device != 0;
  w4a4_status_t st = W4A4_OK;
  // The weight-byte scratch of the context must hold this layer's N x K image.  Growing it is safe between
  // forwards only (synchronise first: a forward of another layer may still be reading the old one).
  const size_t b8_need = static_cast<size_t>(N) * K;
  if (ctx->b8_bytes < b8_need) {
    if (cudaDeviceSynchronize() != cudaSuccess) st = W4A4_ERR_CUDA;
    if (st == W4A4_OK) {
      cudaFree(ctx->b8);
      ctx->bytes -= ctx->b8_bytes;
      ctx->b8_bytes = 0;
      st = dev_alloc(&ctx->b8, b8_need, &ctx->bytes);
      if (st == W4A4_OK) ctx->b8_bytes = b8_need;
    }
  }
  int* d_bad = nullptr;
  if (st == W4A4_OK) st = dev_alloc(&d_bad, 1, nullptr);
  if (st == W4A4_OK && cudaMemset(d_bad, 0, sizeof(int)) != cudaSuccess) st = W4A4_ERR_CUDA;

  for (int ei = 0; st == W4A4_OK && ei < d->num_experts; ++ei) {
    ExpertData& e = h->experts[ei];
    st = dev_alloc(&e.bpacked, static_cast<size_t>(N) * (K / 2), &h->bytes);
    if (st == W4A4_OK) st = dev_alloc(&e.wscale, static_cast<size_t>(G) * N, &h->bytes);
    if (st == W4A4_OK) st = dev_alloc(&e.rlam, static_cast<size_t>(K), &h->bytes);
    if (st == W4A4_OK && r > 0) st = dev_alloc(&e.l1frag, static_cast<size_t>(G) * 4 * (r / 8) * 32, &h->bytes);
    if (st == W4A4_OK && r > 0) st = dev_alloc(&e.l2dup, static_cast<size_t>(N) * 2 * r, &h->bytes);
    const float* bias_src = d->bias ? d->bias[ei] : nullptr;
    if (st == W4A4_OK && bias_src) st = dev_alloc(&e.bias, static_cast<size_t>(N), &h->bytes);
    if (st != W4A4_OK) break;

    const cudaMemcpyKind kind = dev ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice;
    if (cudaMemcpy(e.wscale, d->wscale[ei], sizeof(float) * G * N, kind) != cudaSuccess) st = W4A4_ERR_CUDA;
    const size_t b_sop_bytes = static_cast<size_t>(N / kBN) * ((G + 1) / 2) * kSopBTile;
    if (st == W4A4_OK) st = dev_alloc(&e.b_sop, b_sop_bytes, &h->bytes);
    if (st == W4A4_OK && cudaMemset(e.b_sop, 0, b_sop_bytes) != cudaSuccess) st = W4A4_ERR_CUDA;
    if (st == W4A4_OK) {
      const size_t ns = static_cast<size_t>(G) * N;
      sop_weight_kernel<<<static_cast<unsigned>((ns + 255) / 256), 256>>>(e.wscale, reinterpret_cast<uint4*>(e.b_sop), G, N);
      if (cudaGetLastError() != cudaSuccess) st = W4A4_ERR_CUDA;
    }
    if (st == W4A4_OK && bias_src && cudaMemcpy(e.bias, bias_src, sizeof(float) * N, kind) != cudaSuccess)
      st = W4A4_ERR_CUDA;
    if (st != W4A4_OK) break;

    const int8_t* q_dev = nullptr;
    int8_t* q_own = nullptr;
    const float* lam_dev = nullptr;
    float* lam_own = nullptr;
    const uint16_t *l1_dev = nullptr, *l2_dev = nullptr;
    uint16_t *l1_own = nullptr, *l2_own = nullptr;
    st = stage_in(d->qweight[ei], static_cast<size_t>(K) * N, dev, &q_dev, &q_own);
    if (st == W4A4_OK) st = stage_in(d->lambda[ei], static_cast<size_t>(K), dev, &lam_dev, &lam_own);
    if (st == W4A4_OK && r > 0) st = stage_in(d->L1[ei], static_cast<size_t>(K) * r, dev, &l1_dev, &l1_own);
    if (st == W4A4_OK && r > 0) st = stage_in(d->L2[ei], static_cast<size_t>(r) * N, dev, &l2_dev, &l2_own);
    if (st == W4A4_OK) {
      reciprocal_kernel<<<(K + 255) / 256, 256>>>(lam_dev, e.rlam, K);
      pack_weight_kernel<<<dim3((N + 127) / 128, K / 32), 128>>>(q_dev, e.bpacked, K, N, d_bad);
      if (r > 0) {
        const size_t nf = static_cast<size_t>(G) * 4 * (r / 8) * 32;
        l1_fragment_kernel<<<static_cast<unsigned>((nf + 255) / 256), 256>>>(l1_dev, e.l1frag, K, r);
        const size_t nl = static_cast<size_t>(N) * 2 * r;
        l2_dup_kernel<<<static_cast<unsigned>((nl + 255) / 256), 256>>>(l2_dev, e.l2dup, r, N);
      }
      if (cudaGetLastError() != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess) st = W4A4_ERR_CUDA;
    }
    cudaFree(q_own);
    cudaFree(lam_own);
    cudaFree(l1_own);
    cudaFree(l2_own);
    if (st != W4A4_OK) break;

    // Scale operand images as rows of 32-bit words (one row per 128 output channels), fetched in boxes of 1 KiB.
    if (!encode_2d(ctx->encode, &e.tmSopB, CU_TENSOR_MAP_DATA_TYPE_UINT32, 4, e.b_sop, static_cast<uint64_t>((G + 1) / 2) * (kSopBTile / 4),
                   N / kBN, static_cast<uint64_t>((G + 1) / 2) * kSopBTile, 256, 1, CU_TENSOR_MAP_SWIZZLE_NONE))
      st = W4A4_ERR_CUDA;
    if (st == W4A4_OK && r > 0 &&
        !encode_2d(ctx->encode, &e.tmL2, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, e.l2dup, 2 * r, N, 4 * r, 64, kBN,
                   CU_TENSOR_MAP_SWIZZLE_128B))
      st = W4A4_ERR_CUDA;
  }
  if (st == W4A4_OK) {
    int bad = 0;
    if (cudaMemcpy(&bad, d_bad, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) st = W4A4_ERR_CUDA;
    else if (bad) st = W4A4_ERR_INVALID_ARG;  // a residual code outside [-8, 7]
  }
  cudaFree(d_bad);
  if (st == W4A4_OK &&
      !encode_2d(ctx->encode, &h->tmA, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, ctx->codes, K, ctx->max_M, K, kBK, kBM,
                 CU_TENSOR_MAP_SWIZZLE_128B))
    st = W4A4_ERR_CUDA;
  if (st == W4A4_OK &&
      !encode_2d(ctx->encode, &h->tmSopA, CU_TENSOR_MAP_DATA_TYPE_UINT32, 4, ctx->a_sop, static_cast<uint64_t>((G + 1) / 2) * (kSopATile / 4),
                 (ctx->max_M + kBM - 1) / kBM, static_cast<uint64_t>((G + 1) / 2) * kSopATile, 256, 1, CU_TENSOR_MAP_SWIZZLE_NONE))
    st = W4A4_ERR_CUDA;
  if (st == W4A4_OK && r > 0 &&
      !encode_2d(ctx->encode, &h->tmT, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, ctx->t_hilo, 2 * r, ctx->max_M, 4 * r, 64,
                 kBM, CU_TENSOR_MAP_SWIZZLE_128B))
    st = W4A4_ERR_CUDA;
  if (st != W4A4_OK) {
    cudaGetLastError();
    w4a4_destroy(h);
    return st;
  }
  *out = h;
  return W4A4_OK;
}

w4a4_status_t w4a4_quantize_activations(w4a4_handle_t h, const void* X, int M, int expert_id, int timestep_bin,
                                        const float* clip_table, void* stream) {
  w4a4_status_t st = check_forward_args(h, X, M, expert_id, timestep_bin, clip_table, true);
  if (st != W4A4_OK) return st;
  DeviceGuard guard(h->ctx->device);
  return launch_quantize(h, X, M, expert_id, timestep_bin, clip_table, static_cast<cudaStream_t>(stream));
}

w4a4_status_t w4a4_gemm_from_workspace(w4a4_handle_t h, int M, int expert_id, void* Y, void* stream) {
  w4a4_status_t st = check_forward_args(h, nullptr, M, expert_id, 0, nullptr, false);
  if (st != W4A4_OK) return st;
  if (M > 0 && (!Y || !aligned16(Y))) return W4A4_ERR_INVALID_ARG;
  DeviceGuard guard(h->ctx->device);
  return launch_gemm(h, M, expert_id, Y, static_cast<cudaStream_t>(stream), nullptr, 0, 0);
}

w4a4_status_t w4a4_clip_search(w4a4_handle_t h, const void* const* X_samples, const void* const* Yref_samples,
                               int num_samples, int M, int expert_id, int timestep_bin, const float* candidates,
                               int num_candidates, float* clip_table, double* errors_out, int* best_out,
                               void* stream) {
  if (!h || !h->ctx) return W4A4_ERR_INVALID_ARG;
  if (num_samples < 1 || num_candidates < 1 || num_candidates > 256 || M < 1) return W4A4_ERR_INVALID_ARG;
  if (!X_samples || !Yref_samples || !candidates || !clip_table) return W4A4_ERR_INVALID_ARG;
  for (int c = 0; c < num_candidates; ++c) {
    if (!(candidates[c] >= 1e-4f && candidates[c] <= 1.0f)) return W4A4_ERR_INVALID_ARG;
  }
  for (int s = 0; s < num_samples; ++s) {
    w4a4_status_t st = check_forward_args(h, X_samples[s], M, expert_id, timestep_bin, clip_table, true);
    if (st != W4A4_OK) return st;
    if (!Yref_samples[s] || !aligned16(Yref_samples[s])) return W4A4_ERR_INVALID_ARG;
  }
  DeviceGuard guard(h->ctx->device);
  if (!guard.ok) return W4A4_ERR_CUDA;
  cudaStream_t st_ = static_cast<cudaStream_t>(stream);
  double* d_err = nullptr;
  float* d_cand = nullptr;
  int* d_best = nullptr;
  w4a4_status_t st = dev_alloc(&d_err, static_cast<size_t>(num_candidates), nullptr);
  if (st == W4A4_OK) st = dev_alloc(&d_cand, static_cast<size_t>(num_candidates), nullptr);
  if (st == W4A4_OK) st = dev_alloc(&d_best, 1, nullptr);
  if (st == W4A4_OK &&
      (cudaMemsetAsync(d_err, 0, sizeof(double) * num_candidates, st_) != cudaSuccess ||
       cudaMemcpyAsync(d_cand, candidates, sizeof(float) * num_candidates, cudaMemcpyHostToDevice, st_) != cudaSuccess))
    st = W4A4_ERR_CUDA;
  // Every candidate runs the real forward (kernel 1 with that ratio, kernel 2 on the same weight image, which
  // is expanded once) and leaves only its squared error behind.
  bool expanded = false;
  for (int s = 0; st == W4A4_OK && s < num_samples; ++s) {
    for (int c = 0; st == W4A4_OK && c < num_candidates; ++c) {
      st = launch_quantize_at(h, X_samples[s], M, expert_id, d_cand, c, st_);
      if (st == W4A4_OK)
        st = launch_gemm(h, M, expert_id, nullptr, st_, nullptr, 0, 0, Yref_samples[s], d_err + c, !expanded);
      expanded = true;
    }
  }
  int best = 0;
  if (st == W4A4_OK) {
    clip_argmin_kernel<<<1, 32, 0, st_>>>(d_err, d_cand, num_candidates,
                                          clip_table + clip_table_index(h, expert_id, timestep_bin), d_best);
    if (cudaGetLastError() != cudaSuccess) st = W4A4_ERR_CUDA;
  }
  if (st == W4A4_OK && errors_out &&
      cudaMemcpyAsync(errors_out, d_err, sizeof(double) * num_candidates, cudaMemcpyDeviceToHost, st_) != cudaSuccess)
    st = W4A4_ERR_CUDA;
  if (st == W4A4_OK && cudaMemcpyAsync(&best, d_best, sizeof(int), cudaMemcpyDeviceToHost, st_) != cudaSuccess)
    st = W4A4_ERR_CUDA;
  if (cudaStreamSynchronize(st_) != cudaSuccess && st == W4A4_OK) st = W4A4_ERR_CUDA;
  if (st == W4A4_OK && best_out) *best_out = best;
  cudaFree(d_err);
  cudaFree(d_cand);
  cudaFree(d_best);
  if (st != W4A4_OK) cudaGetLastError();
  return st;
}

w4a4_status_t w4a4_linear_forward(w4a4_handle_t h, const void* X, int M, int expert_id, int timestep_bin,
                                  const float* clip_table, void* Y, void* stream) {
  w4a4_status_t st = check_forward_args(h, X, M, expert_id, timestep_bin, clip_table, true);
  if (st != W4A4_OK) return st;
  if (M > 0 && (!Y || !aligned16(Y))) return W4A4_ERR_INVALID_ARG;
  DeviceGuard guard(h->ctx->device);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  st = launch_quantize(h, X, M, expert_id, timestep_bin, clip_table, s);
  if (st != W4A4_OK) return st;
  return launch_gemm(h, M, expert_id, Y, s, nullptr, 0, 0);
}

w4a4_status_t w4a4_ctx_enable_host_io(w4a4_ctx_t ctx, int chunk_rows, int max_N) {
  if (!ctx) return W4A4_ERR_INVALID_ARG;
  if (chunk_rows <= 0 || chunk_rows > ctx->max_M || max_N <= 0) return W4A4_ERR_SHAPE;
  if (ctx->host_chunk_rows != 0) return W4A4_ERR_INVALID_ARG;  // already enabled
  DeviceGuard guard(ctx->device);
  w4a4_status_t st = W4A4_OK;
  for (int i = 0; st == W4A4_OK && i < 2; ++i) {
    st = dev_alloc(&ctx->hx[i], static_cast<size_t>(chunk_rows) * ctx->max_K, &ctx->bytes);
    if (st == W4A4_OK) st = dev_alloc(&ctx->hy[i], static_cast<size_t>(chunk_rows) * max_N, &ctx->bytes);
    if (st == W4A4_OK && (cudaEventCreateWithFlags(&ctx->ev_in[i], cudaEventDisableTiming) != cudaSuccess ||
                          cudaEventCreateWithFlags(&ctx->ev_done[i], cudaEventDisableTiming) != cudaSuccess ||
                          cudaEventCreateWithFlags(&ctx->ev_out[i], cudaEventDisableTiming) != cudaSuccess))
      st = W4A4_ERR_CUDA;
  }
  if (st == W4A4_OK && (cudaStreamCreateWithFlags(&ctx->s_h2d, cudaStreamNonBlocking) != cudaSuccess ||
                        cudaStreamCreateWithFlags(&ctx->s_compute, cudaStreamNonBlocking) != cudaSuccess ||
                        cudaStreamCreateWithFlags(&ctx->s_d2h, cudaStreamNonBlocking) != cudaSuccess ||
                        cudaEventCreateWithFlags(&ctx->ev_begin, cudaEventDisableTiming) != cudaSuccess ||
                        cudaEventCreateWithFlags(&ctx->ev_end, cudaEventDisableTiming) != cudaSuccess))
    st = W4A4_ERR_CUDA;
  if (st != W4A4_OK) {
    cudaGetLastError();
    return st;
  }
  ctx->host_chunk_rows = chunk_rows;
  ctx->host_max_N = max_N;
  return W4A4_OK;
}

w4a4_status_t w4a4_linear_forward_host(w4a4_handle_t h, const void* X_host, int M, int expert_id, int timestep_bin,
                                       const float* clip_table, void* Y_host, void* stream) {
  w4a4_status_t st = check_forward_args(h, X_host, M, expert_id, timestep_bin, clip_table, true);
  if (st != W4A4_OK) return st;
  w4a4_ctx* ctx = h->ctx;
  if (ctx->host_chunk_rows == 0) return W4A4_ERR_INVALID_ARG;  // w4a4_ctx_enable_host_io was not called
  if (h->N > ctx->host_max_N) return W4A4_ERR_SHAPE;
  if (M > 0 && !Y_host) return W4A4_ERR_INVALID_ARG;
  if (M == 0) return W4A4_OK;
  DeviceGuard guard(ctx->device);
  cudaStream_t user = static_cast<cudaStream_t>(stream);
  const int C = ctx->host_chunk_rows;
  const int chunks = (M + C - 1) / C;
  const uint16_t* xh = static_cast<const uint16_t*>(X_host);
  uint16_t* yh = static_cast<uint16_t*>(Y_host);
  bool ok = cudaEventRecord(ctx->ev_begin, user) == cudaSuccess &&
            cudaStreamWaitEvent(ctx->s_h2d, ctx->ev_begin, 0) == cudaSuccess &&
            cudaStreamWaitEvent(ctx->s_compute, ctx->ev_begin, 0) == cudaSuccess &&
            cudaStreamWaitEvent(ctx->s_d2h, ctx->ev_begin, 0) == cudaSuccess;
  // Three streams: chunk i is copied in while chunk i-1 is computed and chunk i-2 is copied out.
  for (int i = 0; ok && i < chunks; ++i) {
    const int b = i & 1;
    const int rows = (i + 1 < chunks) ? C : M - i * C;
    if (i >= 2) ok = cudaStreamWaitEvent(ctx->s_h2d, ctx->ev_done[b], 0) == cudaSuccess;  // staging X[b] consumed
    ok = ok && cudaMemcpyAsync(ctx->hx[b], xh + static_cast<size_t>(i) * C * h->K, sizeof(uint16_t) * rows * h->K,
                               cudaMemcpyHostToDevice, ctx->s_h2d) == cudaSuccess &&
         cudaEventRecord(ctx->ev_in[b], ctx->s_h2d) == cudaSuccess &&
         cudaStreamWaitEvent(ctx->s_compute, ctx->ev_in[b], 0) == cudaSuccess;
    if (ok && i >= 2) ok = cudaStreamWaitEvent(ctx->s_compute, ctx->ev_out[b], 0) == cudaSuccess;  // staging Y[b] drained
    if (!ok) break;
    st = launch_quantize(h, ctx->hx[b], rows, expert_id, timestep_bin, clip_table, ctx->s_compute);
    // The weight byte image is the same for every chunk: expand it with the first one only.
    if (st == W4A4_OK) st = launch_gemm(h, rows, expert_id, ctx->hy[b], ctx->s_compute, nullptr, 0, 0, nullptr, nullptr, i == 0);
    if (st != W4A4_OK) return st;
    ok = cudaEventRecord(ctx->ev_done[b], ctx->s_compute) == cudaSuccess &&
         cudaStreamWaitEvent(ctx->s_d2h, ctx->ev_done[b], 0) == cudaSuccess &&
         cudaMemcpyAsync(yh + static_cast<size_t>(i) * C * h->N, ctx->hy[b], sizeof(uint16_t) * rows * h->N,
                         cudaMemcpyDeviceToHost, ctx->s_d2h) == cudaSuccess &&
         cudaEventRecord(ctx->ev_out[b], ctx->s_d2h) == cudaSuccess;
  }
  ok = ok && cudaEventRecord(ctx->ev_end, ctx->s_d2h) == cudaSuccess &&
       cudaStreamWaitEvent(user, ctx->ev_end, 0) == cudaSuccess;
  if (!ok) {
    cudaGetLastError();
    return W4A4_ERR_CUDA;
  }
  return W4A4_OK;
}

w4a4_status_t w4a4_debug_quantize(w4a4_handle_t h, const void* X, int M, int expert_id, int timestep_bin,
                                  const float* clip_table, int8_t* codes, float* scales, float* T, void* stream) {
  w4a4_status_t st = check_forward_args(h, X, M, expert_id, timestep_bin, clip_table, true);
  if (st != W4A4_OK) return st;
  if (M > 0 && (!codes || !scales)) return W4A4_ERR_INVALID_ARG;
  DeviceGuard guard(h->ctx->device);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  st = launch_quantize(h, X, M, expert_id, timestep_bin, clip_table, s);
  if (st != W4A4_OK || M == 0) return st;
  const size_t nc = static_cast<size_t>(M) * h->K;
  decode_codes_kernel<<<static_cast<unsigned>((nc + 255) / 256), 256, 0, s>>>(h->ctx->codes, codes, M, h->K);
  const size_t ns = static_cast<size_t>(M) * (h->K / 64);
  decode_scales_kernel<<<static_cast<unsigned>((ns + 255) / 256), 256, 0, s>>>(h->ctx->scales, h->ctx->scales_ld, scales, M,
                                                                               h->K / 64);
  if (T && h->r > 0) {
    const size_t nt = static_cast<size_t>(M) * h->r;
    decode_t_kernel<<<static_cast<unsigned>((nt + 255) / 256), 256, 0, s>>>(h->ctx->t_hilo, T, M, h->r);
  }
  return cudaGetLastError() == cudaSuccess ? W4A4_OK : W4A4_ERR_CUDA;
}

w4a4_status_t w4a4_debug_partials(w4a4_handle_t h, const void* X, int M, int expert_id, int timestep_bin,
                                  const float* clip_table, void* Y, int m0, int n0, int32_t* P, void* stream) {
  w4a4_status_t st = check_forward_args(h, X, M, expert_id, timestep_bin, clip_table, true);
  if (st != W4A4_OK) return st;
  if (M > 0 && (!Y || !aligned16(Y) || !P)) return W4A4_ERR_INVALID_ARG;
  if (m0 < 0 || n0 < 0 || m0 % kBM != 0 || n0 % kBN != 0 || n0 >= h->N || (M > 0 && m0 >= M)) return W4A4_ERR_INVALID_ARG;
  DeviceGuard guard(h->ctx->device);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  st = launch_quantize(h, X, M, expert_id, timestep_bin, clip_table, s);
  if (st != W4A4_OK) return st;
  return launch_gemm(h, M, expert_id, Y, s, P, m0, n0);
}

w4a4_status_t w4a4_query_status(w4a4_ctx_t ctx) {
  if (!ctx) return W4A4_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  if (cudaDeviceSynchronize() != cudaSuccess) return W4A4_ERR_CUDA;
  int err = 0;
  if (cudaMemcpy(&err, ctx->d_err, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return W4A4_ERR_CUDA;
  if (err != 0) {
    cudaMemset(ctx->d_err, 0, sizeof(int));
    return W4A4_ERR_TIMEOUT;
  }
  return W4A4_OK;
}

w4a4_status_t w4a4_debug_wait_probe(w4a4_ctx_t ctx, uint64_t limit_ns, void* stream) {
  if (!ctx) return W4A4_ERR_INVALID_ARG;
  if (limit_ns == 0 || limit_ns > 100000000ull) return W4A4_ERR_INVALID_ARG;  // at most 0.1 s
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return W4A4_ERR_CUDA;
  wait_probe_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(ctx->d_err, limit_ns);
  return cudaGetLastError() == cudaSuccess ? W4A4_OK : W4A4_ERR_CUDA;
}

w4a4_status_t w4a4_debug_stalled_gemm(w4a4_handle_t h, int M, int expert_id, void* Y, int stall_stage,
                                      uint64_t limit_ns, void* stream) {
  w4a4_status_t st = check_forward_args(h, nullptr, M, expert_id, 0, nullptr, false);
  if (st != W4A4_OK) return st;
  if (!Y || !aligned16(Y) || stall_stage < 0) return W4A4_ERR_INVALID_ARG;
  if (limit_ns == 0 || limit_ns > 100000000ull) return W4A4_ERR_INVALID_ARG;  // at most 0.1 s
  DeviceGuard guard(h->ctx->device);
  if (!guard.ok) return W4A4_ERR_CUDA;
  return launch_gemm(h, M, expert_id, Y, static_cast<cudaStream_t>(stream), nullptr, 0, 0, nullptr, nullptr, true,
                     stall_stage, limit_ns);
}

w4a4_status_t w4a4_debug_set_tile_order(w4a4_ctx_t ctx, int super_column_tiles) {
  if (!ctx || super_column_tiles < 0) return W4A4_ERR_INVALID_ARG;
  ctx->debug_sc_tiles = super_column_tiles;
  return W4A4_OK;
}

void w4a4_debug_fail_allocation_after(int n) { g_w4a4_alloc_countdown.store(n < 0 ? -1 : n); }

}  // extern "C"

#include "w4a4_mx_api.cuh"
