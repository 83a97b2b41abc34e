// C-ABI entry points of the MXFP4 variant of the layer (included at the end of w4a4_api.cu, whose set-up
// kernels and host helpers it shares).  Same structure as the INT4 path: pack once, then two kernels per forward.
#pragma once

#include "mx_gemm_kernel.cuh"

struct MxExpertData {
  uint8_t* bpacked = nullptr;  // [N, K/2] two E2M1 codes per byte
  uint8_t* sfb = nullptr;      // weight scale atoms [N/128][K/128][512]
  float* rlam = nullptr;       // [K]
  uint2* l1frag = nullptr;
  uint16_t* l2dup = nullptr;   // [N, 2r]
  float* bias = nullptr;       // [N] or null
  CUtensorMap tmB, tmL2;
  CUtensorMap tmBhalf, tmL2half;   // 128-row boxes: what one CTA of a pair fetches (mx_gemm2_kernel)
  CUtensorMap tmSFB;               // scale atoms as 32-bit words: [N/128] rows of K words, boxes of 1 KiB
  uint16_t* l1t = nullptr;         // L1 transposed, BF16 [r, K]: B operand of the fused producer's T MMA
  CUtensorMap tmL1T;               // boxes of 64 channels x r/2 rows
};

struct w4a4_mx_layer {
  w4a4_ctx* ctx = nullptr;
  int K = 0, N = 0, r = 0, E = 0, B = 0, L = 0, layer_id = 0, act = 0;
  std::vector<MxExpertData> experts;
  CUtensorMap tmA, tmT;
  CUtensorMap tmSFA;               // activation scale atoms as 32-bit words: [max_M/128] rows of K words
  CUtensorMap tmA2, tmT2, tmSFA2;  // the same three on the context's second workspace (input written by a fused producer)
  size_t bytes = 0;
};

namespace {

void mx_free_expert(MxExpertData& e) {
  cudaFree(e.bpacked);
  cudaFree(e.sfb);
  cudaFree(e.rlam);
  cudaFree(e.l1frag);
  cudaFree(e.l2dup);
  cudaFree(e.bias);
  cudaFree(e.l1t);
  e = MxExpertData();
}

size_t mx_sfa_bytes(int max_M, int K) { return static_cast<size_t>((max_M + 127) / 128) * (K / 128) * 512; }

w4a4_status_t mx_check_forward_args(w4a4_mx_handle_t h, const void* X, int M, int expert_id, int bin,
                                    const float* clip_table, bool need_x) {
  if (!h || !h->ctx) return W4A4_ERR_INVALID_ARG;
  if (M < 0 || expert_id < 0 || expert_id >= h->E) return W4A4_ERR_INVALID_ARG;
  if (M > h->ctx->max_M) return W4A4_ERR_SHAPE;
  if (need_x) {
    if (bin < 0 || bin >= h->B) return W4A4_ERR_INVALID_ARG;
    if (M > 0 && (!X || !aligned16(X))) return W4A4_ERR_INVALID_ARG;
    if (!clip_table) return W4A4_ERR_INVALID_ARG;
  }
  return W4A4_OK;
}

w4a4_status_t mx_launch_quantize_at(w4a4_mx_handle_t h, const void* X, int M, int expert_id, const float* clip_table,
                                    int clip_index, cudaStream_t stream) {
  if (M == 0) return W4A4_OK;
  w4a4_ctx* ctx = h->ctx;
  const MxExpertData& e = h->experts[expert_id];
  const int rows_per_cta = kQuantRows * quantize_warps(h->r);
  const int row_ctas = (M + rows_per_cta - 1) / rows_per_cta;
  const int splits = quantize_k_splits(row_ctas, h->K / 64, M, ctx->num_sms);
  const dim3 grid(row_ctas, splits), block(32 * quantize_warps(h->r));
  const uint16_t* x = static_cast<const uint16_t*>(X);
  float* sf = reinterpret_cast<float*>(ctx->mx_sfa);
#define W4A4_LAUNCH_MXQ(R)                                                                                             \
  quantize_kernel<R, quantize_warps(R), kCodesMxfp4><<<grid, block, quantize_smem_bytes(R), stream>>>(                 \
      x, M, h->K, e.rlam, clip_table, clip_index, e.l1frag, ctx->codes, sf, h->K / 128, ctx->t_hilo, ctx->t_partial, nullptr)
  switch (h->r) {
    case 0: W4A4_LAUNCH_MXQ(0); break;
    case 16: W4A4_LAUNCH_MXQ(16); break;
    case 32: W4A4_LAUNCH_MXQ(32); break;
    case 64: W4A4_LAUNCH_MXQ(64); break;
    default: return W4A4_ERR_SHAPE;
  }
#undef W4A4_LAUNCH_MXQ
  if (splits > 1 && h->r > 0) {
    const size_t nt = static_cast<size_t>(M) * h->r;
    t_reduce_kernel<<<static_cast<unsigned>((nt + 255) / 256), 256, 0, stream>>>(ctx->t_partial, splits, M, h->r, ctx->t_hilo);
  }
  return cudaGetLastError() == cudaSuccess ? W4A4_OK : W4A4_ERR_CUDA;
}

w4a4_status_t mx_launch_quantize(w4a4_mx_handle_t h, const void* X, int M, int expert_id, int bin, const float* clip_table,
                                 cudaStream_t stream) {
  return mx_launch_quantize_at(h, X, M, expert_id, clip_table, (expert_id * h->L + h->layer_id) * h->B + bin, stream);
}

// `second_ws`: the layer's input (codes, scale atoms, T) lies in the context's second workspace.  `next` / `next_e`:
// fused form, the epilogue quantizes the output for that layer into the second workspace instead of storing Y.
w4a4_status_t mx_launch_gemm(w4a4_mx_handle_t h, int M, int expert_id, void* Y, cudaStream_t stream,
                             const void* yref = nullptr, double* sq_err = nullptr, bool second_ws = false,
                             w4a4_mx_handle_t next = nullptr, const float* next_rho = nullptr) {
  if (M == 0) return W4A4_OK;
  w4a4_ctx* ctx = h->ctx;
  const MxExpertData& e = h->experts[expert_id];
  MxGemmParams p;
  p.bias = e.bias;
  p.Y = static_cast<uint16_t*>(Y);
  p.sfa = second_ws ? ctx->mx_sfa2 : ctx->mx_sfa;
  p.sfb = e.sfb;
  p.M = M;
  p.N = h->N;
  p.K = h->K;
  p.r = h->r;
  p.tiles_m = (M + kBM - 1) / kBM;
  p.tiles_n = (h->N + kMxBN - 1) / kMxBN;
  p.err = ctx->d_err;
  p.yref = static_cast<const uint16_t*>(yref);
  p.sq_err = sq_err;
  p.act = h->act;
  // Runs of column tiles per cluster: 1 = interleave; the fused form takes six at a time (T stays in TMEM over a
  // run, and the 74 clusters of a wave then cover about a dozen row pairs whose A rows they share in L2).
  p.run = next ? (p.tiles_n < 6 ? p.tiles_n : 6) : 1;
  const int num_tiles = p.tiles_m * p.tiles_n;
  const dim3 grid(num_tiles < ctx->num_sms ? num_tiles : ctx->num_sms), block(kMxThreads);
  const CUtensorMap& tmA = second_ws ? h->tmA2 : h->tmA;
  const CUtensorMap& tmSFA = second_ws ? h->tmSFA2 : h->tmSFA;
  const CUtensorMap& tmT = h->r > 0 ? (second_ws ? h->tmT2 : h->tmT) : tmA;  // unused when r == 0
  const CUtensorMap& tmL2 = h->r > 0 ? e.tmL2 : e.tmB;
  // CTA pairs (cta_group::2) need at least two row tiles and an even number of CTAs.
  if (p.tiles_m >= 2 && ctx->num_sms >= 2) {
    const int runs = ((p.tiles_m + 1) / 2) * ((p.tiles_n + p.run - 1) / p.run);
    const int ctas = 2 * runs < ctx->num_sms ? 2 * runs : (ctx->num_sms & ~1);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(ctas);
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = kMx2SmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const CUtensorMap& tmL2h = h->r > 0 ? e.tmL2half : e.tmBhalf;
    MxNextParams nx = {};
    cudaError_t le;
    if (next) {
      const MxExpertData& ne = next->experts[expert_id];
      nx.rlam = ne.rlam;
      nx.rho = next_rho;
      nx.codes = ctx->mx_codes2;
      nx.sfa = ctx->mx_sfa2;
      nx.t32 = ctx->mx_t32;
      nx.r2 = next->r;
      cfg.dynamicSmemBytes = kMx2FuseSmemBytes;
      const CUtensorMap& tmL1T = next->r > 0 ? ne.tmL1T : e.tmBhalf;
      le = cudaLaunchKernelEx(&cfg, mx_gemm2_kernel<true>, tmA, e.tmBhalf, tmT, tmL2h, tmSFA, e.tmSFB, tmL1T, p, nx);
    } else {
      le = cudaLaunchKernelEx(&cfg, mx_gemm2_kernel<false>, tmA, e.tmBhalf, tmT, tmL2h, tmSFA, e.tmSFB, e.tmBhalf, p, nx);
    }
    if (le != cudaSuccess) {
      cudaGetLastError();
      return W4A4_ERR_CUDA;
    }
    return W4A4_OK;
  }
  if (next) return W4A4_ERR_SHAPE;   // the fused form runs on CTA pairs only
  mx_gemm_kernel<<<grid, block, kMxSmemBytes, stream>>>(tmA, e.tmB, tmT, tmL2, p);
  return cudaGetLastError() == cudaSuccess ? W4A4_OK : W4A4_ERR_CUDA;
}

}  // namespace

extern "C" {

void w4a4_mx_destroy(w4a4_mx_handle_t h) {
  if (!h) return;
  if (h->ctx) {
    DeviceGuard guard(h->ctx->device);
    for (auto& e : h->experts) mx_free_expert(e);
  }
  delete h;
}

size_t w4a4_mx_handle_bytes(w4a4_mx_handle_t h) { return h ? h->bytes : 0; }

w4a4_status_t w4a4_mx_pack_weights(w4a4_ctx_t ctx, const w4a4_mx_weight_desc_t* d, w4a4_mx_handle_t* out) {
  if (!out) return W4A4_ERR_INVALID_ARG;
  *out = nullptr;
  if (!ctx || !d) return W4A4_ERR_INVALID_ARG;
  if (d->K <= 0 || d->K % kMxBK != 0 || d->N <= 0 || d->N % kBN != 0) return W4A4_ERR_SHAPE;
  if (!(d->r == 0 || d->r == 16 || d->r == 32 || d->r == 64)) return W4A4_ERR_SHAPE;
  if (d->K > ctx->max_K || d->r > ctx->max_r) return W4A4_ERR_SHAPE;
  if (d->num_experts < 1 || d->num_bins < 1 || d->num_layers < 1 || d->layer_id < 0 || d->layer_id >= d->num_layers)
    return W4A4_ERR_INVALID_ARG;
  if (!d->wcodes || !d->wexps || !d->lambda || (d->r > 0 && (!d->L1 || !d->L2))) return W4A4_ERR_INVALID_ARG;
  if (d->output_activation != W4A4_ACT_NONE && d->output_activation != W4A4_ACT_GELU_TANH) return W4A4_ERR_INVALID_ARG;
  for (int e = 0; e < d->num_experts; ++e) {
    if (!d->wcodes[e] || !d->wexps[e] || !d->lambda[e] || (d->r > 0 && (!d->L1[e] || !d->L2[e]))) return W4A4_ERR_INVALID_ARG;
  }
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return W4A4_ERR_CUDA;

  w4a4_mx_layer* h = new (std::nothrow) w4a4_mx_layer();
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

  // The activation scale atoms live in the context (zero-filled once: rows past M of the last row block are
  // read by the tensor core and must not hold E8M0's NaN byte).
  if (!ctx->mx_sfa) {
    const size_t nb = mx_sfa_bytes(ctx->max_M, ctx->max_K);
    st = dev_alloc(&ctx->mx_sfa, nb, &ctx->bytes);
    if (st == W4A4_OK && cudaMemset(ctx->mx_sfa, 0, nb) != cudaSuccess) st = W4A4_ERR_CUDA;
    if (st == W4A4_OK)
      cudaFuncSetAttribute(mx_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kMxSmemBytes));
    if (st == W4A4_OK)
      cudaFuncSetAttribute(mx_gemm2_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kMx2SmemBytes));
    if (st == W4A4_OK)
      cudaFuncSetAttribute(mx_gemm2_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kMx2FuseSmemBytes));
    // Second workspace of the fused FFN.
    const size_t codes2 = static_cast<size_t>(ctx->max_M) * (ctx->max_K / 2);
    const int rr = ctx->max_r > 0 ? ctx->max_r : 8;
    if (st == W4A4_OK) st = dev_alloc(&ctx->mx_codes2, codes2, &ctx->bytes);
    if (st == W4A4_OK && cudaMemset(ctx->mx_codes2, 0, codes2) != cudaSuccess) st = W4A4_ERR_CUDA;
    if (st == W4A4_OK) st = dev_alloc(&ctx->mx_sfa2, nb, &ctx->bytes);
    if (st == W4A4_OK && cudaMemset(ctx->mx_sfa2, 0, nb) != cudaSuccess) st = W4A4_ERR_CUDA;
    if (st == W4A4_OK) st = dev_alloc(&ctx->mx_t32, static_cast<size_t>(ctx->max_M) * rr, &ctx->bytes);
    if (st == W4A4_OK) st = dev_alloc(&ctx->t_hilo2, static_cast<size_t>(ctx->max_M) * 2 * rr, &ctx->bytes);
    if (st == W4A4_OK && cudaMemset(ctx->t_hilo2, 0, sizeof(uint16_t) * ctx->max_M * 2 * rr) != cudaSuccess) st = W4A4_ERR_CUDA;

    if (st == W4A4_OK)
      cudaFuncSetAttribute(quantize_kernel<64, quantize_warps(64), kCodesMxfp4>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           static_cast<int>(quantize_smem_bytes(64)));
  }
  int* d_bad = nullptr;
  if (st == W4A4_OK) st = dev_alloc(&d_bad, 1, nullptr);
  if (st == W4A4_OK && cudaMemset(d_bad, 0, sizeof(int)) != cudaSuccess) st = W4A4_ERR_CUDA;

  for (int ei = 0; st == W4A4_OK && ei < d->num_experts; ++ei) {
    MxExpertData& e = h->experts[ei];
    st = dev_alloc(&e.bpacked, static_cast<size_t>(N) * (K / 2), &h->bytes);
    if (st == W4A4_OK) st = dev_alloc(&e.sfb, static_cast<size_t>(N / 128) * (K / 128) * 512, &h->bytes);
    if (st == W4A4_OK) st = dev_alloc(&e.rlam, static_cast<size_t>(K), &h->bytes);
    if (st == W4A4_OK && r > 0) st = dev_alloc(&e.l1frag, static_cast<size_t>(G) * 4 * (r / 8) * 32, &h->bytes);
    if (st == W4A4_OK && r > 0) st = dev_alloc(&e.l2dup, static_cast<size_t>(N) * 2 * r, &h->bytes);
    if (st == W4A4_OK && r > 0) st = dev_alloc(&e.l1t, static_cast<size_t>(r) * K, &h->bytes);
    const float* bias_src = d->bias ? d->bias[ei] : nullptr;
    if (st == W4A4_OK && bias_src) st = dev_alloc(&e.bias, static_cast<size_t>(N), &h->bytes);
    if (st != W4A4_OK) break;
    const cudaMemcpyKind kind = dev ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice;
    if (bias_src && cudaMemcpy(e.bias, bias_src, sizeof(float) * N, kind) != cudaSuccess) st = W4A4_ERR_CUDA;
    if (st != W4A4_OK) break;

    const uint8_t *c_dev = nullptr, *x_dev = nullptr;
    uint8_t *c_own = nullptr, *x_own = nullptr;
    const float* lam_dev = nullptr;
    float* lam_own = nullptr;
    const uint16_t *l1_dev = nullptr, *l2_dev = nullptr;
    uint16_t *l1_own = nullptr, *l2_own = nullptr;
    st = stage_in(d->wcodes[ei], static_cast<size_t>(K) * N, dev, &c_dev, &c_own);
    if (st == W4A4_OK) st = stage_in(d->wexps[ei], static_cast<size_t>(K / 32) * N, dev, &x_dev, &x_own);
    if (st == W4A4_OK) st = stage_in(d->lambda[ei], static_cast<size_t>(K), dev, &lam_dev, &lam_own);
    if (st == W4A4_OK && r > 0) st = stage_in(d->L1[ei], static_cast<size_t>(K) * r, dev, &l1_dev, &l1_own);
    if (st == W4A4_OK && r > 0) st = stage_in(d->L2[ei], static_cast<size_t>(r) * N, dev, &l2_dev, &l2_own);
    if (st == W4A4_OK) {
      reciprocal_kernel<<<(K + 255) / 256, 256>>>(lam_dev, e.rlam, K);
      mx_pack_weight_kernel<<<dim3((N + 127) / 128, K / 32), 128>>>(c_dev, e.bpacked, K, N, d_bad);
      const size_t ns = static_cast<size_t>(K / 32) * N;
      mx_pack_wscale_kernel<<<static_cast<unsigned>((ns + 255) / 256), 256>>>(x_dev, e.sfb, K, N, d_bad);
      if (r > 0) {
        const size_t nf = static_cast<size_t>(G) * 4 * (r / 8) * 32;
        l1_fragment_kernel<<<static_cast<unsigned>((nf + 255) / 256), 256>>>(l1_dev, e.l1frag, K, r);
        const size_t nl = static_cast<size_t>(N) * 2 * r;
        l2_dup_kernel<<<static_cast<unsigned>((nl + 255) / 256), 256>>>(l2_dev, e.l2dup, r, N);
        const size_t nt = static_cast<size_t>(K) * r;
        mx_transpose_l1_kernel<<<static_cast<unsigned>((nt + 255) / 256), 256>>>(l1_dev, e.l1t, K, r);
      }
      if (cudaGetLastError() != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess) st = W4A4_ERR_CUDA;
    }
    cudaFree(c_own);
    cudaFree(x_own);
    cudaFree(lam_own);
    cudaFree(l1_own);
    cudaFree(l2_own);
    if (st != W4A4_OK) break;
    if (!encode_2d(ctx->encode, &e.tmB, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, e.bpacked, K / 2, N, K / 2, 128, kMxBN,
                   CU_TENSOR_MAP_SWIZZLE_128B))
      st = W4A4_ERR_CUDA;
    if (st == W4A4_OK &&
        !encode_2d(ctx->encode, &e.tmBhalf, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, e.bpacked, K / 2, N, K / 2, 128, kMxBN / 2,
                   CU_TENSOR_MAP_SWIZZLE_128B))
      st = W4A4_ERR_CUDA;
    if (st == W4A4_OK &&
        !encode_2d(ctx->encode, &e.tmSFB, CU_TENSOR_MAP_DATA_TYPE_UINT32, 4, e.sfb, K, N / 128, 4 * static_cast<uint64_t>(K), 256,
                   1, CU_TENSOR_MAP_SWIZZLE_NONE))
      st = W4A4_ERR_CUDA;
    if (st == W4A4_OK && r > 0 &&
        !encode_2d(ctx->encode, &e.tmL1T, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, e.l1t, K, r, 2 * static_cast<uint64_t>(K), 64, r / 2,
                   CU_TENSOR_MAP_SWIZZLE_128B))
      st = W4A4_ERR_CUDA;
    if (st == W4A4_OK && r > 0 &&
        !encode_2d(ctx->encode, &e.tmL2half, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, e.l2dup, 2 * r, N, 4 * r, 64, kMxBN / 2,
                   CU_TENSOR_MAP_SWIZZLE_128B))
      st = W4A4_ERR_CUDA;
    if (st == W4A4_OK && r > 0 &&
        !encode_2d(ctx->encode, &e.tmL2, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, e.l2dup, 2 * r, N, 4 * r, 64, kMxBN,
                   CU_TENSOR_MAP_SWIZZLE_128B))
      st = W4A4_ERR_CUDA;
  }
  if (st == W4A4_OK) {
    int bad = 0;
    if (cudaMemcpy(&bad, d_bad, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) st = W4A4_ERR_CUDA;
    else if (bad) st = W4A4_ERR_INVALID_ARG;  // a code above 15 or the NaN scale byte
  }
  cudaFree(d_bad);
  if (st == W4A4_OK &&
      !encode_2d(ctx->encode, &h->tmA, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, ctx->codes, K / 2, ctx->max_M, K / 2, 128, kBM,
                 CU_TENSOR_MAP_SWIZZLE_128B))
    st = W4A4_ERR_CUDA;
  if (st == W4A4_OK &&
      !encode_2d(ctx->encode, &h->tmSFA, CU_TENSOR_MAP_DATA_TYPE_UINT32, 4, ctx->mx_sfa, K, (ctx->max_M + 127) / 128,
                 4 * static_cast<uint64_t>(K), 256, 1, CU_TENSOR_MAP_SWIZZLE_NONE))
    st = W4A4_ERR_CUDA;
  if (st == W4A4_OK &&
      !encode_2d(ctx->encode, &h->tmA2, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, ctx->mx_codes2, K / 2, ctx->max_M, K / 2, 128, kBM,
                 CU_TENSOR_MAP_SWIZZLE_128B))
    st = W4A4_ERR_CUDA;
  if (st == W4A4_OK &&
      !encode_2d(ctx->encode, &h->tmSFA2, CU_TENSOR_MAP_DATA_TYPE_UINT32, 4, ctx->mx_sfa2, K, (ctx->max_M + 127) / 128,
                 4 * static_cast<uint64_t>(K), 256, 1, CU_TENSOR_MAP_SWIZZLE_NONE))
    st = W4A4_ERR_CUDA;
  if (st == W4A4_OK && r > 0 &&
      !encode_2d(ctx->encode, &h->tmT2, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, ctx->t_hilo2, 2 * r, ctx->max_M, 4 * r, 64,
                 kBM, CU_TENSOR_MAP_SWIZZLE_128B))
    st = W4A4_ERR_CUDA;
  if (st == W4A4_OK && r > 0 &&
      !encode_2d(ctx->encode, &h->tmT, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, ctx->t_hilo, 2 * r, ctx->max_M, 4 * r, 64,
                 kBM, CU_TENSOR_MAP_SWIZZLE_128B))
    st = W4A4_ERR_CUDA;
  if (st != W4A4_OK) {
    cudaGetLastError();
    w4a4_mx_destroy(h);
    return st;
  }
  *out = h;
  return W4A4_OK;
}

w4a4_status_t w4a4_mx_quantize_activations(w4a4_mx_handle_t h, const void* X, int M, int expert_id, int timestep_bin,
                                           const float* clip_table, void* stream) {
  w4a4_status_t st = mx_check_forward_args(h, X, M, expert_id, timestep_bin, clip_table, true);
  if (st != W4A4_OK) return st;
  DeviceGuard guard(h->ctx->device);
  return mx_launch_quantize(h, X, M, expert_id, timestep_bin, clip_table, static_cast<cudaStream_t>(stream));
}

w4a4_status_t w4a4_mx_gemm_from_workspace(w4a4_mx_handle_t h, int M, int expert_id, void* Y, void* stream) {
  w4a4_status_t st = mx_check_forward_args(h, nullptr, M, expert_id, 0, nullptr, false);
  if (st != W4A4_OK) return st;
  if (M > 0 && (!Y || !aligned16(Y))) return W4A4_ERR_INVALID_ARG;
  DeviceGuard guard(h->ctx->device);
  return mx_launch_gemm(h, M, expert_id, Y, static_cast<cudaStream_t>(stream));
}

w4a4_status_t w4a4_mx_linear_forward(w4a4_mx_handle_t h, const void* X, int M, int expert_id, int timestep_bin,
                                     const float* clip_table, void* Y, void* stream) {
  w4a4_status_t st = mx_check_forward_args(h, X, M, expert_id, timestep_bin, clip_table, true);
  if (st != W4A4_OK) return st;
  if (M > 0 && (!Y || !aligned16(Y))) return W4A4_ERR_INVALID_ARG;
  DeviceGuard guard(h->ctx->device);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  st = mx_launch_quantize(h, X, M, expert_id, timestep_bin, clip_table, s);
  if (st != W4A4_OK) return st;
  return mx_launch_gemm(h, M, expert_id, Y, s);
}

w4a4_status_t w4a4_mx_clip_search(w4a4_mx_handle_t h, const void* const* X_samples, const void* const* Yref_samples,
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
    w4a4_status_t st = mx_check_forward_args(h, X_samples[s], M, expert_id, timestep_bin, clip_table, true);
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
  for (int s = 0; st == W4A4_OK && s < num_samples; ++s) {
    for (int c = 0; st == W4A4_OK && c < num_candidates; ++c) {
      st = mx_launch_quantize_at(h, X_samples[s], M, expert_id, d_cand, c, st_);
      if (st == W4A4_OK) st = mx_launch_gemm(h, M, expert_id, nullptr, st_, Yref_samples[s], d_err + c);
    }
  }
  int best = 0;
  if (st == W4A4_OK) {
    clip_argmin_kernel<<<1, 32, 0, st_>>>(d_err, d_cand, num_candidates,
                                          clip_table + (expert_id * h->L + h->layer_id) * h->B + timestep_bin, d_best);
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

w4a4_status_t w4a4_mx_debug_quantize(w4a4_mx_handle_t h, const void* X, int M, int expert_id, int timestep_bin,
                                     const float* clip_table, uint8_t* codes, uint8_t* exps, float* T, void* stream) {
  w4a4_status_t st = mx_check_forward_args(h, X, M, expert_id, timestep_bin, clip_table, true);
  if (st != W4A4_OK) return st;
  if (M > 0 && (!codes || !exps)) return W4A4_ERR_INVALID_ARG;
  if (M == 0) return W4A4_OK;
  DeviceGuard guard(h->ctx->device);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  st = mx_launch_quantize(h, X, M, expert_id, timestep_bin, clip_table, s);
  if (st != W4A4_OK) return st;
  const size_t nc = static_cast<size_t>(M) * h->K, ns = static_cast<size_t>(M) * (h->K / 32);
  mx_decode_codes_kernel<<<static_cast<unsigned>((nc + 255) / 256), 256, 0, s>>>(h->ctx->codes, codes, M, h->K);
  mx_decode_exps_kernel<<<static_cast<unsigned>((ns + 255) / 256), 256, 0, s>>>(h->ctx->mx_sfa, h->K / 128, exps, M, h->K / 32);
  if (T && h->r > 0) {
    const size_t nt = static_cast<size_t>(M) * h->r;
    decode_t_kernel<<<static_cast<unsigned>((nt + 255) / 256), 256, 0, s>>>(h->ctx->t_hilo, T, M, h->r);
  }
  return cudaGetLastError() == cudaSuccess ? W4A4_OK : W4A4_ERR_CUDA;
}

// Fused pair of layers (Sec. III, the FFN): `up` runs as usual except that its GEMM's epilogue applies bias and
// activation, rounds to BF16 and quantizes the result for `down` (codes, block exponents, the low-rank projection T)
// straight into the context's second workspace; `down`'s GEMM then reads its operands from there.  The hidden
// activation never reaches memory and `down`'s activation kernel does not run.
w4a4_status_t w4a4_mx_ffn_forward(w4a4_mx_handle_t up, w4a4_mx_handle_t down, const void* X, int M, int expert_id,
                                  int timestep_bin, const float* clip_table, void* Y, void* stream) {
  w4a4_status_t st = mx_check_forward_args(up, X, M, expert_id, timestep_bin, clip_table, true);
  if (st != W4A4_OK) return st;
  st = mx_check_forward_args(down, X, M, expert_id, timestep_bin, clip_table, true);
  if (st != W4A4_OK) return st;
  if (up->ctx != down->ctx || up->N != down->K) return W4A4_ERR_SHAPE;
  if (M > 0 && (!Y || !aligned16(Y))) return W4A4_ERR_INVALID_ARG;
  if (M == 0) return W4A4_OK;
  if (M <= kBM) return W4A4_ERR_SHAPE;   // the fused epilogue exists in the CTA-pair kernel only (two row tiles)
  w4a4_ctx* ctx = up->ctx;
  DeviceGuard guard(ctx->device);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  st = mx_launch_quantize(up, X, M, expert_id, timestep_bin, clip_table, s);
  if (st != W4A4_OK) return st;
  if (down->r > 0 &&
      cudaMemsetAsync(ctx->mx_t32, 0, sizeof(float) * static_cast<size_t>(M) * down->r, s) != cudaSuccess)
    return W4A4_ERR_CUDA;
  const float* rho2 = clip_table + (static_cast<size_t>(expert_id) * down->L + down->layer_id) * down->B + timestep_bin;
  st = mx_launch_gemm(up, M, expert_id, nullptr, s, nullptr, nullptr, false, down, rho2);
  if (st != W4A4_OK) return st;
  if (down->r > 0) {
    const size_t nt = static_cast<size_t>(M) * down->r;
    t_reduce_kernel<<<static_cast<unsigned>((nt + 255) / 256), 256, 0, s>>>(ctx->mx_t32, 1, M, down->r, ctx->t_hilo2);
    if (cudaGetLastError() != cudaSuccess) return W4A4_ERR_CUDA;
  }
  return mx_launch_gemm(down, M, expert_id, Y, s, nullptr, nullptr, true);
}

// Parity tap of the fused form: decodes what the last w4a4_mx_ffn_forward left in the second workspace for `down`.
w4a4_status_t w4a4_mx_debug_fused_input(w4a4_mx_handle_t down, int M, uint8_t* codes, uint8_t* exps, float* T, void* stream) {
  if (!down || !down->ctx || M < 0 || M > down->ctx->max_M) return W4A4_ERR_INVALID_ARG;
  if (M > 0 && (!codes || !exps)) return W4A4_ERR_INVALID_ARG;
  if (M == 0) return W4A4_OK;
  DeviceGuard guard(down->ctx->device);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const size_t nc = static_cast<size_t>(M) * down->K, ns = static_cast<size_t>(M) * (down->K / 32);
  mx_decode_codes_kernel<<<static_cast<unsigned>((nc + 255) / 256), 256, 0, s>>>(down->ctx->mx_codes2, codes, M, down->K);
  mx_decode_exps_kernel<<<static_cast<unsigned>((ns + 255) / 256), 256, 0, s>>>(down->ctx->mx_sfa2, down->K / 128, exps, M, down->K / 32);
  if (T && down->r > 0) {
    const size_t nt = static_cast<size_t>(M) * down->r;
    decode_t_kernel<<<static_cast<unsigned>((nt + 255) / 256), 256, 0, s>>>(down->ctx->t_hilo2, T, M, down->r);
  }
  return cudaGetLastError() == cudaSuccess ? W4A4_OK : W4A4_ERR_CUDA;
}

}  // extern "C"
