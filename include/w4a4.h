/*
 * libw4a4 -- W4A4 + low-rank linear layer forward for NVIDIA B200 (sm_100a).
 *
 * The layer computed here is the inference-time form of the paper's quantized linear (Eq. 7 and
 * Eq. 11 of "Timestep-Aware SVDQuant-GPTQ for W4A4 Quantization of Wan2.2-I2V"):
 *
 *     Y = Q_A(Xh; rho[expert, layer, bin]) * Qw  +  (Xh * L1) * L2  +  b ,     Xh = X * diag(lambda)^-1
 *
 * Xh is the smoothed activation (Eq. 5), Q_A the symmetric 4-bit quantizer of Eq. 3-4 applied per
 * token and per group of 64 consecutive input channels with the clip threshold of Eq. 8-9
 * (threshold = rho * group absolute maximum, scale = threshold / 7, codes clipped to [-8, 7],
 * round half to even), Qw the 4-bit residual weight with one FP32 scale per (64-row group, output
 * column) (Eq. 6), and L1 (K x r), L2 (r x N) the BF16 low-rank pair (Eq. 6).  rho is fetched on the
 * device from a table indexed by (expert, layer, timestep bin) (Sec. III-C, last paragraph).
 *
 * sm_100a has no 4-bit integer tensor-core instruction.  The 4-bit codes (integers -8 .. 7) are fed to the
 * tensor core as E4M3 bytes, which represent them exactly; products and 64-term group sums are exact in the
 * FP32 accumulator, so Eq. 7's integer partial sums come out bit for bit.
 *
 * Every step runs in hand-written CUDA kernels; there is no CPU fallback.  All entry points return
 * a status code, never throw and never abort.  Unless stated otherwise pointers are DEVICE pointers
 * owned by the caller, 16-byte aligned, and only read/written during the call (asynchronously, on
 * the given stream, for the forward calls).
 */
#ifndef W4A4_H_
#define W4A4_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  W4A4_OK = 0,
  W4A4_ERR_INVALID_ARG = 1, /* NULL pointer, out-of-range expert / bin / layer, misaligned buffer */
  W4A4_ERR_SHAPE = 2,       /* unsupported K, N, r, group or M beyond the context's limits */
  W4A4_ERR_ALLOC = 3,       /* device or host allocation failed (setup calls only) */
  W4A4_ERR_CUDA = 4,        /* a CUDA runtime / driver call or a kernel launch failed */
  W4A4_ERR_ARCH = 5,        /* the device is not compute capability 10.x */
  W4A4_ERR_TIMEOUT = 6      /* a kernel gave up on a bounded wait and returned early (see w4a4_query_status) */
} w4a4_status_t;

/* Activation fused into the output of a layer (no counterpart in the paper's equations; it is the producer-side
 * fusion for the FFN, whose second linear consumes GELU of the first one's output: applying it in the GEMM's
 * epilogue saves the element-wise pass over the 13824-wide hidden activations).  GELU_TANH is
 * 0.5 y (1 + tanh(sqrt(2/pi) (y + 0.044715 y^3))) evaluated in FP32 on y = Eq. 11's value before the BF16 rounding. */
#define W4A4_ACT_NONE 0
#define W4A4_ACT_GELU_TANH 1

typedef struct w4a4_ctx* w4a4_ctx_t;      /* per-stream workspace: activation codes, scales, low-rank intermediate */
typedef struct w4a4_layer* w4a4_handle_t; /* one layer position: packed constants of all its experts */

/*
 * Constants of one layer position for all experts (Eq. 5-6; Sec. I: one weight set per expert).
 * Arrays are indexed by expert.  With pointers_on_device == 0 the inner pointers are HOST pointers,
 * with 1 they are DEVICE pointers; the outer arrays are always host arrays.  Everything is copied /
 * repacked during w4a4_pack_weights and may be freed when it returns.
 */
typedef struct {
  int K;           /* input channels C_in, multiple of 64 */
  int N;           /* output channels C_out, multiple of 128 */
  int r;           /* low-rank width: 0, 16, 32, 64 or 96 (96: three rank-32 projections packed along N) */
  int group;       /* quantization group along K: must be 64 */
  int num_experts; /* >= 1 */
  int num_bins;    /* timestep bins per (expert, layer) in the clip table */
  int num_layers;  /* layers per expert in the clip table */
  int layer_id;    /* this layer's index into the clip table */
  int pointers_on_device;
  int output_activation; /* W4A4_ACT_NONE, or W4A4_ACT_GELU_TANH: the layer returns GELU(Y) (see below) */
  const int8_t* const* qweight;  /* [E] -> K x N row-major, one code per byte, values in [-8, 7] */
  const float* const* wscale;    /* [E] -> (K/64) x N row-major FP32 */
  const float* const* lambda;    /* [E] -> K FP32, > 0 (diagonal of the smoothing matrix D_l) */
  const uint16_t* const* L1;     /* [E] -> K x r row-major BF16 bit patterns (ignored if r == 0) */
  const uint16_t* const* L2;     /* [E] -> r x N row-major BF16 bit patterns (ignored if r == 0) */
  const float* const* bias;      /* [E] -> N FP32; the array or an entry may be NULL (no bias) */
} w4a4_weight_desc_t;

/* Creates a context on `device` whose workspace fits M <= max_M tokens, K <= max_K, r <= max_r.
 * One context serves one stream at a time (calls on it reuse the same workspace in stream order).
 * Sec. III (whole forward) -- the workspace holds Q_A(Xh) (one byte per code), its scales and Xh*L1 between
 * the kernels, and the 8-bit image of the running layer's weights (N x K bytes, sized by w4a4_pack_weights
 * for the largest layer packed on the context). */
w4a4_status_t w4a4_ctx_create(int device, int max_M, int max_K, int max_r, w4a4_ctx_t* out);
void w4a4_ctx_destroy(w4a4_ctx_t ctx);

/* Copies and repacks one layer's constants (Eq. 5-6) into the library's own device layout:
 * reciprocal smoothing vector, nibble-packed residual codes (4 bits per weight at rest), scales, low-rank
 * factors in tensor-core order, bias.  Synchronous; allocates device memory owned by the handle, and grows
 * the context's weight-image scratch if this layer is the largest so far (it synchronises the device first). */
w4a4_status_t w4a4_pack_weights(w4a4_ctx_t ctx, const w4a4_weight_desc_t* desc, w4a4_handle_t* out);
void w4a4_destroy(w4a4_handle_t h);

/* The layer forward, Eq. 11:  Y = Q_A(Xh; rho) Qw + (Xh L1) L2 + b  with rho =
 * clip_table[(expert_id * num_layers + layer_id) * num_bins + timestep_bin], read on the device.
 *   X   device BF16 [M, K] row-major (leading dimension K), 16-byte aligned
 *   Y   device BF16 [M, N] row-major, 16-byte aligned
 *   clip_table  device FP32 [num_experts, num_layers, num_bins], values in [1e-4, 1]
 *   stream      a cudaStream_t (as void*); three kernels are enqueued (activation quantization, expansion of
 *               the layer's 4-bit weights to bytes, GEMM), no host synchronisation.
 * M may be 0 (nothing is launched).  Errors: INVALID_ARG, SHAPE (M > max_M), CUDA.  A pipeline wait that
 * gives up on the device is not visible here (the call does not synchronise): see w4a4_query_status. */
w4a4_status_t w4a4_linear_forward(w4a4_handle_t h, const void* X, int M, int expert_id, int timestep_bin,
                                  const float* clip_table, void* Y, void* stream);

/* The same layer (Eq. 11) with X and Y in HOST memory (pinned memory recommended; pageable works but the
 * copies then serialise).  M is split into chunks of `chunk_rows` tokens that flow through three internal
 * streams -- host-to-device copy, the two kernels, device-to-host copy -- so that the copies of neighbouring
 * chunks overlap the kernels (rows are independent, so chunking does not change any result).  The whole
 * operation is ordered after the work already enqueued on `stream`, and `stream` waits for its completion;
 * the call itself does not synchronise the host.  w4a4_ctx_enable_host_io must have been called once on the
 * context (it allocates the staging buffers: 2 x chunk_rows x (max_K + max_N) BF16 values, plus streams and
 * events); the forward itself allocates nothing.  clip_table stays a DEVICE pointer.
 * Errors: INVALID_ARG (host I/O not enabled, NULL pointers), SHAPE (M > max_M, N > max_N), CUDA. */
w4a4_status_t w4a4_ctx_enable_host_io(w4a4_ctx_t ctx, int chunk_rows, int max_N);
w4a4_status_t w4a4_linear_forward_host(w4a4_handle_t h, const void* X_host, int M, int expert_id, int timestep_bin,
                                       const float* clip_table, void* Y_host, void* stream);

/* The two halves of w4a4_linear_forward, exposed so that each kernel can be timed on its own.
 * w4a4_quantize_activations: Eq. 3-5, 8-9 and the first factor of Eq. 7's low-rank term, into the
 * context workspace.  w4a4_gemm_from_workspace: the rest of Eq. 7/11 from that workspace into Y. */
w4a4_status_t w4a4_quantize_activations(w4a4_handle_t h, const void* X, int M, int expert_id, int timestep_bin,
                                        const float* clip_table, void* stream);
w4a4_status_t w4a4_gemm_from_workspace(w4a4_handle_t h, int M, int expert_id, void* Y, void* stream);

/* Timestep-wise clipping-ratio search for one (expert, layer, timestep bin), Sec. III-C, Eq. 8-10:
 *     rho* = argmin over rho in R of  sum over calibration samples t in the bin of  || Y(t) - Y_hat(t; rho) ||_2^2
 * Y(t) is the full-precision layer output supplied by the caller, Y_hat(t; rho) the output of this quantized
 * layer (Eq. 11) with ratio rho, rounded to BF16 as the forward stores it.  Every candidate runs the real
 * forward kernels; the GEMM epilogue accumulates the squared error instead of storing Y_hat (FP32 inside a
 * warp and tile, FP64 across them).  The winning ratio (the first one on ties) is written into
 * clip_table[(expert_id * num_layers + layer_id) * num_bins + timestep_bin]; no other entry is touched.
 *   X_samples     host array of num_samples DEVICE pointers, each BF16 [M, K] (calibration activations of the bin)
 *   Yref_samples  host array of num_samples DEVICE pointers, each BF16 [M, N] (full-precision outputs)
 *   candidates    HOST array of num_candidates ratios in [1e-4, 1]  (1 <= num_candidates <= 256)
 *   clip_table    device FP32 table as in w4a4_linear_forward (read-modify-write of one entry)
 *   errors_out    HOST array of num_candidates doubles (the objective per candidate) or NULL
 *   best_out      HOST int (index of the winner) or NULL
 * A calibration-time call: it allocates a few hundred bytes of device scratch, enqueues
 * num_samples x num_candidates forwards on `stream` and synchronises the stream before returning.
 * Errors: INVALID_ARG (NULL / misaligned pointers, candidate out of range, M < 1), SHAPE (M > max_M), ALLOC, CUDA. */
w4a4_status_t w4a4_clip_search(w4a4_handle_t h, const void* const* X_samples, const void* const* Yref_samples,
                               int num_samples, int M, int expert_id, int timestep_bin, const float* candidates,
                               int num_candidates, float* clip_table, double* errors_out, int* best_out,
                               void* stream);

/* Parity taps (tests only; same kernels, extra stores).
 * w4a4_debug_quantize: runs the activation kernel and decodes its outputs to plain layouts:
 *   codes  device int8 [M, K] (logical 4-bit codes, Eq. 3), scales device FP32 [M, K/64] (Eq. 9),
 *   T      device FP32 [M, r] (Xh L1 as the GEMM will see it: the sum of its BF16 high and low parts); may be NULL.
 * w4a4_debug_partials: runs the whole forward and additionally stores the per-group integer partial
 *   sums (Eq. 7's 4-bit product before rescaling) of the output tile whose first row is m0 and first
 *   column is n0 (multiples of the tile sizes reported by w4a4_tile_shape):
 *   P device int32 [tile_m, K/64, tile_n];  Y as in the forward. */
w4a4_status_t w4a4_debug_quantize(w4a4_handle_t h, const void* X, int M, int expert_id, int timestep_bin,
                                  const float* clip_table, int8_t* codes, float* scales, float* T, void* stream);
w4a4_status_t w4a4_debug_partials(w4a4_handle_t h, const void* X, int M, int expert_id, int timestep_bin,
                                  const float* clip_table, void* Y, int m0, int n0, int32_t* P, void* stream);
void w4a4_tile_shape(int* tile_m, int* tile_n);

/* Activation quantization for callers that cannot allocate (the paper has no counterpart: this entry
 * point exists for deployment, not for the method).  Code that runs in a host callback, under a runtime
 * whose memory pool owns the whole device, or on a latency-critical path where the implicit device
 * synchronisation of cudaMalloc is not acceptable cannot create a context or a handle.  This call needs
 * neither: it computes Xh = X / lambda, the per-(token, 64-channel group) scales and the 4-bit codes
 * (Eq. 3-5, 8-9; no low-rank branch) with its scratch held in a fixed array inside the library image
 * (about 2.3 MiB of device memory on every GPU that loads the library, for the life of the process).
 *   X       device BF16 [M, K] row-major, 16-byte aligned          lambda  device FP32 [K], > 0
 *   clip_table / clip_index   device FP32 table and the index of the ratio to use (read on the device)
 *   codes   device int8 [M, K], one code per byte in [-8, 7]       scales  device FP32 [M, K/64]
 * Limits: K a multiple of 64, K <= 16384 and M * K <= 4194304; anything larger returns W4A4_ERR_SHAPE.
 * It calls no cudaMalloc / cudaFree and no allocating library routine.  The first call on each device
 * looks up the scratch's device address (cudaGetSymbolAddress) with that device current, so make that
 * first call outside any stream capture.  All calls share the one scratch array: every byte a call reads
 * it has written itself first (nothing relies on old contents or on zeros), but two calls that overlap
 * on the GPU (different streams, or threads) race on it -- serialise them.  Work is enqueued on `stream`;
 * the call does not synchronise. */
w4a4_status_t w4a4_quantize_noalloc(const void* X, int M, int K, const float* lambda, const float* clip_table,
                                    int clip_index, int8_t* codes, float* scales, void* stream);

/* ---- MXFP4 variant of the same layer -------------------------------------------------------------------------
 * The caption of the paper's Table 1 states that all its 4-bit runs use the MXFP4 data format, and Sec. IV-D names
 * the hardware's own 4-bit floating-point tensor path as the way forward.  This variant computes Eq. 11 with both 4-bit operands in MXFP4 as
 * the OCP Microscaling Formats specification v1.0 defines it: E2M1 elements (+-{0, 0.5, 1, 1.5, 2, 3, 4, 6}), one
 * E8M0 scale (a byte e, value 2^(e-127)) per block of 32 consecutive input channels, conversion by shared exponent
 * floor(log2(block maximum)) - 2 and round-to-nearest-even with saturation.  The clipping ratio of Eq. 8-9 scales the
 * block maximum before the shared exponent is taken (threshold = rho * max|Xh|).  Smoothing (Eq. 5), the BF16
 * low-rank branch (Eq. 6-7), the (expert, layer, bin) clip table and the bias are as in the INT4 entry points.
 * The block scales are applied inside the tensor core (tcgen05.mma kind::mxf4.block_scale), FP32 accumulation.
 * K must be a multiple of 256, N of 128; r in {0, 16, 32, 64}.  A context serves both variants. */
typedef struct w4a4_mx_layer* w4a4_mx_handle_t;

typedef struct {
  int K, N, r;
  int num_experts, num_bins, num_layers, layer_id;
  int pointers_on_device;
  int output_activation; /* W4A4_ACT_NONE or W4A4_ACT_GELU_TANH, as in w4a4_weight_desc_t */
  const uint8_t* const* wcodes; /* [E] -> K x N row-major, one E2M1 code per byte: bit 3 sign, bits 0-2 magnitude index */
  const uint8_t* const* wexps;  /* [E] -> (K/32) x N row-major E8M0 bytes (0xFF, the NaN encoding, is rejected) */
  const float* const* lambda;   /* [E] -> K FP32, > 0 */
  const uint16_t* const* L1;    /* [E] -> K x r BF16 bit patterns (ignored if r == 0) */
  const uint16_t* const* L2;    /* [E] -> r x N BF16 bit patterns (ignored if r == 0) */
  const float* const* bias;     /* [E] -> N FP32; the array or an entry may be NULL */
} w4a4_mx_weight_desc_t;

/* Copies and repacks one layer's MXFP4 constants (two codes per byte, scale bytes in the tensor core's atom
 * layout).  Synchronous; allocates device memory owned by the handle (and, once per context, the activation
 * scale workspace and the second workspace of w4a4_mx_ffn_forward: max_M x max_K / 2 bytes of codes, scale atoms,
 * and max_M x max_r FP32 + BF16 pairs).  Errors: SHAPE, INVALID_ARG (also: a code above 15, a 0xFF scale byte),
 * ALLOC, CUDA. */
w4a4_status_t w4a4_mx_pack_weights(w4a4_ctx_t ctx, const w4a4_mx_weight_desc_t* desc, w4a4_mx_handle_t* out);
void w4a4_mx_destroy(w4a4_mx_handle_t h);
size_t w4a4_mx_handle_bytes(w4a4_mx_handle_t h);

/* Eq. 11 in MXFP4: arguments, layouts, ownership and errors exactly as w4a4_linear_forward.  Two kernels are
 * enqueued on `stream`; no host synchronisation. */
w4a4_status_t w4a4_mx_linear_forward(w4a4_mx_handle_t h, const void* X, int M, int expert_id, int timestep_bin,
                                     const float* clip_table, void* Y, void* stream);
/* Its two halves, for per-kernel timing. */
w4a4_status_t w4a4_mx_quantize_activations(w4a4_mx_handle_t h, const void* X, int M, int expert_id, int timestep_bin,
                                           const float* clip_table, void* stream);
w4a4_status_t w4a4_mx_gemm_from_workspace(w4a4_mx_handle_t h, int M, int expert_id, void* Y, void* stream);
/* Clipping-ratio search (Eq. 8-10) for the MXFP4 variant: arguments, behaviour and errors exactly as
 * w4a4_clip_search.  Because the shared exponent is a floor of log2(rho * block maximum), candidates act only
 * through the blocks whose threshold they move across a power of two. */
w4a4_status_t w4a4_mx_clip_search(w4a4_mx_handle_t h, const void* const* X_samples, const void* const* Yref_samples,
                                  int num_samples, int M, int expert_id, int timestep_bin, const float* candidates,
                                  int num_candidates, float* clip_table, double* errors_out, int* best_out,
                                  void* stream);
/* Parity tap: runs the activation kernel and decodes its outputs: codes device uint8 [M, K] (E2M1 codes),
 * exps device uint8 [M, K/32] (E8M0), T device FP32 [M, r] or NULL. */
w4a4_status_t w4a4_mx_debug_quantize(w4a4_mx_handle_t h, const void* X, int M, int expert_id, int timestep_bin,
                                     const float* clip_table, uint8_t* codes, uint8_t* exps, float* T, void* stream);

/* Two consecutive layers of the MXFP4 variant in one call (Sec. III: the FFN, whose second linear reads the
 * activation of the first; Eq. 7 and Eq. 8-9 for both).  `up` runs as w4a4_mx_linear_forward does, except that the
 * epilogue of its GEMM applies bias and output activation, rounds to BF16 and then does the work of `down`'s
 * activation kernel on the result (smoothing by `down`'s lambda, MXFP4 codes and block exponents with `down`'s clip
 * ratio, the low-rank projection onto `down`'s L1) into a second workspace of the context; `down`'s GEMM reads it
 * from there and writes Y.  The intermediate activation [M, up.N] is never stored.  The result equals
 * w4a4_mx_linear_forward(up) followed by w4a4_mx_linear_forward(down) except for the summation order of T.
 *   X  device BF16 [M, up.K], 16-byte aligned;  Y  device BF16 [M, down.N], 16-byte aligned;  both handles on the
 *   same context with up.N == down.K; expert_id, timestep_bin, clip_table as for the single layer (each layer
 *   reads its own entry).  M > 128 (else W4A4_ERR_SHAPE).  Asynchronous on `stream`; errors as the single layer. */
w4a4_status_t w4a4_mx_ffn_forward(w4a4_mx_handle_t up, w4a4_mx_handle_t down, const void* X, int M, int expert_id,
                                  int timestep_bin, const float* clip_table, void* Y, void* stream);
/* Parity tap: decodes what the last w4a4_mx_ffn_forward left for `down` in the second workspace: codes device
 * uint8 [M, down.K], exps device uint8 [M, down.K/32], T device FP32 [M, down.r] or NULL. */
w4a4_status_t w4a4_mx_debug_fused_input(w4a4_mx_handle_t down, int M, uint8_t* codes, uint8_t* exps, float* T, void* stream);

/*
 * GPTQ on the residual branch (Sec. III-B: the residual weights are quantized with GPTQ, not round-to-nearest;
 * the algorithm is Frantar et al., 2023, Algorithm 1 with the Cholesky reformulation of its Sec. 4).  Offline
 * step: produces the qweight / wscale inputs of w4a4_pack_weights for one expert of one layer.
 *   R       device FP32 [K, N] row-major: residual weights, input channels along rows.
 *   Xhat    device BF16 bit patterns [M_cal, K]: smoothed calibration activations; H = Xhat^T Xhat in FP64; or NULL
 *   H_in    device FP64 [K, K] row-major, symmetric: the statistic itself (only its upper triangle is read); or NULL.
 *           Exactly one of Xhat and H_in is given (else W4A4_ERR_INVALID_ARG); M_cal is ignored with H_in.
 *   percdamp  damping: percdamp * mean(diag H) is added to the diagonal (after dead channels, H_kk = 0, were given
 *           H_kk = 1 and zero weights).  >= 0.
 *   codes   device int8 [K, N] (values in [-8, 7]) and scales device FP32 [K/64, N]: outputs.  Group scale =
 *           FP32(max |w| / 7) over the group's 64 error-compensated input channels when the sweep enters the group;
 *           code = round-half-even(w / scale) clamped to [-8, 7]; an all-zero group has scale 0 and codes 0.
 *   workspace  device memory for the temporaries (FP64 copies of the statistic, its factor, the weights), 256-byte
 *           aligned, at least w4a4_gptq_workspace_bytes(K, N, M_cal) bytes (M_cal = 0 with H_in), owned by the caller
 *           and free again when the call returns; too small or misaligned returns W4A4_ERR_INVALID_ARG.  NULL: the
 *           call allocates and frees the same amount itself (W4A4_ERR_ALLOC if that fails).
 * All arithmetic is FP64.  K a multiple of 64, K <= 16384, N <= 65536, M_cal <= 2^20 (else W4A4_ERR_SHAPE;
 * w4a4_gptq_workspace_bytes returns 0 for such a shape).  The workspace is about 16 K^2 + 8 K N + 8 M_cal K bytes.
 * Runs on `stream` and returns after the stream has drained.  A statistic that is not positive definite after
 * damping returns W4A4_ERR_INVALID_ARG with the outputs undefined.  No context is needed.
 */
size_t w4a4_gptq_workspace_bytes(int K, int N, int M_cal);
w4a4_status_t w4a4_gptq_quantize(int device, const float* R, const uint16_t* Xhat, int M_cal, const double* H_in,
                                 int K, int N, double percdamp, int8_t* codes, float* scales, void* workspace,
                                 size_t workspace_bytes, void* stream);

/* The statistic of GPTQ over several batches of calibration tokens (Sec. III-B; Frantar et al., 2023, Sec. 3: the
 * layer-wise Hessian is a sum over calibration inputs): H += Xhat^T Xhat in FP64.  Xhat device BF16 bit patterns
 * [M_cal, K]; H device FP64 [K, K] row-major, zeroed by the caller before the first batch.  Only the tiles on and above
 * the diagonal are updated (64 x 128 granularity), which is the part w4a4_gptq_quantize reads from H_in.  K a multiple
 * of 64, K <= 16384, 0 < M_cal <= 2^20 (W4A4_ERR_SHAPE).  Allocates and frees 8 * min(M_cal, 4096) * K bytes
 * (W4A4_ERR_ALLOC); runs on `stream` and returns after it has drained. */
w4a4_status_t w4a4_gptq_accumulate(int device, const uint16_t* Xhat, int M_cal, int K, double* H, void* stream);

/* The same step on the MX variant's grid (Sec. III-B with the MXFP4 quantizer of w4a4_mx_pack_weights; OCP MX v1.0):
 * codes device uint8 [K, N] (E2M1: bit 3 sign, bits 0-2 magnitude index of {0, 0.5, 1, 1.5, 2, 3, 4, 6}) and exps
 * device uint8 [K/32, N] (E8M0: scale 2^(e - 127)).  A block's exponent is floor(log2 max|w|) - 2 over its 32
 * error-compensated input channels when the sweep enters the block (an all-zero block: 0); elements are the nearest
 * E2M1 value of w / 2^e, ties to the even code, saturating at 6, sign bit from the compensated weight.  Everything
 * else (arguments, workspace, limits, errors) as w4a4_gptq_quantize. */
w4a4_status_t w4a4_mx_gptq_quantize(int device, const float* R, const uint16_t* Xhat, int M_cal, const double* H_in,
                                    int K, int N, double percdamp, uint8_t* codes, uint8_t* exps, void* workspace,
                                    size_t workspace_bytes, void* stream);

/* Synchronises the context's device and reports W4A4_ERR_TIMEOUT if any kernel launched through this
 * context gave up on a bounded wait since the last query (the flag is cleared), else W4A4_OK / ERR_CUDA.
 * The flag is sticky on the device: from the moment one CTA records a give-up, every other CTA of that kernel
 * and every GEMM launched on the context afterwards leaves its pipeline at its next wait (within microseconds)
 * and stores nothing more, so outputs enqueued between the failure and this query are undefined.  A caller
 * that must trust an output queries the status after the work that produced it; a W4A4_ERR_TIMEOUT answer means
 * "re-run everything enqueued since the last W4A4_OK".  The context stays usable after the query. */
w4a4_status_t w4a4_query_status(w4a4_ctx_t ctx);

/* Test hooks for the two failure paths that no healthy run reaches (no counterpart in the paper).
 * w4a4_debug_wait_probe enqueues a one-warp kernel that waits, with the library's bounded wait, for an mbarrier
 * phase nobody completes; it uses no copy engine, tensor core or tensor memory.  After limit_ns (1 .. 1e8, else
 * W4A4_ERR_INVALID_ARG) the wait gives up and sets the context's device error word exactly as a stuck GEMM
 * pipeline would: the next w4a4_query_status returns W4A4_ERR_TIMEOUT, the one after it W4A4_OK.
 * w4a4_debug_fail_allocation_after(n) makes the (n + 1)-th device allocation that w4a4_ctx_create,
 * w4a4_ctx_enable_host_io, w4a4_pack_weights, w4a4_mx_pack_weights or the clip-ratio searches attempt from now on
 * fail once, as if cudaMalloc had refused it (the call then returns W4A4_ERR_ALLOC after releasing what it had
 * allocated); n < 0 disarms.  Process-wide; not for use while other threads call the library.
 * w4a4_debug_stalled_gemm runs the GEMM of w4a4_gemm_from_workspace (its parity-tap instantiation) on whatever the
 * workspace holds, with the wait limit set to limit_ns (1 .. 1e8) and with one operand stage (number stall_stage >= 0
 * of every CTA's sequence) never loaded: the consumers of that stage run into the limit, every role of the CTA
 * leaves through the kernel's common tail (error word, a drain period for copies in flight, release of tensor
 * memory), and Y is left partly written.  The next w4a4_query_status returns W4A4_ERR_TIMEOUT, and the context must
 * compute correctly afterwards.  Nothing faults or traps.
 * w4a4_debug_set_tile_order forces the width, in 128-channel column tiles, of the super-columns in which the INT4
 * GEMM walks its output tiles (all row blocks of one super-column before the next; the width is otherwise chosen so
 * that a super-column's weight bytes take about two ninths of the L2); 0 restores the automatic choice.  Results do
 * not depend on it; the tests use it to run every shape of the order on small layers. */
w4a4_status_t w4a4_debug_wait_probe(w4a4_ctx_t ctx, uint64_t limit_ns, void* stream);
w4a4_status_t w4a4_debug_set_tile_order(w4a4_ctx_t ctx, int super_column_tiles);
w4a4_status_t w4a4_debug_stalled_gemm(w4a4_handle_t h, int M, int expert_id, void* Y, int stall_stage,
                                      uint64_t limit_ns, void* stream);
void w4a4_debug_fail_allocation_after(int n);

/* Bytes of device memory held by a handle / a context. */
size_t w4a4_handle_bytes(w4a4_handle_t h);
size_t w4a4_ctx_bytes(w4a4_ctx_t ctx);

const char* w4a4_status_string(w4a4_status_t s);

#ifdef __cplusplus
}
#endif
#endif /* W4A4_H_ */
