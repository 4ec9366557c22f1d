/*
 * libkop — fused pointwise+reduction segments for NVIDIA B200 (sm_100a), C ABI.
 *
 * These are the memory-bound sub-kernels a model compiler emits between vendor
 * GEMM / convolution calls: bias / scale / activation / residual chains that end in a
 * row- or channel-wise reduction. The paper's problem formulation (Definition 1)
 * keeps the vendor calls fixed and speeds up exactly these sub-kernels; its fusion
 * agent's technique list and planner strategies 8-9 name the classes implemented
 * here (fused softmax, single-pass LayerNorm / RMSNorm, activation + bias fusion,
 * residual + norm, reduction + pointwise, LogSumExp reductions). The paper never
 * prints their formulas; each entry point below states the one it computes.
 *
 * Conventions shared by every entry point
 *   pointers   All data / parameter / output / workspace pointers are DEVICE pointers
 *              on the current device, owned by the caller. Shape arrays passed by
 *              pointer (strides of kop_bn_relu_avgpool) are HOST pointers.
 *   dtype      `dtype` is the element type of the data tensors (inputs and the main
 *              output): KOP_F32, KOP_BF16 or KOP_F16 (IEEE binary16; results beyond
 *              65504 in magnitude are stored as infinity). Parameter vectors (bias, gamma, beta,
 *              scale, shift, weight) are fp32; the *_ex entry points also take them in the
 *              data type; statistics outputs (mean, rstd, pooled, loss) are
 *              always fp32. All arithmetic is fp32; the only rounding to
 *              bf16 / fp16 is the final store (round to nearest even), as the paper's
 *              numerics rule requires (accumulate in fp32, cast only at the store).
 *   strides    In elements. The innermost stride is 1 by contract; a row stride
 *              must be >= the row length.
 *   alignment  16-byte-aligned bases, row strides and row lengths take the 128-bit
 *              vector kernels; anything else runs a GPU kernel of the same arithmetic
 *              with narrower accesses (the cross-entropy, softmax and GroupNorm entry
 *              points keep 128-bit accesses for any length and alignment). There is no
 *              CPU path.
 *   aliasing   Where stated, the output may be exactly the input (same pointer and
 *              stride). Any other overlap returns KOP_ERR_BAD_ALIAS when detectable
 *              and is undefined otherwise.
 *   stream     Work is enqueued on `stream`; nothing synchronises, allocates or frees,
 *              and the library keeps no state between calls (kop_mlp_handle_* aside,
 *              which only wrap cuBLAS handle creation).
 *   threads    Any entry point may be called from several host threads at once, on the
 *              same or different streams, as long as concurrent calls do not share an
 *              output, a workspace or a kop_mlp_handle (kop_ce_loss_rowwise_static's
 *              built-in scratch counts as a shared workspace). Results do not depend on
 *              what else runs.
 *   errors     Static validation (the paper's Gate 1: structural checks before any
 *              numerics) runs first and touches no CUDA API: a call that fails
 *              validation launches nothing. rows == 0 (or N == 0) returns KOP_OK
 *              without a launch. Launch failures are reported as KOP_ERR_CUDA.
 *              Device code never traps or asserts.
 */
#ifndef KOP_H_
#define KOP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Same type as the CUDA runtime's cudaStream_t (a pointer to CUstream_st). */
typedef struct CUstream_st* kop_stream_t;

typedef enum {
    KOP_OK = 0,
    KOP_ERR_NULL_POINTER = 1,
    KOP_ERR_BAD_SHAPE = 2,
    KOP_ERR_BAD_STRIDE = 3,
    KOP_ERR_UNSUPPORTED_DTYPE = 4,
    KOP_ERR_MISALIGNED = 5,
    KOP_ERR_BAD_ALIAS = 6,
    KOP_ERR_WORKSPACE_TOO_SMALL = 7,
    KOP_ERR_UNSUPPORTED_DEVICE = 8,
    KOP_ERR_CUDA = 9,
    KOP_ERR_CUBLAS = 10
} kop_status_t;

typedef enum { KOP_F32 = 0, KOP_BF16 = 1, KOP_F16 = 2 } kop_dtype_t;

/* Library version as major * 10000 + minor * 100 + patch. */
int kop_version(void);

/* Static, NUL-terminated name of a status code ("KOP_OK", ...); never NULL. */
const char* kop_status_string(kop_status_t status);

/*
 * Row softmax of a scaled, biased matrix ("fused softmax", planner strategy 9):
 *   z[i,j] = x[i,j] * scale + bias[j];  y[i,j] = exp(z[i,j] - max_j z) / sum_j exp(z[i,j] - max_j z)
 * x, y: [rows, cols] of `dtype`, row strides x_row_stride / y_row_stride.
 * bias: fp32 [cols], or NULL for no bias; -inf entries mask a column (output 0);
 *       a row whose z are all -inf yields NaN (the definition's 0/0).
 * y may alias x exactly. Element size must divide the alignment of x / y
 * (else KOP_ERR_MISALIGNED).
 */
kop_status_t kop_softmax_scale_bias(const void* x, const float* bias, void* y,
                                    int64_t rows, int64_t cols,
                                    int64_t x_row_stride, int64_t y_row_stride,
                                    float scale, kop_dtype_t dtype, kop_stream_t stream);

/*
 * Softmax variants (planner strategy 9 "fused softmax" / "online softmax"; the LogSoftmax row of the results
 * table): the same z = x * scale + bias, then
 *   log_output == 0:  y = exp(z - m) / sum_j exp(z_j - m)            (as kop_softmax_scale_bias)
 *   log_output != 0:  y = z - m - ln sum_j exp(z_j - m)               (log-softmax)
 * with m = max_j z_j, and, when causal_period > 0, causal rows: row i keeps the columns
 * j <= (i mod causal_period) + (cols - causal_period) and every other column counts as z = -inf (output 0, or
 * -inf in the log form). causal_period == cols is the square mask of attention scores stored as
 * [batch * heads * cols, cols]; a smaller period leaves a prefix of cols - causal_period columns visible to every
 * row (queries behind a cache). 0 <= causal_period <= cols, else KOP_ERR_BAD_SHAPE. Everything else as in
 * kop_softmax_scale_bias.
 */
kop_status_t kop_softmax_opts(const void* x, const float* bias, void* y, int64_t rows, int64_t cols,
                              int64_t x_row_stride, int64_t y_row_stride, float scale, int log_output,
                              int64_t causal_period, kop_dtype_t dtype, kop_stream_t stream);

/*
 * Bias-add, tanh-form GELU, residual add and LayerNorm in one pass (fusion agent:
 * "activation + bias fusion" and "residual + norm: one kernel, one memory pass";
 * codegen agent: "single-pass LayerNorm instead of 3 kernels"):
 *   u = x + bias;  g = 0.5 u (1 + tanh(sqrt(2/pi) (u + 0.044715 u^3)));  v = residual + g
 *   mu = mean_j v;  var = mean_j (v - mu)^2 (biased);  r = 1 / sqrt(var + eps)
 *   y = (v - mu) * r * gamma + beta;   mean[i] = mu;  rstd[i] = r
 * x, residual, y: [rows, hidden] of `dtype`; bias, gamma, beta: fp32 [hidden];
 * mean, rstd: fp32 [rows], each may be NULL. v is kept in fp32 (never rounded).
 * y may alias x or residual exactly.
 */
kop_status_t kop_bias_gelu_residual_layernorm(const void* x, const void* residual,
                                              const float* bias, const float* gamma,
                                              const float* beta, void* y,
                                              float* mean, float* rstd,
                                              int64_t rows, int64_t hidden,
                                              int64_t x_row_stride, int64_t res_row_stride,
                                              int64_t y_row_stride, float eps,
                                              kop_dtype_t dtype, kop_stream_t stream);

/*
 * The same segment with the error-function GELU (the exact form, as in BERT- and ViT-style blocks; one of
 * the coverage variants of the benchmark segment):
 *   g = 0.5 u (1 + erf(u / sqrt 2)),  u = x + bias;  everything else as in kop_bias_gelu_residual_layernorm.
 */
kop_status_t kop_bias_erfgelu_residual_layernorm(const void* x, const void* residual,
                                                 const float* bias, const float* gamma,
                                                 const float* beta, void* y,
                                                 float* mean, float* rstd,
                                                 int64_t rows, int64_t hidden,
                                                 int64_t x_row_stride, int64_t res_row_stride,
                                                 int64_t y_row_stride, float eps,
                                                 kop_dtype_t dtype, kop_stream_t stream);

/*
 * Inference BatchNorm (pre-folded per-channel affine), ReLU and global average pool
 * (fusion agent: "reduction + pointwise"; the BN / pooling epilogues of the paper's
 * CNN models, next to preserved cuDNN convolutions):
 *   a[n,c,h,w] = max(x[n,c,h,w] * scale[c] + shift[c], 0)   (NaN stays NaN)
 *   pooled[n,c] = (1 / (H W)) sum_{h,w} a[n,c,h,w]          (sum of unrounded fp32 a)
 * x, y: indexed [n,c,h,w], of `dtype`; x_strides / y_strides are HOST arrays of 4 element
 * strides (for n, c, h, w) and must both describe the same one of two dense layouts:
 * contiguous NCHW ({C*H*W, H*W, W, 1}) or channels-last, i.e. NHWC memory
 * ({H*W*C, 1, W*C, C}); strides of extent-1 dimensions are ignored; anything else
 * returns KOP_ERR_BAD_STRIDE. scale, shift: fp32 [C]; pooled: fp32 [N, C].
 * y may alias x exactly. Each pooled value is summed by one CTA in a fixed order.
 */
kop_status_t kop_bn_relu_avgpool(const void* x, const float* scale, const float* shift,
                                 void* y, float* pooled,
                                 int64_t N, int64_t C, int64_t H, int64_t W,
                                 const int64_t x_strides[4], const int64_t y_strides[4],
                                 kop_dtype_t dtype, kop_stream_t stream);

/*
 * Row-wise cross-entropy in a single pass over the logits ("LogSumExp reductions";
 * planner strategy 8 "single-pass reductions"; "online softmax"):
 *   loss[i] = ln sum_j exp(z[i,j]) - z[i, labels[i]];   *mean_loss = (1/rows) sum_i loss[i]
 * logits: [rows, vocab] of `dtype`, row stride row_stride; labels: int32 [rows];
 * loss: fp32 [rows]; mean_loss: fp32 [1] or NULL; bad_label_count: int32 [1] or NULL.
 * A label outside [0, vocab) gives loss NaN for that row and is counted in
 * *bad_label_count (then *mean_loss is NaN). The mean is summed in a fixed order:
 * results are bit-identical run to run.
 * Non-finite logits follow the max-shifted definition lse = m + ln sum_j exp(z_j - m): -inf entries
 * are ordinary (they add 0); a NaN anywhere in a row, or a +inf logit (exp(inf - inf)), makes that
 * row's loss NaN (and with it the mean); a row of nothing but -inf is NaN too. Other rows are unaffected.
 * workspace: device scratch of at least kop_ce_loss_rowwise_workspace_bytes() bytes,
 * 16-byte aligned, contents irrelevant on entry (the call clears what it needs on
 * `stream`); calls sharing one workspace must not overlap on the GPU.
 */
kop_status_t kop_ce_loss_rowwise(const void* logits, const int32_t* labels,
                                 float* loss, float* mean_loss, int32_t* bad_label_count,
                                 int64_t rows, int64_t vocab, int64_t row_stride,
                                 void* workspace, size_t workspace_bytes,
                                 kop_dtype_t dtype, kop_stream_t stream);

/* Scratch bytes kop_ce_loss_rowwise needs for this shape (0 on invalid arguments). */
size_t kop_ce_loss_rowwise_workspace_bytes(int64_t rows, int64_t vocab, kop_dtype_t dtype);

/*
 * kop_ce_loss_rowwise for callers that cannot allocate. (The paper has no counterpart: this is a
 * packaging variant of the entry point above, same arithmetic, same kernels.)
 *
 * Who needs it: code that has no allocator to turn to at the point of the call — a plug-in inside
 * another runtime's operator that cannot reach that runtime's memory pool (and where a raw
 * cudaMalloc would synchronise the device and take memory the pool does not know about), a server
 * whose memory plan is frozen after start-up, a C caller on a latency-critical path. Instead of a
 * caller-supplied workspace, the scratch of the mean reduction (tickets and per-group partials) is
 * a fixed device array inside the library: 65,552 bytes that every GPU which loads the library
 * holds until the process exits.
 *
 * Arguments, outputs, results and error behaviour are those of kop_ce_loss_rowwise without the
 * workspace pair, with these additions:
 *   limit     rows <= kop_ce_loss_rowwise_static_max_rows() (1,048,576). More rows return
 *             KOP_ERR_WORKSPACE_TOO_SMALL before anything is launched; use the workspace variant.
 *             Like every entry point it checks all of its arguments before its first CUDA call.
 *   set-up    The first call on each device looks up the device address of the built-in array
 *             (once per device, with that device current). Make that first call outside any
 *             stream capture. The call itself never calls cudaMalloc, cudaFree or any allocating
 *             library routine; it clears the tickets it needs on `stream`.
 *   sharing   Every call on a device uses the same array, which keeps the previous call's
 *             contents. Calls that may overlap on the GPU (different streams, different threads)
 *             race on it and give wrong means: serialise them, or use kop_ce_loss_rowwise with
 *             one workspace per concurrent call.
 */
kop_status_t kop_ce_loss_rowwise_static(const void* logits, const int32_t* labels,
                                        float* loss, float* mean_loss, int32_t* bad_label_count,
                                        int64_t rows, int64_t vocab, int64_t row_stride,
                                        kop_dtype_t dtype, kop_stream_t stream);

/* Largest `rows` kop_ce_loss_rowwise_static accepts. */
int64_t kop_ce_loss_rowwise_static_max_rows(void);

/*
 * kop_ce_loss_rowwise with ignore_index, label smoothing and all three reductions (coverage variant of the
 * same segment; the reductions are the "none" / "mean" / "sum" forms of the loss):
 *   loss[i] = (1 - s) (lse_i - z[i, label_i]) + s (lse_i - (1/vocab) sum_j z[i,j]),  s = label_smoothing in [0, 1)
 * Rows whose label equals ignore_index get loss 0, are not read, and do not count;
 * *sum_loss = sum of the counted losses (0 when no row counts); *mean_loss = *sum_loss / *counted_rows (NaN
 * when no row counts); both come from one fixed-order sum, so they are bit-identical run to run. A label
 * outside [0, vocab) that is not ignore_index is a bad label as above (sum and mean NaN). loss: fp32 [rows]
 * ("none"); mean_loss, sum_loss: fp32 [1] or NULL; counted_rows: int32 [1] or NULL. Workspace as for
 * kop_ce_loss_rowwise (same size function).
 */
kop_status_t kop_ce_loss_rowwise_opts(const void* logits, const int32_t* labels,
                                      float* loss, float* mean_loss, float* sum_loss,
                                      int32_t* bad_label_count,
                                      int32_t* counted_rows, int64_t rows, int64_t vocab, int64_t row_stride,
                                      int32_t ignore_index, float label_smoothing,
                                      void* workspace, size_t workspace_bytes,
                                      kop_dtype_t dtype, kop_stream_t stream);

/*
 * Residual add + LayerNorm, the fusion agent's "residual + norm" pattern without a bias / activation
 * prologue ("x = residual + x; x = LayerNorm(x): one kernel, one memory pass"), or plain LayerNorm:
 *   v = x + residual (residual may be NULL: v = x);  y = (v - mean v) / sqrt(var v + eps) * gamma + beta
 * Same statistics outputs, strides and aliasing rules as kop_bias_gelu_residual_layernorm.
 */
kop_status_t kop_residual_layernorm(const void* x, const void* residual,
                                    const float* gamma, const float* beta, void* y,
                                    float* mean, float* rstd, int64_t rows, int64_t hidden,
                                    int64_t x_row_stride, int64_t res_row_stride, int64_t y_row_stride,
                                    float eps, kop_dtype_t dtype, kop_stream_t stream);

/*
 * RMSNorm (fusion agent: "normalization fusion (LayerNorm/RMSNorm sequences)"):
 *   y[i,j] = x[i,j] / sqrt(mean_j x[i,j]^2 + eps) * weight[j]
 * x, y: [rows, hidden] of `dtype`; weight: fp32 [hidden]. y may alias x exactly.
 */
kop_status_t kop_rmsnorm(const void* x, const float* weight, void* y,
                         int64_t rows, int64_t hidden,
                         int64_t x_row_stride, int64_t y_row_stride,
                         float eps, kop_dtype_t dtype, kop_stream_t stream);

/*
 * Residual add and RMSNorm in one pass (fusion agent: "residual + norm: one kernel, one memory pass", for the
 * RMSNorm sequences of pre-norm transformer blocks: the add that ends one sub-layer and the norm that opens
 * the next):
 *   v = x + residual;   h = v (rounded to `dtype`);   y = v / sqrt(mean_j v^2 + eps) * weight
 * The normalisation uses the unrounded fp32 v. x, residual, h, y: [rows, hidden] of `dtype`; weight: fp32
 * [hidden]. h and y may each be x or residual exactly; h and y must be different tensors. Against
 * kop_residual_add followed by kop_rmsnorm this saves one write-then-read of h (4 instead of 5 tensor passes).
 */
kop_status_t kop_residual_rmsnorm(const void* x, const void* residual, const float* weight, void* h, void* y,
                                  int64_t rows, int64_t hidden, int64_t x_row_stride, int64_t res_row_stride,
                                  int64_t h_row_stride, int64_t y_row_stride, float eps, kop_dtype_t dtype,
                                  kop_stream_t stream);

/*
 * The LayerNorm and RMSNorm entry points above with the parameter vectors in either fp32 or the data type
 * (models held in bf16 / fp16 keep their norm weights in that type; 16-bit parameters also halve the
 * parameter bytes every row re-reads from L1, which is what bounds the LayerNorm kernel). param_dtype is
 * KOP_F32 or equal to `dtype`; anything else returns KOP_ERR_UNSUPPORTED_DTYPE. A 16-bit parameter is
 * widened exactly to fp32 and the arithmetic is the same.
 *
 * kop_layernorm_ex: `prologue` selects what precedes the normalisation:
 *   0  v = residual + gelu_tanh(x + bias)      (kop_bias_gelu_residual_layernorm)
 *   1  v = x + residual                        (kop_residual_layernorm with a residual; bias ignored)
 *   2  v = x                                   (kop_residual_layernorm without; residual and bias ignored)
 *   3  v = residual + gelu_erf(x + bias)       (kop_bias_erfgelu_residual_layernorm)
 * bias, gamma, beta: [hidden] of param_dtype. Everything else as in those entry points.
 *
 * kop_rmsnorm_ex: residual == NULL gives kop_rmsnorm (h and the two residual strides are ignored), otherwise
 * kop_residual_rmsnorm. weight: [hidden] of param_dtype.
 */
kop_status_t kop_layernorm_ex(const void* x, const void* residual, const void* bias, const void* gamma,
                              const void* beta, void* y, float* mean, float* rstd, int64_t rows, int64_t hidden,
                              int64_t x_row_stride, int64_t res_row_stride, int64_t y_row_stride, float eps,
                              int prologue, kop_dtype_t dtype, kop_dtype_t param_dtype, kop_stream_t stream);
kop_status_t kop_rmsnorm_ex(const void* x, const void* residual, const void* weight, void* h, void* y, int64_t rows,
                            int64_t hidden, int64_t x_row_stride, int64_t res_row_stride, int64_t h_row_stride,
                            int64_t y_row_stride, float eps, kop_dtype_t dtype, kop_dtype_t param_dtype,
                            kop_stream_t stream);

/*
 * SwiGLU epilogue of a preserved GEMM (fusion agent: "activation fusion
 * (GELU/SiLU/ReLU)"; codegen agent: keep the matmul as a library call and fuse only
 * the epilogue):
 *   out[i,j] = gate / (1 + exp(-gate)) * up,  gate = gate_up[i,j],  up = gate_up[i, inter + j]
 * gate_up: [rows, 2*inter] of `dtype` (two contiguous halves per row), row stride
 * in_row_stride; out: [rows, inter], row stride out_row_stride. No aliasing.
 */
kop_status_t kop_silu_mul(const void* gate_up, void* out, int64_t rows, int64_t inter,
                          int64_t in_row_stride, int64_t out_row_stride,
                          kop_dtype_t dtype, kop_stream_t stream);

/*
 * kop_silu_mul for the interleaved layout [g0, u0, g1, u1, ...] (gate_up: [rows, 2*inter]):
 *   out[i,j] = silu(gate_up[i, 2j]) * gate_up[i, 2j+1]
 */
kop_status_t kop_silu_mul_interleaved(const void* gate_up, void* out, int64_t rows, int64_t inter,
                                      int64_t in_row_stride, int64_t out_row_stride,
                                      kop_dtype_t dtype, kop_stream_t stream);

/*
 * Residual add (fusion agent: "pointwise + pointwise: load once, store once"):
 *   out[i,j] = a[i,j] + b[i,j]
 * a, b, out: [rows, cols] of `dtype`. out may alias a or b exactly.
 */
kop_status_t kop_residual_add(const void* a, const void* b, void* out,
                              int64_t rows, int64_t cols,
                              int64_t a_row_stride, int64_t b_row_stride,
                              int64_t out_row_stride, kop_dtype_t dtype, kop_stream_t stream);

/*
 * Row scaling, the O(N^2) form of diag(a) * B that the paper's L1-012 case study (Appendix "Generated
 * Kernel Examples", diagonal matrix multiply) replaces a cuBLAS GEMM with:
 *   out[i,j] = a[i] * b[i,j]
 * a: [rows] of `dtype`; b, out: [rows, cols] of `dtype`. out may alias b exactly; a must not overlap out.
 */
kop_status_t kop_row_scale(const void* a, const void* b, void* out, int64_t rows, int64_t cols,
                           int64_t b_row_stride, int64_t out_row_stride, kop_dtype_t dtype,
                           kop_stream_t stream);

/*
 * Mat-vec with a bias sum, the form the paper's L2-018 case study reduces Linear -> Sum -> Max -> Mean ->
 * LogSumExp -> LogSumExp to (sum_j (x W^T + b)_j = x . colsum(W) + sum(b); the later reductions act on a
 * single element per row and are identities):
 *   out[i] = sum_k x[i,k] * w[k] + b_sum
 * x: [rows, k] of `dtype`; w: fp32 [k] (the caller's precomputed column sums); out: fp32 [rows]. x is read
 * once; products and sums are fp32.
 */
kop_status_t kop_matvec_bias(const void* x, const float* w, float b_sum, float* out, int64_t rows,
                             int64_t k, int64_t x_row_stride, kop_dtype_t dtype, kop_stream_t stream);

/*
 * GroupNorm with optional per-channel affine and activation (the per-kernel results table's InstanceNorm
 * row, L1-034, and GroupNorm row, L1-035, which the paper's system left at its fallback; fusion agent:
 * normalisation followed by a pointwise op is one load and one store). For image n and group g over the
 * (C / groups) * H * W elements of that group:
 *   mu = mean(x), var = mean((x - mu)^2)              (biased variance)
 *   y[n,c,h,w] = act((x[n,c,h,w] - mu) / sqrt(var + eps) * gamma[c] + beta[c])
 * groups == C is InstanceNorm; groups == 1 normalises whole images. act: 0 identity, 1 ReLU (NaN passes),
 * 2 SiLU v / (1 + exp(-v)).
 * x, y: [N, C, H, W] contiguous NCHW of `dtype`; y may be x exactly. gamma, beta: fp32 [C], each may be NULL
 * (1 and 0). mean, rstd: fp32 [N, groups] outputs, each may be NULL. Statistics are fp32, accumulated as
 * (count, mean, M2) triples merged pairwise in a fixed order, so results do not depend on scheduling.
 * Errors: groups must divide C; act outside 0..2 or eps < 0 or NaN is KOP_ERR_BAD_SHAPE. N == 0 is KOP_OK.
 */
kop_status_t kop_groupnorm_act(const void* x, const float* gamma, const float* beta, void* y,
                               float* mean, float* rstd, int64_t N, int64_t C, int64_t H, int64_t W,
                               int64_t groups, float eps, int act, kop_dtype_t dtype, kop_stream_t stream);

/*
 * Per-channel affine, optional ReLU and windowed 2-D pooling in one pass over NCHW planes (the BatchNorm ->
 * ReLU -> Pool epilogues after the preserved convolutions of the paper's CNN problems; "Pool" is the most
 * frequent non-vendor operation of its level-2 / level-3 result tables; fusion agent: pointwise + reduction):
 *   a[n,c,i,j] = x[n,c,i,j] * scale[c] + shift[c]  (scale and shift both NULL: a = x), ReLU if relu != 0
 *   OH = floor((H + 2 ph - kh) / sh) + 1,  OW = floor((W + 2 pw - kw) / sw) + 1
 *   mode 0: y[n,c,oi,oj] = max of a over rows oi*sh - ph + [0, kh), columns oj*sw - pw + [0, kw) that lie
 *           inside the image (padding never wins; a NaN inside the window gives NaN)
 *   mode 1: y = (sum of a over the same positions) / (kh * kw)      (padding counts in the divisor)
 * x: [N, C, H, W] contiguous, y: [N, C, OH, OW] contiguous, both of `dtype`; scale, shift: fp32 [C] or both
 * NULL. Requires ph <= kh / 2 and pw <= kw / 2 (every window touches the image), H + 2 ph >= kh,
 * W + 2 pw >= kw; otherwise KOP_ERR_BAD_SHAPE. The activation a is never written to memory. y must not
 * overlap x.
 */
kop_status_t kop_affine_relu_pool2d(const void* x, const float* scale, const float* shift, void* y,
                                    int64_t N, int64_t C, int64_t H, int64_t W, int kh, int kw, int sh, int sw,
                                    int ph, int pw, int mode, int relu, kop_dtype_t dtype, kop_stream_t stream);

/*
 * Bias + activation epilogue (fusion agent: "activation + bias fusion"; the pointwise tail that follows a
 * preserved Linear / GEMM call in most of the paper's level-2 problems), one load and one store:
 *   u = x[i,j] + bias[j]   (bias NULL: u = x[i,j]);   y[i,j] = act(u)
 * act: 0 identity, 1 relu (NaN stays NaN), 2 leaky_relu (u > 0 ? u : alpha u), 3 gelu, tanh form,
 *      4 gelu, erf form, 5 silu u / (1 + exp(-u)), 6 sigmoid, 7 tanh, 8 mish u tanh(ln(1 + exp(u))),
 *      9 hardswish u min(max(u + 3, 0), 6) / 6, 10 elu (u > 0 ? u : alpha (exp(u) - 1)).
 * alpha is used by leaky_relu and elu only. x, y: [rows, cols] of `dtype`; bias: fp32 [cols] or NULL.
 * y may alias x exactly.
 */
kop_status_t kop_bias_act(const void* x, const float* bias, void* y, int64_t rows, int64_t cols,
                          int64_t x_row_stride, int64_t y_row_stride, int act, float alpha,
                          kop_dtype_t dtype, kop_stream_t stream);

/*
 * Pointwise epilogue chain: the general form of the "several pointwise operations after a vendor GEMM" class
 * (the paper's L2-064 case, whose operations are not listed; fusion agent: "pointwise + pointwise: load once,
 * store once"), one pass:
 *   u = (x[i,j] + bias[j]) * scale + residual[i,j] * residual_scale     (bias / residual NULL: term absent)
 *   u = min(max(u, clamp_lo), clamp_hi)     (NaN stays NaN; -INFINITY / +INFINITY switch a side off)
 *   y[i,j] = act(u)                          (act and alpha as in kop_bias_act)
 * x, residual, y: [rows, cols] of `dtype`; bias: fp32 [cols]. clamp_lo <= clamp_hi, else KOP_ERR_BAD_SHAPE.
 * y may alias x or residual exactly.
 */
kop_status_t kop_epilogue_chain(const void* x, const float* bias, const void* residual, void* y,
                                int64_t rows, int64_t cols, int64_t x_row_stride, int64_t res_row_stride,
                                int64_t y_row_stride, float scale, float residual_scale, float clamp_lo,
                                float clamp_hi, int act, float alpha, kop_dtype_t dtype, kop_stream_t stream);

/*
 * Row reductions (the "Reduction" rows of the paper's result tables and its planner's "single-pass
 * reductions" / "LogSumExp reductions"), one read-only pass:
 *   op 0 sum, 1 mean, 2 max, 3 min, 4 logsumexp = m + ln sum_j exp(x[i,j] - m), m = max_j x[i,j]
 * x: [rows, cols] of `dtype`; out: fp32 [rows]; index: int32 [rows] or NULL, written for max / min only: the
 * position of the first element equal to the result (argmax / argmin). A NaN in a row makes its result NaN;
 * for max / min the index is then the position of the first NaN (a NaN outranks every number). logsumexp
 * of a row of -inf is -inf, a +inf element gives +inf. Sums are fp32 trees in a fixed order; max / min
 * and the indices are exact. cols and rows <= 2^31 - 1. out and index must not overlap x or each other.
 */
kop_status_t kop_reduce_rows(const void* x, float* out, int32_t* index, int64_t rows, int64_t cols,
                             int64_t x_row_stride, int op, kop_dtype_t dtype, kop_stream_t stream);

/*
 * Running sums along each row (the CumSum rows of the paper's per-kernel results table, L1-089 to L1-093:
 * plain, reverse, exclusive and masked cumulative sums; planner strategy "single-pass reductions" applied
 * to a scan). With m[i,k] = 1 when mask is NULL, else (mask[i,k] != 0):
 *   exclusive = 0, reverse = 0:  y[i,j] = sum_{k <= j} x[i,k] m[i,k]
 *   exclusive = 1, reverse = 0:  y[i,j] = sum_{k <  j} x[i,k] m[i,k]      (y[i,0] = 0)
 *   exclusive = 0, reverse = 1:  y[i,j] = sum_{k >= j} x[i,k] m[i,k]
 *   exclusive = 1, reverse = 1:  y[i,j] = sum_{k >  j} x[i,k] m[i,k]      (y[i,cols-1] = 0)
 * x, y: [rows, cols] of `dtype`; mask: uint8 [rows, cols] with row stride mask_row_stride (bytes =
 * elements), or NULL. Sums are fp32 (a tree of partial sums, fixed order: results are bit-identical run
 * to run); a masked-out element contributes 0 even if it is NaN or infinite; a NaN or infinity that is
 * kept affects exactly the outputs whose sums include it. y may alias x exactly; mask must not overlap y.
 * rows <= 2^31 - 1. Nonzero `exclusive` / `reverse` mean "on".
 */
kop_status_t kop_cumsum_rows(const void* x, const unsigned char* mask, void* y, int64_t rows, int64_t cols,
                             int64_t x_row_stride, int64_t mask_row_stride, int64_t y_row_stride,
                             int exclusive, int reverse, kop_dtype_t dtype, kop_stream_t stream);

/*
 * The entry points above with their parameter vectors in fp32 OR in the data type (a model held in bf16 / fp16
 * keeps its biases, folded BatchNorm coefficients and norm weights in that type; the coverage variant "16-bit
 * parameters" of the same segments). param_dtype is KOP_F32 or equal to `dtype`, anything else returns
 * KOP_ERR_UNSUPPORTED_DTYPE; all parameter vectors of one call share it. A 16-bit parameter is widened exactly to
 * fp32 and the arithmetic, the results for fp32 parameters and every other rule are those of the base entry point:
 *   kop_softmax_ex           kop_softmax_scale_bias (log_output == 0 and causal_period == 0) / kop_softmax_opts
 *   kop_bn_relu_avgpool_ex   kop_bn_relu_avgpool      (scale, shift)
 *   kop_groupnorm_act_ex     kop_groupnorm_act        (gamma, beta; each may be NULL)
 *   kop_bias_act_ex          kop_bias_act             (bias; may be NULL)
 *   kop_epilogue_chain_ex    kop_epilogue_chain       (bias; may be NULL)
 *   kop_affine_relu_pool2d_ex  kop_affine_relu_pool2d  (scale, shift; both or neither NULL)
 * Parameter pointers must be aligned to their element size; 16-byte alignment takes the vector kernels.
 */
kop_status_t kop_softmax_ex(const void* x, const void* bias, void* y, int64_t rows, int64_t cols,
                            int64_t x_row_stride, int64_t y_row_stride, float scale, int log_output,
                            int64_t causal_period, kop_dtype_t dtype, kop_dtype_t param_dtype, kop_stream_t stream);
kop_status_t kop_bn_relu_avgpool_ex(const void* x, const void* scale, const void* shift, void* y, float* pooled,
                                    int64_t N, int64_t C, int64_t H, int64_t W, const int64_t x_strides[4],
                                    const int64_t y_strides[4], kop_dtype_t dtype, kop_dtype_t param_dtype,
                                    kop_stream_t stream);
kop_status_t kop_groupnorm_act_ex(const void* x, const void* gamma, const void* beta, void* y, float* mean,
                                  float* rstd, int64_t N, int64_t C, int64_t H, int64_t W, int64_t groups, float eps,
                                  int act, kop_dtype_t dtype, kop_dtype_t param_dtype, kop_stream_t stream);
kop_status_t kop_bias_act_ex(const void* x, const void* bias, void* y, int64_t rows, int64_t cols,
                             int64_t x_row_stride, int64_t y_row_stride, int act, float alpha, kop_dtype_t dtype,
                             kop_dtype_t param_dtype, kop_stream_t stream);
kop_status_t kop_epilogue_chain_ex(const void* x, const void* bias, const void* residual, void* y, int64_t rows,
                                   int64_t cols, int64_t x_row_stride, int64_t res_row_stride, int64_t y_row_stride,
                                   float scale, float residual_scale, float clamp_lo, float clamp_hi, int act,
                                   float alpha, kop_dtype_t dtype, kop_dtype_t param_dtype, kop_stream_t stream);
kop_status_t kop_affine_relu_pool2d_ex(const void* x, const void* scale, const void* shift, void* y, int64_t N,
                                       int64_t C, int64_t H, int64_t W, int kh, int kw, int sh, int sw, int ph,
                                       int pw, int mode, int relu, kop_dtype_t dtype, kop_dtype_t param_dtype,
                                       kop_stream_t stream);

/*
 * Lp normalisation of rows (fusion agent: "normalization fusion", a reduction and the pointwise pass that uses it
 * in one kernel; the vector-norm rows of the paper's level-1 table):
 *   n_i = sum_j |x[i,j]|  (p = 1)   or   sqrt(sum_j x[i,j]^2)  (p = 2);     y[i,j] = x[i,j] / max(n_i, eps)
 * x, y: [rows, cols] of `dtype`; norm_out: fp32 [rows] or NULL, receives n_i (the L1 / L2 norm of every row; a
 * tensor passed as one row gives its Frobenius norm). Sums are fp32 in a fixed order. eps >= 0. A NaN in a row
 * makes its norm and every output of that row NaN; an infinite element gives norm inf and outputs 0 (NaN at the
 * infinite positions). y may alias x exactly; norm_out overlaps neither. rows <= 2^31 - 1.
 */
kop_status_t kop_lp_normalize_rows(const void* x, void* y, float* norm_out, int64_t rows, int64_t cols,
                                   int64_t x_row_stride, int64_t y_row_stride, int p, float eps, kop_dtype_t dtype,
                                   kop_stream_t stream);

/*
 * The pointwise part of one LSTM step (the LSTM models of the paper's level-3 table, L3-035 to L3-038, for
 * which its compiler emitted no kernels and the recurrent layer stayed with the vendor library; here the
 * two gate GEMMs stay with the vendor library and everything after them is one pass). With H = hidden and
 *   a[i, :] = gates[i, :] + gates2[i, :] + bias          (gates2 and bias optional)
 * split into four blocks of H columns in the order input i, forget f, candidate g, output o:
 *   c_out = sigmoid(a_f) * c_prev + sigmoid(a_i) * tanh(a_g)
 *   h_out = sigmoid(a_o) * tanh(c_out)                    (from c_out before it is rounded to `dtype`)
 * gates, gates2: [rows, 4H] of `dtype`, contiguous (the outputs of x W_ih^T and h W_hh^T; pass one and NULL
 * when a single GEMM produced their sum); bias: fp32 [4H] or NULL (b_ih + b_hh); c_prev, h_out, c_out:
 * [rows, H] of `dtype`, contiguous. Arithmetic is fp32. c_out may be c_prev exactly (the state updated in
 * place); otherwise h_out and c_out overlap no input and not each other. hidden <= 2^31 - 1.
 */
kop_status_t kop_lstm_cell(const void* gates, const void* gates2, const float* bias, const void* c_prev,
                           void* h_out, void* c_out, int64_t rows, int64_t hidden, kop_dtype_t dtype,
                           kop_stream_t stream);

/*
 * The pointwise part of one GRU step (the GRU models of the paper's level-3 table, L3-039 to L3-042, which
 * its compiler also left to the vendor library's recurrent layer). With gi = x W_ih^T and gh = h W_hh^T
 * from the two preserved GEMMs, each split into three blocks of H columns in the order reset r, update z,
 * candidate n, and a = gi + bias_i, b = gh + bias_h:
 *   r = sigmoid(a_r + b_r);  z = sigmoid(a_z + b_z);  n = tanh(a_n + r * b_n)
 *   h_out = (1 - z) * n + z * h_prev
 * gi, gh: [rows, 3H] of `dtype`, contiguous; bias_i, bias_h: fp32 [3H] or NULL, independently (they are
 * separate because the candidate's hidden part is gated before the sum); h_prev, h_out: [rows, H] of
 * `dtype`, contiguous. Arithmetic is fp32. h_out may be h_prev exactly (the state updated in place);
 * otherwise it overlaps no input. hidden <= 2^31 - 1.
 */
kop_status_t kop_gru_cell(const void* gi, const void* gh, const float* bias_i, const float* bias_h,
                          const void* h_prev, void* h_out, int64_t rows, int64_t hidden, kop_dtype_t dtype,
                          kop_stream_t stream);

/*
 * Diagnostic for kop_groupnorm_act (no counterpart in the paper): its staged kernel waits for its bulk
 * copies with a bounded number of polls; a CTA whose wait runs out writes nothing, and counts itself here.
 * host_count: HOST pointer, receives the count for the current device since the library was loaded (always
 * 0 on healthy hardware). Blocks until the device is idle (a synchronous copy); not for hot paths.
 */
kop_status_t kop_groupnorm_wait_timeouts(unsigned int* host_count);

/*
 * Transformer MLP segment with the vendor GEMMs preserved between the fused kernels
 * (problem formulation: extern library calls stay fixed; codegen agent: "do not
 * replace cuBLAS"): five operations enqueued on `stream`,
 *   n = rmsnorm(h; rms_weight, eps)            kop_rmsnorm
 *   gu = n * w_gate_up^T                       cuBLAS, [rows, 2*inter]
 *   act = silu(gu[:, :inter]) * gu[:, inter:]  kop_silu_mul
 *   d = act * w_down^T                         cuBLAS, [rows, hidden]
 *   out = h + d                                kop_residual_add
 * h, out: [rows, hidden] contiguous; w_gate_up: [2*inter, hidden]; w_down:
 * [hidden, inter], both row-major (out_features, in_features), all of `dtype`;
 * rms_weight: fp32 [hidden]. GEMMs accumulate in fp32 and store `dtype`.
 * handle: from kop_mlp_handle_create, used by one call at a time.
 * workspace: device scratch of at least kop_rmsnorm_swiglu_residual_workspace_bytes()
 * bytes, 256-byte aligned; holds n, gu, act, d and the cuBLAS workspace, so the call
 * allocates nothing and can be captured into a CUDA graph. out may alias h exactly.
 */
kop_status_t kop_rmsnorm_swiglu_residual(void* handle, const void* h, const float* rms_weight,
                                         const void* w_gate_up, const void* w_down, void* out,
                                         int64_t rows, int64_t hidden, int64_t inter, float eps,
                                         void* workspace, size_t workspace_bytes,
                                         kop_dtype_t dtype, kop_stream_t stream);

/* Scratch bytes kop_rmsnorm_swiglu_residual needs (0 on invalid arguments). */
size_t kop_rmsnorm_swiglu_residual_workspace_bytes(int64_t rows, int64_t hidden, int64_t inter,
                                                   kop_dtype_t dtype);

/*
 * Create / destroy the vendor-GEMM handle used by kop_rmsnorm_swiglu_residual (a
 * cuBLAS handle made by the same cuBLAS this library is linked against, on the current
 * device). Creation allocates; do it outside stream capture. (Part of the preserved
 * vendor-call boundary; the paper has no counterpart beyond "extern_kernels".)
 */
kop_status_t kop_mlp_handle_create(void** handle);
kop_status_t kop_mlp_handle_destroy(void* handle);

/*
 * The same handle around a cuBLAS handle the CALLER owns (problem formulation: the extern library calls and
 * their set-up stay exactly as the surrounding program has them): cublas_handle is a cublasHandle_t created by
 * the caller, on the current device, with the cuBLAS that this library is linked against (a handle from another
 * copy of cuBLAS in the process is undefined). Nothing is created on the device: the call only allocates a
 * few host bytes for the segment's settings. Every kop_rmsnorm_swiglu_residual call sets the handle's stream
 * to its `stream` (and leaves it so), lends it the call's workspace and hands the handle back with cuBLAS's
 * default workspace; its other settings (math mode; pointer mode must be host) are left alone.
 * kop_mlp_handle_destroy frees the wrapper and leaves the caller's cuBLAS handle alive.
 */
kop_status_t kop_mlp_handle_wrap(void* cublas_handle, void** handle);

/*
 * Vendor-library configuration of the segment (the paper's stated future work: besides rewriting the fused
 * kernels, choose how the preserved vendor calls are configured). With enable != 0 the down projection is
 * issued as one cublasLtMatmul with C = h and beta = 1, so that
 *   out = act * w_down^T + h
 * leaves the GEMM's epilogue directly (fp32 sum, one rounding) and neither kop_residual_add nor the
 * intermediate d is used. enable == 0 restores the default five-operation form. The setting belongs to
 * the handle and applies to later kop_rmsnorm_swiglu_residual calls; results differ from the default
 * form by at most one rounding of `dtype`. Calls with out == h keep the default form (the vendor
 * kernel is not used in place). Assess it with the perf gate on whole-segment time.
 */
kop_status_t kop_mlp_handle_set_residual_in_gemm(void* handle, int enable);

#ifdef __cplusplus
}
#endif

#endif /* KOP_H_ */
