/*
 * lite3r.h -- C ABI of the FP8 Sparse Linear Attention (SLA) forward for NVIDIA B200 (sm_100a).
 *
 * The library computes  A_SLA(Q,K,V) = A_sparse(Q,K,V) + Proj(A_lin(Q,K,V))   (paper Eq. 1, Algorithm 1)
 * in its block-level form: tokens of one (batch, head) are cut into blocks of `block` tokens; Q and K are
 * mean-pooled per block, every (query-block, key-block) pair is ranked by the pooled score and classified
 * critical / marginal / negligible; critical pairs run exact softmax attention on the e4m3 operands, marginal
 * pairs feed a linear-attention branch through the feature map phi, negligible pairs are skipped.
 *
 * General conventions (all entry points)
 *   - Every pointer inside a struct or argument marked DEVICE is a CUDA device pointer owned by the caller.
 *     The library never allocates or frees device memory, never synchronises the device and never changes
 *     the current device; work is enqueued on `stream` and the call returns.
 *   - Shapes: B = batch, H = heads, N = tokens, D = head_dim (must be 64), Bs = block (64 or 128),
 *     Nb = ceil(N / Bs).  The last block of a sequence may be ragged; only its valid tokens take part.
 *   - Errors detected on the host (bad argument, unsupported shape, short workspace, failed launch) are
 *     returned as a lite3r_status; nothing has been enqueued when a call returns an error other than
 *     LITE3R_ERR_CUDA.  There is no CPU fallback: without a CUDA device the compute calls fail.
 *   - Same inputs give bit-identical outputs (fixed reduction orders, no floating-point atomics).
 */
#ifndef LITE3R_H
#define LITE3R_H

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define LITE3R_API __attribute__((visibility("default")))
#else
#define LITE3R_API
#endif

typedef enum {
  LITE3R_OK = 0,
  LITE3R_ERR_INVALID_ARG = 1, /* null pointer, non-positive size, misaligned pointer or stride, fraction outside [0,1] */
  LITE3R_ERR_UNSUPPORTED = 2, /* head_dim != 64, block not in {64,128}, unknown dtype / phi, device not compute capability 10.x */
  LITE3R_ERR_WORKSPACE = 3,   /* workspace_bytes smaller than the size query reports */
  LITE3R_ERR_CUDA = 4,        /* a CUDA call failed; see lite3r_last_cuda_error() */
  LITE3R_ERR_TIMEOUT = 5      /* a bounded device-side wait expired (reported through device_status) */
} lite3r_status;

typedef enum { LITE3R_F32 = 0, LITE3R_BF16 = 1, LITE3R_F16 = 2 } lite3r_dtype;

/* Feature map of the linear branch.  SOFTMAX: softmax over the head_dim components (the benchmark
 * contract).  ELU1: ELU(x)+1 (the feature map Algorithm 1 prints). */
typedef enum { LITE3R_PHI_SOFTMAX = 0, LITE3R_PHI_ELU1 = 1 } lite3r_phi;

typedef struct {
  int batch, heads, tokens, head_dim, block;
} lite3r_shape;

/* A source tensor [B, H, N, D] with arbitrary batch/head/token strides (in elements) and contiguous D.
 * DEVICE pointer, 16-byte aligned; every stride must be a multiple of 8 elements. */
typedef struct {
  const void* ptr;
  lite3r_dtype dtype;
  long long stride_b, stride_h, stride_n;
} lite3r_tensor;

/* A block-quantised tensor (all DEVICE pointers, caller-allocated, 16-byte aligned):
 *   codes  uint8 [B, H, Nb*Bs, D]  e4m3 codes, rows past N are zero
 *   scales fp32  [B, H, Nb]        one scale per (b, h, token-block) tile of Bs x D:  x ~= value(code) * scale
 *   colsum int32 [B, H, Nb, D]     per-tile column sums of the code values in units of 2^-9 (exact integers);
 *                                  the pooled block mean is colsum * 2^-9 * scale / valid_tokens. */
typedef struct {
  unsigned char* codes;
  float* scales;
  int* colsum;
} lite3r_fp8;

/* The block plan (all DEVICE pointers, caller-allocated):
 *   cls       int8  [B, H, Nb, Nb]    class of key block j for query block i: 0 negligible, 1 marginal, 2 critical
 *                                     (a plan handed to lite3r_sla_forward must hold no other value: the forward reads
 *                                     bit 0 as "marginal"; the array is read in aligned 32-bit words, so up to three
 *                                     bytes next to either end of it are touched and must be addressable)
 *   crit_idx  int32 [B, H, Nb, k_crit] key-block indices of the critical blocks of row i, ascending
 *   marg_idx  int32 [B, H, Nb, k_marg] same for the marginal blocks; may be NULL (not written then)
 * k_crit / k_marg / k_neg are the per-row counts lite3r_plan_sizes reports. */
typedef struct {
  signed char* cls;
  int* crit_idx;
  int* marg_idx;
  int k_crit, k_marg, k_neg;
} lite3r_plan;

/* Byte sizes of the three buffers of a lite3r_fp8 for `shape`.  Host-only. */
LITE3R_API lite3r_status lite3r_fp8_sizes(const lite3r_shape* shape, size_t* codes_bytes, size_t* scales_bytes,
                               size_t* colsum_bytes);

/* Per-row class counts and plan buffer sizes.  Counts: k_crit = 0 if crit == 0, else
 * min(Nb, max(1, floor(crit*Nb + 0.5))); k_neg = min(Nb - k_crit, floor(neg*Nb + 0.5)); k_marg is the rest
 * (the row-wise TopKMask of Algorithm 1 with its keep ratio, applied to blocks).  Host-only. */
LITE3R_API lite3r_status lite3r_plan_sizes(const lite3r_shape* shape, double crit, double neg, size_t* cls_bytes,
                                size_t* crit_idx_bytes, size_t* marg_idx_bytes, int* k_crit, int* k_marg,
                                int* k_neg);

/* Bytes of scratch lite3r_sla_forward needs for `shape` and these fractions when the caller passes a plan
 * (lite3r_forward_workspace) and when it passes plan == NULL and the plan is built inside the workspace
 * (lite3r_forward_workspace_planned: the class matrix and the critical lists come on top).  Host-only. */
LITE3R_API lite3r_status lite3r_forward_workspace(const lite3r_shape* shape, double crit, double neg, size_t* bytes);
LITE3R_API lite3r_status lite3r_forward_workspace_planned(const lite3r_shape* shape, double crit, double neg, size_t* bytes);

/* Scaled FP8 quantisation (paper appendix "Scaled FP8 Quantization" with the epsilon of "Implementation
 * Details"), one scale per (b, h, token-block) tile, all in fp32:
 *   amax = max |x| over the valid tokens of the tile;  scale = (amax + 1e-8) / 448;
 *   code = e4m3_round_to_nearest_even(clamp(x / scale, -448, 448))   (IEEE fp32 division).
 * Writes out.codes, out.scales and, when out.colsum is not NULL, out.colsum.  x: DEVICE source tensor. */
LITE3R_API lite3r_status lite3r_quantize_fp8(const lite3r_tensor* x, const lite3r_shape* shape, lite3r_fp8 out, void* stream);

/* The same quantisation (same passage of the paper) of Q, K and V of one attention call in a single launch: three
 * lite3r_quantize_fp8 calls cost three launches and three pipeline fill/drain phases, which is a large share of
 * the time at small sequence lengths.  The three sources must have the same dtype (else LITE3R_ERR_UNSUPPORTED);
 * strides may differ.  Results are identical to three separate calls. */
LITE3R_API lite3r_status lite3r_quantize_fp8_qkv(const lite3r_tensor* q, const lite3r_tensor* k, const lite3r_tensor* v,
                                      const lite3r_shape* shape, lite3r_fp8 q_out, lite3r_fp8 k_out, lite3r_fp8 v_out,
                                      void* stream);

/* Pooled scores and row-wise top-k classification (the score and TopKMask steps of Algorithm 1 on block means):
 *   s_ij = mean_i(q_hat) . mean_j(k_hat) / sqrt(D), means over valid tokens of the dequantised blocks;
 *   row i ranks j by (s_ij descending, j ascending); first k_crit critical, last k_neg negligible.
 * Scores are evaluated from the exact integer column sums in fp64, so the ranking can differ from an exact
 * evaluation only between scores that agree to ~1e-15 relative.  q, k need scales and colsum only.
 * Fills plan->cls, plan->crit_idx, plan->marg_idx (if not NULL) and the three counts. */
LITE3R_API lite3r_status lite3r_sla_plan(const lite3r_fp8* q, const lite3r_fp8* k, const lite3r_shape* shape, double crit,
                              double neg, lite3r_plan* plan, void* stream);

/* The SLA forward (Eq. 1; Algorithm 1: Require q, k, v, the projection and the keep ratio; Ensure the output).
 *   sparse branch: per query token, softmax over exactly the valid keys of the critical blocks of
 *     (q_hat . k_hat) / sqrt(D), times v_hat;
 *   linear branch: (phi(q_hat) G_i) / (phi(q_hat) . zeta_i) with G_i = sum over marginal blocks of
 *     phi(K_j)^T V_j and zeta_i = sum of phi(K_j)^T 1;
 *   out = sparse + linear @ proj[h]   (no bias).
 * plan: the block plan of lite3r_sla_plan, or NULL: then the plan is computed first, inside the workspace, from the
 *   column sums of q and k and the fractions crit / neg (the row-wise TopKMask of Algorithm 1 on block means), exactly
 *   as lite3r_sla_plan would; with a plan, crit and neg are not used (the plan's counts are).
 * proj: DEVICE fp32 [H, D, D] row-major [d_in][d_out]; proj_head_stride in elements (D*D for per-head
 * matrices, 0 for one matrix shared by all heads).
 * out: DEVICE [B, H, N, D] of out_dtype (LITE3R_F32, LITE3R_BF16 or LITE3R_F16: the fp32 result rounded to nearest
 * even on the way out) with the given strides in elements (multiples of 4 for fp32, of 8 for the 16-bit types;
 * pointer 16-byte aligned); rows past N are not written.
 * workspace: DEVICE, 256-byte aligned, at least lite3r_forward_workspace() bytes (lite3r_forward_workspace_planned()
 * when plan is NULL); its contents are scratch.
 * device_status: optional DEVICE int, set non-zero by the kernels if a bounded wait expired (read it after
 * synchronising); may be NULL.
 * Value range: the probabilities, phi(K), the per-block summaries and the dequantised V travel as fp16 / bf16 inside
 * (the accumulation is fp32).  |v_hat| must stay below 65504 and the per-block sums |sum_s phi(k_s)[d] v_s[e]| below
 * ~6e4 (softmax phi: |v| up to ~900 per component is always safe; ELU+1: |k| |v| summed over a block must stay below
 * that); beyond it the result holds inf / NaN and device_status stays 0.  Inputs of unit to tens magnitude, the
 * range of transformer activations, are far inside. */
LITE3R_API lite3r_status lite3r_sla_forward(const lite3r_fp8* q, const lite3r_fp8* k, const lite3r_fp8* v, const float* proj,
                                 long long proj_head_stride, const lite3r_shape* shape, double crit, double neg,
                                 lite3r_phi phi, const lite3r_plan* plan, void* out, lite3r_dtype out_dtype,
                                 long long out_stride_b, long long out_stride_h, long long out_stride_n,
                                 void* workspace, size_t workspace_bytes, int* device_status, void* stream);

/* lite3r_sla_forward in two halves, for callers that overlap the block plan with the part of the forward that does
 * not depend on it.  The per-key-block summaries of the linear branch (Algorithm 1's feature map, KV summary and
 * normaliser, with proj folded in) and the fp16 copy of V read only K, V and proj, so
 *     lite3r_sla_forward_begin  (stream A)  may run beside  lite3r_sla_plan  (stream B),
 * and lite3r_sla_forward_finish (aggregation over the marginal blocks, attention, linear output, sum) follows once
 * both have completed (the caller orders the streams).  begin followed by finish on one stream is exactly
 * lite3r_sla_forward: same kernels, same results.  begin takes the three class counts lite3r_plan_sizes reports
 * (they depend on the fractions only) and clears *device_status; finish does not clear it.  Both use the same
 * workspace, which must not be touched in between.  Both need the caller's plan (finish its contents, begin only the
 * three counts).  Arguments otherwise as for lite3r_sla_forward. */
LITE3R_API lite3r_status lite3r_sla_forward_begin(const lite3r_fp8* k, const lite3r_fp8* v, const float* proj,
                                       long long proj_head_stride, const lite3r_shape* shape, lite3r_phi phi,
                                       int k_crit, int k_marg, int k_neg, void* workspace, size_t workspace_bytes,
                                       int* device_status, void* stream);
LITE3R_API lite3r_status lite3r_sla_forward_finish(const lite3r_fp8* q, const lite3r_fp8* k, const lite3r_fp8* v,
                                        const lite3r_shape* shape, lite3r_phi phi, const lite3r_plan* plan,
                                        void* out, lite3r_dtype out_dtype, long long out_stride_b,
                                        long long out_stride_h, long long out_stride_n, void* workspace,
                                        size_t workspace_bytes, int* device_status, void* stream);

/* The same forward for callers that cannot provide scratch memory.  (The paper has no counterpart: this entry
 * point exists for deployments, not for the method.)
 *
 * Who needs it: code that is not allowed to allocate device memory where it calls the library -- a plug-in that
 * lives inside another runtime's pre-planned memory arena, a latency-critical loop that must stay away from the
 * allocator, a process whose memory pool is already sized to the last byte.  Such a caller still owns the inputs
 * and the output, but has nowhere to take the workspace of lite3r_sla_forward from.
 *
 * Here the scratch is a fixed array of LITE3R_STATIC_SCRATCH_BYTES inside the library image.  Arguments are those
 * of lite3r_sla_forward without workspace / workspace_bytes and without the fractions (a plan must be passed), and
 * the results are identical.
 *   - First call per device: CUDA loads device code lazily, so the array takes its 32 MiB of device memory when this
 *     entry point is first called on a device (that call also looks up the array's address; the device must be
 *     current).  Make that call during start-up, outside any stream capture, while memory can still be taken; it may
 *     fail with a CUDA out-of-memory error if 32 MiB are not free.  A call that is then refused for its size (or any
 *     valid call) serves as this warm-up.  Every later call on that device allocates and frees nothing, on the device
 *     or through any library; the memory stays with the process until it exits.
 *   - Limit: if lite3r_forward_workspace() for this shape exceeds LITE3R_STATIC_SCRATCH_BYTES the call returns
 *     LITE3R_ERR_WORKSPACE and enqueues nothing: 32 MiB hold 1344 (batch x head x block) tiles at block 64 (e.g. two
 *     heads of an 8-frame 10992-token sequence) and 1012 tiles at block 128; use lite3r_sla_forward with your own
 *     buffer for larger problems.
 *   - All calls on a device share the one array, and it keeps whatever the previous call left there.  The forward
 *     overwrites every scratch element before reading it, so nothing needs clearing between calls, but two calls
 *     whose kernels may overlap on the GPU (different streams, no ordering between them) race on the array:
 *     serialise them. */
#define LITE3R_STATIC_SCRATCH_BYTES (32u << 20)
LITE3R_API lite3r_status lite3r_sla_forward_static_scratch(const lite3r_fp8* q, const lite3r_fp8* k, const lite3r_fp8* v,
                                                const float* proj, long long proj_head_stride,
                                                const lite3r_shape* shape, lite3r_phi phi, const lite3r_plan* plan,
                                                void* out, lite3r_dtype out_dtype, long long out_stride_b,
                                                long long out_stride_h, long long out_stride_n, int* device_status,
                                                void* stream);

/* ---- The FP8 linear layer in front of the attention (paper Sec. 3.4 Eq. 2; appendix "Per-Tensor Dynamic Scaling" and
 * Algorithm 2 "FP8 fake-quantised linear" in its deployed form: the operands really are e4m3, nothing is faked). ---- */

/* Scaled FP8 quantisation with one scale per row of a matrix [rows, cols] (appendix "Per-Tensor Dynamic Scaling"):
 * per token for an activation matrix, per output row for a weight matrix.  In fp32, as for the block quantiser:
 *   scale_i = (max_j |x_ij| + 1e-8) / 448;  code_ij = e4m3_round_to_nearest_even(clamp(x_ij / scale_i, -448, 448)).
 * x: DEVICE, fp32 or bf16, 16-byte aligned, row_stride in elements (a multiple of 8, >= cols); cols a multiple of 16.
 * codes: DEVICE uint8 [rows, cols] contiguous; scales: DEVICE fp32 [rows]. */
LITE3R_API lite3r_status lite3r_quantize_rows_fp8(const void* x, lite3r_dtype dtype, long long row_stride, int rows, int cols,
                                       unsigned char* codes, float* scales, void* stream);

/* y = x_q W_q^T + b (the linear transformation of Algorithm 2) on quantised operands, e4m3 x e4m3 with fp32
 * accumulation on the tensor cores:  y[n][o] = x_scales[n] * w_scales[o] * sum_k value(x_codes[n][k]) value(w_codes[o][k]) + bias[o].
 * x_codes: DEVICE uint8 [rows, d_in]; w_codes: DEVICE uint8 [d_out, d_in] (the layout of an nn.Linear weight);
 * bias: DEVICE fp32 [d_out] or NULL.  d_in must be a multiple of 128 and d_out of 64 (else LITE3R_ERR_UNSUPPORTED).
 * y: DEVICE [rows, d_out] of y_dtype (fp32, bf16 or fp16), row pitch y_stride elements (a multiple of 8), 16-byte
 * aligned.  device_status as for lite3r_sla_forward (cleared by the call). */
LITE3R_API lite3r_status lite3r_linear_fp8(const unsigned char* x_codes, const float* x_scales, const unsigned char* w_codes,
                                const float* w_scales, const float* bias, int rows, int d_in, int d_out, void* y,
                                lite3r_dtype y_dtype, long long y_stride, int* device_status, void* stream);

/* The qkv projection of an attention block as that FP8 linear layer (Eq. 2), with the block quantiser of
 * lite3r_quantize_fp8 fused into its epilogue: Q, K and V never exist in 16 or 32 bits in memory, they leave the
 * kernel as the lite3r_fp8 tensors lite3r_sla_plan / lite3r_sla_forward take.
 * x_codes: [B * N, d_model] (token-major; row b * N + n); w_codes: [3 * H * 64, d_model] with the output rows ordered
 * (q | k | v) x head x 64; bias [3 * H * 64] or NULL; shape gives B, H, N and the block size; H must be even.
 * Each output value is formed in fp32 (accumulator x (x_scale * w_scale) + bias) and each (b, h, token-block) tile of
 * it is then quantised by the rule of lite3r_quantize_fp8 (tile maximum over the valid tokens, scale, codes, column
 * sums when colsum is not NULL; v_out.colsum may be NULL).  Because the fp32 accumulation order of the tensor cores is
 * not that of an fp64 evaluation, a value may fall on the other side of an e4m3 rounding boundary than a reference
 * computed in higher precision would put it: scales agree to within a few fp32 ulps and codes except for a small
 * fraction that differ by one code step. */
LITE3R_API lite3r_status lite3r_qkv_project_fp8(const unsigned char* x_codes, const float* x_scales, const unsigned char* w_codes,
                                     const float* w_scales, const float* bias, const lite3r_shape* shape, int d_model,
                                     lite3r_fp8 q_out, lite3r_fp8 k_out, lite3r_fp8 v_out, int* device_status,
                                     void* stream);

/* ---- Training side of the linear-branch projection, the only tensor the method trains (Sec. 3.3 "selective
 * freezing": gradients are applied only to the linear-branch projection layers; Sec. 3.5 Eq. 3). ---- */

/* Bytes of scratch that cover lite3r_sla_linear_branch, lite3r_mse_distill and lite3r_proj_lin_backward for `shape`
 * and these fractions.  Host-only. */
LITE3R_API lite3r_status lite3r_train_workspace(const lite3r_shape* shape, double crit, double neg, size_t* bytes);

/* The linear branch alone, before the projection: O_lin = (phi(q_hat) G_i) / (phi(q_hat) . zeta_i) over the marginal
 * blocks of the given plan (Algorithm 1's feature map, KV summary, normaliser and linear output; zero where a query
 * block has no marginal block).  The forward proper never forms it (the projection is folded into the summaries);
 * the backward of the projection needs it.  Arguments as for lite3r_sla_forward with a plan; out may be fp32, bf16
 * or fp16 (lite3r_proj_lin_backward takes bf16, contiguous [B, H, N, 64]).  workspace: lite3r_train_workspace() bytes. */
LITE3R_API lite3r_status lite3r_sla_linear_branch(const lite3r_fp8* q, const lite3r_fp8* k, const lite3r_fp8* v,
                                       const lite3r_shape* shape, lite3r_phi phi, const lite3r_plan* plan, void* out,
                                       lite3r_dtype out_dtype, long long out_stride_b, long long out_stride_h,
                                       long long out_stride_n, void* workspace, size_t workspace_bytes,
                                       int* device_status, void* stream);

/* One module's term of the partial attention distillation loss (Eq. 3):
 *   *loss = mean over all `count` elements of (student - teacher)^2   (the teacher is a constant: stop-gradient),
 *   grad  = 2 (student - teacher) / count, the gradient with respect to the student's attention output, as bf16.
 * student, teacher: DEVICE, contiguous, fp32 or bf16 (same dtype), 16-byte aligned; count a multiple of 8.
 * grad: DEVICE bf16 [count] or NULL; loss: DEVICE double.  The sum is accumulated in fp64 in a fixed order.
 * workspace: DEVICE, 256-byte aligned, at least 16 KiB. */
LITE3R_API lite3r_status lite3r_mse_distill(const void* student, const void* teacher, lite3r_dtype dtype, long long count,
                                 void* grad, double* loss, void* workspace, size_t workspace_bytes, void* stream);

/* Gradient of the loss with respect to the projection: the output is out = sparse + O_lin @ proj[h] (Algorithm 1's
 * last step), hence  d_proj[h] = sum over batch and tokens of O_lin[b,h,t,:]^T d_out[b,h,t,:]   ([d_in][d_out] like proj).
 * o_lin, d_out: DEVICE bf16, contiguous [B, H, N, 64]; d_proj: DEVICE fp32 [H, 64, 64] (overwritten).
 * A contraction over the tokens on the tensor cores (bf16 operands, fp32 accumulation), partial sums added in a fixed
 * order.  workspace: lite3r_train_workspace() bytes. */
LITE3R_API lite3r_status lite3r_proj_lin_backward(const void* o_lin, const void* d_out, const lite3r_shape* shape, float* d_proj,
                                       void* workspace, size_t workspace_bytes, int* device_status, void* stream);

/* Text for a status code; the last CUDA error code (cudaError_t as int) recorded by this thread. */
LITE3R_API const char* lite3r_status_string(lite3r_status status);
LITE3R_API int lite3r_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* LITE3R_H */
