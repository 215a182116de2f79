// Shared host/device helpers of the lite3r library (internal; the public surface is include/lite3r.h).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_fp8.h>
#include <stdint.h>

#include "lite3r.h"

namespace lite3r {

constexpr int kHeadDim = 64;
// One row of per-key-block linear-branch summaries: (H_j W)^T as [e][d] (4096 values) followed by z_j[d] (64).
constexpr int kSummaryRow = kHeadDim * kHeadDim + kHeadDim;

// Records a CUDA error for lite3r_last_cuda_error(); returns LITE3R_ERR_CUDA if err != cudaSuccess.
lite3r_status record_cuda(cudaError_t err);
// Counts one enqueued kernel launch and returns the launch's error state as a status.
lite3r_status after_launch();

// Benchmark stage timing: records event `idx` (0..7; stage s runs from event 2s to 2s+1) on `stream` when
// profiling is enabled.
void profile_mark(int idx, cudaStream_t stream);
bool profile_enabled();

// Number of SMs of the current device (looked up once per device).
lite3r_status sm_count(int* count);
// LITE3R_OK when the current device is a compute-capability 10.x part (the kernels are sm_100a code), else
// LITE3R_ERR_UNSUPPORTED (looked up once per device).
lite3r_status check_device();

// Sets a kernel's dynamic shared-memory limit, but only when this launch needs more than any earlier launch of that
// kernel on that device asked for (the limits already set are remembered per kernel and device; guarded by a mutex so
// that concurrent callers cannot leave a smaller limit behind).
lite3r_status ensure_smem_limit(const void* kernel, int bytes);
template <typename K>
lite3r_status ensure_dynamic_smem(K* kernel, int bytes) {
  return ensure_smem_limit(reinterpret_cast<const void*>(kernel), bytes);
}

inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

struct Counts {
  int k_crit, k_marg, k_neg;
};
Counts class_counts(int nb, double crit, double neg);

// Value of an e4m3 code in units of 2^-9 (an exact integer, |v| <= 448 * 512).
__device__ __forceinline__ int e4m3_units(uint32_t code) {
  const int e = (code >> 3) & 0xF;
  const int m = code & 0x7;
  const int mag = e ? ((8 | m) << (e - 1)) : m;
  return (code & 0x80) ? -mag : mag;
}

// Decodes four packed e4m3 codes to fp32 (exact).
__device__ __forceinline__ void e4m3x4_to_float(uint32_t packed, float out[4]) {
  const __half2_raw lo = __nv_cvt_fp8x2_to_halfraw2(static_cast<__nv_fp8x2_storage_t>(packed & 0xFFFFu), __NV_E4M3);
  const __half2_raw hi = __nv_cvt_fp8x2_to_halfraw2(static_cast<__nv_fp8x2_storage_t>(packed >> 16), __NV_E4M3);
  const float2 a = __half22float2(__half2(lo));
  const float2 b = __half22float2(__half2(hi));
  out[0] = a.x;
  out[1] = a.y;
  out[2] = b.x;
  out[3] = b.y;
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  return v;
}

// Kernel launchers (one per translation unit).  All enqueue on `stream` and return a status.
// One launch quantises `count` (1..3) source tensors of the same shape and dtype.
lite3r_status launch_quantize(const lite3r_tensor* const* x, const lite3r_fp8* out, int count, const lite3r_shape& s,
                              cudaStream_t stream);
void set_plan_variant(int variant);  // test hook, see lite3r_plan_variant
lite3r_status launch_plan(const lite3r_fp8& q, const lite3r_fp8& k, const lite3r_shape& s, const Counts& c,
                          const lite3r_plan& plan, cudaStream_t stream);

struct ForwardArgs {
  lite3r_fp8 q, k, v;
  const float* proj;
  long long proj_head_stride;
  lite3r_shape s;
  int phi;
  lite3r_plan plan;
  void* out;
  int out_dtype;
  long long out_stride_b, out_stride_h, out_stride_n;
  int linear_only;      // 1: the sparse branch is left out (the output is the linear branch through proj alone)
  int plan_inside;      // 1: the plan is built in the workspace from q/k column sums and the fractions below
  double crit, neg;
  void* workspace;
  size_t workspace_bytes;
  int* device_status;
};
struct AttentionLaunch {
  lite3r_shape shape;
  const uint8_t* q_codes;
  const uint8_t* k_codes;
  const float* q_scales;
  const float* k_scales;
  const float* v_scales;
  const __half* v16;          // [tiles*Bs][64] dequantised V as fp16
  const __nv_bfloat16* g16;   // [tiles][64][64] aggregated projected summaries, [e][d]
  const float* zeta;          // [tiles][64]
  const int* crit_idx;
  int k_crit, k_marg, phi;
  void* out;
  int out_dtype;  // lite3r_dtype of the output
  long long out_stride_b, out_stride_h, out_stride_n;
  int* device_status;
  bool overlap_prior;  // the preceding launch in the stream produced only g16 and zeta: start before it has finished
};
lite3r_status launch_attention(const AttentionLaunch& a, cudaStream_t stream);
void set_attention_plain_stores(int on);  // test hook, see lite3r_attention_plain_stores

// Per-key-block summaries ((H_j W)^T | z_j) in bf16, one kSummaryRow-wide row per (b, h, key block).
lite3r_status launch_summary(const lite3r_fp8& k, const lite3r_fp8& v, const float* proj, long long proj_head_stride,
                             const lite3r_shape& s, int phi, __nv_bfloat16* hws, __half* v16, int* device_status,
                             cudaStream_t stream);

// Marginal aggregation G_i = sum over marginal j of the summary rows, as a 0/1-mask GEMM on tensor cores.
lite3r_status launch_aggregate(const __nv_bfloat16* hws, const signed char* cls, const lite3r_shape& s, int nb,
                               __nv_bfloat16* g16, float* zeta, int* device_status, cudaStream_t stream);

// TMA descriptor of a row-major 2-D tensor [rows][inner] (row pitch = inner * elem_bytes, a multiple of 16 bytes)
// with a box of box_inner x box_rows elements.
lite3r_status make_tensor_map_2d(CUtensorMap* map, CUtensorMapDataType type, int elem_bytes, const void* base,
                                 uint64_t inner, uint64_t rows, uint32_t box_inner, uint32_t box_rows,
                                 CUtensorMapSwizzle swizzle);

// The FP8 linear layer in front of the attention (linear.cu).
lite3r_status launch_rowquant(const void* x, int dtype, long long row_stride, int rows, int cols, uint8_t* codes,
                              float* scales, cudaStream_t stream);
lite3r_status launch_linear_fp8(const uint8_t* x_codes, const float* x_scales, const uint8_t* w_codes,
                                const float* w_scales, const float* bias, int rows, int d_in, int d_out, void* y,
                                int y_dtype, long long y_stride, int* device_status, cudaStream_t stream);
lite3r_status launch_qkv_project(const uint8_t* x_codes, const float* x_scales, const uint8_t* w_codes,
                                 const float* w_scales, const float* bias, const lite3r_shape& s, int d_model,
                                 const lite3r_fp8* out, int* device_status, cudaStream_t stream);

// The same for a 3-D tensor [planes][rows][inner] with a box of box_inner x box_rows x 1 (rows past the end of a plane
// are zero-filled, so a tile never runs into the next plane).
lite3r_status make_tensor_map_4d(CUtensorMap* map, CUtensorMapDataType type, const void* base, const uint64_t dims[4],
                                 const uint64_t strides_bytes[3], const uint32_t box[4], CUtensorMapSwizzle swizzle);
lite3r_status make_tensor_map_3d(CUtensorMap* map, CUtensorMapDataType type, int elem_bytes, const void* base,
                                 uint64_t inner, uint64_t rows, uint64_t planes, uint32_t box_inner, uint32_t box_rows,
                                 CUtensorMapSwizzle swizzle);

// Training side of the linear-branch projection (train.cu).
size_t train_workspace_bytes(const lite3r_shape& s);
lite3r_status launch_fill_identity(float* dst, cudaStream_t stream);
lite3r_status launch_mse_distill(const void* student, const void* teacher, int dtype, size_t count, __nv_bfloat16* grad,
                                 double* loss, double* partials, cudaStream_t stream);
lite3r_status launch_proj_lin_backward(const __nv_bfloat16* o_lin, const __nv_bfloat16* d_out, const lite3r_shape& s,
                                       float* d_w, float* partials, int* device_status, cudaStream_t stream);

lite3r_status launch_wait_expiry_probe(int* status, unsigned long long limit_ns, cudaStream_t stream);
size_t forward_workspace_bytes(const lite3r_shape& s, const Counts& c, bool plan_inside = false);
// byte offsets of the workspace's parts: summaries, aggregates, zeta, fp16 V, class bytes, critical lists
void forward_workspace_offsets(const lite3r_shape& s, const Counts& c, bool plan_inside, size_t* offsets);
// phases: 1 = the plan-independent first part, 2 = the rest, 3 = the whole forward
lite3r_status launch_forward(const ForwardArgs& a, int phases, cudaStream_t stream);

}  // namespace lite3r
