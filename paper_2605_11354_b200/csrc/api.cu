// C-ABI entry points of the lite3r library: argument validation, size queries and dispatch.
#include <algorithm>
#include <atomic>
#include <cmath>
#include <mutex>
#include <unordered_map>

#include "common.cuh"
#include "lite3r_debug.h"

namespace lite3r {

static thread_local int g_last_cuda_error = 0;
static std::atomic<long long> g_launches{0};

lite3r_status record_cuda(cudaError_t err) {
  if (err == cudaSuccess) return LITE3R_OK;
  g_last_cuda_error = static_cast<int>(err);
  return LITE3R_ERR_CUDA;
}

lite3r_status after_launch() {
  g_launches.fetch_add(1, std::memory_order_relaxed);
  return record_cuda(cudaGetLastError());
}

// Facts about each device, looked up once (the current device is never changed).
namespace {
constexpr int kMaxDevices = 64;
struct DeviceInfo {
  std::atomic<int> ready{0};
  int sms = 0, cc_major = 0;
};
DeviceInfo g_devices[kMaxDevices];
std::mutex g_device_mutex;

lite3r_status device_info(const DeviceInfo** info, int* device_out = nullptr) {
  int device = 0;
  lite3r_status st = record_cuda(cudaGetDevice(&device));
  if (st != LITE3R_OK) return st;
  if (device < 0 || device >= kMaxDevices) return LITE3R_ERR_UNSUPPORTED;
  DeviceInfo& d = g_devices[device];
  if (d.ready.load(std::memory_order_acquire) == 0) {
    std::lock_guard<std::mutex> lock(g_device_mutex);
    if (d.ready.load(std::memory_order_relaxed) == 0) {
      if ((st = record_cuda(cudaDeviceGetAttribute(&d.sms, cudaDevAttrMultiProcessorCount, device))) != LITE3R_OK) return st;
      if ((st = record_cuda(cudaDeviceGetAttribute(&d.cc_major, cudaDevAttrComputeCapabilityMajor, device))) != LITE3R_OK) return st;
      d.ready.store(1, std::memory_order_release);
    }
  }
  *info = &d;
  if (device_out != nullptr) *device_out = device;
  return LITE3R_OK;
}
}  // namespace

lite3r_status sm_count(int* count) {
  const DeviceInfo* d = nullptr;
  lite3r_status st = device_info(&d);
  if (st != LITE3R_OK) return st;
  *count = d->sms;
  return LITE3R_OK;
}

lite3r_status check_device() {
  const DeviceInfo* d = nullptr;
  lite3r_status st = device_info(&d);
  if (st != LITE3R_OK) return st;
  return d->cc_major == 10 ? LITE3R_OK : LITE3R_ERR_UNSUPPORTED;
}

namespace {
struct SmemLimits {
  int set_bytes[kMaxDevices] = {};
};
std::mutex g_smem_mutex;
std::unordered_map<const void*, SmemLimits> g_smem_limits;
}  // namespace

lite3r_status ensure_smem_limit(const void* kernel, int bytes) {
  const DeviceInfo* d = nullptr;
  int device = 0;
  lite3r_status st = device_info(&d, &device);
  if (st != LITE3R_OK) return st;
  std::lock_guard<std::mutex> lock(g_smem_mutex);
  SmemLimits& limits = g_smem_limits[kernel];
  if (limits.set_bytes[device] >= bytes) return LITE3R_OK;
  st = record_cuda(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
  if (st == LITE3R_OK) limits.set_bytes[device] = bytes;
  return st;
}

static bool g_profile = false;
static cudaEvent_t g_events[8] = {};
static bool g_marked[8] = {};

bool profile_enabled() { return g_profile; }
void profile_mark(int idx, cudaStream_t stream) {
  if (!g_profile) return;
  if (idx == 0)
    for (bool& m : g_marked) m = false;
  if (cudaEventRecord(g_events[idx], stream) == cudaSuccess) g_marked[idx] = true;
}

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver's tensor-map encoder, looked up through the runtime so the library does not link against libcuda.
static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = [] {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult res;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &res) != cudaSuccess ||
        res != cudaDriverEntryPointSuccess)
      ptr = nullptr;
    return reinterpret_cast<EncodeTiledFn>(ptr);
  }();
  return fn;
}

lite3r_status make_tensor_map_2d(CUtensorMap* map, CUtensorMapDataType type, int elem_bytes, const void* base,
                                 uint64_t inner, uint64_t rows, uint32_t box_inner, uint32_t box_rows,
                                 CUtensorMapSwizzle swizzle) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return LITE3R_ERR_CUDA;
  const cuuint64_t dims[2] = {inner, rows};
  const cuuint64_t strides[1] = {inner * static_cast<cuuint64_t>(elem_bytes)};
  const cuuint32_t box[2] = {box_inner, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = fn(map, type, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? LITE3R_OK : LITE3R_ERR_CUDA;
}

lite3r_status make_tensor_map_3d(CUtensorMap* map, CUtensorMapDataType type, int elem_bytes, const void* base,
                                 uint64_t inner, uint64_t rows, uint64_t planes, uint32_t box_inner, uint32_t box_rows,
                                 CUtensorMapSwizzle swizzle) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return LITE3R_ERR_CUDA;
  const cuuint64_t dims[3] = {inner, rows, planes};
  const cuuint64_t strides[2] = {inner * static_cast<cuuint64_t>(elem_bytes),
                                 inner * rows * static_cast<cuuint64_t>(elem_bytes)};
  const cuuint32_t box[3] = {box_inner, box_rows, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  const CUresult r = fn(map, type, 3, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? LITE3R_OK : LITE3R_ERR_CUDA;
}

// Rank-4 map over a tensor whose innermost dimension is contiguous: extents dims[0..3], byte strides of dimensions
// 1..3 (multiples of 16), box of box[0..3] elements.
lite3r_status make_tensor_map_4d(CUtensorMap* map, CUtensorMapDataType type, const void* base, const uint64_t dims[4],
                                 const uint64_t strides_bytes[3], const uint32_t box[4], CUtensorMapSwizzle swizzle) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return LITE3R_ERR_CUDA;
  const cuuint64_t d[4] = {dims[0], dims[1], dims[2], dims[3]};
  const cuuint64_t st[3] = {strides_bytes[0], strides_bytes[1], strides_bytes[2]};
  const cuuint32_t bx[4] = {box[0], box[1], box[2], box[3]};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  const CUresult r = fn(map, type, 4, const_cast<void*>(base), d, st, bx, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle,
                        CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? LITE3R_OK : LITE3R_ERR_CUDA;
}

Counts class_counts(int nb, double crit, double neg) {
  Counts c;
  if (crit == 0.0) {
    c.k_crit = 0;
  } else {
    long long kc = static_cast<long long>(std::floor(crit * nb + 0.5));
    if (kc < 1) kc = 1;
    if (kc > nb) kc = nb;
    c.k_crit = static_cast<int>(kc);
  }
  long long kn = static_cast<long long>(std::floor(neg * nb + 0.5));
  if (kn > nb - c.k_crit) kn = nb - c.k_crit;
  c.k_neg = static_cast<int>(kn);
  c.k_marg = nb - c.k_crit - c.k_neg;
  return c;
}

static lite3r_status check_shape(const lite3r_shape* s) {
  if (s == nullptr) return LITE3R_ERR_INVALID_ARG;
  if (s->batch <= 0 || s->heads <= 0 || s->tokens <= 0) return LITE3R_ERR_INVALID_ARG;
  if (s->head_dim != kHeadDim) return LITE3R_ERR_UNSUPPORTED;
  if (s->block != 64 && s->block != 128) return LITE3R_ERR_UNSUPPORTED;
  const long long rows = static_cast<long long>(s->batch) * s->heads * ceil_div(s->tokens, s->block);
  if (rows > 0x7FFFFFFFLL / 4) return LITE3R_ERR_UNSUPPORTED;  // tile ids are 32-bit
  return LITE3R_OK;
}

static lite3r_status check_fractions(double crit, double neg) {
  if (!(crit >= 0.0 && crit <= 1.0) || !(neg >= 0.0 && neg <= 1.0)) return LITE3R_ERR_INVALID_ARG;
  return LITE3R_OK;
}

static bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

static lite3r_status check_fp8(const lite3r_fp8* t, bool need_codes, bool need_colsum) {
  if (t == nullptr || t->scales == nullptr) return LITE3R_ERR_INVALID_ARG;
  if (need_codes && (t->codes == nullptr || !aligned(t->codes, 16))) return LITE3R_ERR_INVALID_ARG;
  if (need_colsum && t->colsum == nullptr) return LITE3R_ERR_INVALID_ARG;
  if (!aligned(t->scales, 4) || (t->colsum != nullptr && !aligned(t->colsum, 16))) return LITE3R_ERR_INVALID_ARG;
  return LITE3R_OK;
}

}  // namespace lite3r

using namespace lite3r;

extern "C" {

lite3r_status lite3r_fp8_sizes(const lite3r_shape* shape, size_t* codes_bytes, size_t* scales_bytes,
                               size_t* colsum_bytes) {
  lite3r_status st = check_shape(shape);
  if (st != LITE3R_OK) return st;
  const size_t bh = static_cast<size_t>(shape->batch) * shape->heads;
  const size_t nb = ceil_div(shape->tokens, shape->block);
  if (codes_bytes) *codes_bytes = bh * nb * shape->block * kHeadDim;
  if (scales_bytes) *scales_bytes = bh * nb * sizeof(float);
  if (colsum_bytes) *colsum_bytes = bh * nb * kHeadDim * sizeof(int);
  return LITE3R_OK;
}

lite3r_status lite3r_plan_sizes(const lite3r_shape* shape, double crit, double neg, size_t* cls_bytes,
                                size_t* crit_idx_bytes, size_t* marg_idx_bytes, int* k_crit, int* k_marg,
                                int* k_neg) {
  lite3r_status st = check_shape(shape);
  if (st != LITE3R_OK) return st;
  st = check_fractions(crit, neg);
  if (st != LITE3R_OK) return st;
  const size_t bh = static_cast<size_t>(shape->batch) * shape->heads;
  const size_t nb = ceil_div(shape->tokens, shape->block);
  const Counts c = class_counts(static_cast<int>(nb), crit, neg);
  if (cls_bytes) *cls_bytes = bh * nb * nb;
  if (crit_idx_bytes) *crit_idx_bytes = bh * nb * c.k_crit * sizeof(int);
  if (marg_idx_bytes) *marg_idx_bytes = bh * nb * c.k_marg * sizeof(int);
  if (k_crit) *k_crit = c.k_crit;
  if (k_marg) *k_marg = c.k_marg;
  if (k_neg) *k_neg = c.k_neg;
  return LITE3R_OK;
}

static lite3r_status workspace_query(const lite3r_shape* shape, double crit, double neg, bool plan_inside, size_t* bytes) {
  lite3r_status st = check_shape(shape);
  if (st != LITE3R_OK) return st;
  st = check_fractions(crit, neg);
  if (st != LITE3R_OK) return st;
  if (bytes == nullptr) return LITE3R_ERR_INVALID_ARG;
  *bytes = forward_workspace_bytes(*shape, class_counts(ceil_div(shape->tokens, shape->block), crit, neg), plan_inside);
  return LITE3R_OK;
}

lite3r_status lite3r_forward_workspace(const lite3r_shape* shape, double crit, double neg, size_t* bytes) {
  return workspace_query(shape, crit, neg, false, bytes);
}

lite3r_status lite3r_forward_workspace_planned(const lite3r_shape* shape, double crit, double neg, size_t* bytes) {
  return workspace_query(shape, crit, neg, true, bytes);
}

static lite3r_status check_source(const lite3r_tensor* x) {
  if (x == nullptr || x->ptr == nullptr || !aligned(x->ptr, 16)) return LITE3R_ERR_INVALID_ARG;
  if (x->dtype != LITE3R_F32 && x->dtype != LITE3R_BF16) return LITE3R_ERR_UNSUPPORTED;
  if (x->stride_n < kHeadDim || x->stride_b < 0 || x->stride_h < 0) return LITE3R_ERR_INVALID_ARG;
  if ((x->stride_b % 8) || (x->stride_h % 8) || (x->stride_n % 8)) return LITE3R_ERR_INVALID_ARG;
  return LITE3R_OK;
}

lite3r_status lite3r_quantize_fp8(const lite3r_tensor* x, const lite3r_shape* shape, lite3r_fp8 out, void* stream) {
  lite3r_status st = check_shape(shape);
  if (st != LITE3R_OK) return st;
  if ((st = check_source(x)) != LITE3R_OK) return st;
  st = check_fp8(&out, true, false);
  if (st != LITE3R_OK) return st;
  if ((st = check_device()) != LITE3R_OK) return st;
  return launch_quantize(&x, &out, 1, *shape, static_cast<cudaStream_t>(stream));
}

lite3r_status lite3r_quantize_fp8_qkv(const lite3r_tensor* q, const lite3r_tensor* k, const lite3r_tensor* v,
                                      const lite3r_shape* shape, lite3r_fp8 q_out, lite3r_fp8 k_out, lite3r_fp8 v_out,
                                      void* stream) {
  lite3r_status st = check_shape(shape);
  if (st != LITE3R_OK) return st;
  const lite3r_tensor* x[3] = {q, k, v};
  const lite3r_fp8 out[3] = {q_out, k_out, v_out};
  for (int n = 0; n < 3; ++n) {
    if ((st = check_source(x[n])) != LITE3R_OK) return st;
    if ((st = check_fp8(&out[n], true, false)) != LITE3R_OK) return st;
    if (x[n]->dtype != x[0]->dtype) return LITE3R_ERR_UNSUPPORTED;
  }
  if ((st = check_device()) != LITE3R_OK) return st;
  return launch_quantize(x, out, 3, *shape, static_cast<cudaStream_t>(stream));
}

lite3r_status lite3r_sla_plan(const lite3r_fp8* q, const lite3r_fp8* k, const lite3r_shape* shape, double crit,
                              double neg, lite3r_plan* plan, void* stream) {
  lite3r_status st = check_shape(shape);
  if (st != LITE3R_OK) return st;
  st = check_fractions(crit, neg);
  if (st != LITE3R_OK) return st;
  if ((st = check_fp8(q, false, true)) != LITE3R_OK) return st;
  if ((st = check_fp8(k, false, true)) != LITE3R_OK) return st;
  if (plan == nullptr || plan->cls == nullptr) return LITE3R_ERR_INVALID_ARG;
  const Counts c = class_counts(ceil_div(shape->tokens, shape->block), crit, neg);
  if (c.k_crit > 0 && plan->crit_idx == nullptr) return LITE3R_ERR_INVALID_ARG;
  plan->k_crit = c.k_crit;
  plan->k_marg = c.k_marg;
  plan->k_neg = c.k_neg;
  if ((st = check_device()) != LITE3R_OK) return st;
  return launch_plan(*q, *k, *shape, c, *plan, static_cast<cudaStream_t>(stream));
}

// Shared argument checks and launch of lite3r_sla_forward and its two halves (phases as in launch_forward).
static lite3r_status forward_phases(int phases, const lite3r_fp8* q, const lite3r_fp8* k, const lite3r_fp8* v,
                                    const float* proj, long long proj_head_stride, const lite3r_shape* shape,
                                    double crit, double neg, lite3r_phi phi, const lite3r_plan* plan, void* out,
                                    lite3r_dtype out_dtype, long long out_stride_b, long long out_stride_h,
                                    long long out_stride_n, void* workspace, size_t workspace_bytes,
                                    int* device_status, void* stream, int linear_only = 0) {
  lite3r_status st = check_shape(shape);
  if (st != LITE3R_OK) return st;
  if ((st = check_fp8(k, true, false)) != LITE3R_OK) return st;
  if ((st = check_fp8(v, true, false)) != LITE3R_OK) return st;
  if (phi != LITE3R_PHI_SOFTMAX && phi != LITE3R_PHI_ELU1) return LITE3R_ERR_UNSUPPORTED;
  const int nb = ceil_div(shape->tokens, shape->block);
  const bool plan_inside = plan == nullptr;
  lite3r_plan effective = {};
  if (plan_inside) {
    if (phases != 3) return LITE3R_ERR_INVALID_ARG;  // the two halves take the plan from the caller
    if ((st = check_fractions(crit, neg)) != LITE3R_OK) return st;
    if ((st = check_fp8(q, true, true)) != LITE3R_OK) return st;  // pooled scores need the column sums
    if ((st = check_fp8(k, true, true)) != LITE3R_OK) return st;
    const Counts c = class_counts(nb, crit, neg);
    effective.k_crit = c.k_crit;
    effective.k_marg = c.k_marg;
    effective.k_neg = c.k_neg;
  } else {
    effective = *plan;
    if (plan->k_crit < 0 || plan->k_marg < 0 || plan->k_neg < 0 || plan->k_crit + plan->k_marg + plan->k_neg != nb)
      return LITE3R_ERR_INVALID_ARG;
  }
  if (phases & 1) {
    if (proj == nullptr || !aligned(proj, 16) || proj_head_stride < 0 || (proj_head_stride % 4)) return LITE3R_ERR_INVALID_ARG;
  }
  if (phases & 2) {
    if ((st = check_fp8(q, true, false)) != LITE3R_OK) return st;
    if (out_dtype != LITE3R_F32 && out_dtype != LITE3R_BF16 && out_dtype != LITE3R_F16) return LITE3R_ERR_UNSUPPORTED;
    const int vec = out_dtype == LITE3R_F32 ? 4 : 8;  // elements per 16-byte store
    if (out == nullptr || !aligned(out, 16)) return LITE3R_ERR_INVALID_ARG;
    if (out_stride_n < kHeadDim || out_stride_b < 0 || out_stride_h < 0) return LITE3R_ERR_INVALID_ARG;
    if ((out_stride_b % vec) || (out_stride_h % vec) || (out_stride_n % vec)) return LITE3R_ERR_INVALID_ARG;
    if (!plan_inside) {
      if (plan->cls == nullptr) return LITE3R_ERR_INVALID_ARG;
      if (plan->k_crit > 0 && plan->crit_idx == nullptr) return LITE3R_ERR_INVALID_ARG;
    }
  }
  const Counts c{effective.k_crit, effective.k_marg, effective.k_neg};
  if (workspace == nullptr || !aligned(workspace, 256)) return LITE3R_ERR_INVALID_ARG;
  if (workspace_bytes < forward_workspace_bytes(*shape, c, plan_inside)) return LITE3R_ERR_WORKSPACE;
  if ((st = check_device()) != LITE3R_OK) return st;
  ForwardArgs a = {};
  if (q != nullptr) a.q = *q;
  a.k = *k;
  a.v = *v;
  a.proj = proj;
  a.proj_head_stride = proj_head_stride;
  a.s = *shape;
  a.phi = static_cast<int>(phi);
  a.plan = effective;
  a.plan_inside = plan_inside ? 1 : 0;
  a.linear_only = linear_only;
  a.crit = crit;
  a.neg = neg;
  a.out = out;
  a.out_dtype = static_cast<int>(out_dtype);
  a.out_stride_b = out_stride_b;
  a.out_stride_h = out_stride_h;
  a.out_stride_n = out_stride_n;
  a.workspace = workspace;
  a.workspace_bytes = workspace_bytes;
  a.device_status = device_status;
  return launch_forward(a, phases, static_cast<cudaStream_t>(stream));
}

lite3r_status lite3r_sla_forward(const lite3r_fp8* q, const lite3r_fp8* k, const lite3r_fp8* v, const float* proj,
                                 long long proj_head_stride, const lite3r_shape* shape, double crit, double neg,
                                 lite3r_phi phi, const lite3r_plan* plan, void* out, lite3r_dtype out_dtype,
                                 long long out_stride_b, long long out_stride_h, long long out_stride_n,
                                 void* workspace, size_t workspace_bytes, int* device_status, void* stream) {
  return forward_phases(3, q, k, v, proj, proj_head_stride, shape, crit, neg, phi, plan, out, out_dtype, out_stride_b,
                        out_stride_h, out_stride_n, workspace, workspace_bytes, device_status, stream);
}

lite3r_status lite3r_sla_forward_begin(const lite3r_fp8* k, const lite3r_fp8* v, const float* proj,
                                       long long proj_head_stride, const lite3r_shape* shape, lite3r_phi phi,
                                       int k_crit, int k_marg, int k_neg, void* workspace, size_t workspace_bytes,
                                       int* device_status, void* stream) {
  lite3r_plan counts = {};
  counts.k_crit = k_crit;
  counts.k_marg = k_marg;
  counts.k_neg = k_neg;
  return forward_phases(1, nullptr, k, v, proj, proj_head_stride, shape, 0.0, 0.0, phi, &counts, nullptr, LITE3R_F32,
                        0, 0, 0, workspace, workspace_bytes, device_status, stream);
}

lite3r_status lite3r_sla_forward_finish(const lite3r_fp8* q, const lite3r_fp8* k, const lite3r_fp8* v,
                                        const lite3r_shape* shape, lite3r_phi phi, const lite3r_plan* plan,
                                        void* out, lite3r_dtype out_dtype, long long out_stride_b,
                                        long long out_stride_h, long long out_stride_n, void* workspace,
                                        size_t workspace_bytes, int* device_status, void* stream) {
  if (plan == nullptr) return LITE3R_ERR_INVALID_ARG;
  return forward_phases(2, q, k, v, nullptr, 0, shape, 0.0, 0.0, phi, plan, out, out_dtype, out_stride_b,
                        out_stride_h, out_stride_n, workspace, workspace_bytes, device_status, stream);
}

lite3r_status lite3r_train_workspace(const lite3r_shape* shape, double crit, double neg, size_t* bytes) {
  size_t fwd = 0;
  lite3r_status st = workspace_query(shape, crit, neg, false, &fwd);
  if (st != LITE3R_OK) return st;
  *bytes = std::max(fwd + kHeadDim * kHeadDim * sizeof(float), train_workspace_bytes(*shape));
  return LITE3R_OK;
}

lite3r_status lite3r_sla_linear_branch(const lite3r_fp8* q, const lite3r_fp8* k, const lite3r_fp8* v,
                                       const lite3r_shape* shape, lite3r_phi phi, const lite3r_plan* plan, void* out,
                                       lite3r_dtype out_dtype, long long out_stride_b, long long out_stride_h,
                                       long long out_stride_n, void* workspace, size_t workspace_bytes,
                                       int* device_status, void* stream) {
  lite3r_status st = check_shape(shape);
  if (st != LITE3R_OK) return st;
  if (plan == nullptr || workspace == nullptr || !aligned(workspace, 256)) return LITE3R_ERR_INVALID_ARG;
  const size_t fwd = forward_workspace_bytes(*shape, Counts{plan->k_crit, plan->k_marg, plan->k_neg});
  if (workspace_bytes < fwd + kHeadDim * kHeadDim * sizeof(float)) return LITE3R_ERR_WORKSPACE;
  if ((st = check_device()) != LITE3R_OK) return st;
  // the projection is left out by running the forward with the identity in its place (exact in every format used)
  float* identity = reinterpret_cast<float*>(static_cast<char*>(workspace) + fwd);
  if ((st = launch_fill_identity(identity, static_cast<cudaStream_t>(stream))) != LITE3R_OK) return st;
  return forward_phases(3, q, k, v, identity, 0, shape, 0.0, 0.0, phi, plan, out, out_dtype, out_stride_b, out_stride_h,
                        out_stride_n, workspace, fwd, device_status, stream, 1);
}

lite3r_status lite3r_mse_distill(const void* student, const void* teacher, lite3r_dtype dtype, long long count,
                                 void* grad, double* loss, void* workspace, size_t workspace_bytes, void* stream) {
  if (student == nullptr || teacher == nullptr || loss == nullptr || workspace == nullptr || count <= 0)
    return LITE3R_ERR_INVALID_ARG;
  if (dtype != LITE3R_F32 && dtype != LITE3R_BF16) return LITE3R_ERR_UNSUPPORTED;
  if ((count % 8) || !aligned(student, 16) || !aligned(teacher, 16) || (grad != nullptr && !aligned(grad, 16)) ||
      !aligned(loss, 8) || !aligned(workspace, 256))
    return LITE3R_ERR_INVALID_ARG;
  if (workspace_bytes < 2048 * sizeof(double)) return LITE3R_ERR_WORKSPACE;
  lite3r_status st = check_device();
  if (st != LITE3R_OK) return st;
  return launch_mse_distill(student, teacher, static_cast<int>(dtype), static_cast<size_t>(count),
                            static_cast<__nv_bfloat16*>(grad), loss, static_cast<double*>(workspace),
                            static_cast<cudaStream_t>(stream));
}

lite3r_status lite3r_proj_lin_backward(const void* o_lin, const void* d_out, const lite3r_shape* shape, float* d_proj,
                                       void* workspace, size_t workspace_bytes, int* device_status, void* stream) {
  lite3r_status st = check_shape(shape);
  if (st != LITE3R_OK) return st;
  if (o_lin == nullptr || d_out == nullptr || d_proj == nullptr || workspace == nullptr) return LITE3R_ERR_INVALID_ARG;
  if (!aligned(o_lin, 16) || !aligned(d_out, 16) || !aligned(d_proj, 16) || !aligned(workspace, 256)) return LITE3R_ERR_INVALID_ARG;
  if (workspace_bytes < train_workspace_bytes(*shape)) return LITE3R_ERR_WORKSPACE;
  if ((st = check_device()) != LITE3R_OK) return st;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  if (device_status != nullptr && (st = record_cuda(cudaMemsetAsync(device_status, 0, sizeof(int), cs))) != LITE3R_OK) return st;
  return launch_proj_lin_backward(static_cast<const __nv_bfloat16*>(o_lin), static_cast<const __nv_bfloat16*>(d_out), *shape,
                                  d_proj, static_cast<float*>(workspace), device_status, cs);
}

lite3r_status lite3r_workspace_layout(const lite3r_shape* shape, double crit, double neg, int plan_inside,
                                      size_t* offsets) {
  lite3r_status st = check_shape(shape);
  if (st != LITE3R_OK) return st;
  if ((st = check_fractions(crit, neg)) != LITE3R_OK) return st;
  if (offsets == nullptr) return LITE3R_ERR_INVALID_ARG;
  forward_workspace_offsets(*shape, class_counts(ceil_div(shape->tokens, shape->block), crit, neg), plan_inside != 0,
                            offsets);
  return LITE3R_OK;
}

lite3r_status lite3r_quantize_rows_fp8(const void* x, lite3r_dtype dtype, long long row_stride, int rows, int cols,
                                       unsigned char* codes, float* scales, void* stream) {
  if (x == nullptr || codes == nullptr || scales == nullptr || rows <= 0 || cols <= 0) return LITE3R_ERR_INVALID_ARG;
  if (dtype != LITE3R_F32 && dtype != LITE3R_BF16) return LITE3R_ERR_UNSUPPORTED;
  if ((cols % 16) || row_stride < cols || (row_stride % 8) || !aligned(x, 16) || !aligned(codes, 16) || !aligned(scales, 4))
    return LITE3R_ERR_INVALID_ARG;
  lite3r_status st = check_device();
  if (st != LITE3R_OK) return st;
  return launch_rowquant(x, static_cast<int>(dtype), row_stride, rows, cols, codes, scales, static_cast<cudaStream_t>(stream));
}

static lite3r_status check_linear_operands(const unsigned char* x_codes, const float* x_scales, const unsigned char* w_codes,
                                           const float* w_scales, const float* bias, long long rows, int d_in, int d_out) {
  if (x_codes == nullptr || x_scales == nullptr || w_codes == nullptr || w_scales == nullptr) return LITE3R_ERR_INVALID_ARG;
  if (rows <= 0 || rows > 0x7FFFFFFFLL - 256 || d_in <= 0 || d_out <= 0) return LITE3R_ERR_INVALID_ARG;
  if ((d_in % 128) || (d_out % 64)) return LITE3R_ERR_UNSUPPORTED;
  if (!aligned(x_codes, 16) || !aligned(w_codes, 16) || !aligned(x_scales, 4) || !aligned(w_scales, 4) ||
      (bias != nullptr && !aligned(bias, 4)))
    return LITE3R_ERR_INVALID_ARG;
  return LITE3R_OK;
}

lite3r_status lite3r_linear_fp8(const unsigned char* x_codes, const float* x_scales, const unsigned char* w_codes,
                                const float* w_scales, const float* bias, int rows, int d_in, int d_out, void* y,
                                lite3r_dtype y_dtype, long long y_stride, int* device_status, void* stream) {
  lite3r_status st = check_linear_operands(x_codes, x_scales, w_codes, w_scales, bias, rows, d_in, d_out);
  if (st != LITE3R_OK) return st;
  if (y_dtype != LITE3R_F32 && y_dtype != LITE3R_BF16 && y_dtype != LITE3R_F16) return LITE3R_ERR_UNSUPPORTED;
  if (y == nullptr || !aligned(y, 16) || y_stride < d_out || (y_stride % 8)) return LITE3R_ERR_INVALID_ARG;
  if ((st = check_device()) != LITE3R_OK) return st;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  if (device_status != nullptr && (st = record_cuda(cudaMemsetAsync(device_status, 0, sizeof(int), cs))) != LITE3R_OK) return st;
  return launch_linear_fp8(x_codes, x_scales, w_codes, w_scales, bias, rows, d_in, d_out, y, static_cast<int>(y_dtype),
                           y_stride, device_status, cs);
}

lite3r_status lite3r_qkv_project_fp8(const unsigned char* x_codes, const float* x_scales, const unsigned char* w_codes,
                                     const float* w_scales, const float* bias, const lite3r_shape* shape, int d_model,
                                     lite3r_fp8 q_out, lite3r_fp8 k_out, lite3r_fp8 v_out, int* device_status,
                                     void* stream) {
  lite3r_status st = check_shape(shape);
  if (st != LITE3R_OK) return st;
  if (shape->heads % 2) return LITE3R_ERR_UNSUPPORTED;  // an output tile of 128 columns is two whole heads
  const long long rows = static_cast<long long>(shape->batch) * shape->tokens;
  st = check_linear_operands(x_codes, x_scales, w_codes, w_scales, bias, rows, d_model, 3 * shape->heads * kHeadDim);
  if (st != LITE3R_OK) return st;
  const lite3r_fp8 out[3] = {q_out, k_out, v_out};
  for (int i = 0; i < 3; ++i)
    if ((st = check_fp8(&out[i], true, false)) != LITE3R_OK) return st;
  if ((st = check_device()) != LITE3R_OK) return st;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  if (device_status != nullptr && (st = record_cuda(cudaMemsetAsync(device_status, 0, sizeof(int), cs))) != LITE3R_OK) return st;
  return launch_qkv_project(x_codes, x_scales, w_codes, w_scales, bias, *shape, d_model, out, device_status, cs);
}

lite3r_status lite3r_selftest_wait_expiry(int* device_status, unsigned long long limit_ns, void* stream) {
  if (device_status == nullptr || limit_ns == 0 || limit_ns > 1000000000ull) return LITE3R_ERR_INVALID_ARG;
  return launch_wait_expiry_probe(device_status, limit_ns, static_cast<cudaStream_t>(stream));
}

lite3r_status lite3r_profile_enable(int enable) {
  if (enable && !g_profile) {
    for (cudaEvent_t& e : g_events) {
      lite3r_status st = record_cuda(cudaEventCreate(&e));
      if (st != LITE3R_OK) return st;
    }
  } else if (!enable && g_profile) {
    for (cudaEvent_t& e : g_events) cudaEventDestroy(e);
  }
  g_profile = enable != 0;
  return LITE3R_OK;
}

lite3r_status lite3r_profile_stage_ms(float* ms) {
  if (ms == nullptr || !g_profile) return LITE3R_ERR_INVALID_ARG;
  for (int s = 0; s < 4; ++s) {
    ms[s] = 0.f;
    if (g_marked[2 * s] && g_marked[2 * s + 1]) {
      lite3r_status st = record_cuda(cudaEventSynchronize(g_events[2 * s + 1]));
      if (st != LITE3R_OK) return st;
      st = record_cuda(cudaEventElapsedTime(&ms[s], g_events[2 * s], g_events[2 * s + 1]));
      if (st != LITE3R_OK) return st;
    }
  }
  return LITE3R_OK;
}

const char* lite3r_status_string(lite3r_status status) {
  switch (status) {
    case LITE3R_OK: return "ok";
    case LITE3R_ERR_INVALID_ARG: return "invalid argument";
    case LITE3R_ERR_UNSUPPORTED: return "unsupported shape, dtype or option";
    case LITE3R_ERR_WORKSPACE: return "workspace too small";
    case LITE3R_ERR_CUDA: return "CUDA error";
    case LITE3R_ERR_TIMEOUT: return "device-side wait timed out";
  }
  return "unknown status";
}

int lite3r_last_cuda_error(void) { return g_last_cuda_error; }

long long lite3r_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

lite3r_status lite3r_attention_plain_stores(int on) {
  lite3r::set_attention_plain_stores(on != 0 ? 1 : 0);
  return LITE3R_OK;
}

lite3r_status lite3r_plan_variant(int variant) {
  if (variant < 0 || variant > 4) return LITE3R_ERR_INVALID_ARG;
  lite3r::set_plan_variant(variant);
  return LITE3R_OK;
}

}  // extern "C"
