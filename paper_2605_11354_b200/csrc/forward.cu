// K3 / K3b / K4: the SLA forward for a given block plan (Eq. 1; Algorithm 1 lines 4-10).
//
//   K3  summary.cu        per key block j:  H_j = phi(K_j)^T V_j, z_j = phi(K_j)^T 1  (lines 7-8 per block), stored as
//                         (H_j W)^T and z_j in bf16 (output projection folded in early).
//   K3b aggregate.cu      per query block i:  G_i = sum over marginal j of (H_j W)^T,  zeta_i = sum of z_j.
//   K4  attention.cu      per query block i: online-softmax attention over the critical key blocks (lines 4-5),
//                         then the linear branch (line 9) phi(q) G_i / (phi(q) . zeta_i), the sum of the two
//                         (line 10) and the store.
//   prep_kernel           V code values as fp16 and the per-head reference V scale for the attention kernel.
#include <algorithm>

#include "common.cuh"

namespace lite3r {

namespace {

// ------------------------------------------------------------------------------------------------ prep
// V code values as fp16 (exact) for the P V tensor-core product, and the largest V block scale of every head.
__global__ void __launch_bounds__(256) prep_kernel(const uint8_t* __restrict__ v_codes, const float* __restrict__ v_scales,
                                                   size_t words, int tiles, int nb, __half* __restrict__ v16,
                                                   float* __restrict__ vref) {
  const size_t stride = static_cast<size_t>(gridDim.x) * blockDim.x;
  for (size_t w = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x; w < words; w += stride) {
    const uint32_t packed = __ldg(reinterpret_cast<const uint32_t*>(v_codes) + w);
    const __half2_raw lo = __nv_cvt_fp8x2_to_halfraw2(static_cast<__nv_fp8x2_storage_t>(packed & 0xFFFFu), __NV_E4M3);
    const __half2_raw hi = __nv_cvt_fp8x2_to_halfraw2(static_cast<__nv_fp8x2_storage_t>(packed >> 16), __NV_E4M3);
    uint2 out;
    out.x = static_cast<uint32_t>(lo.x) | (static_cast<uint32_t>(lo.y) << 16);
    out.y = static_cast<uint32_t>(hi.x) | (static_cast<uint32_t>(hi.y) << 16);
    reinterpret_cast<uint2*>(v16)[w] = out;
  }
  // scales are positive, so their bit patterns order like integers; max is order-independent (deterministic)
  for (int t = blockIdx.x * blockDim.x + threadIdx.x; t < tiles; t += static_cast<int>(stride))
    atomicMax(reinterpret_cast<int*>(vref) + t / nb, __float_as_int(v_scales[t]));
}

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct Workspace {
  __nv_bfloat16* hws;  // [tiles][4160]   per-key-block summaries
  __nv_bfloat16* g16;  // [tiles][64][64] aggregated summaries, [e][d]
  float* zeta;         // [tiles][64]
  __half* v16;         // [tiles*Bs][64]  V code values as fp16
  float* vref;         // [B*H]
  size_t bytes;
};

Workspace carve(void* base, const lite3r_shape& s) {
  const size_t tiles = static_cast<size_t>(s.batch) * s.heads * ceil_div(s.tokens, s.block);
  char* p = static_cast<char*>(base);
  size_t off = 0;
  Workspace w;
  auto take = [&](size_t bytes) {
    char* r = p + off;
    off += align_up(bytes, 1024);
    return r;
  };
  w.hws = reinterpret_cast<__nv_bfloat16*>(take(tiles * kSummaryRow * sizeof(__nv_bfloat16)));
  w.g16 = reinterpret_cast<__nv_bfloat16*>(take(tiles * kHeadDim * kHeadDim * sizeof(__nv_bfloat16)));
  w.zeta = reinterpret_cast<float*>(take(tiles * kHeadDim * sizeof(float)));
  w.v16 = reinterpret_cast<__half*>(take(tiles * s.block * kHeadDim * sizeof(__half)));
  w.vref = reinterpret_cast<float*>(take(static_cast<size_t>(s.batch) * s.heads * sizeof(float)));
  w.bytes = off;
  return w;
}

template <int BS>
lite3r_status run_forward(const ForwardArgs& a, cudaStream_t stream) {
  const lite3r_shape& s = a.s;
  const int nb = ceil_div(s.tokens, BS);
  const int rows = s.batch * s.heads * nb;
  const Workspace w = carve(a.workspace, s);
  lite3r_status st;
  profile_mark(0, stream);
  if (a.plan.k_crit > 0) {
    st = record_cuda(cudaMemsetAsync(w.vref, 0, static_cast<size_t>(s.batch) * s.heads * sizeof(float), stream));
    if (st != LITE3R_OK) return st;
    const size_t words = static_cast<size_t>(rows) * BS * kHeadDim / 4;
    const int blocks = static_cast<int>(std::min<size_t>((words + 255) / 256, 148 * 16));
    prep_kernel<<<blocks, 256, 0, stream>>>(a.v.codes, a.v.scales, words, rows, nb, w.v16, w.vref);
    if ((st = after_launch()) != LITE3R_OK) return st;
    profile_mark(1, stream);
  }
  if (a.plan.k_marg > 0) {
    profile_mark(2, stream);
    st = launch_summary(a.k, a.v, a.proj, a.proj_head_stride, s, a.phi, w.hws, a.device_status, stream);
    if (st != LITE3R_OK) return st;
    profile_mark(3, stream);
    profile_mark(4, stream);
    if ((st = launch_aggregate(w.hws, a.plan.cls, s, nb, w.g16, w.zeta, a.device_status, stream)) != LITE3R_OK) return st;
    profile_mark(5, stream);
  }
  AttentionLaunch att;
  att.shape = s;
  att.q_codes = a.q.codes;
  att.k_codes = a.k.codes;
  att.q_scales = a.q.scales;
  att.k_scales = a.k.scales;
  att.v_scales = a.v.scales;
  att.v16 = w.v16;
  att.g16 = w.g16;
  att.zeta = w.zeta;
  att.vref = w.vref;
  att.crit_idx = a.plan.crit_idx;
  att.k_crit = a.plan.k_crit;
  att.k_marg = a.plan.k_marg;
  att.phi = a.phi;
  att.out = a.out;
  att.out_stride_b = a.out_stride_b;
  att.out_stride_h = a.out_stride_h;
  att.out_stride_n = a.out_stride_n;
  att.device_status = a.device_status;
  profile_mark(6, stream);
  st = launch_attention(att, stream);
  profile_mark(7, stream);
  return st;
}

}  // namespace

size_t forward_workspace_bytes(const lite3r_shape& s, const Counts& c) {
  (void)c;
  return carve(nullptr, s).bytes;
}

lite3r_status launch_forward(const ForwardArgs& a, cudaStream_t stream) {
  if (a.device_status != nullptr) {
    lite3r_status st = record_cuda(cudaMemsetAsync(a.device_status, 0, sizeof(int), stream));
    if (st != LITE3R_OK) return st;
  }
  return a.s.block == 64 ? run_forward<64>(a, stream) : run_forward<128>(a, stream);
}

}  // namespace lite3r
