// K3 / K3b / K4: the SLA forward for a given block plan (Eq. 1; Algorithm 1 from the sparse softmax on).
//
//   K3  summary.cu        per key block j:  H_j = phi(K_j)^T V_j, z_j = phi(K_j)^T 1  (KV summary and normaliser, per block), stored as
//                         (H_j W)^T and z_j in bf16 (output projection folded in early).
//   K3b aggregate.cu      per query block i:  G_i = sum over marginal j of (H_j W)^T,  zeta_i = sum of z_j.
//   K4  attention.cu      per query block i: online-softmax attention over the critical key blocks (sparse branch),
//                         then the linear output phi(q) G_i / (phi(q) . zeta_i), the sum of the two
//                         and the store.
//   prep_kernel           dequantised V as fp16 for the attention kernel's P V product.
#include <algorithm>

#include "common.cuh"
#include "sm100.cuh"

namespace lite3r {

namespace {

// ------------------------------------------------------------------------------------------------ prep
// Dequantised V (code value x block scale) as fp16, the B operand of the P V tensor-core product.
__global__ void __launch_bounds__(256) prep_kernel(const uint8_t* __restrict__ v_codes, const float* __restrict__ v_scales,
                                                   size_t words, int words_per_tile, __half* __restrict__ v16) {
  const size_t stride = static_cast<size_t>(gridDim.x) * blockDim.x;
  for (size_t w = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x; w < words; w += stride) {
    const uint4 packed = __ldg(reinterpret_cast<const uint4*>(v_codes) + w);
    const float sv = __ldg(v_scales + w / words_per_tile);
    const uint32_t in[4] = {packed.x, packed.y, packed.z, packed.w};
    uint32_t out[8];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      float f[4];
      e4m3x4_to_float(in[q], f);
      const __half2 lo = __floats2half2_rn(f[0] * sv, f[1] * sv), hi = __floats2half2_rn(f[2] * sv, f[3] * sv);
      out[2 * q] = *reinterpret_cast<const uint32_t*>(&lo);
      out[2 * q + 1] = *reinterpret_cast<const uint32_t*>(&hi);
    }
    uint4* dst = reinterpret_cast<uint4*>(v16) + 2 * w;
    dst[0] = make_uint4(out[0], out[1], out[2], out[3]);
    dst[1] = make_uint4(out[4], out[5], out[6], out[7]);
  }
}

// Self-test of the bounded waits: one thread waits on a barrier that nothing ever arrives on.  The wait must give up
// after limit_ns, write its code to *status and let the kernel end normally.
__global__ void wait_expiry_probe_kernel(int* status, unsigned long long limit_ns) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    sm100::mbar_init(&bar, 1);
    abort_flag = 0;
    sm100::mbar_fence_init();
    sm100::mbar_wait(&bar, 0, &abort_flag, status, 999, 0, limit_ns);
  }
}

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct Workspace {
  __nv_bfloat16* hws;  // [tiles][4160]   per-key-block summaries
  __nv_bfloat16* g16;  // [tiles][64][64] aggregated summaries, [e][d]
  float* zeta;         // [tiles][64]
  __half* v16;         // [tiles*Bs][64]  dequantised V as fp16
  signed char* cls;    // [tiles][Nb]     block classes, only when the plan is built inside the workspace
  int* crit_idx;       // [tiles][k_crit] critical lists, likewise
  size_t bytes;
  size_t offsets[6];
};

Workspace carve(void* base, const lite3r_shape& s, int k_crit = 0, bool plan_inside = false) {
  const size_t tiles = static_cast<size_t>(s.batch) * s.heads * ceil_div(s.tokens, s.block);
  char* p = static_cast<char*>(base);
  size_t off = 0;
  Workspace w;
  auto take = [&](size_t bytes) {
    char* r = p + off;
    off += align_up(bytes, 1024);
    return r;
  };
  w.offsets[0] = off;
  w.hws = reinterpret_cast<__nv_bfloat16*>(take(tiles * kSummaryRow * sizeof(__nv_bfloat16)));
  w.offsets[1] = off;
  w.g16 = reinterpret_cast<__nv_bfloat16*>(take(tiles * kHeadDim * kHeadDim * sizeof(__nv_bfloat16)));
  w.offsets[2] = off;
  w.zeta = reinterpret_cast<float*>(take(tiles * kHeadDim * sizeof(float)));
  w.offsets[3] = off;
  w.v16 = reinterpret_cast<__half*>(take(tiles * s.block * kHeadDim * sizeof(__half)));
  w.cls = nullptr;
  w.crit_idx = nullptr;
  w.offsets[4] = w.offsets[5] = off;
  if (plan_inside) {
    const size_t nb = ceil_div(s.tokens, s.block);
    w.offsets[4] = off;
    w.cls = reinterpret_cast<signed char*>(take(tiles * nb + 16));  // the class bytes are read in aligned 32-bit words
    w.offsets[5] = off;
    w.crit_idx = reinterpret_cast<int*>(take(tiles * static_cast<size_t>(k_crit) * sizeof(int) + 16));
  }
  w.bytes = off;
  return w;
}

// phases: bit 0 = the part that does not depend on the plan's contents (summaries, fp16 V operand), bit 1 = the rest.
template <int BS>
lite3r_status run_forward(const ForwardArgs& a, int phases, cudaStream_t stream) {
  const lite3r_shape& s = a.s;
  const int nb = ceil_div(s.tokens, BS);
  const int rows = s.batch * s.heads * nb;
  const Workspace w = carve(a.workspace, s, a.plan.k_crit, a.plan_inside != 0);
  lite3r_status st = LITE3R_OK;
  lite3r_plan plan = a.plan;
  if (a.plan_inside) {  // the block plan is built first, into the tail of the workspace
    plan.cls = w.cls;
    plan.crit_idx = w.crit_idx;
    plan.marg_idx = nullptr;
    const Counts c{plan.k_crit, plan.k_marg, plan.k_neg};
    if ((st = launch_plan(a.q, a.k, s, c, plan, stream)) != LITE3R_OK) return st;
  }
  if (phases & 1) profile_mark(0, stream);
  // With a linear branch the summary kernel reads every V row anyway and writes the fp16 operand on the way; the
  // stand-alone pass runs only when there is no linear branch.
  const bool v16_from_summary = a.plan.k_marg > 0;
  if ((phases & 1) && a.plan.k_crit > 0 && !v16_from_summary && !a.linear_only) {
    const size_t words = static_cast<size_t>(rows) * BS * kHeadDim / 16;  // 16 codes per thread and pass
    int sms = 0;
    if ((st = sm_count(&sms)) != LITE3R_OK) return st;
    const int blocks = static_cast<int>(std::min<size_t>((words + 255) / 256, static_cast<size_t>(sms) * 8));
    prep_kernel<<<blocks, 256, 0, stream>>>(a.v.codes, a.v.scales, words, BS * kHeadDim / 16, w.v16);
    if ((st = after_launch()) != LITE3R_OK) return st;
    profile_mark(1, stream);
  }
  if ((phases & 1) && a.plan.k_marg > 0) {
    profile_mark(2, stream);
    st = launch_summary(a.k, a.v, a.proj, a.proj_head_stride, s, a.phi, w.hws, a.plan.k_crit > 0 ? w.v16 : nullptr,
                        a.device_status, stream);
    if (st != LITE3R_OK) return st;
    profile_mark(3, stream);
  }
  if (!(phases & 2)) return st;
  if (a.plan.k_marg > 0) {
    profile_mark(4, stream);
    if ((st = launch_aggregate(w.hws, plan.cls, s, nb, w.g16, w.zeta, a.device_status, stream)) != LITE3R_OK) return st;
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
  att.crit_idx = plan.crit_idx;
  att.k_crit = a.linear_only ? 0 : a.plan.k_crit;
  att.k_marg = a.plan.k_marg;
  att.phi = a.phi;
  att.out = a.out;
  att.out_dtype = a.out_dtype;
  att.out_stride_b = a.out_stride_b;
  att.out_stride_h = a.out_stride_h;
  att.out_stride_n = a.out_stride_n;
  att.device_status = a.device_status;
  // With a linear branch the kernel enqueued just before the attention kernel is the aggregation, whose results the
  // attention kernel needs only in its tail: the two may overlap (not while stage events sit between them).
  att.overlap_prior = a.plan.k_marg > 0 && !profile_enabled();
  profile_mark(6, stream);
  st = launch_attention(att, stream);
  profile_mark(7, stream);
  return st;
}

}  // namespace

lite3r_status launch_wait_expiry_probe(int* status, unsigned long long limit_ns, cudaStream_t stream) {
  lite3r_status st = record_cuda(cudaMemsetAsync(status, 0, sizeof(int), stream));
  if (st != LITE3R_OK) return st;
  wait_expiry_probe_kernel<<<1, 32, 0, stream>>>(status, limit_ns);
  return after_launch();
}

size_t forward_workspace_bytes(const lite3r_shape& s, const Counts& c, bool plan_inside) {
  return carve(nullptr, s, c.k_crit, plan_inside).bytes;
}

void forward_workspace_offsets(const lite3r_shape& s, const Counts& c, bool plan_inside, size_t* offsets) {
  const Workspace w = carve(nullptr, s, c.k_crit, plan_inside);
  for (int i = 0; i < 6; ++i) offsets[i] = w.offsets[i];
}

lite3r_status launch_forward(const ForwardArgs& a, int phases, cudaStream_t stream) {
  if ((phases & 1) && a.device_status != nullptr) {  // the status word is cleared where the forward begins
    lite3r_status st = record_cuda(cudaMemsetAsync(a.device_status, 0, sizeof(int), stream));
    if (st != LITE3R_OK) return st;
  }
  return a.s.block == 64 ? run_forward<64>(a, phases, stream) : run_forward<128>(a, phases, stream);
}

}  // namespace lite3r
