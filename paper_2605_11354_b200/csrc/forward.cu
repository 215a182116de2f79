// K3 / K3b / K4: the SLA forward for a given block plan (Eq. 1; Algorithm 1 lines 4-10).
//
//   K3  summary_kernel    per key block j:  H_j = phi(K_j)^T V_j, z_j = phi(K_j)^T 1  (lines 7-8 per block), with the
//                         output projection folded in early: the kernel stores (H_j W)^T and z_j in bf16.  Folding
//                         is exact algebra: (phi(q) sum_j H_j) W = phi(q) sum_j (H_j W).
//   K3b aggregate_kernel  per query block i:  G_i = sum over marginal j of (H_j W)^T,  zeta_i = sum of z_j  (fp32).
//   K4  attention_kernel  per query block i: online-softmax attention over the critical key blocks (lines 4-5),
//                         then the linear branch (line 9) phi(q) G_i / (phi(q) . zeta_i), the sum of the two
//                         (line 10) and the store.
#include "common.cuh"

namespace lite3r {

namespace {

constexpr float kLog2e = 1.4426950408889634f;

__device__ __forceinline__ float phi_elu1(float x) { return x > 0.f ? x + 1.f : expf(x); }

// ------------------------------------------------------------------------------------------------ K3
constexpr int kSumThreads = 256;

template <int BS>
__global__ void __launch_bounds__(kSumThreads) summary_kernel(const uint8_t* __restrict__ k_codes,
                                                              const float* __restrict__ k_scales,
                                                              const uint8_t* __restrict__ v_codes,
                                                              const float* __restrict__ v_scales,
                                                              const float* __restrict__ proj,
                                                              long long proj_head_stride, int heads, int tokens, int nb,
                                                              int phi, __nv_bfloat16* __restrict__ hws) {
  extern __shared__ __align__(16) float smem_f[];
  float* s_phi = smem_f;                 // [BS][64]
  float* s_v = s_phi + BS * kHeadDim;    // [BS][64]
  float* s_h = s_v + BS * kHeadDim;      // [64][68]
  float* s_w = s_h + kHeadDim * 68;      // [64][64]

  const int tile = blockIdx.x;  // (b*H + h) * nb + j
  const int j = tile % nb;
  const int h = (tile / nb) % heads;
  const int valid = min(BS, tokens - j * BS);
  const float sk = k_scales[tile];
  const float sv = v_scales[tile];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  const uint8_t* kc = k_codes + static_cast<size_t>(tile) * BS * kHeadDim;
  const uint8_t* vc = v_codes + static_cast<size_t>(tile) * BS * kHeadDim;
  for (int r = warp; r < BS; r += kSumThreads / 32) {
    float p0 = 0.f, p1 = 0.f;
    if (r < valid) {
      const uint32_t two = *reinterpret_cast<const uint16_t*>(kc + r * kHeadDim + 2 * lane);
      float x[4];
      e4m3x4_to_float(two, x);
      const float x0 = x[0] * sk, x1 = x[1] * sk;
      if (phi == LITE3R_PHI_SOFTMAX) {
        const float m = warp_max(fmaxf(x0, x1));
        const float e0 = expf(x0 - m), e1 = expf(x1 - m);
        const float inv = 1.f / warp_sum(e0 + e1);
        p0 = e0 * inv;
        p1 = e1 * inv;
      } else {
        p0 = phi_elu1(x0);
        p1 = phi_elu1(x1);
      }
    }
    *reinterpret_cast<float2*>(s_phi + r * kHeadDim + 2 * lane) = make_float2(p0, p1);
  }
  for (int w = threadIdx.x; w < BS * kHeadDim / 4; w += kSumThreads) {
    float x[4];
    e4m3x4_to_float(*reinterpret_cast<const uint32_t*>(vc + 4 * w), x);
    *reinterpret_cast<float4*>(s_v + 4 * w) = make_float4(x[0] * sv, x[1] * sv, x[2] * sv, x[3] * sv);
  }
  const float* w_h = proj + h * proj_head_stride;
  for (int w = threadIdx.x; w < kHeadDim * kHeadDim / 4; w += kSumThreads) {
    *reinterpret_cast<float4*>(s_w + 4 * w) = __ldg(reinterpret_cast<const float4*>(w_h) + w);
  }
  __syncthreads();

  const int d0 = (threadIdx.x >> 4) * 4, e0 = (threadIdx.x & 15) * 4;
  float acc[4][4] = {};
  float z[4] = {};
  for (int s = 0; s < valid; ++s) {
    const float4 a = *reinterpret_cast<const float4*>(s_phi + s * kHeadDim + d0);
    const float4 b = *reinterpret_cast<const float4*>(s_v + s * kHeadDim + e0);
    const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
    for (int x = 0; x < 4; ++x) {
      z[x] += av[x];
#pragma unroll
      for (int y = 0; y < 4; ++y) acc[x][y] = fmaf(av[x], bv[y], acc[x][y]);
    }
  }
#pragma unroll
  for (int x = 0; x < 4; ++x)
    *reinterpret_cast<float4*>(s_h + (d0 + x) * 68 + e0) = make_float4(acc[x][0], acc[x][1], acc[x][2], acc[x][3]);
  __syncthreads();

  float out[4][4] = {};
  for (int f = 0; f < kHeadDim; ++f) {
    const float4 b = *reinterpret_cast<const float4*>(s_w + f * kHeadDim + e0);
    const float bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
    for (int x = 0; x < 4; ++x) {
      const float a = s_h[(d0 + x) * 68 + f];
#pragma unroll
      for (int y = 0; y < 4; ++y) out[x][y] = fmaf(a, bv[y], out[x][y]);
    }
  }
  __nv_bfloat16* dst = hws + static_cast<size_t>(tile) * kSummaryRow;
#pragma unroll
  for (int y = 0; y < 4; ++y) {  // row e0+y of (H W)^T holds d0..d0+3 contiguously
    __nv_bfloat162 lo = __floats2bfloat162_rn(out[0][y], out[1][y]);
    __nv_bfloat162 hi = __floats2bfloat162_rn(out[2][y], out[3][y]);
    uint2 pk;
    pk.x = *reinterpret_cast<uint32_t*>(&lo);
    pk.y = *reinterpret_cast<uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(dst + (e0 + y) * kHeadDim + d0) = pk;
  }
  if ((threadIdx.x & 15) == 0) {
    __nv_bfloat162 lo = __floats2bfloat162_rn(z[0], z[1]);
    __nv_bfloat162 hi = __floats2bfloat162_rn(z[2], z[3]);
    uint2 pk;
    pk.x = *reinterpret_cast<uint32_t*>(&lo);
    pk.y = *reinterpret_cast<uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(dst + kHeadDim * kHeadDim + d0) = pk;
  }
}

// ------------------------------------------------------------------------------------------------ K3b
constexpr int kAggThreads = 256;
constexpr int kAggPer = (kSummaryRow / 2 + kAggThreads - 1) / kAggThreads;  // bf16 pairs per thread

__global__ void __launch_bounds__(kAggThreads) aggregate_kernel(const __nv_bfloat16* __restrict__ hws,
                                                                const int* __restrict__ marg_idx,
                                                                const signed char* __restrict__ cls, int nb, int k_marg,
                                                                float* __restrict__ g) {
  extern __shared__ int s_list[];  // [k_marg]
  const int row = blockIdx.x;      // (b*H + h) * nb + i
  const size_t bh_rows = static_cast<size_t>(row / nb) * nb;
  if (marg_idx != nullptr) {
    for (int t = threadIdx.x; t < k_marg; t += kAggThreads) s_list[t] = marg_idx[static_cast<size_t>(row) * k_marg + t];
  } else if (threadIdx.x == 0) {  // rebuild the ascending list from the class row
    int n = 0;
    const signed char* c = cls + static_cast<size_t>(row) * nb;
    for (int j = 0; j < nb; ++j)
      if (c[j] == 1) s_list[n++] = j;
  }
  __syncthreads();
  float2 acc[kAggPer];
#pragma unroll
  for (int x = 0; x < kAggPer; ++x) acc[x] = make_float2(0.f, 0.f);
  for (int t = 0; t < k_marg; ++t) {
    const __nv_bfloat162* src = reinterpret_cast<const __nv_bfloat162*>(hws + (bh_rows + s_list[t]) * kSummaryRow);
#pragma unroll
    for (int x = 0; x < kAggPer; ++x) {
      const int n = threadIdx.x + x * kAggThreads;
      if (n < kSummaryRow / 2) {
        const float2 v = __bfloat1622float2(src[n]);
        acc[x].x += v.x;
        acc[x].y += v.y;
      }
    }
  }
  float2* dst = reinterpret_cast<float2*>(g + static_cast<size_t>(row) * kSummaryRow);
#pragma unroll
  for (int x = 0; x < kAggPer; ++x) {
    const int n = threadIdx.x + x * kAggThreads;
    if (n < kSummaryRow / 2) dst[n] = acc[x];
  }
}

// ------------------------------------------------------------------------------------------------ K4
template <int BS>
__global__ void __launch_bounds__(BS) attention_kernel(const uint8_t* __restrict__ q_codes,
                                                       const float* __restrict__ q_scales,
                                                       const uint8_t* __restrict__ k_codes,
                                                       const float* __restrict__ k_scales,
                                                       const uint8_t* __restrict__ v_codes,
                                                       const float* __restrict__ v_scales,
                                                       const int* __restrict__ crit_idx, const float* __restrict__ g,
                                                       int heads, int tokens, int nb, int k_crit, int k_marg, int phi,
                                                       float* __restrict__ out, long long out_stride_b,
                                                       long long out_stride_h, long long out_stride_n) {
  extern __shared__ __align__(16) float smem_f[];
  float* s_k = smem_f;               // [BS][64]
  float* s_v = s_k + BS * kHeadDim;  // [BS][64]

  const int row_tile = blockIdx.x;  // (b*H + h) * nb + i
  const int i = row_tile % nb;
  const int bh = row_tile / nb;
  const int h = bh % heads, b = bh / heads;
  const size_t bh_rows = static_cast<size_t>(bh) * nb;
  const int t = threadIdx.x;
  const int token = i * BS + t;
  const bool live = token < tokens;

  // The query row: decoded codes times scale^Q, kept twice: plain (for phi) and pre-multiplied by log2(e)/sqrt(D).
  float qv[kHeadDim];
  {
    const uint4* src = reinterpret_cast<const uint4*>(q_codes + (static_cast<size_t>(row_tile) * BS + t) * kHeadDim);
    const float sq = q_scales[row_tile];
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      const uint4 raw = __ldg(src + w);
      const uint32_t words[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
      for (int x = 0; x < 4; ++x) {
        float f[4];
        e4m3x4_to_float(words[x], f);
#pragma unroll
        for (int y = 0; y < 4; ++y) qv[w * 16 + x * 4 + y] = f[y] * sq;
      }
    }
  }
  const float qk_scale = kLog2e * 0.125f;  // 1/sqrt(64) in the base-2 exponent domain

  float o[kHeadDim];
#pragma unroll
  for (int e = 0; e < kHeadDim; ++e) o[e] = 0.f;
  float m = -INFINITY, l = 0.f;

  for (int c = 0; c < k_crit; ++c) {
    const int j = crit_idx[static_cast<size_t>(row_tile) * k_crit + c];
    const float sk = k_scales[bh_rows + j], sv = v_scales[bh_rows + j];
    const int valid = min(BS, tokens - j * BS);
    const uint32_t* kc = reinterpret_cast<const uint32_t*>(k_codes + (bh_rows + j) * BS * kHeadDim);
    const uint32_t* vc = reinterpret_cast<const uint32_t*>(v_codes + (bh_rows + j) * BS * kHeadDim);
    __syncthreads();
#pragma unroll 4
    for (int w = t; w < BS * kHeadDim / 4; w += BS) {
      float f[4];
      e4m3x4_to_float(__ldg(kc + w), f);
      *reinterpret_cast<float4*>(s_k + 4 * w) = make_float4(f[0] * sk, f[1] * sk, f[2] * sk, f[3] * sk);
      e4m3x4_to_float(__ldg(vc + w), f);
      *reinterpret_cast<float4*>(s_v + 4 * w) = make_float4(f[0] * sv, f[1] * sv, f[2] * sv, f[3] * sv);
    }
    __syncthreads();
    for (int s = 0; s < valid; ++s) {
      const float4* kr = reinterpret_cast<const float4*>(s_k + s * kHeadDim);
      float acc = 0.f;
#pragma unroll
      for (int d4 = 0; d4 < kHeadDim / 4; ++d4) {
        const float4 kk = kr[d4];
        acc = fmaf(qv[4 * d4], kk.x, acc);
        acc = fmaf(qv[4 * d4 + 1], kk.y, acc);
        acc = fmaf(qv[4 * d4 + 2], kk.z, acc);
        acc = fmaf(qv[4 * d4 + 3], kk.w, acc);
      }
      acc *= qk_scale;
      if (acc > m) {
        const float corr = exp2f(m - acc);
        l *= corr;
#pragma unroll
        for (int e = 0; e < kHeadDim; ++e) o[e] *= corr;
        m = acc;
      }
      const float p = exp2f(acc - m);
      l += p;
      const float4* vr = reinterpret_cast<const float4*>(s_v + s * kHeadDim);
#pragma unroll
      for (int e4 = 0; e4 < kHeadDim / 4; ++e4) {
        const float4 vv = vr[e4];
        o[4 * e4] = fmaf(p, vv.x, o[4 * e4]);
        o[4 * e4 + 1] = fmaf(p, vv.y, o[4 * e4 + 1]);
        o[4 * e4 + 2] = fmaf(p, vv.z, o[4 * e4 + 2]);
        o[4 * e4 + 3] = fmaf(p, vv.w, o[4 * e4 + 3]);
      }
    }
  }
  if (k_crit > 0) {
    const float inv = 1.f / l;
#pragma unroll
    for (int e = 0; e < kHeadDim; ++e) o[e] *= inv;
  }

  if (k_marg > 0) {
    __syncthreads();
    const float4* src = reinterpret_cast<const float4*>(g + static_cast<size_t>(row_tile) * kSummaryRow);
    for (int w = t; w < kSummaryRow / 4; w += BS) reinterpret_cast<float4*>(smem_f)[w] = __ldg(src + w);
    __syncthreads();
    if (phi == LITE3R_PHI_SOFTMAX) {
      float mx = qv[0];
#pragma unroll
      for (int d = 1; d < kHeadDim; ++d) mx = fmaxf(mx, qv[d]);
#pragma unroll
      for (int d = 0; d < kHeadDim; ++d) qv[d] = expf(qv[d] - mx);  // normalisation cancels in the ratio
    } else {
#pragma unroll
      for (int d = 0; d < kHeadDim; ++d) qv[d] = phi_elu1(qv[d]);
    }
    float den = 0.f;
    const float* zeta = smem_f + kHeadDim * kHeadDim;
#pragma unroll
    for (int d = 0; d < kHeadDim; ++d) den = fmaf(qv[d], zeta[d], den);
    const float inv = 1.f / den;
#pragma unroll
    for (int e = 0; e < kHeadDim; ++e) {
      const float4* gr = reinterpret_cast<const float4*>(smem_f + e * kHeadDim);
      float num = 0.f;
#pragma unroll
      for (int d4 = 0; d4 < kHeadDim / 4; ++d4) {
        const float4 gg = gr[d4];
        num = fmaf(qv[4 * d4], gg.x, num);
        num = fmaf(qv[4 * d4 + 1], gg.y, num);
        num = fmaf(qv[4 * d4 + 2], gg.z, num);
        num = fmaf(qv[4 * d4 + 3], gg.w, num);
      }
      o[e] = fmaf(num, inv, o[e]);
    }
  }
  if (live) {
    float4* dst = reinterpret_cast<float4*>(out + b * out_stride_b + h * out_stride_h + token * out_stride_n);
#pragma unroll
    for (int e4 = 0; e4 < kHeadDim / 4; ++e4) dst[e4] = make_float4(o[4 * e4], o[4 * e4 + 1], o[4 * e4 + 2], o[4 * e4 + 3]);
  }
}

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

template <int BS>
lite3r_status run_forward(const ForwardArgs& a, cudaStream_t stream) {
  const lite3r_shape& s = a.s;
  const int nb = ceil_div(s.tokens, BS);
  const int rows = s.batch * s.heads * nb;
  __nv_bfloat16* hws = static_cast<__nv_bfloat16*>(a.workspace);
  float* g = reinterpret_cast<float*>(static_cast<char*>(a.workspace) +
                                      align_up(static_cast<size_t>(rows) * kSummaryRow * sizeof(__nv_bfloat16), 256));
  lite3r_status st;
  if (a.plan.k_marg > 0) {
    const size_t smem = (2 * BS * kHeadDim + kHeadDim * 68 + kHeadDim * kHeadDim) * sizeof(float);
    st = record_cuda(cudaFuncSetAttribute(summary_kernel<BS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          static_cast<int>(smem)));
    if (st != LITE3R_OK) return st;
    profile_mark(0, stream);
    summary_kernel<BS><<<rows, kSumThreads, smem, stream>>>(a.k.codes, a.k.scales, a.v.codes, a.v.scales, a.proj,
                                                            a.proj_head_stride, s.heads, s.tokens, nb, a.phi, hws);
    if ((st = after_launch()) != LITE3R_OK) return st;
    profile_mark(1, stream);
    profile_mark(2, stream);
    aggregate_kernel<<<rows, kAggThreads, a.plan.k_marg * sizeof(int), stream>>>(hws, a.plan.marg_idx, a.plan.cls, nb,
                                                                                   a.plan.k_marg, g);
    if ((st = after_launch()) != LITE3R_OK) return st;
    profile_mark(3, stream);
  }
  const size_t smem = align_up(2 * BS * kHeadDim * sizeof(float), 16) + 1024;
  st = record_cuda(cudaFuncSetAttribute(attention_kernel<BS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        static_cast<int>(smem)));
  if (st != LITE3R_OK) return st;
  profile_mark(4, stream);
  attention_kernel<BS><<<rows, BS, smem, stream>>>(a.q.codes, a.q.scales, a.k.codes, a.k.scales, a.v.codes, a.v.scales,
                                                   a.plan.crit_idx, g, s.heads, s.tokens, nb, a.plan.k_crit,
                                                   a.plan.k_marg, a.phi, a.out, a.out_stride_b, a.out_stride_h,
                                                   a.out_stride_n);
  st = after_launch();
  profile_mark(5, stream);
  return st;
}

}  // namespace

size_t forward_workspace_bytes(const lite3r_shape& s, const Counts& c) {
  (void)c;
  const size_t rows = static_cast<size_t>(s.batch) * s.heads * ceil_div(s.tokens, s.block);
  return align_up(rows * kSummaryRow * sizeof(__nv_bfloat16), 256) + align_up(rows * kSummaryRow * sizeof(float), 256);
}

lite3r_status launch_forward(const ForwardArgs& a, cudaStream_t stream) {
  if (a.device_status != nullptr) {
    lite3r_status st = record_cuda(cudaMemsetAsync(a.device_status, 0, sizeof(int), stream));
    if (st != LITE3R_OK) return st;
  }
  return a.s.block == 64 ? run_forward<64>(a, stream) : run_forward<128>(a, stream);
}

}  // namespace lite3r
