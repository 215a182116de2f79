// K1: scaled FP8 (e4m3) quantisation, one scale per (b, h, token-block) tile of Bs x 64
// (paper appendix "Scaled FP8 Quantization"; epsilon from "Implementation Details").
//
// One CTA per tile.  The tile (8-32 KB) is read once into registers with 16-byte loads, the tile maximum is
// reduced through shuffles and shared memory, then every value is divided by the scale (IEEE fp32 division,
// so the codes equal a plain fp32 program's bit for bit), clamped, cast to e4m3 with round-to-nearest-even
// and written with 8-byte stores.  The same pass emits the per-tile column sums of the code values as exact
// integers (units of 2^-9), which is all the block plan needs.  HBM-bound: 2 (bf16) or 4 (fp32) bytes read
// and 1 byte written per element.
#include "common.cuh"

namespace lite3r {

namespace {

constexpr int kThreads = 256;
constexpr int kRowsPerPass = kThreads / 8;  // a thread owns one 8-column segment of one row per pass

__device__ __forceinline__ void load8(const float* p, float v[8]) {
  const float4 a = __ldg(reinterpret_cast<const float4*>(p));
  const float4 b = __ldg(reinterpret_cast<const float4*>(p) + 1);
  v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
  v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}

__device__ __forceinline__ void load8(const __nv_bfloat16* p, float v[8]) {
  const uint4 raw = __ldg(reinterpret_cast<const uint4*>(p));
  const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    v[2 * i] = __uint_as_float(w[i] << 16);
    v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
  }
}

template <int BS, typename SrcT>
__global__ void __launch_bounds__(kThreads) quantize_kernel(const SrcT* __restrict__ x, long long stride_b,
                                                            long long stride_h, long long stride_n, int heads,
                                                            int tokens, int nb, uint8_t* __restrict__ codes,
                                                            float* __restrict__ scales, int* __restrict__ colsum) {
  constexpr int kPasses = BS / kRowsPerPass;
  __shared__ float s_max[kThreads / 32];
  __shared__ int s_col[kHeadDim];

  const int tile = blockIdx.x;
  const int i = tile % nb;
  const int bh = tile / nb;
  const int h = bh % heads;
  const int b = bh / heads;
  const int valid = min(BS, tokens - i * BS);
  const int seg = threadIdx.x & 7;
  const int row0 = threadIdx.x >> 3;

  const SrcT* src = x + b * stride_b + h * stride_h + static_cast<long long>(i) * BS * stride_n + seg * 8;

  float v[kPasses][8];
  float amax = 0.f;
#pragma unroll
  for (int p = 0; p < kPasses; ++p) {
    const int r = row0 + p * kRowsPerPass;
    if (r < valid) {
      load8(src + r * stride_n, v[p]);
    } else {
#pragma unroll
      for (int c = 0; c < 8; ++c) v[p][c] = 0.f;
    }
#pragma unroll
    for (int c = 0; c < 8; ++c) amax = fmaxf(amax, fabsf(v[p][c]));
  }
  amax = warp_max(amax);
  if (threadIdx.x < kHeadDim) s_col[threadIdx.x] = 0;
  if ((threadIdx.x & 31) == 0) s_max[threadIdx.x >> 5] = amax;
  __syncthreads();
  amax = s_max[0];
#pragma unroll
  for (int w = 1; w < kThreads / 32; ++w) amax = fmaxf(amax, s_max[w]);

  const float scale = __fdiv_rn(__fadd_rn(amax, 1e-8f), 448.0f);
  if (threadIdx.x == 0) scales[tile] = scale;

  int sums[8] = {0, 0, 0, 0, 0, 0, 0, 0};
  uint8_t* dst = codes + (static_cast<size_t>(tile) * BS) * kHeadDim + seg * 8;
#pragma unroll
  for (int p = 0; p < kPasses; ++p) {
    const int r = row0 + p * kRowsPerPass;
    uint32_t packed[2];
#pragma unroll
    for (int c = 0; c < 8; c += 2) {
      float y0 = fminf(fmaxf(__fdiv_rn(v[p][c], scale), -448.0f), 448.0f);
      float y1 = fminf(fmaxf(__fdiv_rn(v[p][c + 1], scale), -448.0f), 448.0f);
      const uint32_t two = __nv_cvt_float2_to_fp8x2(make_float2(y0, y1), __NV_SATFINITE, __NV_E4M3);
      sums[c] += e4m3_units(two & 0xFFu);
      sums[c + 1] += e4m3_units(two >> 8);
      if ((c & 2) == 0) {
        packed[c >> 2] = two;
      } else {
        packed[c >> 2] |= two << 16;
      }
    }
    *reinterpret_cast<uint2*>(dst + static_cast<size_t>(r) * kHeadDim) = make_uint2(packed[0], packed[1]);
  }
  if (colsum != nullptr) {
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      int s = sums[c];
      s += __shfl_xor_sync(0xFFFFFFFFu, s, 8);
      s += __shfl_xor_sync(0xFFFFFFFFu, s, 16);
      if ((threadIdx.x & 31) < 8) atomicAdd(&s_col[seg * 8 + c], s);
    }
    __syncthreads();
    if (threadIdx.x < kHeadDim) colsum[static_cast<size_t>(tile) * kHeadDim + threadIdx.x] = s_col[threadIdx.x];
  }
}

template <int BS, typename SrcT>
lite3r_status launch(const lite3r_tensor& x, const lite3r_shape& s, const lite3r_fp8& out, cudaStream_t stream) {
  const int nb = ceil_div(s.tokens, BS);
  const int tiles = s.batch * s.heads * nb;
  quantize_kernel<BS, SrcT><<<tiles, kThreads, 0, stream>>>(static_cast<const SrcT*>(x.ptr), x.stride_b, x.stride_h,
                                                             x.stride_n, s.heads, s.tokens, nb, out.codes,
                                                             out.scales, out.colsum);
  return after_launch();
}

}  // namespace

lite3r_status launch_quantize(const lite3r_tensor& x, const lite3r_shape& s, const lite3r_fp8& out,
                              cudaStream_t stream) {
  if (x.dtype == LITE3R_BF16) {
    return s.block == 64 ? launch<64, __nv_bfloat16>(x, s, out, stream) : launch<128, __nv_bfloat16>(x, s, out, stream);
  }
  return s.block == 64 ? launch<64, float>(x, s, out, stream) : launch<128, float>(x, s, out, stream);
}

}  // namespace lite3r
