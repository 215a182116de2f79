// Training side of the linear-branch projection, the only tensor Lite3R trains (Sec. 3.3 "selective freezing"):
//   mse_distill         one module's term of the partial attention distillation loss (Eq. 3), MSE(A_student, A_teacher),
//                       and its gradient 2 (A_s - A_t) / numel with respect to the student's attention output
//   proj_lin_backward   dW_h = sum over batch and tokens of O_lin^T dO  (O = O_sparse + O_lin W_h, Algorithm 1's last step)
// The gradient is a dense contraction over the tokens (64 x T x 64 per head): tokens are split over CTAs, each
// accumulates its chunk on tcgen05 (bf16 operands, both token-major as they lie in memory: A M-major, B N-major; fp32
// accumulator in TMEM), writes a 64 x 64 partial, and a second kernel adds the partials of a head in a fixed order
// (no floating-point atomics: results are bit-identical from run to run).
#include <algorithm>

#include "common.cuh"
#include "sm100.cuh"

namespace lite3r {

namespace {

using namespace sm100;

// ------------------------------------------------------------------------------------------------ identity (64 x 64)
__global__ void fill_identity_kernel(float* dst) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < kHeadDim * kHeadDim) dst[i] = (i / kHeadDim == i % kHeadDim) ? 1.f : 0.f;
}

// ------------------------------------------------------------------------------------------------ MSE term
constexpr int kMseThreads = 256;
constexpr int kMaxMseBlocks = 2048;

__device__ __forceinline__ void load8f(const float* p, float v[8]) {
  const float4 a = *reinterpret_cast<const float4*>(p);
  const float4 b = *reinterpret_cast<const float4*>(p + 4);
  v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
  v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}
__device__ __forceinline__ void load8f(const __nv_bfloat16* p, float v[8]) {
  const uint4 w = *reinterpret_cast<const uint4*>(p);
  const uint32_t x[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    v[2 * i] = __uint_as_float(x[i] << 16);
    v[2 * i + 1] = __uint_as_float(x[i] & 0xFFFF0000u);
  }
}

template <typename T>
__global__ void __launch_bounds__(kMseThreads) mse_kernel(const T* __restrict__ student, const T* __restrict__ teacher,
                                                          size_t groups, float grad_scale, __nv_bfloat16* __restrict__ grad,
                                                          double* __restrict__ partials) {
  __shared__ double s_sum[kMseThreads / 32];
  double acc = 0.0;
  const size_t stride = static_cast<size_t>(gridDim.x) * blockDim.x;
  for (size_t g = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x; g < groups; g += stride) {
    float a[8], b[8];
    load8f(student + g * 8, a);
    load8f(teacher + g * 8, b);
    uint32_t out[4];
    float sq = 0.f;
#pragma unroll
    for (int i = 0; i < 8; i += 2) {
      const float d0 = a[i] - b[i], d1 = a[i + 1] - b[i + 1];
      sq = fmaf(d0, d0, fmaf(d1, d1, sq));
      __nv_bfloat162 h = __floats2bfloat162_rn(d0 * grad_scale, d1 * grad_scale);
      out[i >> 1] = *reinterpret_cast<uint32_t*>(&h);
    }
    acc += static_cast<double>(sq);
    if (grad != nullptr) *reinterpret_cast<uint4*>(grad + g * 8) = make_uint4(out[0], out[1], out[2], out[3]);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
  if ((threadIdx.x & 31) == 0) s_sum[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    double t = 0.0;
    for (int w = 0; w < kMseThreads / 32; ++w) t += s_sum[w];
    partials[blockIdx.x] = t;
  }
}

__global__ void mse_finish_kernel(const double* __restrict__ partials, int n, double inv_count, double* __restrict__ loss) {
  if (threadIdx.x == 0 && blockIdx.x == 0) {
    double t = 0.0;
    for (int i = 0; i < n; ++i) t += partials[i];  // fixed order
    *loss = t * inv_count;
  }
}

// ------------------------------------------------------------------------------------------------ dW = O_lin^T dO
constexpr int kStages = 4;
constexpr int kTileTok = 64;
constexpr uint32_t kTileBytes = kTileTok * kHeadDim * 2;  // 8 KB per operand tile
constexpr uint32_t kStageBytes = 2 * kTileBytes;
constexpr uint32_t kOffBar = kStages * kStageBytes;
constexpr uint32_t kSmemBytes = kOffBar + 256;
constexpr int kThreads = 256;
constexpr uint32_t kTmemCols = 64;

struct Bars {
  uint64_t full[kStages], empty[kStages], acc_full;
  uint32_t tmem_base;
  int abort;
};

// CTA c of head-plane bh (b * H + h) handles the token tiles [c * tiles_per_cta, ...) of that plane.
__global__ void __launch_bounds__(kThreads, 2)
projgrad_kernel(const __grid_constant__ CUtensorMap map_o, const __grid_constant__ CUtensorMap map_g, int tokens,
                int chunks, int tiles_per_cta, float* __restrict__ partials, int* status) {
  extern __shared__ __align__(1024) uint8_t smem[];
  Bars* bars = reinterpret_cast<Bars*>(smem + kOffBar);
  volatile int* abort_flag = &bars->abort;
  if ((smem_u32(smem) & 1023u) != 0) {
    if (threadIdx.x == 0 && status != nullptr) atomicCAS(status, 0, 900);
    return;
  }
  if (status != nullptr && *reinterpret_cast<volatile int*>(status) != 0) return;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int bh = blockIdx.x / chunks, chunk = blockIdx.x % chunks;
  const int total_tiles = (tokens + kTileTok - 1) / kTileTok;
  const int t_begin = chunk * tiles_per_cta;
  const int t_end = min(total_tiles, t_begin + tiles_per_cta);
  const int n_tiles = max(0, t_end - t_begin);

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&bars->full[s], 1);
      mbar_init(&bars->empty[s], 1);
    }
    mbar_init(&bars->acc_full, 1);
    bars->abort = 0;
    mbar_fence_init();
  }
  if (warp == 1) {
    tmem_alloc(&bars->tmem_base, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_base;

  if (warp == 0) {
    if (lane == 0) {
      tma_prefetch_desc(&map_o);
      tma_prefetch_desc(&map_g);
      bool ok = true;
      for (int i = 0; ok && i < n_tiles; ++i) {
        const int st = i % kStages;
        if (i >= kStages) ok = mbar_wait(&bars->empty[st], ((i - kStages) / kStages) & 1, abort_flag, status, 701, 32);
        if (!ok) break;
        mbar_arrive_expect_tx(&bars->full[st], kStageBytes);
        tma_load_3d(smem + st * kStageBytes, &map_o, &bars->full[st], 0, (t_begin + i) * kTileTok, bh);
        tma_load_3d(smem + st * kStageBytes + kTileBytes, &map_g, &bars->full[st], 0, (t_begin + i) * kTileTok, bh);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = instr_desc(1, 64, 64, 1, 1);  // bf16, A M-major (O_lin^T), B N-major (dO)
      const uint32_t base = smem_u32(smem);
      bool ok = true;
      for (int i = 0; ok && i < n_tiles; ++i) {
        const int st = i % kStages;
        ok = mbar_wait(&bars->full[st], (i / kStages) & 1, abort_flag, status, 702);
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {  // 16 tokens per product
          const uint64_t a = smem_desc(base + st * kStageBytes + kk * 2048, 8192, 1024, kSwizzle128);
          const uint64_t b = smem_desc(base + st * kStageBytes + kTileBytes + kk * 2048, 8192, 1024, kSwizzle128);
          mma_f16(tmem, a, b, idesc, (i > 0 || kk > 0) ? 1u : 0u);
        }
        mma_commit(&bars->empty[st]);
      }
      if (ok) mma_commit(&bars->acc_full);
    }
  } else if (warp >= 4) {
    // rows of an M = 64 accumulator sit in lanes 0..15 of each 32-lane sub-partition
    const int quarter = warp & 3;
    const bool live = lane < 16;
    const int row = quarter * 16 + (lane & 15);
    float* dst = partials + (static_cast<size_t>(blockIdx.x) * kHeadDim + row) * kHeadDim;
    bool ok = true;
    if (n_tiles > 0) {
      ok = mbar_wait(&bars->acc_full, 0, abort_flag, status, 703);
      tc_fence_after();
    }
    ok = __all_sync(0xFFFFFFFFu, ok);
    if (ok) {
      const uint32_t lane_addr = tmem + ((static_cast<uint32_t>(quarter) * 32u) << 16);
#pragma unroll 1
      for (int cb = 0; cb < 64; cb += 32) {
        uint32_t v[32];
        if (n_tiles > 0) {
          tmem_ld32(lane_addr + cb, v);
          tmem_wait_ld();
        } else {
#pragma unroll
          for (int c = 0; c < 32; ++c) v[c] = 0u;
        }
        if (live) {
#pragma unroll
          for (int c = 0; c < 8; ++c)
            reinterpret_cast<uint4*>(dst + cb)[c] = make_uint4(v[4 * c], v[4 * c + 1], v[4 * c + 2], v[4 * c + 3]);
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, kTmemCols);
  }
}

// dW[h] = sum over batch entries and chunks of the partials, in a fixed order
__global__ void projgrad_reduce_kernel(const float* __restrict__ partials, int batch, int heads, int chunks,
                                       float* __restrict__ d_w) {
  const int h = blockIdx.x;
  for (int e = threadIdx.x; e < kHeadDim * kHeadDim; e += blockDim.x) {
    float acc = 0.f;
    for (int b = 0; b < batch; ++b)
      for (int c = 0; c < chunks; ++c)
        acc += partials[(static_cast<size_t>(b * heads + h) * chunks + c) * kHeadDim * kHeadDim + e];
    d_w[static_cast<size_t>(h) * kHeadDim * kHeadDim + e] = acc;
  }
}

int projgrad_chunks(const lite3r_shape& s, int sms) {
  const int planes = s.batch * s.heads;
  const int total_tiles = ceil_div(s.tokens, kTileTok);
  int chunks = std::max(1, (2 * sms + planes - 1) / planes);  // about two CTAs per SM
  return std::min(chunks, total_tiles);
}

}  // namespace

size_t train_workspace_bytes(const lite3r_shape& s) {
  // partials of the gradient for the largest chunk count any device could ask for (4 CTAs per plane-SM pair bound),
  // and the partial sums of the MSE term
  const size_t planes = static_cast<size_t>(s.batch) * s.heads;
  const size_t total_tiles = ceil_div(s.tokens, kTileTok);
  const size_t chunks = std::min<size_t>(total_tiles, std::max<size_t>(1, (2 * 256 + planes - 1) / planes));
  return planes * chunks * kHeadDim * kHeadDim * sizeof(float) + kMaxMseBlocks * sizeof(double) + 1024;
}

lite3r_status launch_fill_identity(float* dst, cudaStream_t stream) {
  fill_identity_kernel<<<(kHeadDim * kHeadDim + 255) / 256, 256, 0, stream>>>(dst);
  return after_launch();
}

lite3r_status launch_mse_distill(const void* student, const void* teacher, int dtype, size_t count, __nv_bfloat16* grad,
                                 double* loss, double* partials, cudaStream_t stream) {
  int sms = 0;
  lite3r_status st = sm_count(&sms);
  if (st != LITE3R_OK) return st;
  const size_t groups = count / 8;
  const int blocks = static_cast<int>(std::min<size_t>(std::min(kMaxMseBlocks, sms * 8), (groups + kMseThreads - 1) / kMseThreads));
  const float grad_scale = static_cast<float>(2.0 / static_cast<double>(count));
  if (dtype == LITE3R_BF16)
    mse_kernel<<<blocks, kMseThreads, 0, stream>>>(static_cast<const __nv_bfloat16*>(student),
                                                   static_cast<const __nv_bfloat16*>(teacher), groups, grad_scale, grad, partials);
  else
    mse_kernel<<<blocks, kMseThreads, 0, stream>>>(static_cast<const float*>(student), static_cast<const float*>(teacher),
                                                   groups, grad_scale, grad, partials);
  if ((st = after_launch()) != LITE3R_OK) return st;
  mse_finish_kernel<<<1, 32, 0, stream>>>(partials, blocks, 1.0 / static_cast<double>(count), loss);
  return after_launch();
}

lite3r_status launch_proj_lin_backward(const __nv_bfloat16* o_lin, const __nv_bfloat16* d_out, const lite3r_shape& s,
                                       float* d_w, float* partials, int* device_status, cudaStream_t stream) {
  int sms = 0;
  lite3r_status st = sm_count(&sms);
  if (st != LITE3R_OK) return st;
  const int planes = s.batch * s.heads;
  const int chunks = projgrad_chunks(s, sms);
  const int tiles_per_cta = ceil_div(ceil_div(s.tokens, kTileTok), chunks);
  alignas(64) CUtensorMap map_o, map_g;
  if ((st = make_tensor_map_3d(&map_o, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, o_lin, kHeadDim, s.tokens, planes, kHeadDim,
                               kTileTok, CU_TENSOR_MAP_SWIZZLE_128B)) != LITE3R_OK) return st;
  if ((st = make_tensor_map_3d(&map_g, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, d_out, kHeadDim, s.tokens, planes, kHeadDim,
                               kTileTok, CU_TENSOR_MAP_SWIZZLE_128B)) != LITE3R_OK) return st;
  if ((st = ensure_dynamic_smem(projgrad_kernel, static_cast<int>(kSmemBytes))) != LITE3R_OK) return st;
  projgrad_kernel<<<planes * chunks, kThreads, kSmemBytes, stream>>>(map_o, map_g, s.tokens, chunks, tiles_per_cta, partials,
                                                                     device_status);
  if ((st = after_launch()) != LITE3R_OK) return st;
  projgrad_reduce_kernel<<<s.heads, 256, 0, stream>>>(partials, s.batch, s.heads, chunks, d_w);
  return after_launch();
}

}  // namespace lite3r
