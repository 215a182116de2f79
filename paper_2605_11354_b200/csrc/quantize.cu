// K1: scaled FP8 (e4m3) quantisation, one scale per (b, h, token-block) tile of Bs x 64
// (paper appendix "Scaled FP8 Quantization"; epsilon from "Implementation Details").
//
// One CTA per tile at a time (persistent CTAs of 64 or 128 threads, 64 values per thread).  Tiles travel global ->
// shared memory by asynchronous 16-byte copies, a few tiles ahead of the one being processed; the tile maximum is
// reduced through shuffles and shared memory, then every value is divided by the scale (with the result of an
// IEEE fp32 division, so the codes equal a plain fp32 program's bit for bit), clamped, cast to e4m3 with
// round-to-nearest-even and written with 8-byte stores.  The same pass emits, where asked for, the per-tile column
// sums of the code values as exact integers (units of 2^-9), which is all the block plan needs.  HBM traffic: 2
// (bf16) or 4 (fp32) bytes read and 1 byte written per element; the instruction count per element decides how
// close the kernel gets to that, hence the packed fp32x2 arithmetic.
#include <atomic>

#include "common.cuh"
#include "sm100.cuh"

namespace lite3r {

namespace {

using sm100::add_f32x2;
using sm100::fma_f32x2;
using sm100::pack_f32x2;
using sm100::unpack_f32x2;

constexpr int kQuantThreadsSmall = 64;  // CTA size for 8 KB tiles

// Threads per CTA (= per tile).  The per-tile work that does not shrink with the tile (address arithmetic, the two
// reductions, barriers) is paid per thread, so few threads with many values each keep the instruction count per
// value low: the kernel is otherwise bound by instruction issue, not by HBM.
__host__ __device__ constexpr int cta_threads(int tile_bytes) { return tile_bytes <= 8192 ? kQuantThreadsSmall : 128; }
// Ring depth for a tile size and CTA size: enough CTAs per SM to cover the arithmetic, at least two tiles each.
__host__ __device__ constexpr int ring_depth(int tile_bytes, int threads) {
  const int budget = threads * 256;
  return budget / tile_bytes >= 2 ? budget / tile_bytes : 2;
}

// Asynchronous 16-byte copy global -> shared; with src_bytes = 0 the destination is zero-filled.
__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc, uint32_t src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(static_cast<uint32_t>(__cvta_generic_to_shared(smem_dst))),
               "l"(gsrc), "r"(src_bytes)
               : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

__device__ __forceinline__ void unpack8(const __nv_bfloat16* p, float v[8]) {
  const uint4 w = *reinterpret_cast<const uint4*>(p);
  const uint32_t x[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    v[2 * i] = __uint_as_float(x[i] << 16);
    v[2 * i + 1] = __uint_as_float(x[i] & 0xFFFF0000u);
  }
}
__device__ __forceinline__ void unpack8(const float* p, float v[8]) {
  const float4 a = *reinterpret_cast<const float4*>(p);
  const float4 b = *reinterpret_cast<const float4*>(p + 4);
  v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
  v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}

// Persistent CTAs walk the tiles with a stride of the grid size.  Tiles travel global -> shared memory through
// asynchronous copies, kDepth tiles ahead of the one being processed, so the bytes a CTA keeps in flight are set by
// its shared-memory ring and not by its registers: that, not the arithmetic, is what the HBM rate depends on.  Every
// thread copies and later reads only its own 8-value segments, so the ring needs no barrier.
// Up to three tensors of one shape (Q, K, V) quantised by one launch: the tiles of all of them form one walk.
struct QuantBatch {
  const void* x[3];
  long long stride_b[3], stride_h[3], stride_n[3];
  uint8_t* codes[3];
  float* scales[3];
  int* colsum[3];
  int count;
};

template <int BS, typename SrcT, int kThreads>
__global__ void __launch_bounds__(kThreads) quantize_kernel(const __grid_constant__ QuantBatch batch, int heads, int tokens,
                                                            int nb, int tiles) {
  constexpr int kRowsPerPass = kThreads / 8;  // a thread owns one 8-column segment of one row per pass
  constexpr int kPasses = BS / kRowsPerPass;
  constexpr bool kKeep = kPasses <= 8;  // the tile stays in registers between the two sweeps, else it is re-read
  constexpr int kSegBytes = 8 * sizeof(SrcT);                 // one thread's 8 values of one row
  constexpr int kTileBytes = kPasses * kThreads * kSegBytes;  // = BS * 64 * sizeof(SrcT)
  constexpr int kDepth = ring_depth(kTileBytes, kThreads);
  extern __shared__ __align__(16) uint8_t ring[];
  __shared__ float s_max[(kThreads + 31) / 32];
  __shared__ int s_col[kHeadDim];

  const int seg = threadIdx.x & 7;
  const int row0 = threadIdx.x >> 3;
  const int stride = static_cast<int>(gridDim.x);

  // Copies this thread's segments of the next tile of the walk into ring slot `slot` (nothing once the walk has
  // ended).  A position of the walk is (tensor, (b h), block); it advances by the grid size, which is split into whole
  // (b h) and blocks once, so that no division sits in the per-tile path.  A full tile is copied with one running
  // source pointer (one 64-bit add per pass); only a ragged last block takes the row-by-row form.
  const int bh_total = tiles / nb;
  const int step_bh = stride / nb, step_i = stride - step_bh * nb;
  int f_which = 0, f_bh = static_cast<int>(blockIdx.x) / nb, f_i = static_cast<int>(blockIdx.x) - f_bh * nb;
  while (f_bh >= bh_total && f_which < batch.count) {
    f_bh -= bh_total;
    ++f_which;
  }
  auto fetch = [&](int slot) {
    if (f_which < batch.count) {
      const int valid = min(BS, tokens - f_i * BS);
      const int b = f_bh / heads;
      const long long stride_n = batch.stride_n[f_which];
      const SrcT* src = static_cast<const SrcT*>(batch.x[f_which]) + b * batch.stride_b[f_which] +
                        (f_bh - b * heads) * batch.stride_h[f_which] + static_cast<long long>(f_i) * BS * stride_n + seg * 8;
      uint8_t* const dst0 = ring + slot * kTileBytes + threadIdx.x * kSegBytes;
      if (valid == BS) {
        const uint8_t* g = reinterpret_cast<const uint8_t*>(src + row0 * stride_n);
        const long long row_step = kRowsPerPass * stride_n * static_cast<long long>(sizeof(SrcT));
#pragma unroll
        for (int p = 0; p < kPasses; ++p) {
#pragma unroll
          for (int q = 0; q < kSegBytes / 16; ++q) cp_async16(dst0 + p * kThreads * kSegBytes + 16 * q, g + 16 * q, 16u);
          g += row_step;
        }
      } else {
#pragma unroll
        for (int p = 0; p < kPasses; ++p) {
          const int r = row0 + p * kRowsPerPass;
          const SrcT* g = src + (r < valid ? r : 0) * stride_n;  // rows past the end are zero-filled, not read
#pragma unroll
          for (int q = 0; q < kSegBytes / 16; ++q)
            cp_async16(dst0 + p * kThreads * kSegBytes + 16 * q, reinterpret_cast<const uint8_t*>(g) + 16 * q, r < valid ? 16u : 0u);
        }
      }
    }
    cp_async_commit();
    f_i += step_i;
    f_bh += step_bh;
    if (f_i >= nb) {
      f_i -= nb;
      ++f_bh;
    }
    while (f_bh >= bh_total && f_which < batch.count) {
      f_bh -= bh_total;
      ++f_which;
    }
  };

#pragma unroll
  for (int d = 0; d < kDepth - 1; ++d) fetch(d);

  int slot = 0;
  int which = 0, tile = blockIdx.x;
  while (tile >= tiles && which < batch.count) {
    tile -= tiles;
    ++which;
  }
  for (; which < batch.count;) {
    uint8_t* const codes = batch.codes[which];
    float* const scales = batch.scales[which];
    int* const colsum = batch.colsum[which];
    fetch(slot == 0 ? kDepth - 1 : slot - 1);
    cp_async_wait<kDepth - 1>();  // all but the kDepth-1 newest groups are complete: this tile has landed
    float v[kKeep ? kPasses : 1][8];
    const uint8_t* const mine = ring + slot * kTileBytes + threadIdx.x * kSegBytes;
    float amax = 0.f;
#pragma unroll
    for (int p = 0; p < kPasses; ++p) {
      float* const vp = v[kKeep ? p : 0];
      unpack8(reinterpret_cast<const SrcT*>(mine + p * kThreads * kSegBytes), vp);
#pragma unroll
      for (int c = 0; c < 8; ++c) amax = fmaxf(amax, fabsf(vp[c]));
    }
    slot = slot + 1 == kDepth ? 0 : slot + 1;

    amax = warp_max(amax);
    for (int c = threadIdx.x; c < kHeadDim; c += kThreads) s_col[c] = 0;
    if (kThreads > 32) {
      if ((threadIdx.x & 31) == 0) s_max[threadIdx.x >> 5] = amax;
      __syncthreads();
      amax = s_max[0];
#pragma unroll
      for (int w = 1; w < kThreads / 32; ++w) amax = fmaxf(amax, s_max[w]);
    } else {
      __syncwarp();
    }

    const float scale = __fdiv_rn(__fadd_rn(amax, 1e-8f), 448.0f);
    if (threadIdx.x == 0) scales[tile] = scale;
    // x / scale must be the IEEE quotient, but only its e4m3 rounding is kept.  The quotient lies strictly between
    // x * r_lo and x * r_hi with r = 1 / scale widened by 2^-20 either way (the reciprocal, the product and the
    // quotient itself are each rounded by at most 2^-24), and rounding to e4m3 is monotone: when both products give
    // the same code, that is the code of the quotient.  Otherwise (next to, or exactly on, a rounding boundary of the
    // e4m3 grid) the pair is redone with the division.
    const float r = __frcp_rn(scale);
    const float r_lo = r * (1.0f - 0x1p-20f), r_hi = r * (1.0f + 0x1p-20f);

    // fp32 sums of code values are exact (at most 16 values of at most 448 in units of 2^-9: 22 bits); two columns
    // per packed-pair instruction, like the two products
    uint64_t sums2[4] = {0ull, 0ull, 0ull, 0ull};
    const uint64_t r_lo2 = pack_f32x2(r_lo, r_lo), r_hi2 = pack_f32x2(r_hi, r_hi), neg0 = pack_f32x2(-0.f, -0.f);
    uint8_t* dst = codes + (static_cast<size_t>(tile) * BS) * kHeadDim + seg * 8;
#pragma unroll
    for (int p = 0; p < kPasses; ++p) {
      const int row = row0 + p * kRowsPerPass;
      float* const vp = v[kKeep ? p : 0];
      if (!kKeep) unpack8(reinterpret_cast<const SrcT*>(mine + p * kThreads * kSegBytes), vp);
      uint32_t two[4];
#pragma unroll
      for (int c = 0; c < 8; c += 2) {
        // the saturating conversion clamps to +-448 exactly like clamp-then-cast
        // x * r + (-0) is x * r, signed zeros included
        const uint64_t x2 = pack_f32x2(vp[c], vp[c + 1]);
        float2 y_lo, y_hi;
        unpack_f32x2(fma_f32x2(x2, r_lo2, neg0), y_lo.x, y_lo.y);
        unpack_f32x2(fma_f32x2(x2, r_hi2, neg0), y_hi.x, y_hi.y);
        const uint32_t lo = __nv_cvt_float2_to_fp8x2(y_lo, __NV_SATFINITE, __NV_E4M3);
        two[c >> 1] = __nv_cvt_float2_to_fp8x2(y_hi, __NV_SATFINITE, __NV_E4M3);
        // bf16 sources put about one quotient in a thousand exactly on a rounding boundary of the e4m3 grid, so some
        // lane of a warp gets here every few passes: only the pair in question is redone with the division
        if (lo != two[c >> 1])
          two[c >> 1] = __nv_cvt_float2_to_fp8x2(make_float2(__fdiv_rn(vp[c], scale), __fdiv_rn(vp[c + 1], scale)),
                                                 __NV_SATFINITE, __NV_E4M3);
      }
      if (colsum != nullptr) {
#pragma unroll
        for (int c = 0; c < 8; c += 2) {
          const __half2_raw back = __nv_cvt_fp8x2_to_halfraw2(static_cast<__nv_fp8x2_storage_t>(two[c >> 1]), __NV_E4M3);
          const float2 f = __half22float2(__half2(back));
          sums2[c >> 1] = add_f32x2(sums2[c >> 1], pack_f32x2(f.x, f.y));
        }
      }
      *reinterpret_cast<uint2*>(dst + static_cast<size_t>(row) * kHeadDim) =
          make_uint2(two[0] | (two[1] << 16), two[2] | (two[3] << 16));
    }
    if (colsum != nullptr) {
      // Column sums over the four row groups of the warp (lanes that differ in bits 3 and 4): each exchange halves
      // the number of columns a lane still carries, so eight columns take six shuffles instead of sixteen.
      int s8[8];
#pragma unroll
      for (int c = 0; c < 8; c += 2) {  // exact integers, units of 2^-9
        float lo, hi;
        unpack_f32x2(sums2[c >> 1], lo, hi);
        s8[c] = __float2int_rn(lo * 512.0f);
        s8[c + 1] = __float2int_rn(hi * 512.0f);
      }
      const bool up16 = (threadIdx.x & 16) != 0, up8 = (threadIdx.x & 8) != 0;
      int s4[4], s2[2];
#pragma unroll
      for (int c = 0; c < 4; ++c) {  // lanes with bit 4 clear keep columns 0-3, the others columns 4-7
        const int give = up16 ? s8[c] : s8[c + 4];
        const int keep = up16 ? s8[c + 4] : s8[c];
        s4[c] = keep + __shfl_xor_sync(0xFFFFFFFFu, give, 16);
      }
#pragma unroll
      for (int c = 0; c < 2; ++c) {  // lanes with bit 3 clear keep the lower two of those
        const int give = up8 ? s4[c] : s4[c + 2];
        const int keep = up8 ? s4[c + 2] : s4[c];
        s2[c] = keep + __shfl_xor_sync(0xFFFFFFFFu, give, 8);
      }
      const int col = seg * 8 + (up16 ? 4 : 0) + (up8 ? 2 : 0);
      atomicAdd(&s_col[col], s2[0]);
      atomicAdd(&s_col[col + 1], s2[1]);
      __syncthreads();
      for (int c = threadIdx.x; c < kHeadDim; c += kThreads) colsum[static_cast<size_t>(tile) * kHeadDim + c] = s_col[c];
    }
    __syncthreads();  // s_max and s_col are reused by the next tile
    tile += stride;
    while (tile >= tiles && which < batch.count) {
      tile -= tiles;
      ++which;
    }
  }
}

template <int BS, typename SrcT>
lite3r_status launch(const QuantBatch& batch, const lite3r_shape& s, cudaStream_t stream) {
  const int nb = ceil_div(s.tokens, BS);
  const int tiles = s.batch * s.heads * nb;
  constexpr int kTileBytes = BS * kHeadDim * static_cast<int>(sizeof(SrcT));
  constexpr int kThreads = cta_threads(kTileBytes);
  constexpr int kSmem = ring_depth(kTileBytes, kThreads) * kTileBytes;
  int sms = 0;
  lite3r_status st = sm_count(&sms);
  if (st != LITE3R_OK) return st;
  st = ensure_dynamic_smem(quantize_kernel<BS, SrcT, kThreads>, kSmem);
  if (st != LITE3R_OK) return st;
  // resident CTAs per SM: a property of the kernel and the part (every supported device is the same part), asked once
  static std::atomic<int> per_sm_cached{0};
  int per_sm = per_sm_cached.load(std::memory_order_relaxed);
  if (per_sm == 0) {
    st = record_cuda(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, quantize_kernel<BS, SrcT, kThreads>, kThreads, kSmem));
    if (st != LITE3R_OK) return st;
    if (per_sm < 1) per_sm = 1;
    per_sm_cached.store(per_sm, std::memory_order_relaxed);
  }
  const long long all = static_cast<long long>(tiles) * batch.count;
  const int grid = static_cast<int>(all < static_cast<long long>(sms) * per_sm ? all : static_cast<long long>(sms) * per_sm);
  quantize_kernel<BS, SrcT, kThreads><<<grid, kThreads, kSmem, stream>>>(batch, s.heads, s.tokens, nb, tiles);
  return after_launch();
}

}  // namespace

lite3r_status launch_quantize(const lite3r_tensor* const* x, const lite3r_fp8* out, int count, const lite3r_shape& s,
                              cudaStream_t stream) {
  QuantBatch batch = {};
  batch.count = count;
  for (int n = 0; n < count; ++n) {
    batch.x[n] = x[n]->ptr;
    batch.stride_b[n] = x[n]->stride_b;
    batch.stride_h[n] = x[n]->stride_h;
    batch.stride_n[n] = x[n]->stride_n;
    batch.codes[n] = out[n].codes;
    batch.scales[n] = out[n].scales;
    batch.colsum[n] = out[n].colsum;
  }
  if (x[0]->dtype == LITE3R_BF16) {
    return s.block == 64 ? launch<64, __nv_bfloat16>(batch, s, stream) : launch<128, __nv_bfloat16>(batch, s, stream);
  }
  return s.block == 64 ? launch<64, float>(batch, s, stream) : launch<128, float>(batch, s, stream);
}

}  // namespace lite3r
