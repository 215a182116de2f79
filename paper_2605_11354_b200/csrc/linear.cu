// The FP8 linear layer in front of the attention (Algorithm 2 "FP8 fake-quantised linear" in its deployed form; Eq. 2):
//   quantise_rows   per-token (activations) / per-output-row (weights) scaled e4m3 quantiser
//   linear_fp8      y = x_q W_q^T + b on tcgen05 (e4m3 x e4m3, fp32 accumulation in TMEM), scales applied in the epilogue
//   qkv_project     the same product for the qkv projection, with the block quantiser of the attention path fused into
//                   its epilogue: Q, K and V leave the kernel as e4m3 codes + per-(b, h, token-block) scales + column
//                   sums in the library's own layout, so the separate quantiser pass over Q, K, V disappears.
//
// GEMM kernel: persistent CTAs (one per SM) over 128 x 256 output tiles (128 tokens x 256 output columns = four heads
// of the projection).  Warp 0 = TMA producer (A = activation codes, B = weight codes, both K-major rows of 128 bytes,
// 128B swizzle, ring of four stages), warp 1 = MMA issuer (four kind::f8f6f4 products of K = 32 per stage into one of
// two accumulators), warps 4-19 = four epilogue warpgroups, one per 64 columns of the tile (thread = token row = TMEM
// lane; two passes over the accumulator, maximum then codes, so that a row of 64 values never has to stay in
// registers).  The products of the next tile run under the epilogue of this one.
// Every mbarrier wait is bounded; on expiry the CTA sets *device_status and its roles leave their loops.
#include <algorithm>

#include "common.cuh"
#include "sm100.cuh"

namespace lite3r {

namespace {

using namespace sm100;

// ------------------------------------------------------------------------------------------------ row quantiser
__device__ __forceinline__ void load8(const __nv_bfloat16* p, float v[8]) {
  const uint4 w = *reinterpret_cast<const uint4*>(p);
  const uint32_t x[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    v[2 * i] = __uint_as_float(x[i] << 16);
    v[2 * i + 1] = __uint_as_float(x[i] & 0xFFFF0000u);
  }
}
__device__ __forceinline__ void load8(const float* p, float v[8]) {
  const float4 a = *reinterpret_cast<const float4*>(p);
  const float4 b = *reinterpret_cast<const float4*>(p + 4);
  v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
  v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}
// e4m3 codes of x / scale (IEEE fp32 division, saturation at +-448, round to nearest even), two values per call
__device__ __forceinline__ uint32_t quantise_pair(float a, float b, float scale) {
  return __nv_cvt_float2_to_fp8x2(make_float2(__fdiv_rn(a, scale), __fdiv_rn(b, scale)), __NV_SATFINITE, __NV_E4M3);
}

// One warp per row.  Rows of up to 1024 values are held in registers; longer ones are read twice (maximum, then codes;
// the second read comes from L1 / L2).
template <typename SrcT>
__global__ void __launch_bounds__(256) rowquant_kernel(const SrcT* __restrict__ x, long long row_stride, int rows, int cols,
                                                       uint8_t* __restrict__ codes, float* __restrict__ scales) {
  const int lane = threadIdx.x & 31;
  const int warps = (gridDim.x * blockDim.x) >> 5;
  const int segs = cols >> 3;
  for (int row = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; row < rows; row += warps) {
    const SrcT* src = x + static_cast<long long>(row) * row_stride;
    if (segs <= 4 * 32) {
      // rows of up to 1024 values stay in registers between the two sweeps (four 8-value segments per lane, all
      // requested before the first is used): one pass over memory
      float v[4][8];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        if (lane + 32 * q < segs) {
          load8(src + (lane + 32 * q) * 8, v[q]);
        } else {
#pragma unroll
          for (int c = 0; c < 8; ++c) v[q][c] = 0.f;
        }
      }
      float amax = 0.f;
#pragma unroll
      for (int q = 0; q < 4; ++q)
#pragma unroll
        for (int c = 0; c < 8; ++c) amax = fmaxf(amax, fabsf(v[q][c]));
      amax = warp_max(amax);
      const float scale = __fdiv_rn(__fadd_rn(amax, 1e-8f), 448.0f);
      if (lane == 0) scales[row] = scale;
      uint8_t* dst = codes + static_cast<size_t>(row) * cols;
      const float rcp = __frcp_rn(scale);
      const uint64_t r_lo2 = pack_f32x2(rcp * (1.0f - 0x1p-20f), rcp * (1.0f - 0x1p-20f));
      const uint64_t r_hi2 = pack_f32x2(rcp * (1.0f + 0x1p-20f), rcp * (1.0f + 0x1p-20f));
      const uint64_t neg0 = pack_f32x2(-0.f, -0.f);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        if (lane + 32 * q >= segs) continue;
        uint32_t two[4], differ = 0u;
#pragma unroll
        for (int c = 0; c < 8; c += 2) {
          const uint64_t x2 = pack_f32x2(v[q][c], v[q][c + 1]);
          float2 q_lo, q_hi;
          unpack_f32x2(fma_f32x2(x2, r_lo2, neg0), q_lo.x, q_lo.y);
          unpack_f32x2(fma_f32x2(x2, r_hi2, neg0), q_hi.x, q_hi.y);
          const uint32_t lo = __nv_cvt_float2_to_fp8x2(q_lo, __NV_SATFINITE, __NV_E4M3);
          two[c >> 1] = __nv_cvt_float2_to_fp8x2(q_hi, __NV_SATFINITE, __NV_E4M3);
          differ |= lo ^ two[c >> 1];
        }
        if (differ != 0u) {  // next to a rounding boundary of the e4m3 grid: redone with the division
#pragma unroll
          for (int c = 0; c < 8; c += 2) two[c >> 1] = quantise_pair(v[q][c], v[q][c + 1], scale);
        }
        *reinterpret_cast<uint2*>(dst + (lane + 32 * q) * 8) = make_uint2(two[0] | (two[1] << 16), two[2] | (two[3] << 16));
      }
      continue;
    }
    float amax = 0.f;
    for (int s = lane; s < segs; s += 32) {
      float v[8];
      load8(src + s * 8, v);
#pragma unroll
      for (int c = 0; c < 8; ++c) amax = fmaxf(amax, fabsf(v[c]));
    }
    amax = warp_max(amax);
    const float scale = __fdiv_rn(__fadd_rn(amax, 1e-8f), 448.0f);
    if (lane == 0) scales[row] = scale;
    uint8_t* dst = codes + static_cast<size_t>(row) * cols;
    // x / scale must be the IEEE quotient, but only its e4m3 rounding is kept: the quotient lies between x * r_lo and
    // x * r_hi (r = 1 / scale widened by 2^-20 either way) and rounding is monotone, so equal codes of the two products
    // are the quotient's code; otherwise the eight values are redone with the division.
    const float rcp = __frcp_rn(scale);
    const uint64_t r_lo2 = pack_f32x2(rcp * (1.0f - 0x1p-20f), rcp * (1.0f - 0x1p-20f));
    const uint64_t r_hi2 = pack_f32x2(rcp * (1.0f + 0x1p-20f), rcp * (1.0f + 0x1p-20f));
    const uint64_t neg0 = pack_f32x2(-0.f, -0.f);
    for (int s = lane; s < segs; s += 32) {
      float v[8];
      load8(src + s * 8, v);
      uint32_t two[4], differ = 0u;
#pragma unroll
      for (int c = 0; c < 8; c += 2) {
        const uint64_t x2 = pack_f32x2(v[c], v[c + 1]);
        float2 q_lo, q_hi;
        unpack_f32x2(fma_f32x2(x2, r_lo2, neg0), q_lo.x, q_lo.y);
        unpack_f32x2(fma_f32x2(x2, r_hi2, neg0), q_hi.x, q_hi.y);
        const uint32_t lo = __nv_cvt_float2_to_fp8x2(q_lo, __NV_SATFINITE, __NV_E4M3);
        two[c >> 1] = __nv_cvt_float2_to_fp8x2(q_hi, __NV_SATFINITE, __NV_E4M3);
        differ |= lo ^ two[c >> 1];
      }
      if (differ != 0u) {
#pragma unroll
        for (int c = 0; c < 8; c += 2) two[c >> 1] = quantise_pair(v[c], v[c + 1], scale);
      }
      *reinterpret_cast<uint2*>(dst + s * 8) = make_uint2(two[0] | (two[1] << 16), two[2] | (two[3] << 16));
    }
  }
}

// ------------------------------------------------------------------------------------------------ GEMM
constexpr int kStages = 4;
constexpr int kTileM = 128, kTileN = 256, kTileK = 128;  // K in bytes = e4m3 elements
constexpr int kEpiGroups = kTileN / 64;                   // epilogue warpgroups, one per 64 columns (one head) of the tile
constexpr int kThreads = 128 + kEpiGroups * 128;          // 4 control warps + the epilogue warpgroups
constexpr uint32_t kStageBytes = kTileM * kTileK + kTileN * kTileK;  // 48 KB
constexpr uint32_t kOffB = kTileM * kTileK;
constexpr uint32_t kOffMisc = kStages * kStageBytes;  // column scales (1 KB), bias (1 KB), reduction slots, column sums
constexpr uint32_t kOffBar = kOffMisc + 5120;  // + column sums (2 KB)
constexpr uint32_t kSmemBytes = kOffBar + 256;  // 201984 B: one CTA per SM
constexpr uint32_t kAccCols = kTileN;           // one accumulator (128 x 256 fp32)
constexpr uint32_t kTmemCols = 2 * kAccCols;    // two of them (all of tensor memory): the products of the next tile run
                                                // under this tile's epilogue

struct Bars {
  uint64_t full[kStages], empty[kStages];
  uint64_t acc_full[2], acc_empty[2];  // accumulator written (issuer -> epilogue) / read out (epilogue -> issuer)
  uint32_t tmem_base;
  int abort;
};

struct LinearParams {
  const float* x_scales;  // [rows]
  const float* w_scales;  // [d_out]
  const float* bias;      // [d_out] or null
  int rows, d_in, d_out;
  int col_tiles, tiles;   // output tiles per row of tiles, and in all
  // plain output
  void* y;
  long long y_stride;  // elements
  int y_dtype;
  // fused qkv output: rows = batch * tokens, d_out = 3 * heads * 64
  int fused, batch, tokens, heads, block, nb;
  uint8_t* codes[3];
  float* scales[3];
  int* colsum[3];
  int* status;
};

__device__ __forceinline__ void named_barrier_sync(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// Persistent CTAs (one per SM) walk the output tiles blockIdx.x, blockIdx.x + gridDim.x, ... (tiles of one row of
// tiles are neighbours, so the CTAs running at any time share their activation rows in L2).  The operand ring and the
// two accumulators are never re-initialised: ring stages and barrier parities continue on a running count of K steps,
// the accumulators alternate with the CTA's tile count.  The producer and the issuer run ahead into the next tile
// while the epilogue warps drain the previous accumulator: with one tile per CTA the operand loads stopped during
// every epilogue and the kernel was bound by the latency of its loads, not by the tensor pipe or the epilogue.
__global__ void __launch_bounds__(kThreads, 1)
linear_fp8_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                  const LinearParams p) {
  extern __shared__ __align__(1024) uint8_t smem[];
  Bars* bars = reinterpret_cast<Bars*>(smem + kOffBar);
  volatile int* abort_flag = &bars->abort;
  if ((smem_u32(smem) & 1023u) != 0) {
    if (threadIdx.x == 0 && p.status != nullptr) atomicCAS(p.status, 0, 900);
    return;
  }
  if (p.status != nullptr && *reinterpret_cast<volatile int*>(p.status) != 0) return;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // row tiles never run through a batch boundary in the fused form (a tile belongs to one sequence)
  const int tiles_per_seq = ((p.fused ? p.tokens : p.rows) + kTileM - 1) / kTileM;
  const int k_steps = p.d_in / kTileK;
  struct TileAt {
    int seq, tile_in_seq, row0, rows_valid, col0;
  };
  auto tile_at = [&](int tile_id) {
    TileAt t;
    const int row_tile = tile_id / p.col_tiles;
    t.col0 = (tile_id - row_tile * p.col_tiles) * kTileN;
    t.seq = row_tile / tiles_per_seq;
    t.tile_in_seq = row_tile - t.seq * tiles_per_seq;
    t.row0 = p.fused ? t.seq * p.tokens + t.tile_in_seq * kTileM : row_tile * kTileM;
    t.rows_valid = min(kTileM, (p.fused ? p.tokens : p.rows) - t.tile_in_seq * kTileM);
    return t;
  };

  float* const s_wscale = reinterpret_cast<float*>(smem + kOffMisc);
  float* const s_bias = s_wscale + kTileN;
  float* const s_red = s_bias + kTileN;  // 4 floats per epilogue warpgroup
  int* const s_colsum = reinterpret_cast<int*>(s_red + 4 * kEpiGroups);  // 128 ints per epilogue warpgroup

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&bars->full[s], 1);
      mbar_init(&bars->empty[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&bars->acc_full[b], 1);
      mbar_init(&bars->acc_empty[b], kEpiGroups * 128);
    }
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
      tma_prefetch_desc(&map_x);
      tma_prefetch_desc(&map_w);
      bool ok = true;
      int kc = 0;  // K steps issued so far, through all tiles
      for (int tile_id = blockIdx.x; ok && tile_id < p.tiles; tile_id += gridDim.x) {
        const TileAt t = tile_at(tile_id);
        for (int k = 0; ok && k < k_steps; ++k, ++kc) {
          const int st = kc % kStages;
          if (kc >= kStages)
            ok = mbar_wait(&bars->empty[st], ((kc - kStages) / kStages) & 1, abort_flag, p.status, 601, 32);
          if (!ok) break;
          mbar_arrive_expect_tx(&bars->full[st], kStageBytes);
          tma_load_2d(smem + st * kStageBytes, &map_x, &bars->full[st], k * kTileK, t.row0);
          tma_load_2d(smem + st * kStageBytes + kOffB, &map_w, &bars->full[st], k * kTileK, t.col0);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = instr_desc(0, kTileM, kTileN, 0, 0);  // e4m3 x e4m3, both K-major
      const uint64_t a_desc0 = smem_desc(smem_u32(smem), 16, 1024, kSwizzle128);
      const uint64_t b_desc0 = smem_desc(smem_u32(smem) + kOffB, 16, 1024, kSwizzle128);
      bool ok = true;
      int kc = 0, it = 0;
      for (int tile_id = blockIdx.x; ok && tile_id < p.tiles; tile_id += gridDim.x, ++it) {
        const int ab = it & 1;
        // the accumulator was last used two tiles ago: wait until the epilogue warps have read it out
        if (it >= 2) ok = mbar_wait(&bars->acc_empty[ab], ((it - 2) >> 1) & 1, abort_flag, p.status, 604);
        tc_fence_after();
        for (int k = 0; ok && k < k_steps; ++k, ++kc) {
          const int st = kc % kStages;
          ok = mbar_wait(&bars->full[st], (kc / kStages) & 1, abort_flag, p.status, 602);
          if (!ok) break;
          tc_fence_after();
          const uint64_t off = static_cast<uint64_t>((st * kStageBytes) >> 4);
#pragma unroll
          for (int kk = 0; kk < 4; ++kk)
            mma_f8(tmem + ab * kAccCols, a_desc0 + off + ((kk * 32) >> 4), b_desc0 + off + ((kk * 32) >> 4), idesc,
                   (k > 0 || kk > 0) ? 1u : 0u);
          mma_commit(&bars->empty[st]);
        }
        if (ok) mma_commit(&bars->acc_full[ab]);
      }
    }
  } else if (warp >= 4) {
    // ------------------------------------------------------------------------------------------ epilogue
    const int quarter = warp & 3;
    const int hh = (warp - 4) >> 2;     // which 64 columns of the tile this warpgroup owns
    const int r = quarter * 32 + lane;  // row of the tile = TMEM lane
    const int tid = threadIdx.x - (4 + hh * 4) * 32;  // thread of the warpgroup
    float* const wsc = s_wscale + hh * 64;
    float* const bia = s_bias + hh * 64;
    const int bar_id = 1 + hh;
    bool ok = true;
    int it = 0;
    for (int tile_id = blockIdx.x; ok && tile_id < p.tiles; tile_id += gridDim.x, ++it) {
    const TileAt ta = tile_at(tile_id);
    const int row0 = ta.row0, rows_valid = ta.rows_valid, seq = ta.seq, tile_in_seq = ta.tile_in_seq;
    const int ab = it & 1;
    const bool row_ok = r < rows_valid;
    const uint32_t acc_addr = tmem + ((static_cast<uint32_t>(quarter) * 32u) << 16) + ab * kAccCols + hh * 64;
    const float sx = row_ok ? __ldg(p.x_scales + row0 + r) : 0.f;
    const int col = ta.col0 + hh * 64;
    // this warpgroup's 64 column scales and biases (the previous tile's were released by the barrier that ends a tile)
    if (tid < 64) {
      wsc[tid] = col + tid < p.d_out ? __ldg(p.w_scales + col + tid) : 0.f;
      bia[tid] = (p.bias != nullptr && col + tid < p.d_out) ? __ldg(p.bias + col + tid) : 0.f;
    }
    named_barrier_sync(bar_id, 128);
    ok = mbar_wait(&bars->acc_full[ab], (it >> 1) & 1, abort_flag, p.status, 603);
    tc_fence_after();
    ok = __all_sync(0xFFFFFFFFu, ok);
    if (!ok) break;
    if (col < p.d_out && !p.fused) {
      // y = acc * (sx * sw) + b, written row by row (a thread owns 128 contiguous bytes per 32 fp32 columns)
      uint8_t* const yrow = static_cast<uint8_t*>(p.y) +
                            static_cast<long long>(row0 + r) * p.y_stride * (p.y_dtype == LITE3R_F32 ? 4 : 2);
#pragma unroll 1
      for (int cb = 0; cb < 64; cb += 32) {
        uint32_t v[32];
        tmem_ld32(acc_addr + cb, v);
        tmem_wait_ld();
        if (cb == 32) {  // the accumulator is in registers: the issuer may reuse it
          tc_fence_before();
          mbar_arrive(&bars->acc_empty[ab]);
        }
        if (!row_ok) continue;
        float y[32];
#pragma unroll
        for (int c = 0; c < 32; ++c) y[c] = fmaf(__uint_as_float(v[c]), sx * wsc[cb + c], bia[cb + c]);
        if (p.y_dtype == LITE3R_F32) {
          float4* dst = reinterpret_cast<float4*>(yrow + static_cast<size_t>(col + cb) * 4);
#pragma unroll
          for (int c = 0; c < 8; ++c) dst[c] = make_float4(y[4 * c], y[4 * c + 1], y[4 * c + 2], y[4 * c + 3]);
        } else {
          uint4* dst = reinterpret_cast<uint4*>(yrow + static_cast<size_t>(col + cb) * 2);
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            uint32_t w[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              if (p.y_dtype == LITE3R_BF16) {
                __nv_bfloat162 h = __floats2bfloat162_rn(y[8 * c + 2 * q], y[8 * c + 2 * q + 1]);
                w[q] = *reinterpret_cast<uint32_t*>(&h);
              } else {
                __half2 h = __floats2half2_rn(y[8 * c + 2 * q], y[8 * c + 2 * q + 1]);
                w[q] = *reinterpret_cast<uint32_t*>(&h);
              }
            }
            dst[c] = make_uint4(w[0], w[1], w[2], w[3]);
          }
        }
      }
    } else if (col < p.d_out) {
      // Fused block quantiser: this warpgroup's 64 columns are one head; each (head, token block) sub-tile gets its
      // maximum, scale, codes and column sums exactly as the stand-alone quantiser computes them from fp32 values.
      const int hd = p.heads * kHeadDim;
      const int part = col / hd, head = (col - part * hd) / kHeadDim;  // 0 q, 1 k, 2 v
      const int blocks_in_tile = kTileM / p.block;            // 2 at block 64, 1 at block 128
      const int my_block = r / p.block;                       // token block of the tile this row is in
      const int block_first_warp = my_block * (p.block / 32);  // first warp (0..3) of that block in the warpgroup
      float* const red = s_red + hh * 4;
      // pass 1: the row's largest magnitude, then the block's
      // (two columns per instruction: sx * sw and acc * (sx sw) + b as packed fp32 pairs, each lane rounded exactly
      // as the scalar expression would be)
      const uint64_t sx2 = pack_f32x2(sx, sx), neg0 = pack_f32x2(-0.f, -0.f);
      float amax = 0.f;
#pragma unroll 1
      for (int cb = 0; cb < 64; cb += 32) {
        uint32_t v[32];
        tmem_ld32(acc_addr + cb, v);
        tmem_wait_ld();
#pragma unroll
        for (int c = 0; c < 32; c += 4) {
          const ulonglong2 sw4 = *reinterpret_cast<const ulonglong2*>(wsc + cb + c);
          const ulonglong2 b4 = *reinterpret_cast<const ulonglong2*>(bia + cb + c);
          float y0, y1, y2, y3;
          unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(v[c]), __uint_as_float(v[c + 1])), fma_f32x2(sx2, sw4.x, neg0), b4.x), y0, y1);
          unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(v[c + 2]), __uint_as_float(v[c + 3])), fma_f32x2(sx2, sw4.y, neg0), b4.y), y2, y3);
          amax = fmaxf(amax, fmaxf(fmaxf(fabsf(y0), fabsf(y1)), fmaxf(fabsf(y2), fabsf(y3))));
        }
      }
      amax = warp_max(row_ok ? amax : 0.f);
      if (lane == 0) red[quarter] = amax;
      named_barrier_sync(bar_id, 128);
      amax = 0.f;
      for (int wq = 0; wq < p.block / 32; ++wq) amax = fmaxf(amax, red[block_first_warp + wq]);
      const float scale = __fdiv_rn(__fadd_rn(amax, 1e-8f), 448.0f);
      const int token_block = tile_in_seq * blocks_in_tile + my_block;
      const bool block_ok = token_block < p.nb;
      const size_t tile_out = (static_cast<size_t>(seq) * p.heads + head) * p.nb + token_block;
      if (block_ok && (r % p.block) == 0) p.scales[part][tile_out] = scale;
      // pass 2: codes.  x / scale must be the IEEE quotient, but only its e4m3 rounding is kept: the quotient lies
      // between x * r_lo and x * r_hi (r = 1 / scale widened by 2^-20 either way) and rounding is monotone, so equal
      // codes of the two products are the quotient's code; otherwise the pair is redone with the division.
      const float rcp = __frcp_rn(scale);
      const float r_lo = rcp * (1.0f - 0x1p-20f), r_hi = rcp * (1.0f + 0x1p-20f);
      const uint64_t r_lo2 = pack_f32x2(r_lo, r_lo), r_hi2 = pack_f32x2(r_hi, r_hi);
      const bool want_colsum = p.colsum[part] != nullptr;
      uint4* const gdst = reinterpret_cast<uint4*>(p.codes[part] + (tile_out * p.block + (r % p.block)) * kHeadDim);
#pragma unroll 1
      for (int cb = 0; cb < 64; cb += 32) {
        uint32_t v[32], packed[8];
        tmem_ld32(acc_addr + cb, v);
        tmem_wait_ld();
        if (cb == 32) {  // the accumulator is in registers: the issuer may reuse it
          tc_fence_before();
          mbar_arrive(&bars->acc_empty[ab]);
        }
#pragma unroll
        for (int c = 0; c < 32; c += 4) {
          const ulonglong2 sw4 = *reinterpret_cast<const ulonglong2*>(wsc + cb + c);
          const ulonglong2 b4 = *reinterpret_cast<const ulonglong2*>(bia + cb + c);
          const unsigned long long sws[2] = {sw4.x, sw4.y}, bs[2] = {b4.x, b4.y};
          uint32_t two[2];
#pragma unroll
          for (int h2 = 0; h2 < 2; ++h2) {
            const uint64_t y2 = fma_f32x2(pack_f32x2(__uint_as_float(v[c + 2 * h2]), __uint_as_float(v[c + 2 * h2 + 1])),
                                          fma_f32x2(sx2, sws[h2], neg0), bs[h2]);
            float2 q_lo, q_hi;
            unpack_f32x2(fma_f32x2(y2, r_lo2, neg0), q_lo.x, q_lo.y);
            unpack_f32x2(fma_f32x2(y2, r_hi2, neg0), q_hi.x, q_hi.y);
            const uint32_t lo = __nv_cvt_float2_to_fp8x2(q_lo, __NV_SATFINITE, __NV_E4M3);
            uint32_t hi = __nv_cvt_float2_to_fp8x2(q_hi, __NV_SATFINITE, __NV_E4M3);
            if (lo != hi) {
              float y0, y1;
              unpack_f32x2(y2, y0, y1);
              hi = quantise_pair(y0, y1, scale);
            }
            two[h2] = hi;
          }
          packed[c >> 2] = row_ok ? (two[0] | (two[1] << 16)) : 0u;
        }
        if (block_ok) {  // rows past the sequence end inside an existing block are written as zeros
          gdst[cb / 16] = make_uint4(packed[0], packed[1], packed[2], packed[3]);
          gdst[cb / 16 + 1] = make_uint4(packed[4], packed[5], packed[6], packed[7]);
        }
      }
      if (want_colsum) {
        // Column sums of the code values (exact integers in units of 2^-9) from the codes the warpgroup has just written
        // (the barrier orders them; the loads go to L2, past the first-level cache): a thread adds four columns over 16
        // rows in fp32 (exact: at most 16 x 448 in steps of 2^-9), the eight row groups of the tile meet in shared memory.
        int* const cs = s_colsum + hh * 128;  // [token block of the tile][64]
        cs[tid] = 0;
        named_barrier_sync(bar_id, 128);
        {
          const int cg = tid & 15, row_first = (tid >> 4) * 16;
          const int blk = row_first / p.block;
          const int tb = tile_in_seq * blocks_in_tile + blk;
          if (tb < p.nb) {
            const size_t out_tile = (static_cast<size_t>(seq) * p.heads + head) * p.nb + tb;
            const uint32_t* src =
                reinterpret_cast<const uint32_t*>(p.codes[part] + (out_tile * p.block + (row_first % p.block)) * kHeadDim) + cg;
            float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll 4
            for (int rr = 0; rr < 16; ++rr) {
              const uint32_t w4 = __ldcg(src + rr * (kHeadDim / 4));
              const __half2_raw lo = __nv_cvt_fp8x2_to_halfraw2(static_cast<__nv_fp8x2_storage_t>(w4 & 0xFFFFu), __NV_E4M3);
              const __half2_raw hi = __nv_cvt_fp8x2_to_halfraw2(static_cast<__nv_fp8x2_storage_t>(w4 >> 16), __NV_E4M3);
              const float2 f01 = __half22float2(__half2(lo)), f23 = __half22float2(__half2(hi));
              a0 += f01.x;
              a1 += f01.y;
              a2 += f23.x;
              a3 += f23.y;
            }
            int* dst = cs + blk * 64 + cg * 4;
            atomicAdd(dst, __float2int_rn(a0 * 512.f));
            atomicAdd(dst + 1, __float2int_rn(a1 * 512.f));
            atomicAdd(dst + 2, __float2int_rn(a2 * 512.f));
            atomicAdd(dst + 3, __float2int_rn(a3 * 512.f));
          }
        }
        named_barrier_sync(bar_id, 128);
        if (tid < blocks_in_tile * 64) {
          const int blk = tid >> 6, cc = tid & 63;
          const int tb = tile_in_seq * blocks_in_tile + blk;
          if (tb < p.nb)
            p.colsum[part][((static_cast<size_t>(seq) * p.heads + head) * p.nb + tb) * kHeadDim + cc] = cs[tid];
        }
      }
    } else {
      tc_fence_before();
      mbar_arrive(&bars->acc_empty[ab]);  // nothing to do for columns past the output
    }
    named_barrier_sync(bar_id, 128);  // the column scales, biases and reduction slots are rewritten for the next tile
    }  // tiles
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, kTmemCols);
  }
}

lite3r_status launch_gemm(const uint8_t* x_codes, const uint8_t* w_codes, const LinearParams& p, cudaStream_t stream) {
  alignas(64) CUtensorMap map_x, map_w;
  lite3r_status st;
  if ((st = make_tensor_map_2d(&map_x, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, x_codes, p.d_in, p.rows, kTileK, kTileM,
                               CU_TENSOR_MAP_SWIZZLE_128B)) != LITE3R_OK) return st;
  if ((st = make_tensor_map_2d(&map_w, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, w_codes, p.d_in, p.d_out, kTileK, kTileN,
                               CU_TENSOR_MAP_SWIZZLE_128B)) != LITE3R_OK) return st;
  if ((st = ensure_dynamic_smem(linear_fp8_kernel, static_cast<int>(kSmemBytes))) != LITE3R_OK) return st;
  const int row_tiles = p.fused ? p.batch * ceil_div(p.tokens, kTileM) : ceil_div(p.rows, kTileM);
  LinearParams q = p;
  q.col_tiles = ceil_div(p.d_out, kTileN);
  q.tiles = q.col_tiles * row_tiles;
  int sms = 0;
  if ((st = sm_count(&sms)) != LITE3R_OK) return st;
  const int grid = q.tiles < sms ? q.tiles : sms;
  linear_fp8_kernel<<<grid, kThreads, kSmemBytes, stream>>>(map_x, map_w, q);
  return after_launch();
}

}  // namespace

lite3r_status launch_rowquant(const void* x, int dtype, long long row_stride, int rows, int cols, uint8_t* codes,
                              float* scales, cudaStream_t stream) {
  int sms = 0;
  lite3r_status st = sm_count(&sms);
  if (st != LITE3R_OK) return st;
  const int blocks = std::min(ceil_div(rows, 8), sms * 8);
  if (dtype == LITE3R_BF16)
    rowquant_kernel<<<blocks, 256, 0, stream>>>(static_cast<const __nv_bfloat16*>(x), row_stride, rows, cols, codes, scales);
  else
    rowquant_kernel<<<blocks, 256, 0, stream>>>(static_cast<const float*>(x), row_stride, rows, cols, codes, scales);
  return after_launch();
}

lite3r_status launch_linear_fp8(const uint8_t* x_codes, const float* x_scales, const uint8_t* w_codes,
                                const float* w_scales, const float* bias, int rows, int d_in, int d_out, void* y,
                                int y_dtype, long long y_stride, int* device_status, cudaStream_t stream) {
  LinearParams p = {};
  p.x_scales = x_scales;
  p.w_scales = w_scales;
  p.bias = bias;
  p.rows = rows;
  p.d_in = d_in;
  p.d_out = d_out;
  p.y = y;
  p.y_stride = y_stride;
  p.y_dtype = y_dtype;
  p.fused = 0;
  p.status = device_status;
  return launch_gemm(x_codes, w_codes, p, stream);
}

lite3r_status launch_qkv_project(const uint8_t* x_codes, const float* x_scales, const uint8_t* w_codes,
                                 const float* w_scales, const float* bias, const lite3r_shape& s, int d_model,
                                 const lite3r_fp8* out, int* device_status, cudaStream_t stream) {
  LinearParams p = {};
  p.x_scales = x_scales;
  p.w_scales = w_scales;
  p.bias = bias;
  p.rows = s.batch * s.tokens;
  p.d_in = d_model;
  p.d_out = 3 * s.heads * kHeadDim;
  p.fused = 1;
  p.batch = s.batch;
  p.tokens = s.tokens;
  p.heads = s.heads;
  p.block = s.block;
  p.nb = ceil_div(s.tokens, s.block);
  for (int i = 0; i < 3; ++i) {
    p.codes[i] = out[i].codes;
    p.scales[i] = out[i].scales;
    p.colsum[i] = out[i].colsum;
  }
  p.status = device_status;
  return launch_gemm(x_codes, w_codes, p, stream);
}

}  // namespace lite3r
