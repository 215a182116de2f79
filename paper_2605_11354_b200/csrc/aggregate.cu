// K3b: marginal aggregation as a mask-GEMM on tcgen05 tensor cores.
//
// For one (b, h):  G[i, n] = sum_j M[i, j] * S[j, n],  M[i, j] = 1 if key block j is marginal for query block i, else 0,
// S[j, :] = the 4160-wide bf16 summary row of key block j ((H_j W)^T | z_j).  0/1 is exact in bf16 and the
// accumulation is fp32 in TMEM, so this equals the gather-and-add of the summaries while reading each summary once per
// 128 query blocks instead of once per query block.
//
// One CTA computes a 128 (query blocks) x 256 (summary columns) tile; the reduction runs over key blocks in chunks of
// 64.  Per chunk: TMA brings the 64 x 256 slab of summaries (MN-major B operand, four 64-column boxes, 128B swizzle);
// 128 threads expand the class bytes of their query-block row into the bf16 0/1 A tile (K-major, 128B swizzle); one
// thread issues four 128x256x16 MMAs.  Epilogue: the same 128 threads read their accumulator row from TMEM and store
// the first 4096 columns as bf16 (the attention kernel's B operand) and the last 64 (zeta) as fp32.
#include "common.cuh"
#include "sm100.cuh"

namespace lite3r {

namespace {

using namespace sm100;

constexpr int kStages = 2;  // 96 KB of operand stages: two CTAs per SM, one's epilogue overlaps the other's main loop
constexpr int kThreads = 192;
constexpr int kTileM = 128, kTileN = 256, kChunk = 64;
constexpr uint32_t kABytes = kTileM * kChunk * 2;   // 16 KB
constexpr uint32_t kBBytes = kChunk * kTileN * 2;   // 32 KB
constexpr uint32_t kOffA = 0;
constexpr uint32_t kOffB = kStages * kABytes;
constexpr uint32_t kOffBar = kOffB + kStages * kBBytes;
constexpr uint32_t kSmemBytes = kOffBar + 128;
constexpr uint32_t kTmemCols = 256;

struct Bars {
  uint64_t a_full[kStages], b_full[kStages], empty[kStages], acc_full;
  uint32_t tmem_base;
  int abort;
};

__global__ void __launch_bounds__(kThreads, 2)
aggregate_mma_kernel(const __grid_constant__ CUtensorMap map_s, const signed char* __restrict__ cls, int nb,
                     __nv_bfloat16* __restrict__ g16, float* __restrict__ zeta, int* status) {
  extern __shared__ __align__(1024) uint8_t smem[];
  Bars* bars = reinterpret_cast<Bars*>(smem + kOffBar);
  volatile int* abort_flag = &bars->abort;
  if (status != nullptr && *reinterpret_cast<volatile int*>(status) != 0) return;
  if ((smem_u32(smem) & 1023u) != 0) {
    if (threadIdx.x == 0 && status != nullptr) atomicCAS(status, 0, 901);
    return;
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_tile = blockIdx.x;           // 0..16, 256 summary columns each (the last one holds zeta)
  const int i0 = blockIdx.y * kTileM;      // first query block of the tile
  const int bh = blockIdx.z;
  const size_t bh_rows = static_cast<size_t>(bh) * nb;
  const int chunks = (nb + kChunk - 1) / kChunk;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&bars->a_full[s], 128);
      mbar_init(&bars->b_full[s], 1);
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
      tma_prefetch_desc(&map_s);
      for (int c = 0; c < chunks; ++c) {
        const int st = c % kStages;
        if (!mbar_wait(&bars->empty[st], ((c / kStages) & 1) ^ 1, abort_flag, status, 401)) break;
        mbar_arrive_expect_tx(&bars->b_full[st], kBBytes);
        const int row = static_cast<int>(bh_rows) + c * kChunk;
        for (int q = 0; q < 4; ++q)  // columns past 4160 and rows past the tensor are zero-filled by TMA
          tma_load_2d(smem + kOffB + st * kBBytes + q * 8192, &map_s, &bars->b_full[st], n_tile * kTileN + q * 64, row);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = instr_desc(1, kTileM, kTileN, 0, 1);  // bf16, A K-major, B MN-major
      const uint32_t a_addr = smem_u32(smem + kOffA), b_addr = smem_u32(smem + kOffB);
      bool ok = true;
      for (int c = 0; c < chunks && ok; ++c) {
        const int st = c % kStages;
        const uint32_t par = (c / kStages) & 1;
        ok = mbar_wait(&bars->a_full[st], par, abort_flag, status, 402) &&
             mbar_wait(&bars->b_full[st], par, abort_flag, status, 403);
        if (!ok) break;
        tc_fence_after();
        for (int kk = 0; kk < 4; ++kk) {
          const uint64_t a = smem_desc(a_addr + st * kABytes + kk * 32, 16, 1024, kSwizzle128);
          const uint64_t b = smem_desc(b_addr + st * kBBytes + kk * 2048, 8192, 1024, kSwizzle128);
          mma_f16(tmem, a, b, idesc, (c > 0 || kk > 0) ? 1u : 0u);
        }
        mma_commit(&bars->empty[st]);
      }
      if (ok) mma_commit(&bars->acc_full);
    }
  } else {
    const int quarter = warp & 3;
    const int r = quarter * 32 + lane;  // accumulator row = TMEM lane = query block i0 + r
    const int i = i0 + r;
    const bool row_ok = i < nb;
    const signed char* row_ptr = cls + (bh_rows + (row_ok ? i : 0)) * nb;
    bool ok = true;
    // The 64 class bytes of this row for chunk c, as the 17 aligned 32-bit words that hold them (rows start at any
    // byte); fetched one chunk ahead, so that the latency hides behind the wait for the stage and the expansion.
    auto fetch = [&](int c, uint32_t w[17]) {
      const int j0 = c * kChunk;
      const uintptr_t addr = reinterpret_cast<uintptr_t>(row_ptr + j0);
      const uint32_t* wp = reinterpret_cast<const uint32_t*>(addr & ~uintptr_t(3));
      const int len = min(kChunk, nb - j0);                            // in-range class bytes of this chunk
      const int words = (static_cast<int>(addr & 3u) + len + 3) / 4;   // aligned words that hold them
#pragma unroll
      for (int k = 0; k < 17; ++k) w[k] = (row_ok && c < chunks && k < words) ? __ldg(wp + k) : 0u;
    };
    uint32_t w[17];
    fetch(0, w);
    for (int c = 0; c < chunks; ++c) {
      const int st = c % kStages;
      const int j0 = c * kChunk;
      const uint32_t shift = static_cast<uint32_t>(reinterpret_cast<uintptr_t>(row_ptr + j0) & 3u) * 8u;
      const int len = min(kChunk, nb - j0);
      // realigned class bytes; bit 0 of a class (0 negligible, 1 marginal, 2 critical) says "marginal"
      uint32_t m[16];
#pragma unroll
      for (int k = 0; k < 16; ++k) m[k] = __funnelshift_r(w[k], w[k + 1], shift) & 0x01010101u;
      if (len < kChunk) {  // last chunk: the bytes past the row belong to the next row
#pragma unroll
        for (int k = 0; k < 16; ++k) {
          const int left = len - 4 * k;  // in-range bytes of this word
          m[k] = left >= 4 ? m[k] : (left <= 0 ? 0u : (m[k] & (0xFFFFFFFFu >> (32 - 8 * left))));
        }
      }
      fetch(c + 1, w);
      if (!(ok = mbar_wait(&bars->empty[st], ((c / kStages) & 1) ^ 1, abort_flag, status, 404))) break;
      uint8_t* arow = smem + kOffA + st * kABytes + r * 128;
#pragma unroll
      for (int ch = 0; ch < 8; ++ch) {  // 8 mask entries (two class words) per 16-byte chunk
        // bytes (b0 b1 b2 b3) of 0/1 -> bf16 pairs: (b0 | b1 << 16) * 0x3F80 has 1.0 where the byte is 1
        const uint32_t lo = m[2 * ch], hi = m[2 * ch + 1];
        const uint32_t o0 = __byte_perm(lo, 0u, 0x4140) * 0x3F80u, o1 = __byte_perm(lo, 0u, 0x4342) * 0x3F80u;
        const uint32_t o2 = __byte_perm(hi, 0u, 0x4140) * 0x3F80u, o3 = __byte_perm(hi, 0u, 0x4342) * 0x3F80u;
        *reinterpret_cast<uint4*>(arow + ((ch ^ (r & 7)) << 4)) = make_uint4(o0, o1, o2, o3);
      }
      fence_proxy_async_smem();
      mbar_arrive(&bars->a_full[st]);
    }
    if (ok && (ok = mbar_wait(&bars->acc_full, 0, abort_flag, status, 405))) {
      tc_fence_after();
      const uint32_t lane_addr = tmem + ((static_cast<uint32_t>(quarter) * 32u) << 16);
      const size_t out_row = bh_rows + i;
      // A thread owns one accumulator row, so direct stores would touch 32 different lines per instruction.  Each
      // warp turns its 32 rows x 128 bytes (64 bf16 columns) around in shared memory (the operand stages are free:
      // every MMA has completed) and stores whole 128-byte row segments, four rows per instruction.
      uint8_t* const stage = smem + quarter * 4096;
#pragma unroll 1
      for (int pp = 0; pp < kTileN / 64; ++pp) {
        const int n = n_tile * kTileN + pp * 64;
        if (n >= kSummaryRow) break;
        if (n < kHeadDim * kHeadDim) {
          uint32_t pk[32];
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            uint32_t v[32];
            tmem_ld32(lane_addr + pp * 64 + half * 32, v);
            tmem_wait_ld();
#pragma unroll
            for (int x = 0; x < 16; ++x) {
              __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(v[2 * x]), __uint_as_float(v[2 * x + 1]));
              pk[half * 16 + x] = *reinterpret_cast<uint32_t*>(&h);
            }
          }
#pragma unroll
          for (int ch = 0; ch < 8; ++ch)
            *reinterpret_cast<uint4*>(stage + lane * 128 + ((ch ^ (lane & 7)) << 4)) =
                make_uint4(pk[4 * ch], pk[4 * ch + 1], pk[4 * ch + 2], pk[4 * ch + 3]);
          __syncwarp();
          const int ch = lane & 7;
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            const int rr = 4 * k + (lane >> 3);
            const int ir = i0 + quarter * 32 + rr;
            const uint4 val = *reinterpret_cast<const uint4*>(stage + rr * 128 + ((ch ^ (rr & 7)) << 4));
            if (ir < nb)
              *reinterpret_cast<uint4*>(g16 + (bh_rows + ir) * kHeadDim * kHeadDim + n + ch * 8) = val;
          }
          __syncwarp();
        } else {
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            uint32_t v[32];
            tmem_ld32(lane_addr + pp * 64 + half * 32, v);
            tmem_wait_ld();
            if (!row_ok) continue;
            float4* dst = reinterpret_cast<float4*>(zeta + out_row * kHeadDim + (n - kHeadDim * kHeadDim) + half * 32);
#pragma unroll
            for (int q = 0; q < 8; ++q)
              dst[q] = make_float4(__uint_as_float(v[4 * q]), __uint_as_float(v[4 * q + 1]),
                                   __uint_as_float(v[4 * q + 2]), __uint_as_float(v[4 * q + 3]));
          }
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

}  // namespace

lite3r_status launch_aggregate(const __nv_bfloat16* hws, const signed char* cls, const lite3r_shape& s, int nb,
                               __nv_bfloat16* g16, float* zeta, int* device_status, cudaStream_t stream) {
  alignas(64) CUtensorMap map_s;
  const uint64_t rows = static_cast<uint64_t>(s.batch) * s.heads * nb;
  lite3r_status st = make_tensor_map_2d(&map_s, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, hws, kSummaryRow, rows, 64, 64,
                                        CU_TENSOR_MAP_SWIZZLE_128B);
  if (st != LITE3R_OK) return st;
  st = record_cuda(cudaFuncSetAttribute(aggregate_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        static_cast<int>(kSmemBytes)));
  if (st != LITE3R_OK) return st;
  const dim3 grid(ceil_div(kSummaryRow, kTileN), ceil_div(nb, kTileM), s.batch * s.heads);
  aggregate_mma_kernel<<<grid, kThreads, kSmemBytes, stream>>>(map_s, cls, nb, g16, zeta, device_status);
  return after_launch();
}

}  // namespace lite3r
