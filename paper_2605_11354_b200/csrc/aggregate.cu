// K3b: marginal aggregation as a mask-GEMM on tcgen05 tensor cores.
//
// For one (b, h):  G[i, n] = sum_j M[i, j] * S[j, n],  M[i, j] = 1 if key block j is marginal for query block i, else 0,
// S[j, :] = the 4160-wide bf16 summary row of key block j ((H_j W)^T | z_j).  0/1 is exact in bf16 and the
// accumulation is fp32 in TMEM, so this equals the gather-and-add of the summaries while reading each summary once per
// 128 query blocks instead of once per query block.
//
// One CTA computes a 128 (rows) x 256 (summary columns) tile; the reduction runs over key blocks in chunks of 64.  Rows
// and keys are numbered through all (b, h).  Tiles either stay inside one (b, h), or, for short sequences, run through
// the (b, h) boundaries so that several small problems share a tile (the mask is then block-diagonal); the launcher
// takes the cheaper tiling.  Per chunk: TMA brings the 64 x 256 slab of summaries (MN-major B operand, four 64-column
// boxes, 128B swizzle); 128 threads expand the class bytes of their row (fetched a chunk ahead) into the bf16 0/1 A
// tile (K-major, 128B swizzle) with byte permutes; one thread issues four 128x256x16 MMAs.  Epilogue: the same 128
// threads read their accumulator row from TMEM, turn the rows around in shared memory so that stores write whole
// 128-byte segments, and store the first 4096 columns as bf16 (the attention kernel's B operand) and the last 64
// (zeta) as fp32.
#include <algorithm>

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
                     int total_rows, int flat, __nv_bfloat16* __restrict__ g16, float* __restrict__ zeta, int* status) {
  extern __shared__ __align__(1024) uint8_t smem[];
  Bars* bars = reinterpret_cast<Bars*>(smem + kOffBar);
  volatile int* abort_flag = &bars->abort;
  if (status != nullptr && *reinterpret_cast<volatile int*>(status) != 0) return;
  if ((smem_u32(smem) & 1023u) != 0) {
    if (threadIdx.x == 0 && status != nullptr) atomicCAS(status, 0, 901);
    return;
  }
  // The attention kernel that follows needs this kernel's results only at its very end: it may be scheduled as soon
  // as every CTA of this grid has started (it waits for the grid's completion itself before it reads G and zeta).
  sm100::launch_dependents();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_tile = blockIdx.x;           // 0..16, 256 summary columns each (the last one holds zeta)
  // Rows and keys are numbered through all (b, h): row R = (b h) Nb + i, key (b h) Nb + j, the row numbers of the class
  // matrix, the summaries and the outputs.  A tile is 128 consecutive rows and reduces over the keys of the (b, h) it
  // touches.  Long sequences: the tile stays inside one (b, h) (grid z).  Short ones (flat): tiles run through the
  // (b, h) boundaries, so several small problems share one tile instead of each padding its own; the mask is then
  // block-diagonal, a row only ever selecting keys of its own (b, h).
  int row0, row_limit, key0, key_end;
  if (flat) {
    row0 = blockIdx.y * kTileM;
    row_limit = total_rows;
    key0 = (row0 / nb) * nb;
    key_end = (min(row0 + kTileM, total_rows) - 1) / nb * nb + nb;
  } else {
    key0 = blockIdx.z * nb;
    key_end = key0 + nb;
    row0 = key0 + blockIdx.y * kTileM;
    row_limit = key_end;
  }
  const int chunks = (key_end - key0 + kChunk - 1) / kChunk;

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
        const int row = key0 + c * kChunk;
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
    const int r = quarter * 32 + lane;  // accumulator row = TMEM lane = row row0 + r
    const int row = row0 + r;
    const bool row_ok = row < row_limit;
    const int own0 = row_ok ? row / nb * nb : 0;  // first key of this row's (b, h)
    const signed char* row_ptr = cls + static_cast<size_t>(row_ok ? row : 0) * nb;
    bool ok = true;
    // Chunk c covers keys key0 + 64 c ..; of those, positions p_lo .. p_hi - 1 belong to this row's (b, h) and have a
    // class byte, at row_ptr + (key - own0).  The bytes travel as the aligned 32-bit words that hold them (rows start
    // at any byte; words without an in-range byte are not read), fetched one chunk ahead, so that the latency hides
    // behind the wait for the stage and the expansion.
    auto fetch = [&](int c, uint32_t w[17]) {
      const int j0 = key0 + c * kChunk - own0;  // class-byte index of position 0: negative before the row's keys
      const int p_lo = max(0, -j0), p_hi = min(kChunk, nb - j0);
      const intptr_t addr = reinterpret_cast<intptr_t>(row_ptr) + j0;
      const uint32_t* wp = reinterpret_cast<const uint32_t*>(addr & ~intptr_t(3));
      const int a = static_cast<int>(addr & 3);  // word k holds positions 4 k - a .. 4 k - a + 3
      const int k_lo = (p_lo + a) >> 2;          // first and one-past-last word with an in-range byte
      const int k_n = (row_ok && c < chunks) ? ((p_hi + a + 3) >> 2) - k_lo : 0;
#pragma unroll
      for (int k = 0; k < 17; ++k) w[k] = static_cast<unsigned>(k - k_lo) < static_cast<unsigned>(max(k_n, 0)) ? __ldg(wp + k) : 0u;
    };
    uint32_t w[17];
    fetch(0, w);
    for (int c = 0; c < chunks; ++c) {
      const int st = c % kStages;
      const int j0 = key0 + c * kChunk - own0;
      const int p_lo = max(0, -j0), p_hi = min(kChunk, nb - j0);
      const uint32_t shift = static_cast<uint32_t>((reinterpret_cast<intptr_t>(row_ptr) + j0) & 3) * 8u;
      // realigned class bytes; bit 0 of a class (0 negligible, 1 marginal, 2 critical) says "marginal"
      uint32_t m[16];
#pragma unroll
      for (int k = 0; k < 16; ++k) m[k] = __funnelshift_r(w[k], w[k + 1], shift) & 0x01010101u;
      if (p_lo > 0 || p_hi < kChunk) {  // positions outside the row's keys hold other rows' bytes
#pragma unroll
        for (int k = 0; k < 16; ++k) {
          const int lo = min(max(p_lo - 4 * k, 0), 4), hi = min(max(p_hi - 4 * k, 0), 4);  // bytes lo .. hi - 1 stay
          const uint32_t keep = lo < hi ? (0xFFFFFFFFu >> (32 - 8 * hi)) & (0xFFFFFFFFu << (8 * lo)) : 0u;
          m[k] &= keep;
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
            const int ir = row0 + quarter * 32 + rr;
            const uint4 val = *reinterpret_cast<const uint4*>(stage + rr * 128 + ((ch ^ (rr & 7)) << 4));
            if (ir < row_limit)
              *reinterpret_cast<uint4*>(g16 + static_cast<size_t>(ir) * kHeadDim * kHeadDim + n + ch * 8) = val;
          }
          __syncwarp();
        } else {
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            uint32_t v[32];
            tmem_ld32(lane_addr + pp * 64 + half * 32, v);
            tmem_wait_ld();
            if (!row_ok) continue;
            float4* dst = reinterpret_cast<float4*>(zeta + static_cast<size_t>(row) * kHeadDim + (n - kHeadDim * kHeadDim) + half * 32);
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
  const uint64_t rows = static_cast<uint64_t>(s.batch) * s.heads * nb;
  // the tensor map of the summaries is kept from the calling thread's previous call while buffer and size repeat
  struct MapCache {
    alignas(64) CUtensorMap map;
    const void* base = nullptr;
    uint64_t rows = 0;
  };
  thread_local MapCache cache;
  lite3r_status st;
  if (cache.base != hws || cache.rows != rows) {
    cache.base = nullptr;
    st = make_tensor_map_2d(&cache.map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, hws, kSummaryRow, rows, 64, 64,
                            CU_TENSOR_MAP_SWIZZLE_128B);
    if (st != LITE3R_OK) return st;
    cache.base = hws;
    cache.rows = rows;
  }
  const CUtensorMap& map_s = cache.map;
  st = ensure_dynamic_smem(aggregate_mma_kernel, static_cast<int>(kSmemBytes));
  if (st != LITE3R_OK) return st;
  if (rows > 0x7FFFFFFFull - kTileM) return LITE3R_ERR_UNSUPPORTED;
  const int total_rows = static_cast<int>(rows), bh = s.batch * s.heads;
  // Tiles through the (b, h) boundaries pay with a longer reduction (the keys of every (b, h) a tile touches), tiles
  // inside one (b, h) with padding when Nb is not a multiple of 128.  Estimate of either: waves of CTAs (two per SM)
  // times the cost of a CTA, its set-up and drain counted as three 64-key chunks (at Nb = 172 the two tilings are
  // measured on a par at about that ratio).
  int sms = 0;
  if ((st = sm_count(&sms)) != LITE3R_OK) return st;
  constexpr double kFixed = 3.0;
  const long long slots = 2ll * sms, col_tiles = ceil_div(kSummaryRow, kTileN);
  const long long ctas_inside = col_tiles * bh * ceil_div(nb, kTileM);
  const double time_inside = static_cast<double>((ctas_inside + slots - 1) / slots) * (kFixed + ceil_div(nb, kChunk));
  const long long row_tiles = ceil_div(total_rows, kTileM);
  // chunks of a flat tile: one (b, h) when it starts and ends in the same one, else every (b, h) it touches
  double flat_chunks = 0.0;
  const long long probe = std::min<long long>(row_tiles, 4096);  // the pattern repeats; a prefix is representative
  for (long long t = 0; t < probe; ++t) {
    const int r0 = static_cast<int>(t) * kTileM;
    const int k0 = r0 / nb * nb, k1 = (std::min(r0 + kTileM, total_rows) - 1) / nb * nb + nb;
    flat_chunks += ceil_div(k1 - k0, kChunk);
  }
  flat_chunks /= static_cast<double>(probe);
  const long long ctas_flat = col_tiles * row_tiles;
  const double time_flat = static_cast<double>((ctas_flat + slots - 1) / slots) * (kFixed + flat_chunks);
  const int flat = time_flat < time_inside ? 1 : 0;
  const dim3 grid(ceil_div(kSummaryRow, kTileN), flat ? ceil_div(total_rows, kTileM) : ceil_div(nb, kTileM), flat ? 1 : bh);
  aggregate_mma_kernel<<<grid, kThreads, kSmemBytes, stream>>>(map_s, cls, nb, total_rows, flat, g16, zeta, device_status);
  return after_launch();
}

}  // namespace lite3r
