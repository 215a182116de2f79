// K3: per-key-block summaries of the linear branch (Algorithm 1's feature map, KV summary and normaliser, per block) on tcgen05 tensor cores.
//
// For key block j:  H_j = phi(K_j)^T V_j  (64 x 64),  z_j = phi(K_j)^T 1  (64), with the output projection folded in
// early: the kernel stores (H_j W)^T and z_j in bf16.  Folding is exact algebra:
// (phi(q) sum_j H_j) W = phi(q) sum_j (H_j W).
//
// The kernel is bound by HBM (reads the K and V codes once, writes 8320 bytes per key block); the two 64x64x64
// contractions per block are far too many flops for the CUDA cores at that rate, so they run as tcgen05 MMAs:
//   MMA 1   H[d][e]   = sum_s phi[s][d] * Vc[s][e]     A = phi (fp16, M-major), B = V code values (fp16, N-major)
//   MMA 1z  z[d]      = sum_s phi[s][d] * 1            same A, B = a constant tile of ones (N = 8)
//   MMA 2   HW^T[e'][d] = sum_e W[e][e'] * H[d][e]     A = W (fp16, M-major), B = H * scale_V (fp16, K-major)
// A "round" is 128 token rows: two key blocks at block 64 (two M=64 accumulators in the two 16-lane halves of every
// TMEM sub-partition), one key block at block 128.  Per round the 128 compute threads (one token row each) dequantise
// their K row, apply the feature map, and write phi and the V code values to shared memory in the operands' swizzled
// layouts; one thread of a fifth warp issues the MMAs; the compute threads then move H from TMEM to shared memory
// (scaled, fp16), and finally (H W)^T from TMEM to global memory (rows parked in shared memory first, so that stores
// write whole 128-byte rows).  Next to a sparse branch the kernel also writes the dequantised V rows it has just read
// (fp16, the attention kernel's P V operand), which saves a pass of its own over V.  Rounds of one CTA are serial; four CTAs per SM
// overlap their phases.  Every barrier wait is bounded.
#include "common.cuh"
#include "sm100.cuh"

namespace lite3r {

namespace {

using namespace sm100;

constexpr int kComputeThreads = 128;
constexpr int kThreads = kComputeThreads + 32;
constexpr int kCtasPerSm = 4;
constexpr uint32_t kTmemCols = 128;
constexpr uint32_t kColH = 0, kColZ = 64;
constexpr uint32_t kOffA = 0;            // phi operand (16 KB)
constexpr uint32_t kOffV = 16384;        // V operand, later H operand (16 KB)
constexpr uint32_t kOffW = 32768;        // W operand (8 KB)
constexpr uint32_t kOffOnes = 40960;     // ones operand (1 KB)
constexpr uint32_t kOffBar = 41984;
constexpr uint32_t kSmemBytes = kOffBar + 64;
constexpr float kLog2e = 1.4426950408889634f;

struct Bars {
  uint64_t ab_full, h_done, h_full, hw_done;
  uint32_t tmem_base;
  int abort;
};

struct SummaryParams {
  const uint8_t* k_codes;
  const float* k_scales;
  const uint8_t* v_codes;
  const float* v_scales;
  const float* proj;
  long long proj_head_stride;
  int heads, tokens, nb, phi;
  int rounds_per_head, rounds;
  __nv_bfloat16* hws;
  __half* v16;  // when not NULL: also writes the dequantised V rows (code value x block scale, fp16) read on the way
  int* status;
};

__device__ __forceinline__ uint32_t e4m3x2_to_half2(uint32_t two) {
  const __half2_raw h = __nv_cvt_fp8x2_to_halfraw2(static_cast<__nv_fp8x2_storage_t>(two), __NV_E4M3);
  return static_cast<uint32_t>(h.x) | (static_cast<uint32_t>(h.y) << 16);
}
__device__ __forceinline__ float2 half2_bits_to_float2(uint32_t bits) {
  return __half22float2(*reinterpret_cast<const __half2*>(&bits));
}
__device__ __forceinline__ uint32_t float2_to_half2_bits(float a, float b) {
  const __half2 h = __floats2half2_rn(a, b);
  return *reinterpret_cast<const uint32_t*>(&h);
}
__device__ __forceinline__ uint32_t float2_to_bf162_bits(float a, float b) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<const uint32_t*>(&h);
}

// Writes one 128-byte operand row (64 16-bit values, packed in w[32]) with the 128-byte swizzle.
__device__ __forceinline__ void store_row_swizzled(uint8_t* tile, int row, const uint32_t (&w)[32]) {
  uint8_t* dst = tile + row * 128;
#pragma unroll
  for (int ch = 0; ch < 8; ++ch)
    *reinterpret_cast<uint4*>(dst + ((ch ^ (row & 7)) << 4)) = make_uint4(w[4 * ch], w[4 * ch + 1], w[4 * ch + 2], w[4 * ch + 3]);
}

template <int BS>
__global__ void __launch_bounds__(kThreads, kCtasPerSm) summary_kernel(const SummaryParams p) {
  constexpr int kTilesPerRound = 128 / BS;  // 2 or 1
  constexpr int kKSteps = BS / 16;          // MMA 1 steps of 16 tokens per key block

  extern __shared__ __align__(1024) uint8_t smem[];
  Bars* bars = reinterpret_cast<Bars*>(smem + kOffBar);
  volatile int* abort_flag = &bars->abort;
  if ((smem_u32(smem) & 1023u) != 0) {
    if (threadIdx.x == 0 && p.status != nullptr) atomicCAS(p.status, 0, 902);
    return;
  }
  if (p.status != nullptr && *reinterpret_cast<volatile int*>(p.status) != 0) return;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // contiguous, balanced share of the rounds
  const int r_begin = static_cast<int>(static_cast<long long>(p.rounds) * blockIdx.x / gridDim.x);
  const int r_end = static_cast<int>(static_cast<long long>(p.rounds) * (blockIdx.x + 1) / gridDim.x);

  if (threadIdx.x == 0) {
    mbar_init(&bars->ab_full, kComputeThreads);
    mbar_init(&bars->h_done, 1);
    mbar_init(&bars->h_full, kComputeThreads);
    mbar_init(&bars->hw_done, 1);
    bars->abort = 0;
    mbar_fence_init();
  }
  if (warp == 4) {
    tmem_alloc(&bars->tmem_base, kTmemCols);
    tmem_relinquish();
  }
  // constant B operand of the row-sum MMA: 8 x 64 ones (any layout reads the same)
  for (int t = threadIdx.x; t < 256; t += kThreads) reinterpret_cast<uint32_t*>(smem + kOffOnes)[t] = 0x3C003C00u;
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_base;

  if (warp == 4) {
    // ------------------------------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_h = instr_desc(0, 64, 64, 1, 1);   // phi^T V: A M-major, B N-major
      constexpr uint32_t idesc_z = instr_desc(0, 64, 8, 1, 0);    // phi^T 1: B K-major
      constexpr uint32_t idesc_w = instr_desc(0, 64, 64, 1, 0);   // W^T H^T: A M-major, B K-major
      const uint32_t a_addr = smem_u32(smem + kOffA), v_addr = smem_u32(smem + kOffV);
      const uint32_t w_addr = smem_u32(smem + kOffW), o_addr = smem_u32(smem + kOffOnes);
      bool ok = true;
      for (int r = r_begin; r < r_end && ok; ++r) {
        const uint32_t ph = static_cast<uint32_t>(r - r_begin) & 1u;
        if (!(ok = mbar_wait(&bars->ab_full, ph, abort_flag, p.status, 501))) break;
        tc_fence_after();
#pragma unroll
        for (int hf = 0; hf < kTilesPerRound; ++hf) {
          const uint32_t lane_off = (static_cast<uint32_t>(hf) * 16u) << 16;
          const uint32_t tile_off = kTilesPerRound == 2 ? hf * 8192u : 0u;
#pragma unroll
          for (int kk = 0; kk < kKSteps; ++kk) {
            const uint64_t a = smem_desc(a_addr + tile_off + kk * 2048, 8192, 1024, kSwizzle128);
            const uint64_t b = smem_desc(v_addr + tile_off + kk * 2048, 8192, 1024, kSwizzle128);
            mma_f16(tmem + kColH + lane_off, a, b, idesc_h, kk);
          }
        }
        mma_commit(&bars->h_done);
        // the row sums are only needed at the end of the round: they follow the commit, and run while the compute
        // threads already move H (into the V operand's space, which MMA 1 has finished with; phi stays intact)
#pragma unroll
        for (int hf = 0; hf < kTilesPerRound; ++hf) {
          const uint32_t lane_off = (static_cast<uint32_t>(hf) * 16u) << 16;
          const uint32_t tile_off = kTilesPerRound == 2 ? hf * 8192u : 0u;
#pragma unroll
          for (int kk = 0; kk < kKSteps; ++kk) {
            const uint64_t a = smem_desc(a_addr + tile_off + kk * 2048, 8192, 1024, kSwizzle128);
            const uint64_t o = smem_desc(o_addr + (kk & 3) * 32, 16, 1024, kSwizzle128);
            mma_f16(tmem + kColZ + lane_off, a, o, idesc_z, kk);
          }
        }
        if (!(ok = mbar_wait(&bars->h_full, ph, abort_flag, p.status, 502))) break;
        tc_fence_after();
#pragma unroll
        for (int hf = 0; hf < kTilesPerRound; ++hf) {
          const uint32_t lane_off = (static_cast<uint32_t>(hf) * 16u) << 16;
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) {
            const uint64_t a = smem_desc(w_addr + kk * 2048, 8192, 1024, kSwizzle128);
            const uint64_t b = smem_desc(v_addr + hf * 8192 + kk * 32, 16, 1024, kSwizzle128);
            mma_f16(tmem + kColH + lane_off, a, b, idesc_w, kk);
          }
        }
        mma_commit(&bars->hw_done);
      }
    }
  } else {
    // ------------------------------------------------------------------------------------------ compute threads
    const int t = threadIdx.x;                     // token row of the round
    const int tile_tok = t / BS, s = t % BS;       // key block of the round and token inside it (operand build)
    const int hf = lane >> 4;                      // key block of the round whose accumulator row this thread owns
    const int d_row = warp * 16 + (lane & 15);     // that row (d for H, e' for (H W)^T)
    const bool acc_live = hf < kTilesPerRound;
    const uint32_t lane_addr = tmem + ((static_cast<uint32_t>(warp) * 32u) << 16);
    int w_head = -1;
    bool ok = true;

    for (int r = r_begin; r < r_end; ++r) {
      const uint32_t ph = static_cast<uint32_t>(r - r_begin) & 1u;
      const int bh = r / p.rounds_per_head;
      const int j0 = (r % p.rounds_per_head) * kTilesPerRound;
      const int head = bh % p.heads;
      const size_t bh_rows = static_cast<size_t>(bh) * p.nb;

      // W of this head as the fp16 A operand of MMA 2 (rows e, contiguous along e')
      if (head != w_head) {
        w_head = head;
        const int e = t >> 1, half = t & 1;
        const float4* src = reinterpret_cast<const float4*>(p.proj + head * p.proj_head_stride + e * kHeadDim + half * 32);
        uint8_t* dst = smem + kOffW + e * 128;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const float4 x0 = __ldg(src + 2 * c), x1 = __ldg(src + 2 * c + 1);
          const uint4 v4 = make_uint4(float2_to_half2_bits(x0.x, x0.y), float2_to_half2_bits(x0.z, x0.w),
                                      float2_to_half2_bits(x1.x, x1.y), float2_to_half2_bits(x1.z, x1.w));
          *reinterpret_cast<uint4*>(dst + (((half * 4 + c) ^ (e & 7)) << 4)) = v4;
        }
      }

      // ask L2 for the rows this thread will need in the next round
      if (r + 1 < r_end) {
        const int nbh = (r + 1) / p.rounds_per_head;
        const int nj = ((r + 1) % p.rounds_per_head) * kTilesPerRound + tile_tok;
        if (nj < p.nb && s < min(BS, p.tokens - nj * BS)) {
          const size_t off = ((static_cast<size_t>(nbh) * p.nb + nj) * BS + s) * kHeadDim;
          asm volatile("prefetch.global.L2 [%0];" ::"l"(p.k_codes + off));
          asm volatile("prefetch.global.L2 [%0];" ::"l"(p.v_codes + off));
        }
      }

      // operand rows of this thread's token
      {
        const int j = j0 + tile_tok;
        const int valid = j < p.nb ? min(BS, p.tokens - j * BS) : 0;
        uint32_t pw[32], vw[32];
        if (s < valid) {
          const size_t tile = bh_rows + j;
          const uint4* ksrc = reinterpret_cast<const uint4*>(p.k_codes + (tile * BS + s) * kHeadDim);
          const uint4* vsrc = reinterpret_cast<const uint4*>(p.v_codes + (tile * BS + s) * kHeadDim);
          // both rows are requested before either is used, so that only one memory latency is exposed
          uint4 vraw[4], kraw[4];
#pragma unroll
          for (int c = 0; c < 4; ++c) vraw[c] = __ldg(vsrc + c);
#pragma unroll
          for (int c = 0; c < 4; ++c) kraw[c] = __ldg(ksrc + c);
          {  // V code values are exact in fp16: straight conversion, stored before the K row needs the registers
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              const uint32_t vwd[4] = {vraw[c].x, vraw[c].y, vraw[c].z, vraw[c].w};
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                vw[c * 8 + q * 2] = e4m3x2_to_half2(vwd[q] & 0xFFFFu);
                vw[c * 8 + q * 2 + 1] = e4m3x2_to_half2(vwd[q] >> 16);
              }
            }
            store_row_swizzled(smem + kOffV, t, vw);
          }
          const float sk = __ldg(p.k_scales + tile);
          float x[64];
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const uint32_t kwd[4] = {kraw[c].x, kraw[c].y, kraw[c].z, kraw[c].w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const float2 lo = half2_bits_to_float2(e4m3x2_to_half2(kwd[q] & 0xFFFFu));
              const float2 hi = half2_bits_to_float2(e4m3x2_to_half2(kwd[q] >> 16));
              x[c * 16 + q * 4] = lo.x;
              x[c * 16 + q * 4 + 1] = lo.y;
              x[c * 16 + q * 4 + 2] = hi.x;
              x[c * 16 + q * 4 + 3] = hi.y;
            }
          }
          if (p.phi == LITE3R_PHI_SOFTMAX) {
            // Any common shift of the exponents cancels in the ratio.  448 * scale bounds every component of the block,
            // so it serves as the shift without a pass over the row; only when exponents could then leave the fp32
            // range (block magnitudes in the hundreds) is the row's own maximum looked up.  Arguments, sums and the
            // normalisation run on pairs of components (packed fp32x2).
            const float c = sk * kLog2e;  // sk > 0 commutes with max
            float shift = 448.f * c;
            if (896.f * c > 100.f) {
              float mx4[4] = {x[0], x[1], x[2], x[3]};
#pragma unroll
              for (int d = 4; d < 64; ++d) mx4[d & 3] = fmaxf(mx4[d & 3], x[d]);
              shift = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * c;
            }
            const uint64_t c2 = pack_f32x2(c, c), neg_shift2 = pack_f32x2(-shift, -shift);
            uint64_t sum2[2] = {0ull, 0ull};  // bit pattern of (0.f, 0.f)
#pragma unroll
            for (int d = 0; d < 64; d += 2) {
              float a0, a1;
              unpack_f32x2(fma_f32x2(pack_f32x2(x[d], x[d + 1]), c2, neg_shift2), a0, a1);
              x[d] = ex2(a0);
              x[d + 1] = ex2(a1);
              sum2[(d >> 1) & 1] = add_f32x2(sum2[(d >> 1) & 1], pack_f32x2(x[d], x[d + 1]));
            }
            float s0, s1, s2, s3;
            unpack_f32x2(sum2[0], s0, s1);
            unpack_f32x2(sum2[1], s2, s3);
            const float inv = 1.f / ((s0 + s1) + (s2 + s3));
            const uint64_t inv2 = pack_f32x2(inv, inv), neg0 = pack_f32x2(-0.f, -0.f);  // x * inv + (-0) is x * inv
#pragma unroll
            for (int d = 0; d < 64; d += 2) {
              float y0, y1;
              unpack_f32x2(fma_f32x2(pack_f32x2(x[d], x[d + 1]), inv2, neg0), y0, y1);
              pw[d >> 1] = float2_to_half2_bits(y0, y1);
            }
          } else {
            const float c = sk * kLog2e;
#pragma unroll
            for (int d = 0; d < 64; d += 2) {
              const float a0 = x[d] > 0.f ? fmaf(x[d], sk, 1.f) : ex2(x[d] * c);
              const float a1 = x[d + 1] > 0.f ? fmaf(x[d + 1], sk, 1.f) : ex2(x[d + 1] * c);
              pw[d >> 1] = float2_to_half2_bits(a0, a1);
            }
          }
        } else {
#pragma unroll
          for (int d = 0; d < 32; ++d) {
            pw[d] = 0u;
            vw[d] = 0u;
          }
          store_row_swizzled(smem + kOffV, t, vw);
        }
        store_row_swizzled(smem + kOffA, t, pw);
        if (p.v16 != nullptr && j < p.nb) {
          // The attention kernel's P V operand (code value x block scale as fp16, the stand-alone pass's arithmetic),
          // from the rows this warp has just put into the V operand tile (zeros past the end of the sequence): read
          // back so that a store instruction writes four whole 128-byte rows.
          __syncwarp();
          const float sv = __ldg(p.v_scales + bh_rows + j);
          const int r0 = warp * 32, ch = lane & 7;
          uint4* dst = reinterpret_cast<uint4*>(p.v16 + ((bh_rows + j) * BS + (r0 % BS)) * kHeadDim) + ch;
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            const int rr = 4 * k + (lane >> 3), row = r0 + rr;
            const uint4 raw = *reinterpret_cast<const uint4*>(smem + kOffV + row * 128 + ((ch ^ (row & 7)) << 4));
            const uint32_t in[4] = {raw.x, raw.y, raw.z, raw.w};
            uint32_t o[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const float2 f = half2_bits_to_float2(in[q]);
              o[q] = float2_to_half2_bits(f.x * sv, f.y * sv);
            }
            dst[rr * 8] = make_uint4(o[0], o[1], o[2], o[3]);
          }
        }
      }
      fence_proxy_async_smem();
      mbar_arrive(&bars->ab_full);

      // H row: TMEM -> scaled fp16 -> B operand of MMA 2; z row -> global
      if (!(ok = mbar_wait(&bars->h_done, ph, abort_flag, p.status, 503))) break;
      tc_fence_after();
      {
        uint32_t lo[32], hi[32];
        tmem_ld32(lane_addr + kColH, lo);
        tmem_ld32(lane_addr + kColH + 32, hi);
        tmem_wait_ld();
        tc_fence_before();
        const int j = j0 + hf;
        if (acc_live && j < p.nb) {
          const size_t tile = bh_rows + j;
          const float sv = __ldg(p.v_scales + tile);
          uint32_t hw[32];
#pragma unroll
          const uint64_t sv2 = pack_f32x2(sv, sv), neg0 = pack_f32x2(-0.f, -0.f);  // x * sv + (-0) is x * sv
          for (int e = 0; e < 32; e += 2) {
            float a0, a1, b0, b1;
            unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(lo[e]), __uint_as_float(lo[e + 1])), sv2, neg0), a0, a1);
            unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(hi[e]), __uint_as_float(hi[e + 1])), sv2, neg0), b0, b1);
            hw[e >> 1] = float2_to_half2_bits(a0, a1);
            hw[16 + (e >> 1)] = float2_to_half2_bits(b0, b1);
          }
          store_row_swizzled(smem + kOffV + hf * 8192, d_row, hw);
        }
      }
      fence_proxy_async_smem();
      mbar_arrive(&bars->h_full);

      // (H W)^T row e': TMEM -> bf16 -> global
      if (!(ok = mbar_wait(&bars->hw_done, ph, abort_flag, p.status, 504))) break;
      tc_fence_after();
      {
        uint32_t lo[32], hi[32];
        tmem_ld32(lane_addr + kColH, lo);
        tmem_ld32(lane_addr + kColH + 32, hi);
        const uint32_t zbits = tmem_ld1(lane_addr + kColZ);
        tmem_wait_ld();
        tc_fence_before();
        const int j = j0 + hf;
        if (acc_live && j < p.nb)
          p.hws[(bh_rows + j) * kSummaryRow + kHeadDim * kHeadDim + d_row] = __float2bfloat16_rn(__uint_as_float(zbits));
        // A thread owns one 128-byte row of (H W)^T; stored directly, an instruction would touch 32 lines.  The warp
        // parks its 32 rows in its own part of the V / H operand space (both MMAs have completed; the same threads
        // refill exactly these rows in the next round) and stores four whole rows per instruction.
        uint32_t ow[32];
#pragma unroll
        for (int c = 0; c < 16; ++c) {
          ow[c] = float2_to_bf162_bits(__uint_as_float(lo[2 * c]), __uint_as_float(lo[2 * c + 1]));
          ow[16 + c] = float2_to_bf162_bits(__uint_as_float(hi[2 * c]), __uint_as_float(hi[2 * c + 1]));
        }
        store_row_swizzled(smem + kOffV, warp * 32 + lane, ow);
        __syncwarp();
        const int ch = lane & 7;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const int rr = 4 * k + (lane >> 3), src_row = warp * 32 + rr;
          const uint4 val = *reinterpret_cast<const uint4*>(smem + kOffV + src_row * 128 + ((ch ^ (src_row & 7)) << 4));
          const int hf_r = rr >> 4, j_r = j0 + hf_r;  // lane rr of the warp holds row warp * 16 + (rr & 15) of tile hf_r
          if (hf_r < kTilesPerRound && j_r < p.nb)
            *reinterpret_cast<uint4*>(p.hws + (bh_rows + j_r) * kSummaryRow + (warp * 16 + (rr & 15)) * kHeadDim + ch * 8) = val;
        }
        __syncwarp();
      }
    }
    (void)ok;
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 4) {
    tc_fence_after();
    tmem_dealloc(tmem, kTmemCols);
  }
}

template <int BS>
lite3r_status launch(const SummaryParams& p, int sm_count, cudaStream_t stream) {
  lite3r_status st = ensure_dynamic_smem(summary_kernel<BS>, static_cast<int>(kSmemBytes));
  if (st != LITE3R_OK) return st;
  const int grid = p.rounds < sm_count * kCtasPerSm ? p.rounds : sm_count * kCtasPerSm;
  summary_kernel<BS><<<grid, kThreads, kSmemBytes, stream>>>(p);
  return after_launch();
}

}  // namespace

lite3r_status launch_summary(const lite3r_fp8& k, const lite3r_fp8& v, const float* proj, long long proj_head_stride,
                             const lite3r_shape& s, int phi, __nv_bfloat16* hws, __half* v16, int* device_status,
                             cudaStream_t stream) {
  SummaryParams p;
  p.k_codes = k.codes;
  p.k_scales = k.scales;
  p.v_codes = v.codes;
  p.v_scales = v.scales;
  p.proj = proj;
  p.proj_head_stride = proj_head_stride;
  p.heads = s.heads;
  p.tokens = s.tokens;
  p.nb = ceil_div(s.tokens, s.block);
  p.phi = phi;
  p.rounds_per_head = ceil_div(p.nb, 128 / s.block);
  p.rounds = s.batch * s.heads * p.rounds_per_head;
  p.hws = hws;
  p.v16 = v16;
  p.status = device_status;
  int sms = 0;
  lite3r_status st = sm_count(&sms);
  if (st != LITE3R_OK) return st;
  return s.block == 64 ? launch<64>(p, sms, stream) : launch<128>(p, sms, stream);
}

}  // namespace lite3r
