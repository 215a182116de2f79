// K4: critical-block softmax attention + linear branch + add (Algorithm 1 lines 4-5, 9-10) on tcgen05 / TMEM / TMA.
//
// One CTA owns 128 query rows of one (b, h): at block 64 a PAIR of query blocks (two M=64 accumulators interleaved
// in the two 16-lane halves of every TMEM sub-partition), at block 128 one query block (M=128).  Work advances in
// steps of 64 keys.  Per step t:
//   TMA      K tile(s) (e4m3, 64-byte rows, 64B swizzle) and V tile(s) (code values as fp16, 128B swizzle) -> smem ring
//   tcgen05  S[t&1] = Q K^T        kind::f8f6f4, fp32 accumulators in TMEM (64 columns)
//   softmax  128 threads, one query row each (TMEM lane = thread): scale, mask padded keys, running max with lazy
//            rescale, exp2, row sum; P goes to shared memory as fp16 in the MMA's K-major 128B-swizzled layout
//   tcgen05  O += P V              kind::f16, V as MN-major B operand, fp32 accumulators in TMEM (64 columns)
// P is carried in fp16 (not e4m3): one e4m3 term has a 2.6 % rounding error per probability, which alone is ten
// times the output tolerance; V's code values are exact in fp16, and the V block scale rides on P
// (P' = P * scale_j / scale_ref, row sums corrected by the inverse), so O needs one final scale.
// Tail: phi(Q) (bf16) times the aggregated, projected summaries G_i (bf16) as one more MMA, divided by
// phi(Q) . zeta_i, added to O / l and stored.
//
// Warp roles (192 threads): warp 0 = TMA producer, warp 1 = MMA issuer and TMEM owner, warps 2-5 = softmax/epilogue.
// Every mbarrier wait is bounded (1 s); on expiry the CTA sets *device_status and all roles leave their loops.
#include "common.cuh"
#include "sm100.cuh"

namespace lite3r {

namespace {

using namespace sm100;

constexpr int kStages = 3;
constexpr int kThreads = 192;
constexpr int kStepKeys = 64;
constexpr uint32_t kTmemCols = 256;
constexpr uint32_t kColS = 0, kColO = 128, kColL = 192;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kRescaleThreshold = 8.0f;  // lazy rescale: keep the old reference max until it is beaten by 2^8

// shared-memory map (bytes from a 1024-aligned base)
constexpr uint32_t kQBytes = 8192, kKStage = 8192, kVStage = 16384, kPBuf = 16384;
constexpr uint32_t kOffQ = 0;
constexpr uint32_t kOffK = kOffQ + kQBytes;
constexpr uint32_t kOffV = kOffK + kStages * kKStage;
constexpr uint32_t kOffP = kOffV + kStages * kVStage;
constexpr uint32_t kOffBar = kOffP + 2 * kPBuf;
constexpr uint32_t kSmemBytes = kOffBar + 256;  // two CTAs per SM: 2 * (114944 + 1024 reserved) <= 232448

struct Bars {
  uint64_t q_full, g_full, phi_full, l_full;
  uint64_t k_full[kStages], k_empty[kStages], v_full[kStages], v_empty[kStages];
  uint64_t s_full[2], s_empty[2], p_full[2], p_empty[2];
  uint32_t tmem_base;
  int abort;
};

struct AttnParams {
  const uint8_t* q_codes;
  const float* q_scales;
  const float* k_scales;
  const float* v_scales;
  const float* vref;   // [B*H] largest V block scale of the head
  const int* crit_idx; // [B*H*Nb][k_crit]
  const float* zeta;   // [B*H*Nb][64]
  float* out;
  long long out_stride_b, out_stride_h, out_stride_n;
  int heads, tokens, nb, k_crit, k_marg, phi;
  int* status;
};

__device__ __forceinline__ uint32_t pack_half2(float a, float b) {
  __half2 h = __floats2half2_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ uint32_t pack_bf162(float a, float b) {
  __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&h);
}

template <int BS>
__global__ void __launch_bounds__(kThreads, 2)
attention_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                 const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_g,
                 const AttnParams p) {
  constexpr bool kPair = (BS == 64);
  constexpr int kHalves = kPair ? 2 : 1;             // independent M=64 problems per CTA
  constexpr int kStepsPerBlock = BS / kStepKeys;     // 1 or 2
  constexpr int kM = kPair ? 64 : 128;
  constexpr uint32_t kKTx = kHalves * 4096, kVTx = kHalves * 8192;

  extern __shared__ __align__(1024) uint8_t smem[];
  Bars* bars = reinterpret_cast<Bars*>(smem + kOffBar);
  volatile int* abort_flag = &bars->abort;
  // The swizzled operand tiles need a 1024-byte aligned base; refuse to run on anything else.
  if ((smem_u32(smem) & 1023u) != 0) {
    if (threadIdx.x == 0 && p.status != nullptr) atomicCAS(p.status, 0, 900);
    return;
  }

  // A wait that expired in an earlier CTA of this launch stops the rest of the grid before it touches anything.
  if (p.status != nullptr && *reinterpret_cast<volatile int*>(p.status) != 0) return;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tiles_per_head = kPair ? (p.nb + 1) / 2 : p.nb;
  const int bh = blockIdx.x / tiles_per_head;
  const int tile = blockIdx.x % tiles_per_head;
  const int i_q[2] = {kPair ? 2 * tile : tile, kPair ? min(2 * tile + 1, p.nb - 1) : tile};
  const size_t bh_rows = static_cast<size_t>(bh) * p.nb;
  const int steps = p.k_crit * kStepsPerBlock;

  if (threadIdx.x == 0) {
    mbar_init(&bars->q_full, 1);
    mbar_init(&bars->g_full, 1);
    mbar_init(&bars->phi_full, 128);
    mbar_init(&bars->l_full, 1);
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&bars->k_full[s], 1);
      mbar_init(&bars->k_empty[s], 1);
      mbar_init(&bars->v_full[s], 1);
      mbar_init(&bars->v_empty[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&bars->s_full[b], 1);
      mbar_init(&bars->s_empty[b], 128);
      mbar_init(&bars->p_full[b], 128);
      mbar_init(&bars->p_empty[b], 1);
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
    // ------------------------------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      tma_prefetch_desc(&map_q);
      tma_prefetch_desc(&map_k);
      tma_prefetch_desc(&map_v);
      mbar_arrive_expect_tx(&bars->q_full, kQBytes);
      if (kPair) {
        tma_load_2d(smem + kOffQ, &map_q, &bars->q_full, 0, static_cast<int>((bh_rows + i_q[0]) * 64));
        tma_load_2d(smem + kOffQ + 4096, &map_q, &bars->q_full, 0, static_cast<int>((bh_rows + i_q[1]) * 64));
      } else {
        tma_load_2d(smem + kOffQ, &map_q, &bars->q_full, 0, static_cast<int>((bh_rows + i_q[0]) * 128));
        tma_load_2d(smem + kOffQ + 4096, &map_q, &bars->q_full, 0, static_cast<int>((bh_rows + i_q[0]) * 128 + 64));
      }
      const int* list0 = p.crit_idx + (bh_rows + i_q[0]) * p.k_crit;
      const int* list1 = p.crit_idx + (bh_rows + i_q[1]) * p.k_crit;
      bool ok = true;
      for (int t = 0; t < steps && ok; ++t) {
        const int st = t % kStages;
        const uint32_t par = ((t / kStages) & 1) ^ 1;
        int row[2];
        if (kPair) {
          row[0] = static_cast<int>((bh_rows + __ldg(list0 + t)) * 64);
          row[1] = static_cast<int>((bh_rows + __ldg(list1 + t)) * 64);
        } else {
          row[0] = static_cast<int>((bh_rows + __ldg(list0 + t / 2)) * 128 + (t & 1) * 64);
          row[1] = 0;
        }
        ok = mbar_wait(&bars->k_empty[st], par, abort_flag, p.status, 101);
        if (!ok) break;
        mbar_arrive_expect_tx(&bars->k_full[st], kKTx);
        for (int hf = 0; hf < kHalves; ++hf)
          tma_load_2d(smem + kOffK + st * kKStage + hf * 4096, &map_k, &bars->k_full[st], 0, row[hf]);
        ok = mbar_wait(&bars->v_empty[st], par, abort_flag, p.status, 102);
        if (!ok) break;
        mbar_arrive_expect_tx(&bars->v_full[st], kVTx);
        for (int hf = 0; hf < kHalves; ++hf)
          tma_load_2d(smem + kOffV + st * kVStage + hf * 8192, &map_v, &bars->v_full[st], 0, row[hf]);
      }
      if (ok && p.k_marg > 0) {
        // The aggregated summaries reuse V stage 0; it is free once the last P V product has completed.
        if (steps > 0) {
          const int last = steps - 1;
          ok = mbar_wait(&bars->v_empty[last % kStages], (last / kStages) & 1, abort_flag, p.status, 103);
        }
        if (ok) {
          mbar_arrive_expect_tx(&bars->g_full, kHalves * 8192);
          for (int hf = 0; hf < kHalves; ++hf)
            tma_load_2d(smem + kOffV + hf * 8192, &map_g, &bars->g_full, 0, static_cast<int>((bh_rows + i_q[hf]) * 64));
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_qk = instr_desc(0, kM, 64, 0, 0);   // e4m3 x e4m3, both K-major
      constexpr uint32_t idesc_pv = instr_desc(0, kM, 64, 0, 1);   // f16 x f16, V MN-major
      constexpr uint32_t idesc_lin = instr_desc(1, kM, 64, 0, 0);  // bf16 x bf16, both K-major
      const uint32_t q_addr = smem_u32(smem + kOffQ), k_addr = smem_u32(smem + kOffK);
      const uint32_t v_addr = smem_u32(smem + kOffV), p_addr = smem_u32(smem + kOffP);
      bool ok = mbar_wait(&bars->q_full, 0, abort_flag, p.status, 201);
      auto issue_qk = [&](int t) {
        const int st = t % kStages, buf = t & 1;
        if (!mbar_wait(&bars->k_full[st], (t / kStages) & 1, abort_flag, p.status, 202)) return false;
        if (!mbar_wait(&bars->s_empty[buf], ((t >> 1) & 1) ^ 1, abort_flag, p.status, 203)) return false;
        tc_fence_after();
        for (int hf = 0; hf < kHalves; ++hf) {
          const uint32_t d = tmem + kColS + buf * 64 + ((hf * 16u) << 16);
          for (int kk = 0; kk < 2; ++kk) {
            const uint64_t a = smem_desc(q_addr + (kPair ? hf * 4096 : 0) + kk * 32, 16, 512, kSwizzle64);
            const uint64_t b = smem_desc(k_addr + st * kKStage + hf * 4096 + kk * 32, 16, 512, kSwizzle64);
            mma_f8(d, a, b, idesc_qk, kk);
          }
        }
        mma_commit(&bars->k_empty[st]);
        mma_commit(&bars->s_full[buf]);
        return true;
      };
      auto issue_pv = [&](int t) {
        const int st = t % kStages, buf = t & 1;
        if (!mbar_wait(&bars->v_full[st], (t / kStages) & 1, abort_flag, p.status, 204)) return false;
        if (!mbar_wait(&bars->p_full[buf], (t >> 1) & 1, abort_flag, p.status, 205)) return false;
        tc_fence_after();
        for (int hf = 0; hf < kHalves; ++hf) {
          const uint32_t d = tmem + kColO + ((hf * 16u) << 16);
          for (int kk = 0; kk < 4; ++kk) {
            const uint64_t a = smem_desc(p_addr + buf * kPBuf + (kPair ? hf * 8192 : 0) + kk * 32, 16, 1024, kSwizzle128);
            const uint64_t b = smem_desc(v_addr + st * kVStage + hf * 8192 + kk * 2048, 8192, 1024, kSwizzle128);
            mma_f16(d, a, b, idesc_pv, (t > 0 || kk > 0) ? 1u : 0u);
          }
        }
        mma_commit(&bars->v_empty[st]);
        mma_commit(&bars->p_empty[buf]);
        return true;
      };
      for (int t = 0; t < steps && ok; ++t) {
        ok = issue_qk(t);
        if (ok && t > 0) ok = issue_pv(t - 1);
      }
      if (ok && steps > 0) ok = issue_pv(steps - 1);
      if (ok && p.k_marg > 0) {
        ok = mbar_wait(&bars->g_full, 0, abort_flag, p.status, 206) &&
             mbar_wait(&bars->phi_full, 0, abort_flag, p.status, 207);
        if (ok) {
          tc_fence_after();
          for (int hf = 0; hf < kHalves; ++hf) {
            const uint32_t d = tmem + kColL + ((hf * 16u) << 16);
            for (int kk = 0; kk < 4; ++kk) {
              const uint64_t a = smem_desc(p_addr + (kPair ? hf * 8192 : 0) + kk * 32, 16, 1024, kSwizzle128);
              const uint64_t b = smem_desc(v_addr + hf * 8192 + kk * 32, 16, 1024, kSwizzle128);
              mma_f16(d, a, b, idesc_lin, kk);
            }
          }
          mma_commit(&bars->l_full);
        }
      }
    }
  } else {
    // ------------------------------------------------------------------------------------------ softmax + epilogue
    const int quarter = warp & 3;                       // TMEM sub-partition this warp may touch
    const int hf = kPair ? (lane >> 4) : 0;             // which query block of the pair this thread serves
    const int row_in_block = kPair ? quarter * 16 + (lane & 15) : quarter * 32 + lane;
    const int p_row = kPair ? hf * 64 + row_in_block : row_in_block;  // row inside the P / phi tile
    const int iq = i_q[hf];
    const size_t q_tile = bh_rows + iq;
    const uint32_t lane_addr = tmem + ((static_cast<uint32_t>(quarter) * 32u) << 16);
    const int token = iq * BS + row_in_block;
    const float sq = __ldg(p.q_scales + q_tile);
    const float vref = __ldg(p.vref + bh);
    const float qk_scale = sq * (kLog2e * 0.125f);
    const int* list = p.crit_idx + q_tile * p.k_crit;
    uint8_t* p_tile = smem + kOffP;

    float m_ref = -1.0e30f, l = 0.f;
    bool ok = true;

    // per-step scalars, fetched one step ahead
    int j_next = steps > 0 ? __ldg(list) : 0;
    float sk_next = steps > 0 ? __ldg(p.k_scales + bh_rows + j_next) : 0.f;
    float sv_next = steps > 0 ? __ldg(p.v_scales + bh_rows + j_next) : 1.f;

    for (int t = 0; t < steps; ++t) {
      const int buf = t & 1;
      const int j = j_next;
      const float c = qk_scale * sk_next;
      const float f = sv_next / vref;
      if (t + 1 < steps) {
        j_next = __ldg(list + (t + 1) / kStepsPerBlock);
        sk_next = __ldg(p.k_scales + bh_rows + j_next);
        sv_next = __ldg(p.v_scales + bh_rows + j_next);
      }
      int valid = p.tokens - j * BS - (kPair ? 0 : (t & 1) * kStepKeys);
      valid = max(0, min(kStepKeys, valid));

      if (!(ok = mbar_wait(&bars->s_full[buf], (t >> 1) & 1, abort_flag, p.status, 301))) break;
      tc_fence_after();
      uint32_t s_lo[32], s_hi[32];
      tmem_ld32(lane_addr + kColS + buf * 64, s_lo);
      tmem_ld32(lane_addr + kColS + buf * 64 + 32, s_hi);
      tmem_wait_ld();
      tc_fence_before();
      mbar_arrive(&bars->s_empty[buf]);

      float sv[64];
#pragma unroll
      for (int k = 0; k < 32; ++k) {
        sv[k] = __uint_as_float(s_lo[k]);
        sv[k + 32] = __uint_as_float(s_hi[k]);
      }
      if (valid < kStepKeys) {
#pragma unroll
        for (int k = 0; k < 64; ++k)
          if (k >= valid) sv[k] = -INFINITY;
      }
      // row maximum of the raw scores (c > 0 commutes with max), four independent chains
      float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
      for (int k = 0; k < 64; ++k) mx4[k & 3] = fmaxf(mx4[k & 3], sv[k]);
      const float tile_max = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * c;

      bool need = false;
      float alpha = 1.f;
      if (t == 0) {
        m_ref = fmaxf(tile_max, m_ref);
      } else if (tile_max > m_ref + kRescaleThreshold) {
        need = true;
        alpha = ex2(m_ref - tile_max);
        m_ref = tile_max;
        l *= alpha;
      }
      const float neg_shift = __log2f(f) - m_ref;
      float sum4[4] = {0.f, 0.f, 0.f, 0.f};
      uint32_t packed[32];
#pragma unroll
      for (int k = 0; k < 64; k += 2) {
        const float p0 = ex2(fmaf(sv[k], c, neg_shift)), p1 = ex2(fmaf(sv[k + 1], c, neg_shift));
        sum4[(k >> 1) & 3] += p0 + p1;
        packed[k >> 1] = pack_half2(p0, p1);
      }
      l += ((sum4[0] + sum4[1]) + (sum4[2] + sum4[3])) / f;

      // P[buf] is free once the P V product of step t-2 has completed
      if (!(ok = mbar_wait(&bars->p_empty[buf], ((t >> 1) & 1) ^ 1, abort_flag, p.status, 302))) break;
      uint8_t* prow = p_tile + buf * kPBuf + p_row * 128;
#pragma unroll
      for (int ch = 0; ch < 8; ++ch) {
        const uint4 v4 = make_uint4(packed[4 * ch], packed[4 * ch + 1], packed[4 * ch + 2], packed[4 * ch + 3]);
        *reinterpret_cast<uint4*>(prow + ((ch ^ (p_row & 7)) << 4)) = v4;
      }
      if (__any_sync(0xFFFFFFFFu, need)) {
        // O may only be touched between the P V products of steps t-1 and t
        if (!(ok = mbar_wait(&bars->p_empty[buf ^ 1], ((t - 1) >> 1) & 1, abort_flag, p.status, 303))) break;
        tc_fence_after();
        uint32_t o_lo[32], o_hi[32];
        tmem_ld32(lane_addr + kColO, o_lo);
        tmem_ld32(lane_addr + kColO + 32, o_hi);
        tmem_wait_ld();
#pragma unroll
        for (int k = 0; k < 32; ++k) {
          o_lo[k] = __float_as_uint(__uint_as_float(o_lo[k]) * alpha);
          o_hi[k] = __float_as_uint(__uint_as_float(o_hi[k]) * alpha);
        }
        tmem_st32(lane_addr + kColO, o_lo);
        tmem_st32(lane_addr + kColO + 32, o_hi);
        tmem_wait_st();
        tc_fence_before();
      }
      fence_proxy_async_smem();
      mbar_arrive(&bars->p_full[buf]);
    }

    // wait for the last P V product
    if (ok && steps > 0) {
      const int last = steps - 1;
      ok = mbar_wait(&bars->p_empty[last & 1], (last >> 1) & 1, abort_flag, p.status, 304);
      tc_fence_after();
    }

    // linear branch: phi(q) as bf16 A operand, denominators on the side
    float den = 1.f;
    if (ok && p.k_marg > 0) {
      const uint4* qsrc = reinterpret_cast<const uint4*>(p.q_codes + (q_tile * BS + row_in_block) * kHeadDim);
      const float* zeta = p.zeta + q_tile * kHeadDim;
      float e[64];
      float mx = -INFINITY;
#pragma unroll
      for (int w = 0; w < 4; ++w) {
        const uint4 raw = __ldg(qsrc + w);
        const uint32_t words[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
        for (int xw = 0; xw < 4; ++xw) {
          float fv[4];
          e4m3x4_to_float(words[xw], fv);
#pragma unroll
          for (int y = 0; y < 4; ++y) {
            e[w * 16 + xw * 4 + y] = fv[y] * sq;
            mx = fmaxf(mx, fv[y] * sq);
          }
        }
      }
      uint32_t packed[32];
      den = 0.f;
#pragma unroll
      for (int d = 0; d < 64; d += 2) {
        float e0, e1;
        if (p.phi == LITE3R_PHI_SOFTMAX) {  // the softmax normaliser cancels in the ratio
          e0 = ex2((e[d] - mx) * kLog2e);
          e1 = ex2((e[d + 1] - mx) * kLog2e);
        } else {
          e0 = e[d] > 0.f ? e[d] + 1.f : ex2(e[d] * kLog2e);
          e1 = e[d + 1] > 0.f ? e[d + 1] + 1.f : ex2(e[d + 1] * kLog2e);
        }
        const uint32_t pk = pack_bf162(e0, e1);
        packed[d >> 1] = pk;
        // the denominator uses the same rounded values as the MMA's numerator
        den = fmaf(__uint_as_float(pk << 16), __ldg(zeta + d), den);
        den = fmaf(__uint_as_float(pk & 0xFFFF0000u), __ldg(zeta + d + 1), den);
      }
      uint8_t* prow = p_tile + p_row * 128;
#pragma unroll
      for (int ch = 0; ch < 8; ++ch) {
        const uint4 v4 = make_uint4(packed[4 * ch], packed[4 * ch + 1], packed[4 * ch + 2], packed[4 * ch + 3]);
        *reinterpret_cast<uint4*>(prow + ((ch ^ (p_row & 7)) << 4)) = v4;
      }
      fence_proxy_async_smem();
      mbar_arrive(&bars->phi_full);
      ok = mbar_wait(&bars->l_full, 0, abort_flag, p.status, 305);
      tc_fence_after();
    }

    if (ok) {
      const bool live = token < p.tokens && (!kPair || hf == 0 || i_q[1] != i_q[0]);
      const int b = bh / p.heads, h = bh % p.heads;
      float* dst = p.out + b * p.out_stride_b + h * p.out_stride_h + static_cast<long long>(token) * p.out_stride_n;
      const float o_scale = steps > 0 ? vref / l : 0.f;
      const float l_scale = p.k_marg > 0 ? 1.f / den : 0.f;
#pragma unroll
      for (int part = 0; part < 2; ++part) {
        uint32_t o[32], ln[32];
        if (steps > 0) tmem_ld32(lane_addr + kColO + part * 32, o);
        if (p.k_marg > 0) tmem_ld32(lane_addr + kColL + part * 32, ln);
        tmem_wait_ld();
        if (live) {
#pragma unroll
          for (int k = 0; k < 32; k += 4) {
            float r[4];
#pragma unroll
            for (int y = 0; y < 4; ++y) {
              const float a = steps > 0 ? __uint_as_float(o[k + y]) * o_scale : 0.f;
              const float bb = p.k_marg > 0 ? __uint_as_float(ln[k + y]) * l_scale : 0.f;
              r[y] = a + bb;
            }
            *reinterpret_cast<float4*>(dst + part * 32 + k) = make_float4(r[0], r[1], r[2], r[3]);
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

// ------------------------------------------------------------------------------------------------ host side
template <int BS>
lite3r_status launch(const AttentionLaunch& a, cudaStream_t stream) {
  const lite3r_shape& s = a.shape;
  const int nb = ceil_div(s.tokens, BS);
  const uint64_t tiles = static_cast<uint64_t>(s.batch) * s.heads * nb;
  alignas(64) CUtensorMap map_q, map_k, map_v, map_g;
  lite3r_status st;
  if ((st = make_tensor_map_2d(&map_q, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, a.q_codes, 64, tiles * BS, 64, 64, CU_TENSOR_MAP_SWIZZLE_64B)) != LITE3R_OK) return st;
  if ((st = make_tensor_map_2d(&map_k, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, a.k_codes, 64, tiles * BS, 64, 64, CU_TENSOR_MAP_SWIZZLE_64B)) != LITE3R_OK) return st;
  if ((st = make_tensor_map_2d(&map_v, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, a.v16, 64, tiles * BS, 64, 64, CU_TENSOR_MAP_SWIZZLE_128B)) != LITE3R_OK) return st;
  if ((st = make_tensor_map_2d(&map_g, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, a.g16, 64, tiles * 64, 64, 64, CU_TENSOR_MAP_SWIZZLE_128B)) != LITE3R_OK) return st;
  AttnParams p;
  p.q_codes = a.q_codes;
  p.q_scales = a.q_scales;
  p.k_scales = a.k_scales;
  p.v_scales = a.v_scales;
  p.vref = a.vref;
  p.crit_idx = a.crit_idx;
  p.zeta = a.zeta;
  p.out = a.out;
  p.out_stride_b = a.out_stride_b;
  p.out_stride_h = a.out_stride_h;
  p.out_stride_n = a.out_stride_n;
  p.heads = s.heads;
  p.tokens = s.tokens;
  p.nb = nb;
  p.k_crit = a.k_crit;
  p.k_marg = a.k_marg;
  p.phi = a.phi;
  p.status = a.device_status;
  st = record_cuda(cudaFuncSetAttribute(attention_kernel<BS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        static_cast<int>(kSmemBytes)));
  if (st != LITE3R_OK) return st;
  const int ctas = s.batch * s.heads * (BS == 64 ? (nb + 1) / 2 : nb);
  attention_kernel<BS><<<ctas, kThreads, kSmemBytes, stream>>>(map_q, map_k, map_v, map_g, p);
  return after_launch();
}

}  // namespace

lite3r_status launch_attention(const AttentionLaunch& a, cudaStream_t stream) {
  return a.shape.block == 64 ? launch<64>(a, stream) : launch<128>(a, stream);
}

}  // namespace lite3r
