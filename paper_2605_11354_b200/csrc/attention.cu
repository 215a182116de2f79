// K4: critical-block softmax attention + linear branch + add (Algorithm 1's sparse branch, linear output, projection and sum) on tcgen05 / TMEM / TMA.
//
// One CTA owns 128 query rows of one (b, h): at block 64 a PAIR of query blocks (two M=64 accumulators interleaved
// in the two 16-lane halves of every TMEM sub-partition), at block 128 one query block (M=128).  Work advances in
// steps of 64 keys.  The steps are dealt alternately to two independent "sets" (even steps -> set 0, odd steps ->
// set 1).  A set is 128 softmax threads (one query row each, TMEM lane = thread) plus one MMA-issuing thread, with
// its own score buffer S, probability buffer P, output accumulator O and online-softmax state (reference maximum and
// row sum); the two partial results are merged exactly at the end, O = (w0 O0 + w1 O1) / (w0 l0 + w1 l1) with
// w = 2^(m_set - m).  Because the sets never wait for each other, an SM (two CTAs) always has four softmax streams
// in different phases, which keeps the exponential unit busy while other streams wait on barriers, TMEM loads or
// shared-memory stores.  Per step t of set b = t & 1:
//   TMA      K tile(s) (e4m3, 64-byte rows, 64B swizzle) and V tile(s) (dequantised fp16, 128B swizzle) -> smem ring
//   tcgen05  S_b = Q K^T           kind::f8f6f4, fp32 accumulators in TMEM (64 columns)
//   softmax  pass 1: row maximum of the 64 scores, lazy-rescale decision; pass 2: exp2 and row sum, 32 columns at a
//            time; P goes to shared memory as fp16 in the MMA's K-major 128B-swizzled layout
//   tcgen05  O_b += P V            kind::f16, V as MN-major B operand, fp32 accumulators in TMEM (64 columns)
// P is carried in fp16 (not e4m3): one e4m3 term has a 2.6 % rounding error per probability, which alone is ten
// times the output tolerance.  V travels as the dequantised value in fp16 (2^-12 relative rounding).
// Tail: phi(Q) (bf16) times the aggregated, projected summaries G_i (bf16) as one more MMA, divided by
// phi(Q) . zeta_i, added to the merged softmax output and stored (each set stores 32 of the 64 output columns).
//
// Warp roles (352 threads): warp 0 = TMA producer; warps 1 and 2 = MMA issuers of set 0 and set 1 (a single thread
// can issue a small tcgen05.mma only every ~50 clocks, so each set has its own); warps 3-6 = softmax set 0,
// warps 7-10 = softmax set 1.  "Product of step t done" is one barrier per product (rings of six) on which the
// softmax threads and the TMA producer wait.
// Every mbarrier wait is bounded (1 s); on expiry the CTA sets *device_status and all roles leave their loops.
#include "common.cuh"
#include "sm100.cuh"

namespace lite3r {

namespace {

using namespace sm100;

constexpr int kStages = 3;
constexpr int kSetThreads = 128;
constexpr int kSoftmaxThreads = 2 * kSetThreads;
constexpr int kCtrlWarps = 3;
constexpr int kThreads = kCtrlWarps * 32 + kSoftmaxThreads;
constexpr uint32_t kBackoffNs = 100;  // sleep between polls of the single-thread roles
constexpr int kRing = 6;              // lcm of the two sets and the three K/V stages
constexpr int kStepKeys = 64;
constexpr uint32_t kTmemCols = 256;
constexpr uint32_t kColS = 0, kColO = 128, kColL = 0;  // S_b at 64 b, O_b at 128 + 64 b; the linear branch reuses S_0
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kRescaleThreshold = 8.0f;  // lazy rescale: keep the old reference max until it is beaten by 2^8
constexpr float kNoMax = -1.0e30f;         // reference maximum of a row that has seen no valid key yet
constexpr uint32_t kOffX = 8192;           // epilogue exchange between the sets: reuses K stage 0 (4 KB)

// shared-memory map (bytes from a 1024-aligned base)
constexpr uint32_t kQBytes = 8192, kKStage = 8192, kVStage = 16384, kPBuf = 16384;
constexpr uint32_t kOffQ = 0;
constexpr uint32_t kOffK = kOffQ + kQBytes;
constexpr uint32_t kOffV = kOffK + kStages * kKStage;
constexpr uint32_t kOffP = kOffV + kStages * kVStage;
constexpr uint32_t kOffG = kOffK + kKStage;  // aggregated summaries of the linear branch: K stages 1-2 (16 KB)
constexpr uint32_t kOffZeta = kOffX + 4096;  // their denominators zeta_i (256 B per query block): rest of K stage 0
constexpr uint32_t kOffBar = kOffP + 2 * kPBuf;
constexpr uint32_t kSmemBytes = kOffBar + 256;  // two CTAs per SM: 2 * (114944 + 1024 reserved) <= 232448

struct Bars {
  uint64_t q_full, g_full, phi_full, l_full, x_full;
  uint64_t k_full[kStages], v_full[kStages];  // TMA -> issuers
  uint64_t qk_done[kRing], pv_done[kRing];    // product of step t complete: barrier t % 6, phase (t / 6)
  uint64_t s_empty[2], p_full[2];             // softmax set b -> issuer b
  uint32_t tmem_base;
  int abort;
};

struct AttnParams {
  const uint8_t* q_codes;
  const float* q_scales;
  const float* k_scales;
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
__device__ __forceinline__ float max3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}
__device__ __forceinline__ uint32_t pack_bf162(float a, float b) {
  __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&h);
}

// exp2 of 32 scaled scores, packed to fp16 pairs; returns the sum.  Arguments and sums run on pairs of columns
// (packed fp32x2 fma / add).
__device__ __forceinline__ float exp_half_row(const uint32_t (&x)[32], float c, float neg_ref, uint32_t* packed) {
  const uint64_t c2 = pack_f32x2(c, c), shift2 = pack_f32x2(neg_ref, neg_ref);
  uint64_t sum2[2] = {0ull, 0ull};  // bit pattern of (0.f, 0.f)
#pragma unroll
  for (int k = 0; k < 32; k += 2) {
    float a0, a1;
    unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(x[k]), __uint_as_float(x[k + 1])), c2, shift2), a0, a1);
    const float p0 = ex2(a0), p1 = ex2(a1);
    sum2[(k >> 1) & 1] = add_f32x2(sum2[(k >> 1) & 1], pack_f32x2(p0, p1));
    packed[k >> 1] = pack_half2(p0, p1);
  }
  float s0, s1;
  unpack_f32x2(add_f32x2(sum2[0], sum2[1]), s0, s1);
  return s0 + s1;
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
    mbar_init(&bars->phi_full, kSoftmaxThreads);
    mbar_init(&bars->l_full, 1);
    mbar_init(&bars->x_full, kSoftmaxThreads);
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&bars->k_full[s], 1);
      mbar_init(&bars->v_full[s], 1);
    }
    for (int r = 0; r < kRing; ++r) {
      mbar_init(&bars->qk_done[r], 1);
      mbar_init(&bars->pv_done[r], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&bars->s_empty[b], kSetThreads);
      mbar_init(&bars->p_full[b], kSetThreads);
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
      // tile row (in the code tensors) of step t for query block hf
      auto tile_row = [&](int t, int hf) {
        if (kPair) return static_cast<int>((bh_rows + ldg_pinned((hf ? list1 : list0) + t)) * 64);
        return static_cast<int>((bh_rows + ldg_pinned(list0 + t / 2)) * 128 + (t & 1) * 64);
      };
      // K and V tiles are loaded by two independent cursors: a K stage is free after the Q K^T of three steps
      // earlier, a V stage only after that step's P V, and neither load may wait behind the other's condition.
      // The rows of each cursor's next step are fetched one step ahead.
      int tk = 0, tv = 0;
      int rk[2] = {0, 0}, rv[2] = {0, 0};
      if (steps > 0) {
        for (int hf = 0; hf < kHalves; ++hf) rk[hf] = rv[hf] = tile_row(0, hf);
      }
      IdleGuard guard;
      bool ok = true;
      while (ok && (tk < steps || tv < steps)) {
        bool moved = false;
        if (tk < steps) {
          const int u = tk - kStages;
          if (u < 0 || mbar_test(&bars->qk_done[u % kRing], (u / kRing) & 1)) {
            const int st = tk % kStages;
            mbar_arrive_expect_tx(&bars->k_full[st], kKTx);
            for (int hf = 0; hf < kHalves; ++hf)
              tma_load_2d(smem + kOffK + st * kKStage + hf * 4096, &map_k, &bars->k_full[st], 0, rk[hf]);
            if (++tk < steps) {
              for (int hf = 0; hf < kHalves; ++hf) rk[hf] = tile_row(tk, hf);
            }
            moved = true;
          }
        }
        if (tv < steps) {
          const int u = tv - kStages;
          if (u < 0 || mbar_test(&bars->pv_done[u % kRing], (u / kRing) & 1)) {
            const int st = tv % kStages;
            mbar_arrive_expect_tx(&bars->v_full[st], kVTx);
            for (int hf = 0; hf < kHalves; ++hf)
              tma_load_2d(smem + kOffV + st * kVStage + hf * 8192, &map_v, &bars->v_full[st], 0, rv[hf]);
            if (++tv < steps) {
              for (int hf = 0; hf < kHalves; ++hf) rv[hf] = tile_row(tv, hf);
            }
            moved = true;
          }
        }
        if (moved) {
          guard.progress();
        } else {
          ok = guard.idle(abort_flag, p.status, 101, kBackoffNs);
        }
      }
      if (ok && p.k_marg > 0) {
        // The aggregated summaries go to K stages 1 and 2, which are free once the last three Q K^T products have
        // completed: well before the last P V products, so this load is off the tail's critical path.
        for (int u = max(0, steps - kStages); u < steps && ok; ++u)
          ok = mbar_wait(&bars->qk_done[u % kRing], (u / kRing) & 1, abort_flag, p.status, 103, kBackoffNs);
        if (ok) {
          mbar_arrive_expect_tx(&bars->g_full, kHalves * (8192 + 256));
          for (int hf = 0; hf < kHalves; ++hf) {
            tma_load_2d(smem + kOffG + hf * 8192, &map_g, &bars->g_full, 0, static_cast<int>((bh_rows + i_q[hf]) * 64));
            bulk_load(smem + kOffZeta + hf * 256, p.zeta + (bh_rows + i_q[hf]) * kHeadDim, 256, &bars->g_full);
          }
        }
      }
    }
  } else if (warp < kCtrlWarps) {
    // ------------------------------------------------------------------------------------------ MMA issuer of set b
    if (lane == 0) {
      const int b = warp - 1;
      constexpr uint32_t idesc_qk = instr_desc(0, kM, 64, 0, 0);   // e4m3 x e4m3, both K-major
      constexpr uint32_t idesc_pv = instr_desc(0, kM, 64, 0, 1);   // f16 x f16, V MN-major
      constexpr uint32_t idesc_lin = instr_desc(1, kM, 64, 0, 0);  // bf16 x bf16, both K-major
      const uint32_t q_addr = smem_u32(smem + kOffQ), k_addr = smem_u32(smem + kOffK);
      const uint32_t v_addr = smem_u32(smem + kOffV), p_addr = smem_u32(smem + kOffP) + b * kPBuf;
      const uint32_t s_tmem = tmem + kColS + b * 64, o_tmem = tmem + kColO + b * 64;
      bool ok = mbar_wait(&bars->q_full, 0, abort_flag, p.status, 201, kBackoffNs);
      auto issue_qk = [&](int t) {  // S_b = Q K(t)^T
        const int st = t % kStages;
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < 2; ++kk) {
#pragma unroll
          for (int hf = 0; hf < kHalves; ++hf) {
            const uint64_t a = smem_desc(q_addr + (kPair ? hf * 4096 : 0) + kk * 32, 16, 512, kSwizzle64);
            const uint64_t bd = smem_desc(k_addr + st * kKStage + hf * 4096 + kk * 32, 16, 512, kSwizzle64);
            mma_f8(s_tmem + ((hf * 16u) << 16), a, bd, idesc_qk, kk);
          }
        }
        mma_commit(&bars->qk_done[t % kRing]);
      };
      auto issue_pv = [&](int t) {  // O_b += P(t) V(t)
        const int st = t % kStages;
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
#pragma unroll
          for (int hf = 0; hf < kHalves; ++hf) {
            const uint64_t a = smem_desc(p_addr + (kPair ? hf * 8192 : 0) + kk * 32, 16, 1024, kSwizzle128);
            const uint64_t bd = smem_desc(v_addr + st * kVStage + hf * 8192 + kk * 2048, 8192, 1024, kSwizzle128);
            mma_f16(o_tmem + ((hf * 16u) << 16), a, bd, idesc_pv, (t >= 2 || kk > 0) ? 1u : 0u);
          }
        }
        mma_commit(&bars->pv_done[t % kRing]);
      };
      // Two cursors, polled without blocking, so that neither product waits behind the other's operands:
      //   Q K^T of step tq needs its K tile and S_b drained by the softmax of the set's previous step (tq - 2);
      //   P V of step tp needs its V tile and the probabilities of step tp.
      int tq = b, tp = b;
      IdleGuard guard;
      while (ok && tp < steps) {
        bool moved = false;
        if (mbar_test(&bars->p_full[b], (tp >> 1) & 1) && mbar_test(&bars->v_full[tp % kStages], (tp / kStages) & 1)) {
          issue_pv(tp);
          tp += 2;
          moved = true;
        }
        if (tq < steps && mbar_test(&bars->k_full[tq % kStages], (tq / kStages) & 1) &&
            mbar_test(&bars->s_empty[b], ((tq >> 1) & 1) ^ 1)) {
          issue_qk(tq);
          tq += 2;
          moved = true;
        }
        if (moved) {
          guard.progress();
        } else {
          ok = guard.idle(abort_flag, p.status, 202, 0);
        }
      }
      if (b == 0 && ok && p.k_marg > 0) {
        ok = mbar_wait(&bars->g_full, 0, abort_flag, p.status, 206, kBackoffNs) &&
             mbar_wait(&bars->phi_full, 0, abort_flag, p.status, 207, kBackoffNs);
        if (ok) {
          tc_fence_after();
          const uint32_t phi_addr = smem_u32(smem + kOffP), g_addr = smem_u32(smem + kOffG);
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) {
#pragma unroll
            for (int hf = 0; hf < kHalves; ++hf) {
              const uint64_t a = smem_desc(phi_addr + (kPair ? hf * 8192 : 0) + kk * 32, 16, 1024, kSwizzle128);
              const uint64_t bd = smem_desc(g_addr + hf * 8192 + kk * 32, 16, 1024, kSwizzle128);
              mma_f16(tmem + kColL + ((hf * 16u) << 16), a, bd, idesc_lin, kk);
            }
          }
          mma_commit(&bars->l_full);
        }
      }
    }
  } else {
    // ------------------------------------------------------------------------------------------ softmax + epilogue
    const int quarter = warp & 3;                       // TMEM sub-partition this warp may touch
    const int b = (warp - kCtrlWarps) >> 2;             // set: steps t with (t & 1) == b
    const int hf = kPair ? (lane >> 4) : 0;             // which query block of the pair this thread serves
    const int row_in_block = kPair ? quarter * 16 + (lane & 15) : quarter * 32 + lane;
    const int p_row = kPair ? hf * 64 + row_in_block : row_in_block;  // row inside the P / phi tile
    const int iq = i_q[hf];
    const size_t q_tile = bh_rows + iq;
    const uint32_t lane_addr = tmem + ((static_cast<uint32_t>(quarter) * 32u) << 16);
    const uint32_t s_addr = lane_addr + kColS + b * 64, o_addr = lane_addr + kColO + b * 64;
    const float sq = __ldg(p.q_scales + q_tile);
    const float qk_scale = sq * (kLog2e * 0.125f);
    const int* list = p.crit_idx + q_tile * p.k_crit;
    uint8_t* const prow = smem + kOffP + b * kPBuf + p_row * 128;  // this thread's 128-byte row of P_b
    const int swz = p_row & 7;

    float m_ref = kNoMax, l = 0.f;
    bool ok = true;

    // per-step scalars: the key-block index is fetched two of the set's steps ahead and its scale one ahead, so
    // that no load in the loop waits for the address produced by another load of the same iteration
    int j_cur = b < steps ? ldg_pinned(list + b / kStepsPerBlock) : 0;
    int j_nxt = b + 2 < steps ? ldg_pinned(list + (b + 2) / kStepsPerBlock) : 0;
    float sk_cur = b < steps ? ldg_pinned(p.k_scales + bh_rows + j_cur) : 0.f;

    for (int t = b; t < steps; t += 2) {
      const int j = j_cur;
      const float c = qk_scale * sk_cur;
      j_cur = j_nxt;
      if (t + 2 < steps) sk_cur = ldg_pinned(p.k_scales + bh_rows + j_nxt);
      if (t + 4 < steps) j_nxt = ldg_pinned(list + (t + 4) / kStepsPerBlock);
      int valid = p.tokens - j * BS - (kPair ? 0 : (t & 1) * kStepKeys);
      valid = max(0, min(kStepKeys, valid));

      if (!(ok = mbar_wait(&bars->qk_done[t % kRing], (t / kRing) & 1, abort_flag, p.status, 301))) break;
      tc_fence_after();

      // pass 1: row maximum of the raw scores (c > 0 commutes with max), four independent chains
      float tile_max;
      {
        uint32_t x[32], y[32];
        tmem_ld32(s_addr, x);
        tmem_ld32(s_addr + 32, y);
        tmem_wait_ld();
        if (valid < kStepKeys) {
#pragma unroll
          for (int k = 0; k < 32; ++k) {
            if (k >= valid) x[k] = 0xFF800000u;  // -inf
            if (32 + k >= valid) y[k] = 0xFF800000u;
          }
        }
        float mx4[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) mx4[q] = fmaxf(__uint_as_float(x[q]), __uint_as_float(y[q]));
#pragma unroll
        for (int k = 4; k < 32; k += 4) {
#pragma unroll
          for (int q = 0; q < 4; ++q) mx4[q] = max3(mx4[q], __uint_as_float(x[k + q]), __uint_as_float(y[k + q]));
        }
        // a step without any valid key (second half of a short last block) leaves the reference where it is
        tile_max = fmaxf(max3(fmaxf(mx4[0], mx4[1]), mx4[2], mx4[3]) * c, kNoMax);
      }
      bool need = false;
      float alpha = 1.f;
      if (t < 2) {
        m_ref = tile_max;
      } else if (tile_max > m_ref + kRescaleThreshold) {
        need = true;
        alpha = ex2(m_ref - tile_max);
        m_ref = tile_max;
        l *= alpha;
      }
      // P_b is free once the P V product of the set's previous step has completed; asked now, needed after the
      // first exponentials
      uint64_t* const pv_bar = &bars->pv_done[(t + kRing - 2) % kRing];
      const uint32_t pv_par = static_cast<uint32_t>(((t - 2) / kRing) & 1);
      const bool pv_ok = t < 2 || mbar_try_wait(pv_bar, pv_par);

      // pass 2: exponentials and row sum, 32 columns at a time; each half row of P is stored as soon as it exists
      {
        uint32_t x[32], packed[16];
        tmem_ld32(s_addr, x);
        tmem_wait_ld();
        if (valid < 32) {
#pragma unroll
          for (int k = 0; k < 32; ++k)
            if (k >= valid) x[k] = 0xFF800000u;
        }
        l += exp_half_row(x, c, -m_ref, packed);
        if (!pv_ok && !(ok = mbar_wait(pv_bar, pv_par, abort_flag, p.status, 302))) break;
#pragma unroll
        for (int ch = 0; ch < 4; ++ch)
          *reinterpret_cast<uint4*>(prow + ((ch ^ swz) << 4)) =
              make_uint4(packed[4 * ch], packed[4 * ch + 1], packed[4 * ch + 2], packed[4 * ch + 3]);
        tmem_ld32(s_addr + 32, x);
        tmem_wait_ld();
        tc_fence_before();
        mbar_arrive(&bars->s_empty[b]);  // S_b is in registers: the issuer may overwrite it with the set's next step
        if (valid < kStepKeys) {
#pragma unroll
          for (int k = 0; k < 32; ++k)
            if (32 + k >= valid) x[k] = 0xFF800000u;
        }
        l += exp_half_row(x, c, -m_ref, packed);
#pragma unroll
        for (int ch = 0; ch < 4; ++ch)
          *reinterpret_cast<uint4*>(prow + (((4 + ch) ^ swz) << 4)) =
              make_uint4(packed[4 * ch], packed[4 * ch + 1], packed[4 * ch + 2], packed[4 * ch + 3]);
      }
      if (__any_sync(0xFFFFFFFFu, need)) {
        // O_b is only touched by the set's own P V products: the previous one has completed (pv_bar above) and the
        // next one waits for this thread's arrival below
        tc_fence_after();
#pragma unroll
        for (int part = 0; part < 2; ++part) {
          uint32_t o[32];
          tmem_ld32(o_addr + part * 32, o);
          tmem_wait_ld();
#pragma unroll
          for (int k = 0; k < 32; ++k) o[k] = __float_as_uint(__uint_as_float(o[k]) * alpha);
          tmem_st32(o_addr + part * 32, o);
        }
        tmem_wait_st();
        tc_fence_before();
      }
      fence_proxy_async_smem();
      mbar_arrive(&bars->p_full[b]);
    }

    // linear branch: this thread's 32 columns (set b -> columns 32 b ..) of phi(q) as bf16 A operand, partial
    // denominator on the side; computed in registers while the last P V products are still running.  The query row
    // comes from the Q tile in shared memory (64-byte rows, 64B swizzle: 16-byte chunk c of row r sits at chunk
    // c ^ ((r >> 1) & 3)), zeta_i from the copy that arrived with the aggregated summaries.
    float den = 0.f;
    uint32_t phi_packed[16];
    if (ok && p.k_marg > 0) {
      ok = mbar_wait(&bars->q_full, 0, abort_flag, p.status, 307) && mbar_wait(&bars->g_full, 0, abort_flag, p.status, 308);
      const uint8_t* qrow = smem + kOffQ + p_row * 64;
      const float4* zeta = reinterpret_cast<const float4*>(smem + kOffZeta + hf * 256 + b * 128);
      const int qswz = (p_row >> 1) & 3;
      float e[32];
      float mx = -INFINITY;
#pragma unroll
      for (int w = 0; w < 4; ++w) {
        const uint4 raw = *reinterpret_cast<const uint4*>(qrow + ((w ^ qswz) << 4));
        const uint32_t words[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
        for (int xw = 0; xw < 4; ++xw) {
          float fv[4];
          e4m3x4_to_float(words[xw], fv);
#pragma unroll
          for (int y = 0; y < 4; ++y) {
            mx = fmaxf(mx, fv[y]);
            if ((w >> 1) == b) e[(w & 1) * 16 + xw * 4 + y] = fv[y];
          }
        }
      }
      const float cq = sq * kLog2e, shift = mx * cq;  // sq > 0 commutes with max
#pragma unroll
      for (int d = 0; d < 32; d += 4) {
        const float4 z = zeta[d >> 2];
        const float zz[4] = {z.x, z.y, z.z, z.w};
#pragma unroll
        for (int y = 0; y < 4; y += 2) {
          float e0, e1;
          if (p.phi == LITE3R_PHI_SOFTMAX) {  // the softmax normaliser cancels in the ratio
            e0 = ex2(fmaf(e[d + y], cq, -shift));
            e1 = ex2(fmaf(e[d + y + 1], cq, -shift));
          } else {
            e0 = e[d + y] > 0.f ? fmaf(e[d + y], sq, 1.f) : ex2(e[d + y] * cq);
            e1 = e[d + y + 1] > 0.f ? fmaf(e[d + y + 1], sq, 1.f) : ex2(e[d + y + 1] * cq);
          }
          const uint32_t pk = pack_bf162(e0, e1);
          phi_packed[(d + y) >> 1] = pk;
          // the denominator uses the same rounded values as the MMA's numerator
          den = fmaf(__uint_as_float(pk << 16), zz[y], den);
          den = fmaf(__uint_as_float(pk & 0xFFFF0000u), zz[y + 1], den);
        }
      }
    }

    // both sets' last P V products (the epilogue reads O_0 and O_1, and the phi operand reuses P_0)
    for (int u = max(0, steps - 2); u < steps && ok; ++u)
      ok = mbar_wait(&bars->pv_done[u % kRing], (u / kRing) & 1, abort_flag, p.status, 304);
    tc_fence_after();
    if (ok && p.k_marg > 0) {
      uint8_t* const phirow = smem + kOffP + p_row * 128;
#pragma unroll
      for (int i = 0; i < 4; ++i)
        *reinterpret_cast<uint4*>(phirow + (((b * 4 + i) ^ swz) << 4)) =
            make_uint4(phi_packed[4 * i], phi_packed[4 * i + 1], phi_packed[4 * i + 2], phi_packed[4 * i + 3]);
      fence_proxy_async_smem();
      mbar_arrive(&bars->phi_full);
    }

    // the two threads of a row (one per set) swap reference maximum, row sum and partial denominator (K stage 0 is
    // free by now: every Q K^T product has completed before the last P V products did)
    float w_mine = 0.f, w_other = 0.f, inv_l = 0.f;
    if (ok) {
      float4* xbuf = reinterpret_cast<float4*>(smem + kOffX);
      xbuf[b * 128 + p_row] = make_float4(m_ref, l, den, 0.f);
      mbar_arrive(&bars->x_full);
      ok = mbar_wait(&bars->x_full, 0, abort_flag, p.status, 306);
      if (ok) {
        const float4 other = xbuf[(b ^ 1) * 128 + p_row];
        const float m = fmaxf(m_ref, other.x);
        w_mine = ex2(m_ref - m);    // a set without (valid) steps keeps m_ref = kNoMax and l = 0
        w_other = ex2(other.x - m);
        const float l_tot = w_mine * l + w_other * other.y;
        inv_l = steps > 0 ? 1.f / l_tot : 0.f;
        den += other.z;
      }
    }
    if (ok && p.k_marg > 0) {
      ok = mbar_wait(&bars->l_full, 0, abort_flag, p.status, 305);
      tc_fence_after();
    }

    ok = __all_sync(0xFFFFFFFFu, ok);  // the store below synchronises the warp
    if (ok) {
      const int bb = bh / p.heads, h = bh % p.heads;
      // accumulators of a set that ran no step hold no data: they are not read
      const bool has_mine = steps > b, has_other = steps > (b ^ 1);
      const float l_scale = p.k_marg > 0 ? 1.f / den : 0.f;
      const float s_mine = has_mine ? w_mine * inv_l : 0.f, s_other = has_other ? w_other * inv_l : 0.f;
      float acc[32];
#pragma unroll
      for (int k = 0; k < 32; ++k) acc[k] = 0.f;
      uint32_t v[32];
      if (has_mine) {
        tmem_ld32(lane_addr + kColO + b * 64 + b * 32, v);
        tmem_wait_ld();
#pragma unroll
        for (int k = 0; k < 32; ++k) acc[k] = __uint_as_float(v[k]) * s_mine;
      }
      if (has_other) {
        tmem_ld32(lane_addr + kColO + (b ^ 1) * 64 + b * 32, v);
        tmem_wait_ld();
#pragma unroll
        for (int k = 0; k < 32; ++k) acc[k] = fmaf(__uint_as_float(v[k]), s_other, acc[k]);
      }
      if (p.k_marg > 0) {
        tmem_ld32(lane_addr + kColL + b * 32, v);
        tmem_wait_ld();
#pragma unroll
        for (int k = 0; k < 32; ++k) acc[k] = fmaf(__uint_as_float(v[k]), l_scale, acc[k]);
      }
      // A thread owns 128 bytes of one output row, so a direct store would touch 32 different lines per instruction.
      // The warp's 32 x 128-byte block is turned around in its own rows of P_b (free: P V products and the linear
      // product have completed) so that every store instruction writes four whole 128-byte row segments.
#pragma unroll
      for (int ch = 0; ch < 8; ++ch)
        *reinterpret_cast<float4*>(prow + ((ch ^ swz) << 4)) =
            make_float4(acc[4 * ch], acc[4 * ch + 1], acc[4 * ch + 2], acc[4 * ch + 3]);
      __syncwarp();
      const int ch = lane & 7;
      float* const out_bh = p.out + bb * p.out_stride_b + h * p.out_stride_h + b * 32 + ch * 4;
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int r = 4 * k + (lane >> 3);  // row of this warp's block: the one thread `r` of the warp computed
        const int r_hf = kPair ? (r >> 4) : 0;
        const int r_in_block = kPair ? quarter * 16 + (r & 15) : quarter * 32 + r;
        const int r_p = kPair ? r_hf * 64 + r_in_block : r_in_block;
        const int r_token = i_q[r_hf] * BS + r_in_block;
        const float4 val =
            *reinterpret_cast<const float4*>(smem + kOffP + b * kPBuf + r_p * 128 + ((ch ^ (r_p & 7)) << 4));
        if (r_token < p.tokens && (!kPair || r_hf == 0 || i_q[1] != i_q[0]))
          *reinterpret_cast<float4*>(out_bh + static_cast<long long>(r_token) * p.out_stride_n) = val;
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
