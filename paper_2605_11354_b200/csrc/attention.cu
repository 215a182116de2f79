// K4: critical-block softmax attention + linear branch + add (Algorithm 1's sparse branch, linear output, projection
// and sum) on tcgen05 / TMEM / TMA.
//
// One CTA owns 128 query rows of one (b, h): at block 64 a PAIR of query blocks (two M=64 problems interleaved in the
// two 16-lane halves of every TMEM sub-partition, each with its own list of critical key blocks), at block 128 one
// query block (M=128).  Work advances in steps of 64 keys.  Per step t (w = t & 1):
//   TMA      K tile(s) (e4m3, 64-byte rows, 64B swizzle) and V tile(s) (dequantised fp16, 128B swizzle) -> rings of four
//   tcgen05  S[w] = Q K^T          kind::f8f6f4, fp32 accumulators in TMEM (64 columns, two buffers)
//   softmax  warpgroup w, one thread per query row (TMEM lane = thread): the 64 scores are read once into registers,
//            row maximum, lazy rescale, exp2, row sum; the probabilities go back to TMEM as packed fp16 (P[w], 32 columns)
//   tcgen05  O += P[w] V           kind::f16 with the A operand read from TMEM, V as MN-major B operand from shared
//                                  memory, ONE fp32 accumulator in TMEM (64 columns) for all steps
// The two softmax warpgroups take the even and the odd steps.  Each owns a score buffer and a probability buffer, so
// Q K^T of step t+2 is issued as soon as warpgroup w has read S[w], and P V of step t runs under the exponentials of
// the following steps: the softmax threads do not wait for a product in the steady state, and with two CTAs per SM every
// SM sub-partition holds four softmax warps in different phases, which is what keeps the exponential unit fed.
// Both warpgroups accumulate into the same O, so they share one reference maximum per row: the thread that handles
// step t reads the reference left by step t-1 from a shared-memory slot (written early in that step, right after its
// row maximum is known), applies the lazy-rescale rule and publishes the reference of step t.  Row sums are kept
// per warpgroup, brought to the final reference and added in the epilogue.
// P is carried in fp16 (not e4m3): one e4m3 term has a 2.6 % rounding error per probability, which alone is ten
// times the output tolerance.  V travels as the dequantised value in fp16 (2^-12 relative rounding).
// Tail: phi(Q) (bf16) times the aggregated, projected summaries G_i (bf16) as one more MMA, divided by
// phi(Q) . zeta_i, added to the normalised softmax output and stored (each warpgroup handles 32 of the 64 columns).
//
// Warp roles (384 threads): warp 0 = TMA producer, warp 1 = Q K^T issuer, warp 2 = P V issuer (one thread each; all
// their waits block on mbarriers, nothing polls), warp 3 idle, warps 4-7 / 8-11 = softmax warpgroups 0 / 1.  The
// control warps give registers back (setmaxnreg) so that a softmax thread can hold a whole row of scores.
// Every wait is bounded (1 s); on expiry the CTA sets *device_status and all roles leave their loops.
#include <atomic>
#include <utility>

#include "common.cuh"
#include "sm100.cuh"

namespace lite3r {

namespace {

using namespace sm100;

constexpr int kStages = 4;   // K ring; also the number of P V completion barriers (step t uses number t % 4)
constexpr int kVStages = 3;  // V ring
constexpr int kSetThreads = 128;                 // one softmax warpgroup
constexpr int kSoftmaxThreads = 2 * kSetThreads;
constexpr int kCtrlWarps = 4;
constexpr int kThreads = kCtrlWarps * 32 + kSoftmaxThreads;
constexpr int kCtrlRegs = 32, kSoftmaxRegs = 104;  // 128 * 32 + 256 * 104 = 384 * 80, the launch allocation
constexpr uint32_t kBackoffNs = 64;  // sleep between polls of the single-thread roles
constexpr int kStepKeys = 64;
constexpr uint32_t kTmemCols = 256;
// TMEM columns: S buffers at 0 and 64, O at 128, P buffers (packed fp16, 32 columns each) at 192 and 224; the linear
// branch's product reuses S buffer 0.
constexpr uint32_t kColS = 0, kColO = 128, kColP = 192, kColL = 0;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kRescaleThreshold = 8.0f;  // lazy rescale: keep the old reference max until it is beaten by 2^8
constexpr float kNoMax = -1.0e30f;         // reference maximum of a row that has seen no valid key yet

// shared-memory map (bytes from a 1024-aligned base)
constexpr uint32_t kQBytes = 8192, kKStage = 8192, kVStage = 16384;
constexpr uint32_t kOffQ = 0;
constexpr uint32_t kOffK = kOffQ + kQBytes;
constexpr uint32_t kOffV = kOffK + kStages * kKStage;
constexpr uint32_t kOffPhi = kOffV + kVStages * kVStage;  // phi(Q) as bf16 A operand of the linear product (16 KB)
constexpr uint32_t kOffZeta = kOffPhi + 16384;            // zeta_i of the linear branch (256 B per query block)
constexpr uint32_t kOffRef = kOffZeta + 512;              // per row: {reference maximum, number of steps published}
constexpr uint32_t kOffX = kOffRef + 1024;                // epilogue exchange between the warpgroups (2 x 128 x 8 B)
constexpr uint32_t kOffScal = kOffX + 2048;               // per step and query block: {exponent factor, valid keys}, ring of 8
constexpr uint32_t kOffBar = kOffScal + 128;
constexpr uint32_t kSmemBytes = kOffBar + 512;  // two CTAs per SM: 2 * (110592 + 1024 reserved) <= 232448
// after the main loop the rings are reused: aggregated summaries G_i in K stages 0-1 (16 KB), the output rows in the
// V ring (32 KB)
constexpr uint32_t kOffG = kOffK;
constexpr uint32_t kOffOut = kOffV;

struct Bars {
  uint64_t q_full, z_full, g_full, phi_full, l_full, x_full;
  uint64_t k_full[kStages], v_full[kVStages];  // TMA -> issuer
  uint64_t k_free[kStages];                   // Q K^T of the step in this stage complete -> producer
  uint64_t pv_done[kStages];                  // P V of step t (number t % 4) complete -> producer, softmax
  uint64_t qk_done[2];                        // S buffer written -> softmax
  uint64_t s_empty[2], p_full[2];             // softmax -> issuer
  uint32_t tmem_base;
  int abort;
};

struct AttnParams {
  const float* q_scales;
  const float* k_scales;
  const int* crit_idx;  // [B*H*Nb][k_crit]
  const float* zeta;    // [B*H*Nb][64]
  void* out;
  long long out_stride_b, out_stride_h, out_stride_n;
  int heads, tokens, nb, k_crit, k_marg, phi, out_dtype;
  // output through TMA stores (map_o): position of the token / head / batch dimension among the map's dimensions
  // 1..3 (they are ordered by stride); tma_out = 0: plain stores
  int tma_out, dim_token, dim_head, dim_batch;
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
// D[tmem] (+)= A[tmem] * B[smem], kind::f16: the A operand (M x 16 halves per instruction = 8 columns of packed
// pairs, row = TMEM lane) is read from tensor memory.
__device__ __forceinline__ void mma_f16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                           uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}

// One aligned 8-byte word of shared memory, read / written by a single instruction that the compiler may neither
// drop nor reorder against other volatile accesses.
__device__ __forceinline__ uint2 lds_volatile_v2(uint32_t addr) {
  uint2 v;
  asm volatile("ld.volatile.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ void sts_volatile_v2(uint32_t addr, uint32_t x, uint32_t y) {
  asm volatile("st.volatile.shared.v2.u32 [%0], {%1, %2};" ::"r"(addr), "r"(x), "r"(y) : "memory");
}

// Polls a row's reference slot until `count` steps have been published (bounded like every other wait).
static __device__ __noinline__ bool reference_wait_slow(uint32_t slot, int count, uint2& v, volatile int* abort_flag, int* status) {
  const uint64_t t0 = global_timer_ns();
  uint32_t polls = 0;
  while (true) {
    v = lds_volatile_v2(slot);
    if (static_cast<int>(v.y) == count) return true;
    if ((++polls & 0x3Fu) == 0) {
      if (*abort_flag != 0) return false;
      if (global_timer_ns() - t0 > kWaitLimitNs) {
        *abort_flag = 309;
        if (status != nullptr) atomicCAS(status, 0, 309);
        return false;
      }
    }
  }
}
// Scales the 64 accumulator columns of this thread's TMEM lane by alpha (lazy rescale of O; rare).
static __device__ __noinline__ void rescale_accumulator(uint32_t o_addr, float alpha) {
#pragma unroll 1
  for (int part = 0; part < 4; ++part) {
    uint32_t o[16];
    tmem_ld16(o_addr + part * 16, o);
    tmem_wait_ld();
#pragma unroll
    for (int k = 0; k < 16; ++k) o[k] = __float_as_uint(__uint_as_float(o[k]) * alpha);
    tmem_st16(o_addr + part * 16, o);
  }
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
                 const __grid_constant__ CUtensorMap map_o, const AttnParams p) {
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
    mbar_init(&bars->z_full, 1);
    mbar_init(&bars->x_full, kSoftmaxThreads);
    mbar_init(&bars->g_full, 1);
    mbar_init(&bars->phi_full, kSoftmaxThreads);
    mbar_init(&bars->l_full, 1);
    for (int s = 0; s < kVStages; ++s) mbar_init(&bars->v_full[s], 1);
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&bars->k_full[s], 1);
      mbar_init(&bars->k_free[s], 1);
      mbar_init(&bars->pv_done[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&bars->qk_done[b], 1);
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
  if (threadIdx.x >= kCtrlWarps * 32 && threadIdx.x < kCtrlWarps * 32 + 128)
    reinterpret_cast<uint2*>(smem + kOffRef)[threadIdx.x - kCtrlWarps * 32] = make_uint2(__float_as_uint(kNoMax), 0u);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_base;
  // each branch below starts by giving registers back (control warps) or taking them (softmax warps)

  if (warp < kCtrlWarps) {
  setmaxnreg_dec<kCtrlRegs>();
  if (warp == 0) {
    // ------------------------------------------------------------------------------------------ TMA producer
    // All 32 lanes run the loops and the waits, so that control flow, step counters and addresses are the same in every
    // lane (the compiler can then keep them in the warp's uniform registers, which is where TMA and tcgen05
    // instructions take their operands from); one elected lane issues.
    {
      const bool leader = elect_one();
      if (leader) {
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
      }
      const float sq0 = __ldg(p.q_scales + bh_rows + i_q[0]) * (kLog2e * 0.125f);
      const float sq1 = __ldg(p.q_scales + bh_rows + i_q[1]) * (kLog2e * 0.125f);
      // Key blocks and their scales are fetched 32 steps at a time, lane l holding those of step 32 c + l, and handed
      // to the issuing lane by a shuffle: no global load (let alone two dependent ones) sits in the per-step path.
      int jl[2] = {0, 0};
      float sl[2] = {0.f, 0.f};
      auto refill = [&](int first) {
        const int tt = first + lane;
        if (tt < steps) {
          for (int hf = 0; hf < kHalves; ++hf) {
            jl[hf] = ldg_pinned(p.crit_idx + (bh_rows + i_q[hf]) * p.k_crit + (kPair ? tt : tt / 2));
            sl[hf] = ldg_pinned(p.k_scales + bh_rows + jl[hf]);
          }
        }
      };
      // tile row (in the code tensors) of a step in key block j
      auto tile_row = [&](int t, int j) {
        if (kPair) return static_cast<int>((bh_rows + j) * 64);
        return static_cast<int>((bh_rows + j) * 128 + (t & 1) * 64);
      };
      // The K cursor runs one step ahead of the V cursor (a K stage is free after the Q K^T of four steps earlier,
      // a V stage only after the P V of three steps earlier, and Q K^T of step t is issued before P V of step t-1).
      // The events the two cursors wait for alternate in time in exactly this order, so blocking waits lose nothing.
      // Together with the K tile of a step the producer leaves the step's scalars for the softmax threads: the
      // factor that turns a raw score into a base-2 exponent and the number of valid keys (ring of eight: the slot of
      // step t is rewritten for step t+8, when the softmax threads of step t+2 have long released the scores, which
      // they read after the scalars).
      bool ok = true;
      int sv = 0;              // V stage of the V cursor's step (tv % 3)
      int jv[2] = {0, 0};      // key blocks of the V cursor's step (those of the K cursor one iteration earlier)
      for (int i = 0; ok && i <= steps; ++i) {
        const int tk = i, tv = i - 1;
        int jk[2] = {0, 0};
        if (tk < steps) {
          if ((tk & 31) == 0) refill(tk);
          float sk[2];
          for (int hf = 0; hf < kHalves; ++hf) {
            jk[hf] = __shfl_sync(0xFFFFFFFFu, jl[hf], tk & 31);
            sk[hf] = __shfl_sync(0xFFFFFFFFu, sl[hf], tk & 31);
          }
          const int st = tk % kStages;
          if (tk >= kStages)
            ok = __all_sync(0xFFFFFFFFu, mbar_wait(&bars->k_free[st], ((tk - kStages) / kStages) & 1, abort_flag, p.status, 101, kBackoffNs));
          if (!ok) break;
          if (leader) {
            for (int hf = 0; hf < kHalves; ++hf) {
              int valid = p.tokens - jk[hf] * BS - (kPair ? 0 : (tk & 1) * kStepKeys);
              valid = max(0, min(kStepKeys, valid));
              sts_volatile_v2(smem_u32(smem + kOffScal) + (tk & 7) * 16 + hf * 8,
                              __float_as_uint((hf ? sq1 : sq0) * sk[hf]), static_cast<uint32_t>(valid));
            }
            mbar_arrive_expect_tx(&bars->k_full[st], kKTx);
            for (int hf = 0; hf < kHalves; ++hf)
              tma_load_2d(smem + kOffK + st * kKStage + hf * 4096, &map_k, &bars->k_full[st], 0, tile_row(tk, jk[hf]));
          }
        }
        if (tv >= 0) {
          // the stage of step tv held step tv - 3 before
          if (tv >= kVStages)
            ok = __all_sync(0xFFFFFFFFu, mbar_wait(&bars->pv_done[(tv - kVStages) % kStages], ((tv - kVStages) / kStages) & 1,
                                                   abort_flag, p.status, 102, kBackoffNs));
          if (!ok) break;
          if (leader) {
            mbar_arrive_expect_tx(&bars->v_full[sv], kVTx);
            for (int hf = 0; hf < kHalves; ++hf)
              tma_load_2d(smem + kOffV + sv * kVStage + hf * 8192, &map_v, &bars->v_full[sv], 0, tile_row(tv, jv[hf]));
          }
          if (++sv == kVStages) sv = 0;
        }
        for (int hf = 0; hf < kHalves; ++hf) jv[hf] = jk[hf];
      }
      if (ok && p.k_marg > 0) {
        // The aggregated summaries go to K stages 0 and 1, which are free once the last Q K^T products have
        // completed: well before the last P V products, so this load is off the tail's critical path.
        for (int u = max(0, steps - kStages); u < steps && ok; ++u)
          ok = __all_sync(0xFFFFFFFFu, mbar_wait(&bars->k_free[u % kStages], (u / kStages) & 1, abort_flag, p.status, 103, kBackoffNs));
        // G and zeta come from the kernel enqueued just before this one, which may still be running when this kernel
        // was launched to overlap with it: everything above reads older results only.
        wait_for_prior_grid();
        if (ok && leader) {
          mbar_arrive_expect_tx(&bars->z_full, kHalves * 256);
          for (int hf = 0; hf < kHalves; ++hf)
            bulk_load(smem + kOffZeta + hf * 256, p.zeta + (bh_rows + i_q[hf]) * kHeadDim, 256, &bars->z_full);
          mbar_arrive_expect_tx(&bars->g_full, kHalves * 8192);
          for (int hf = 0; hf < kHalves; ++hf)
            tma_load_2d(smem + kOffG + hf * 8192, &map_g, &bars->g_full, 0, static_cast<int>((bh_rows + i_q[hf]) * 64));
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------------------------------ Q K^T issuer
    // One thread issues a small tcgen05.mma about every 55 clocks and pays some 100 clocks per barrier it looks
    // at, so the two products of a step have an issuing warp each (this one and the next); a single issuer for
    // both was measured to be the bottleneck of the whole kernel.  Operand descriptors are built once and advanced by
    // adding byte offsets (in 16-byte units) to their address field.  As in the producer, all lanes run the loop
    // and one elected lane issues.
    {
      const bool leader = elect_one();
      constexpr uint32_t idesc_qk = instr_desc(0, kM, 64, 0, 0);   // e4m3 x e4m3, both K-major
      constexpr uint32_t idesc_lin = instr_desc(1, kM, 64, 0, 0);  // bf16 x bf16, both K-major
      const uint32_t q_addr = smem_u32(smem + kOffQ);
      const uint64_t k_desc0 = smem_desc(smem_u32(smem + kOffK), 16, 512, kSwizzle64);
      bool ok = __all_sync(0xFFFFFFFFu, mbar_wait(&bars->q_full, 0, abort_flag, p.status, 201, kBackoffNs));
      uint64_t q_desc[2][kHalves];
#pragma unroll
      for (int kk = 0; kk < 2; ++kk)
#pragma unroll
        for (int hf = 0; hf < kHalves; ++hf)
          q_desc[kk][hf] = smem_desc(q_addr + (kPair ? hf * 4096 : 0) + kk * 32, 16, 512, kSwizzle64);
      // S[t&1] = Q K(t)^T needs the K tile of step t and S[t&1] drained by the softmax threads of step t-2; it runs
      // one step ahead of the softmax threads, so the scores of step t are waiting when step t-1 is finished.
      for (int t = 0; ok && t < steps; ++t) {
        const int st = t % kStages;
        ok = mbar_wait(&bars->k_full[st], (t / kStages) & 1, abort_flag, p.status, 202, kBackoffNs);
        if (ok && t >= 2)
          ok = mbar_wait(&bars->s_empty[t & 1], ((t - 2) >> 1) & 1, abort_flag, p.status, 203, kBackoffNs);
        ok = __all_sync(0xFFFFFFFFu, ok);
        if (!ok) break;
        const uint32_t s_tmem = tmem + kColS + (t & 1) * 64;
        const uint64_t k_desc = k_desc0 + static_cast<uint64_t>((st * kKStage) >> 4);
        tc_fence_after();
        if (leader) {
#pragma unroll
          for (int kk = 0; kk < 2; ++kk) {
#pragma unroll
            for (int hf = 0; hf < kHalves; ++hf)
              mma_f8(s_tmem + ((hf * 16u) << 16), q_desc[kk][hf], k_desc + ((hf * 4096 + kk * 32) >> 4), idesc_qk, kk);
          }
          mma_commit(&bars->qk_done[t & 1]);
          mma_commit(&bars->k_free[st]);
        }
      }
      if (ok && p.k_marg > 0) {
        // the linear product lands in score buffer 0: the scores of the last even step must have been read (the loop
        // above has only waited for those of steps up to steps - 3)
        ok = mbar_wait(&bars->g_full, 0, abort_flag, p.status, 206, kBackoffNs) &&
             mbar_wait(&bars->phi_full, 0, abort_flag, p.status, 207, kBackoffNs);
        if (ok && steps > 0) {
          const int t_even = (steps - 1) & ~1;
          ok = mbar_wait(&bars->s_empty[0], (t_even >> 1) & 1, abort_flag, p.status, 208, kBackoffNs);
        }
        ok = __all_sync(0xFFFFFFFFu, ok);
        if (ok) {
          tc_fence_after();
          const uint32_t phi_addr = smem_u32(smem + kOffPhi), g_addr = smem_u32(smem + kOffG);
          if (leader) {
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
    }
  } else if (warp == 2) {
    // ------------------------------------------------------------------------------------------ P V issuer
    {
      const bool leader = elect_one();
      constexpr uint32_t idesc_pv = instr_desc(0, kM, 64, 0, 1);  // f16 x f16, P from TMEM, V MN-major
      const uint64_t v_desc0 = smem_desc(smem_u32(smem + kOffV), 8192, 1024, kSwizzle128);
      const uint32_t o_tmem = tmem + kColO;
      bool ok = true;
      int sv = 0;
      uint32_t v_par = 0;  // V stage of step t (t % 3) and the parity of its barrier ((t / 3) & 1)
      for (int t = 0; ok && t < steps; ++t) {  // O += P[t&1] V(t)
        ok = mbar_wait(&bars->v_full[sv], v_par, abort_flag, p.status, 205, kBackoffNs) &&
             mbar_wait(&bars->p_full[t & 1], (t >> 1) & 1, abort_flag, p.status, 204, kBackoffNs);
        ok = __all_sync(0xFFFFFFFFu, ok);
        if (!ok) break;
        const uint32_t p_tmem = tmem + kColP + (t & 1) * 32;
        const uint64_t v_desc = v_desc0 + static_cast<uint64_t>((sv * kVStage) >> 4);
        tc_fence_after();
        if (leader) {
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) {
#pragma unroll
            for (int hf = 0; hf < kHalves; ++hf)
              mma_f16_ts(o_tmem + ((hf * 16u) << 16), p_tmem + ((hf * 16u) << 16) + kk * 8,
                         v_desc + ((hf * 8192 + kk * 2048) >> 4), idesc_pv, (t > 0 || kk > 0) ? 1u : 0u);
          }
          mma_commit(&bars->pv_done[t % kStages]);
        }
        if (++sv == kVStages) {
          sv = 0;
          v_par ^= 1u;
        }
      }
    }
  }
  } else {
    // ------------------------------------------------------------------------------------------ softmax + epilogue
    setmaxnreg_inc<kSoftmaxRegs>();
    const int quarter = warp & 3;                       // TMEM sub-partition this warp may touch
    const int w = (warp - kCtrlWarps) >> 2;             // warpgroup: steps t with (t & 1) == w
    const int hf = kPair ? (lane >> 4) : 0;             // which query block of the pair this thread serves
    const int row_in_block = kPair ? quarter * 16 + (lane & 15) : quarter * 32 + lane;
    const int p_row = kPair ? hf * 64 + row_in_block : row_in_block;  // row inside the 128-row tile
    const int iq = i_q[hf];
    const size_t q_tile = bh_rows + iq;
    const uint32_t lane_addr = tmem + ((static_cast<uint32_t>(quarter) * 32u) << 16);
    const uint32_t s_addr = lane_addr + kColS + w * 64, p_addr = lane_addr + kColP + w * 32, o_addr = lane_addr + kColO;
    const float sq = __ldg(p.q_scales + q_tile);
    const uint32_t scal_slot = smem_u32(smem + kOffScal) + hf * 8;
    const uint32_t ref_slot = smem_u32(smem + kOffRef) + p_row * 8;

    float m_seen = kNoMax, l = 0.f;  // reference this warpgroup's row sum is relative to; the row sum
    bool ok = true;

    // Waits until `count` steps have published their reference for this row and returns it.  The slot is one aligned
    // 8-byte word written by a single store, so value and count are always seen together.
    auto reference_after = [&](int count, float& m) -> bool {
      uint2 v = lds_volatile_v2(ref_slot);
      if (static_cast<int>(v.y) != count && !reference_wait_slow(ref_slot, count, v, abort_flag, p.status)) return false;
      m = __uint_as_float(v.x);
      return true;
    };

    // linear branch, first part: this thread's 32 columns (warpgroup w -> columns 32 w ..) of phi(q) as bf16 A operand
    // of the linear product.  It needs the Q tile only, so it is computed while the first key tiles are on their way
    // and the softmax threads would be idle; the operand has a shared-memory region of its own and the linear product
    // can then be issued as soon as the aggregated summaries have arrived and the last scores have been read.  The
    // denominators phi(q) . zeta_i follow in the epilogue, from the operand's own rounded values.
    // The query row comes from the Q tile in shared memory (64-byte rows, 64B swizzle: 16-byte chunk c of row r sits at
    // chunk c ^ ((r >> 1) & 3)).
    // The loops over 16-column chunks here and in the epilogue are deliberately NOT unrolled: the kernel's code has to
    // stay within the instruction cache of an SM, which its fully unrolled form exceeded several times over (the
    // kernel was then bound by instruction fetch from the GPC-level cache, not by any arithmetic unit).
    float den = 0.f;
    const int swz = p_row & 7;
    if (p.k_marg > 0) {
      ok = mbar_wait_far(&bars->q_full, 0, abort_flag, p.status, 307);
      const uint8_t* qrow = smem + kOffQ + p_row * 64;
      const int qswz = (p_row >> 1) & 3;
      // phi = softmax over the components: any common shift of the exponents cancels in the ratio numerator /
      // denominator.  448 * scale bounds every component of the block, so it serves as the shift without a pass over
      // the row; only when exponents could then leave the fp32 range (block magnitudes in the hundreds) is the row's
      // own maximum looked up.
      const bool phi_softmax = p.phi == LITE3R_PHI_SOFTMAX;
      const float cq = sq * kLog2e;
      float shift = 448.f * cq;
      if (phi_softmax && 896.f * cq > 100.f) {
        float mxq[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll 1
        for (int c4 = 0; c4 < 4; ++c4) {  // row maximum over the 64 components
          const uint4 raw = *reinterpret_cast<const uint4*>(qrow + ((c4 ^ qswz) << 4));
          const uint32_t words[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
          for (int xw = 0; xw < 4; ++xw) {
            float fv[4];
            e4m3x4_to_float(words[xw], fv);
#pragma unroll
            for (int y = 0; y < 4; ++y) mxq[y] = fmaxf(mxq[y], fv[y]);
          }
        }
        shift = fmaxf(fmaxf(mxq[0], mxq[1]), fmaxf(mxq[2], mxq[3])) * cq;  // sq > 0 commutes with max
      }
      uint8_t* const phirow = smem + kOffPhi + p_row * 128;
#pragma unroll 1
      for (int cc = 0; cc < 2; ++cc) {  // this warpgroup's two chunks of 16 components
        const int c4 = 2 * w + cc;
        const uint4 raw = *reinterpret_cast<const uint4*>(qrow + ((c4 ^ qswz) << 4));
        const uint32_t words[4] = {raw.x, raw.y, raw.z, raw.w};
        uint32_t pk8[8];
#pragma unroll
        for (int xw = 0; xw < 4; ++xw) {
          float fv[4];
          e4m3x4_to_float(words[xw], fv);
#pragma unroll
          for (int y = 0; y < 4; y += 2) {
            float e0, e1;
            if (phi_softmax) {  // the softmax normaliser cancels in the ratio
              e0 = ex2(fmaf(fv[y], cq, -shift));
              e1 = ex2(fmaf(fv[y + 1], cq, -shift));
            } else {
              e0 = fv[y] > 0.f ? fmaf(fv[y], sq, 1.f) : ex2(fv[y] * cq);
              e1 = fv[y + 1] > 0.f ? fmaf(fv[y + 1], sq, 1.f) : ex2(fv[y + 1] * cq);
            }
            pk8[xw * 2 + (y >> 1)] = pack_bf162(e0, e1);
          }
        }
        *reinterpret_cast<uint4*>(phirow + (((c4 * 2) ^ swz) << 4)) = make_uint4(pk8[0], pk8[1], pk8[2], pk8[3]);
        *reinterpret_cast<uint4*>(phirow + (((c4 * 2 + 1) ^ swz) << 4)) = make_uint4(pk8[4], pk8[5], pk8[6], pk8[7]);
      }
      fence_proxy_async_smem();
      mbar_arrive(&bars->phi_full);
    }


    // barrier of the P V product two steps back (the one that frees P[w]): its stage alternates between w and w + 2,
    // its parity flips every second iteration; both are carried along instead of being recomputed from t
    uint64_t* const pv_bar0 = &bars->pv_done[w];
    uint32_t pv_off = 0, pv_par = 0, pv_flip = 0, qk_par = 0;

    for (int t = w; t < steps; t += 2) {
      if (!(ok = mbar_wait_far(&bars->qk_done[w], qk_par, abort_flag, p.status, 301))) break;
      qk_par ^= 1u;
      tc_fence_after();
      // the step's scalars, left by the producer before it requested the K tile
      const uint2 scal = lds_volatile_v2(scal_slot + (t & 7) * 16);
      const float c = __uint_as_float(scal.x);
      const int valid = static_cast<int>(scal.y);
      uint32_t xa[32], xb[32];
      float mx4[4];
      {
        tmem_ld32(s_addr, xa);
        tmem_ld32(s_addr + 32, xb);
        tmem_wait_ld();
        // the whole row of scores is in registers: the issuer may overwrite S[w] with step t+2 right away
        tc_fence_before();
        mbar_arrive(&bars->s_empty[w]);
        if (valid < kStepKeys) {
#pragma unroll
          for (int k = 0; k < 32; ++k) {
            if (k >= valid) xa[k] = 0xFF800000u;  // -inf
            if (32 + k >= valid) xb[k] = 0xFF800000u;
          }
        }
        // row maximum of the raw scores (c > 0 commutes with max), four independent chains
#pragma unroll
        for (int q = 0; q < 4; ++q) mx4[q] = fmaxf(__uint_as_float(xa[q]), __uint_as_float(xb[q]));
#pragma unroll
        for (int k = 4; k < 32; k += 4) {
#pragma unroll
          for (int q = 0; q < 4; ++q) mx4[q] = max3(mx4[q], __uint_as_float(xa[k + q]), __uint_as_float(xb[k + q]));
        }
      }
      // a step without any valid key (second half of a short last block) leaves the reference where it is
      const float tile_max = fmaxf(max3(fmaxf(mx4[0], mx4[1]), mx4[2], mx4[3]) * c, kNoMax);

      // the row's reference after step t-1 (published early in that step by the other warpgroup), the lazy-rescale
      // decision of this step, and its publication for step t+1
      float m_ref = kNoMax;
      if (t > 0 && !(ok = reference_after(t, m_ref))) break;
      if (m_ref != m_seen) l *= ex2(m_seen - m_ref);  // bring this warpgroup's row sum to the current reference
      bool need = false;
      float alpha = 1.f;
      if (t == 0) {
        m_ref = tile_max;
      } else if (tile_max > m_ref + kRescaleThreshold) {
        need = true;
        alpha = ex2(m_ref - tile_max);
        m_ref = tile_max;
        l *= alpha;
      }
      m_seen = m_ref;
      sts_volatile_v2(ref_slot, __float_as_uint(m_ref), static_cast<uint32_t>(t + 1));

      // P[w] is free once the P V product of step t-2 has completed (long ago in the steady state)
      if (t >= 2) {
        if (!(ok = mbar_wait_far(pv_bar0 + pv_off, pv_par, abort_flag, p.status, 302))) break;
        pv_off ^= 2u;
        pv_par ^= pv_flip;
        pv_flip ^= 1u;
      }
      tc_fence_after();
      {
        // the second half of the row is read again instead of being held across the first half's exponentials;
        // S[w] is released once it is in registers
        uint32_t packed[16];
        l += exp_half_row(xa, c, -m_ref, packed);
        tmem_st16(p_addr, packed);
        l += exp_half_row(xb, c, -m_ref, packed);
        tmem_st16(p_addr + 16, packed);
      }
      if (__any_sync(0xFFFFFFFFu, need)) {
        // O is being accumulated into by the P V product of step t-1: wait for it, then scale the rows whose
        // reference moved.  The product of this step waits for this thread's arrival below.
        if (!(ok = mbar_wait_far(&bars->pv_done[(t - 1) % kStages], ((t - 1) / kStages) & 1, abort_flag, p.status, 303))) break;
        tc_fence_after();
        rescale_accumulator(o_addr, alpha);
      }
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(&bars->p_full[w]);
    }

    // linear branch, second part: partial denominator phi(q) . zeta_i over this thread's 32 columns, with the same
    // rounded values as the numerator's operand (read back from shared memory); zeta_i arrives with the aggregated
    // summaries at the end of the producer's work
    if (ok && p.k_marg > 0) {
      ok = mbar_wait_far(&bars->z_full, 0, abort_flag, p.status, 308);
      const uint8_t* const phirow = smem + kOffPhi + p_row * 128;
      float den4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 1
      for (int ch = 0; ch < 4; ++ch) {  // 16-byte chunks of eight components
        const int c8 = 4 * w + ch;
        const uint4 raw = *reinterpret_cast<const uint4*>(phirow + ((c8 ^ swz) << 4));
        const uint32_t words[4] = {raw.x, raw.y, raw.z, raw.w};
        const float4* zeta = reinterpret_cast<const float4*>(smem + kOffZeta + hf * 256 + c8 * 32);
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          const float4 z = zeta[half];
          den4[0] = fmaf(__uint_as_float(words[2 * half] << 16), z.x, den4[0]);
          den4[1] = fmaf(__uint_as_float(words[2 * half] & 0xFFFF0000u), z.y, den4[1]);
          den4[2] = fmaf(__uint_as_float(words[2 * half + 1] << 16), z.z, den4[2]);
          den4[3] = fmaf(__uint_as_float(words[2 * half + 1] & 0xFFFF0000u), z.w, den4[3]);
        }
      }
      den = (den4[0] + den4[1]) + (den4[2] + den4[3]);
    }

    // the two threads of a row (one per warpgroup) bring their row sums to the final reference and swap them together
    // with the partial denominators
    float inv_l = 0.f;
    if (ok) {
      float m_fin = kNoMax;
      if (steps > 0) ok = reference_after(steps, m_fin);
      if (ok) {
        if (m_fin != m_seen) l *= ex2(m_seen - m_fin);
        float2* xbuf = reinterpret_cast<float2*>(smem + kOffX);
        xbuf[w * 128 + p_row] = make_float2(l, den);
        mbar_arrive(&bars->x_full);
        ok = mbar_wait_far(&bars->x_full, 0, abort_flag, p.status, 306);
        if (ok) {
          const float2 other = xbuf[(w ^ 1) * 128 + p_row];
          inv_l = steps > 0 ? 1.f / (l + other.x) : 0.f;
          den += other.y;
        }
      }
    }
    // the last P V product (commits are cumulative: it covers every earlier one), then the linear product
    if (ok && steps > 0)
      ok = mbar_wait_far(&bars->pv_done[(steps - 1) % kStages], ((steps - 1) / kStages) & 1, abort_flag, p.status, 304);
    if (ok && p.k_marg > 0) ok = mbar_wait_far(&bars->l_full, 0, abort_flag, p.status, 305);
    tc_fence_after();

    ok = __all_sync(0xFFFFFFFFu, ok);  // the store below synchronises the warp
    if (ok) {
      const int bb = bh / p.heads, h = bh % p.heads;
      const float l_scale = p.k_marg > 0 ? 1.f / den : 0.f;
      // The thread's 32 output values go to the V ring (free: every P V product has completed), 16-byte chunks
      // swizzled by the row so that neither these writes nor the row-wise reads below conflict; then each store
      // instruction of the warp writes whole half rows (fp32: four rows x 128 bytes, 16-bit: eight rows x 64 bytes).
      const bool wide = p.out_dtype == LITE3R_F32;
      const bool to_bf16 = p.out_dtype == LITE3R_BF16;
      const uint32_t row_bytes = wide ? 256u : 128u;
      // With TMA stores every warp stages its 32 half rows in a tile of its own (row = lane, 128 bytes with the 128B
      // swizzle for fp32, 64 bytes with the 64B swizzle for the 16-bit types), which is the layout the store engine
      // reads; otherwise whole rows of the 128-row tile, chunks swizzled by the row.
      const bool tma_out = p.tma_out != 0;
      const uint32_t half_bytes = wide ? 128u : 64u;
      uint8_t* const warp_tile = smem + kOffOut + (warp - kCtrlWarps) * 4096;
      const int tswz = wide ? (lane & 7) : ((lane >> 1) & 3);
      uint8_t* const orow = tma_out ? warp_tile + lane * half_bytes : smem + kOffOut + p_row * row_bytes;
#pragma unroll 1
      for (int cc = 0; cc < 2; ++cc) {  // 16 columns at a time
        float acc[16];
        uint32_t v[16];
        if (steps > 0) {
          tmem_ld16(o_addr + w * 32 + cc * 16, v);
          tmem_wait_ld();
#pragma unroll
          for (int k = 0; k < 16; ++k) acc[k] = __uint_as_float(v[k]) * inv_l;
        } else {
#pragma unroll
          for (int k = 0; k < 16; ++k) acc[k] = 0.f;
        }
        if (p.k_marg > 0) {
          tmem_ld16(lane_addr + kColL + w * 32 + cc * 16, v);
          tmem_wait_ld();
#pragma unroll
          for (int k = 0; k < 16; ++k) acc[k] = fmaf(__uint_as_float(v[k]), l_scale, acc[k]);
        }
        if (wide) {
#pragma unroll
          for (int ch = 0; ch < 4; ++ch)
            *reinterpret_cast<float4*>(orow + ((tma_out ? ((cc * 4 + ch) ^ tswz) : ((w * 8 + cc * 4 + ch) ^ swz)) << 4)) =
                make_float4(acc[4 * ch], acc[4 * ch + 1], acc[4 * ch + 2], acc[4 * ch + 3]);
        } else {
#pragma unroll
          for (int ch = 0; ch < 2; ++ch) {
            uint32_t pk[4];
#pragma unroll
            for (int y = 0; y < 4; ++y)
              pk[y] = to_bf16 ? pack_bf162(acc[8 * ch + 2 * y], acc[8 * ch + 2 * y + 1])
                              : pack_half2(acc[8 * ch + 2 * y], acc[8 * ch + 2 * y + 1]);
            *reinterpret_cast<uint4*>(orow + ((tma_out ? ((cc * 2 + ch) ^ tswz) : ((w * 4 + cc * 2 + ch) ^ swz)) << 4)) =
                make_uint4(pk[0], pk[1], pk[2], pk[3]);
          }
        }
      }
      if (tma_out) {
        // two boxes of 16 rows x 32 columns per warp: lanes 0-15 and 16-31 hold 16 consecutive tokens each (of the two
        // query blocks of a pair, or of the two halves of the warp's 32 rows); rows past the end of the sequence are
        // clipped by the store engine, the copy of the last block in an odd pair is not stored at all
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
#pragma unroll
          for (int g2 = 0; g2 < 2; ++g2) {
            const int token0 = kPair ? i_q[g2] * BS + quarter * 16 : i_q[0] * BS + quarter * 32 + 16 * g2;
            if (token0 >= p.tokens || (kPair && g2 == 1 && i_q[1] == i_q[0])) continue;
            int c[4] = {w * 32, 0, 0, 0};
            c[p.dim_token] = token0;
            c[p.dim_head] = h;
            c[p.dim_batch] = bb;
            tma_store_4d(&map_o, warp_tile + g2 * 16 * half_bytes, c[0], c[1], c[2], c[3]);
          }
          bulk_commit_group();
          bulk_wait_group_read0();  // the tile must stay in place until the engine has read it
        }
        __syncwarp();
      } else {
      __syncwarp();
      const int chunk_shift = wide ? 3 : 2;       // 8 or 4 chunks of 16 bytes per half row
      const int ch = lane & ((1 << chunk_shift) - 1);
      const int half_chunks = 1 << chunk_shift;
      const int rows_per_pass = 32 >> chunk_shift;  // 4 or 8
      const uint32_t elem = wide ? 4u : 2u;
      uint8_t* const out_bh = static_cast<uint8_t*>(p.out) +
                              (static_cast<long long>(bb) * p.out_stride_b + static_cast<long long>(h) * p.out_stride_h) * elem +
                              w * 32 * elem + ch * 16;
      const long long row_pitch = p.out_stride_n * static_cast<long long>(elem);
      const bool second_block_is_copy = kPair && i_q[1] == i_q[0];
#pragma unroll 1
      for (int r = lane >> chunk_shift; r < 32; r += rows_per_pass) {  // row of this warp's block: thread r computed it
        const int r_hf = kPair ? (r >> 4) : 0;
        const int r_in_block = kPair ? quarter * 16 + (r & 15) : quarter * 32 + r;
        const int r_p = kPair ? r_hf * 64 + r_in_block : r_in_block;
        const int r_token = i_q[r_hf] * BS + r_in_block;
        const uint4 val = *reinterpret_cast<const uint4*>(smem + kOffOut + r_p * row_bytes +
                                                          (((w * half_chunks + ch) ^ (r_p & 7)) << 4));
        if (r_token < p.tokens && !(second_block_is_copy && r_hf == 1))
          *reinterpret_cast<uint4*>(out_bh + r_token * row_pitch) = val;
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
// Test hook: non-zero makes the kernel write its output with plain stores even where a TMA map exists.
std::atomic<int> g_plain_stores{0};

template <int BS>
lite3r_status launch(const AttentionLaunch& a, cudaStream_t stream) {
  const lite3r_shape& s = a.shape;
  const int nb = ceil_div(s.tokens, BS);
  const uint64_t tiles = static_cast<uint64_t>(s.batch) * s.heads * nb;
  // The four tensor maps depend on the buffers and the shape only; a caller that runs the same buffers again (the
  // usual serving loop) reuses the encoded maps of its previous call (one entry per calling thread).
  struct MapCache {
    alignas(64) CUtensorMap q, k, v, g, o;
    const void* key[4] = {nullptr, nullptr, nullptr, nullptr};
    uint64_t tiles = 0;
    int block = 0;
    // the output map
    const void* out = nullptr;
    long long out_strides[3] = {0, 0, 0};
    int out_dims[3] = {0, 0, 0}, out_dtype = -1, out_ok = 0, dim_token = 1, dim_head = 2, dim_batch = 3;
  };
  thread_local MapCache cache;
  lite3r_status st;
  if (cache.key[0] != a.q_codes || cache.key[1] != a.k_codes || cache.key[2] != a.v16 || cache.key[3] != a.g16 ||
      cache.tiles != tiles || cache.block != BS) {
    cache.key[0] = nullptr;  // stays invalid if an encode below fails
    if ((st = make_tensor_map_2d(&cache.q, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, a.q_codes, 64, tiles * BS, 64, 64, CU_TENSOR_MAP_SWIZZLE_64B)) != LITE3R_OK) return st;
    if ((st = make_tensor_map_2d(&cache.k, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, a.k_codes, 64, tiles * BS, 64, 64, CU_TENSOR_MAP_SWIZZLE_64B)) != LITE3R_OK) return st;
    if ((st = make_tensor_map_2d(&cache.v, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, a.v16, 64, tiles * BS, 64, 64, CU_TENSOR_MAP_SWIZZLE_128B)) != LITE3R_OK) return st;
    if ((st = make_tensor_map_2d(&cache.g, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, a.g16, 64, tiles * 64, 64, 64, CU_TENSOR_MAP_SWIZZLE_128B)) != LITE3R_OK) return st;
    cache.key[0] = a.q_codes;
    cache.key[1] = a.k_codes;
    cache.key[2] = a.v16;
    cache.key[3] = a.g16;
    cache.tiles = tiles;
    cache.block = BS;
  }
  // The output goes through TMA stores when a tiled map can describe it: the token, head and batch dimensions ordered
  // by stride (dimensions of extent 1 last), 16 tokens x 32 columns per box.  If the driver refuses the map the kernel
  // falls back to plain stores.
  if (cache.out != a.out || cache.out_dtype != a.out_dtype || cache.out_strides[0] != a.out_stride_n ||
      cache.out_strides[1] != a.out_stride_h || cache.out_strides[2] != a.out_stride_b || cache.out_dims[0] != s.tokens ||
      cache.out_dims[1] != s.heads || cache.out_dims[2] != s.batch) {
    const int elem = a.out_dtype == LITE3R_F32 ? 4 : 2;
    struct Dim {
      long long stride;
      int extent, which;  // which: 0 token, 1 head, 2 batch
    } dm[3] = {{a.out_stride_n, s.tokens, 0}, {a.out_stride_h, s.heads, 1}, {a.out_stride_b, s.batch, 2}};
    // order: extents above 1 by ascending stride, then the extent-1 dimensions (whose stride does not matter)
    auto before = [](const Dim& x, const Dim& y) {
      if ((x.extent > 1) != (y.extent > 1)) return x.extent > 1;
      if (x.extent > 1 && x.stride != y.stride) return x.stride < y.stride;
      return x.which < y.which;
    };
    for (int i = 0; i < 3; ++i)
      for (int j = i + 1; j < 3; ++j)
        if (before(dm[j], dm[i])) std::swap(dm[i], dm[j]);
    uint64_t dims[4] = {kHeadDim, 0, 0, 0}, strides[3];
    uint32_t box[4] = {32, 1, 1, 1};
    uint64_t packed = static_cast<uint64_t>(kHeadDim) * elem;  // stride a dimension would have if packed after the previous ones
    bool ok = (reinterpret_cast<uintptr_t>(a.out) & 15u) == 0;
    for (int i = 0; i < 3; ++i) {
      dims[i + 1] = static_cast<uint64_t>(dm[i].extent);
      strides[i] = dm[i].extent > 1 ? static_cast<uint64_t>(dm[i].stride) * elem : packed;
      ok = ok && strides[i] > 0 && (strides[i] & 15u) == 0;
      packed = strides[i] * dims[i + 1];
      if (dm[i].which == 0) {
        box[i + 1] = 16;
        cache.dim_token = i + 1;
      } else if (dm[i].which == 1) {
        cache.dim_head = i + 1;
      } else {
        cache.dim_batch = i + 1;
      }
    }
    cache.out_ok = 0;
    if (ok) {
      const CUtensorMapDataType type = a.out_dtype == LITE3R_F32    ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32
                                       : a.out_dtype == LITE3R_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16
                                                                    : CU_TENSOR_MAP_DATA_TYPE_FLOAT16;
      const CUtensorMapSwizzle swz = a.out_dtype == LITE3R_F32 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B;
      cache.out_ok = make_tensor_map_4d(&cache.o, type, a.out, dims, strides, box, swz) == LITE3R_OK ? 1 : 0;
    }
    cache.out = a.out;
    cache.out_dtype = a.out_dtype;
    cache.out_strides[0] = a.out_stride_n;
    cache.out_strides[1] = a.out_stride_h;
    cache.out_strides[2] = a.out_stride_b;
    cache.out_dims[0] = s.tokens;
    cache.out_dims[1] = s.heads;
    cache.out_dims[2] = s.batch;
  }
  const CUtensorMap &map_q = cache.q, &map_k = cache.k, &map_v = cache.v, &map_g = cache.g;
  const bool tma_out = cache.out_ok != 0 && g_plain_stores.load(std::memory_order_relaxed) == 0;
  const CUtensorMap& map_o = tma_out ? cache.o : cache.q;  // any valid map when it is not used
  AttnParams p;
  p.tma_out = tma_out ? 1 : 0;
  p.dim_token = cache.dim_token;
  p.dim_head = cache.dim_head;
  p.dim_batch = cache.dim_batch;
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
  p.out_dtype = a.out_dtype;
  p.status = a.device_status;
  st = ensure_dynamic_smem(attention_kernel<BS>, static_cast<int>(kSmemBytes));
  if (st != LITE3R_OK) return st;
  const int ctas = s.batch * s.heads * (BS == 64 ? (nb + 1) / 2 : nb);
  if (a.overlap_prior) {
    // programmatic dependent launch: the kernel may start while the preceding one (which announces it early) is
    // still running, and waits for its completion itself before it reads that kernel's results
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(ctas));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t err = cudaLaunchKernelEx(&cfg, attention_kernel<BS>, map_q, map_k, map_v, map_g, map_o, p);
    if (err != cudaSuccess) return record_cuda(err);
    return after_launch();
  }
  attention_kernel<BS><<<ctas, kThreads, kSmemBytes, stream>>>(map_q, map_k, map_v, map_g, map_o, p);
  return after_launch();
}

}  // namespace

void set_attention_plain_stores(int on) { g_plain_stores.store(on, std::memory_order_relaxed); }

lite3r_status launch_attention(const AttentionLaunch& a, cudaStream_t stream) {
  return a.shape.block == 64 ? launch<64>(a, stream) : launch<128>(a, stream);
}

}  // namespace lite3r
