// K2: pooled scores and row-wise top-k block classification (Algorithm 1 lines 2-3 on block means).
//
// The pooled mean of block i is colsum_i * 2^-9 * scale_i / valid_i with colsum an exact integer vector, so
//   s_ij = (colsum^Q_i . colsum^K_j) * [scale^K_j / valid_j] * [scale^Q_i / (valid_i * 8 * 2^18)].
// The last bracket is a positive constant of row i and cannot change the ranking inside the row, so the
// kernel ranks t_ij = (integer dot product, exact in fp64 below 2^53) * scale^K_j / valid_j.  Two fp64
// roundings separate t_ij from the exact value; the ranking is therefore the exact one except between
// scores that agree to ~1e-15 relative.  Ranking order: score descending, then key-block index ascending.
//
// One CTA of R warps handles R consecutive query blocks (rows) of one (b, h).
//   Phase A (whole CTA): the scores of the R rows against all key blocks, 64 staged key blocks at a time; a lane
//     owns one key block and R/4 rows, so every staged value feeds several fp64 FMAs.  Scores are kept in shared
//     memory as order-preserving 64-bit keys.
//   Phase B (one warp per row): "the k best of the row" is found by a most-significant-digit-first radix select
//     over the 64-bit keys (8-bit digits placed at the highest bit on which the remaining candidates differ,
//     per-warp histogram in shared memory): it yields a key prefix such that
//     every entry above it is selected, and of the entries equal to it the first `take` in index order are.  That
//     is exactly the total order (score descending, index ascending), at O(Nb) work per row.  Two selections
//     give the classes: the best k_crit are critical, the best Nb - k_neg are critical-or-marginal.
//   Phase C (same warp): class row and ascending index lists, written with ballot prefix sums.
#include "common.cuh"

namespace lite3r {

namespace {

constexpr int kChunk = 64;          // key blocks staged per pass (upper bound; the used part is keys_per_warp * R)
constexpr int kPitch = kHeadDim + 4;  // staged row pitch in doubles: 16-byte aligned rows; 8-byte reads of four consecutive
                                      // values from four (eight) rows and 16-byte reads of eight rows fall on different banks

// Maps a double to an unsigned key with the same order (larger double -> larger key).
__device__ __forceinline__ unsigned long long order_key(double v) {
  const unsigned long long u = static_cast<unsigned long long>(__double_as_longlong(v));
  return (u >> 63) ? ~u : (u | 0x8000000000000000ull);
}

struct Selection {
  unsigned long long prefix, mask;  // (key & mask) > prefix: selected; == prefix: the first `take` by index are
  int take;
};

// The k best (largest key, then lowest index) of keys[0..n): warp-collective, hist is this warp's 256 counters.
__device__ Selection select_top(const unsigned long long* keys, int n, int k, unsigned int* hist, int lane) {
  Selection s;
  if (k <= 0) {  // nothing selected: no masked key exceeds or equals the all-ones prefix with take 0
    s.prefix = ~0ull;
    s.mask = ~0ull;
    s.take = 0;
    return s;
  }
  if (k >= n) {  // everything selected
    s.prefix = 0ull;
    s.mask = 0ull;
    s.take = n;
    return s;
  }
  unsigned long long prefix = 0ull, mask = 0ull;
  int remaining = k;
  while (true) {
    // Bits on which the candidates (keys matching the prefix so far) still differ: scores of one row share their
    // sign and leading exponent bits, so fixed digit positions would spend whole passes (and 32-way histogram
    // conflicts) on digits that are equal for everyone.  Each pass starts at the highest differing bit instead.
    unsigned long long all_and = ~0ull, all_or = 0ull;
    for (int j = lane; j < n; j += 32) {
      const unsigned long long key = keys[j];
      if ((key & mask) == prefix) {
        all_and &= key;
        all_or |= key;
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      all_and &= __shfl_xor_sync(0xFFFFFFFFu, all_and, o);
      all_or |= __shfl_xor_sync(0xFFFFFFFFu, all_or, o);
    }
    const unsigned long long diff = all_and ^ all_or;
    if (diff == 0ull) {  // all candidates are equal: the first `remaining` of them by index are selected
      prefix = all_and;
      mask = ~0ull;
      break;
    }
    const int hb = 63 - __clzll(static_cast<long long>(diff));      // highest differing bit
    const int shift = hb >= 7 ? hb - 7 : 0;                          // digit = bits shift .. shift+7
    const unsigned long long above_hb = hb == 63 ? 0ull : ~((2ull << hb) - 1ull);
    prefix |= all_and & above_hb & ~mask;                            // the common leading bits join the prefix
    mask |= above_hb;
#pragma unroll
    for (int b = 0; b < 8; ++b) hist[lane + 32 * b] = 0u;
    __syncwarp();
    for (int j = lane; j < n; j += 32) {
      const unsigned long long key = keys[j];
      if ((key & mask) == prefix) atomicAdd(&hist[static_cast<unsigned int>(key >> shift) & 255u], 1u);
    }
    __syncwarp();
    // lane L owns the digits 255-8L .. 248-8L, visited in descending order
    int cnt[8], tot = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      cnt[i] = static_cast<int>(hist[255 - 8 * lane - i]);
      tot += cnt[i];
    }
    int incl = tot;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
      if (lane >= o) incl += up;
    }
    const int excl = incl - tot;
    const bool mine = excl < remaining && remaining <= incl;
    int digit = 0, above = 0, bin = 0;
    if (mine) {
      int run = excl;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        if (bin == 0 && run + cnt[i] >= remaining) {
          digit = 255 - 8 * lane - i;
          above = run;
          bin = cnt[i];
        }
        run += cnt[i];
      }
    }
    const int src = __ffs(__ballot_sync(0xFFFFFFFFu, mine)) - 1;
    digit = __shfl_sync(0xFFFFFFFFu, digit, src);
    above = __shfl_sync(0xFFFFFFFFu, above, src);
    bin = __shfl_sync(0xFFFFFFFFu, bin, src);
    remaining -= above;
    const unsigned long long field = 0xFFull << shift;
    prefix = (prefix & ~field) | (static_cast<unsigned long long>(digit) << shift);
    mask |= field;
    __syncwarp();
    if (bin == remaining || shift == 0) break;  // the whole bin is selected, or every bit has been decided
  }
  s.prefix = prefix;
  s.mask = mask;
  s.take = remaining;
  return s;
}

template <int R>
__global__ void __launch_bounds__(R * 32) plan_kernel(const int* __restrict__ q_colsum, const int* __restrict__ k_colsum,
                                                       const float* __restrict__ k_scales, int tokens, int block,
                                                       int nb, int k_crit, int k_marg, int k_neg,
                                                       signed char* __restrict__ cls, int* __restrict__ crit_idx,
                                                       int* __restrict__ marg_idx) {
  constexpr int kThreads = R * 32;
  constexpr int kGroups = R >= 4 ? 4 : R;        // row groups inside a warp
  constexpr int kRowsPerLane = R / kGroups;       // rows whose score one lane accumulates
  constexpr int kKeysPerWarp = 32 / kGroups;
  constexpr int kStep = kKeysPerWarp * R;         // key blocks per staged pass (<= kChunk)
  static_assert(kStep <= kChunk, "staging buffer too small");

  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int pitch = (nb + 1) & ~1;  // key-row pitch: keeps everything behind the keys 16-byte aligned
  unsigned long long* s_key = reinterpret_cast<unsigned long long*>(smem_raw);        // [R][pitch]
  double* s_q = reinterpret_cast<double*>(s_key + static_cast<size_t>(R) * pitch);    // [R][kPitch]
  double* s_k = s_q + R * kPitch;                                                     // [kChunk][kPitch]
  unsigned int* s_hist = reinterpret_cast<unsigned int*>(s_k + kChunk * kPitch);      // [R][256]

  const int row_tiles = (nb + R - 1) / R;
  const int bh = blockIdx.x / row_tiles;
  const int i0 = (blockIdx.x % row_tiles) * R;
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const size_t bh_rows = static_cast<size_t>(bh) * nb;

  for (int t = threadIdx.x; t < R * kHeadDim; t += kThreads) {
    const int r = t / kHeadDim, d = t % kHeadDim;
    s_q[r * kPitch + d] = (i0 + r < nb) ? static_cast<double>(q_colsum[(bh_rows + i0 + r) * kHeadDim + d]) : 0.0;
  }

  // Phase A.  The column sums of the next kStep key blocks are fetched (16-byte loads) into registers before the
  // current ones are multiplied, so their latency hides behind the fp64 work; both staged arrays use a row pitch
  // of 66 doubles, which keeps the 16-byte reads of the eight key rows and of the four row groups of a warp on
  // different banks.
  constexpr int kLoads = kStep * (kHeadDim / 4) / kThreads;  // int4 loads per thread and pass
  const int kl = lane % kKeysPerWarp, rg = lane / kKeysPerWarp;
  const int jj = warp * kKeysPerWarp + kl;
  int4 pre[kLoads];
  auto prefetch = [&](int j0) {
    const int4* src = reinterpret_cast<const int4*>(k_colsum + (bh_rows + j0) * kHeadDim);
    const int n4 = min(kStep, nb - j0) * (kHeadDim / 4);
#pragma unroll
    for (int q = 0; q < kLoads; ++q) {
      const int v = threadIdx.x + q * kThreads;
      pre[q] = v < n4 ? __ldg(src + v) : make_int4(0, 0, 0, 0);
    }
  };
  prefetch(0);
  double q_frag[R == 8 ? kHeadDim / 4 : 1] = {};
  if constexpr (R == 8) {
    __syncthreads();  // s_q is complete
#pragma unroll
    for (int st = 0; st < kHeadDim / 4; ++st) q_frag[st] = s_q[(lane >> 2) * kPitch + 4 * st + (lane & 3)];
  }
  for (int j0 = 0; j0 < nb; j0 += kStep) {
    __syncthreads();
    const int nj = min(kStep, nb - j0);
#pragma unroll
    for (int q = 0; q < kLoads; ++q) {
      const int v = threadIdx.x + q * kThreads;
      double* dst = s_k + (v / (kHeadDim / 4)) * kPitch + (v % (kHeadDim / 4)) * 4;
      *reinterpret_cast<double2*>(dst) = make_double2(static_cast<double>(pre[q].x), static_cast<double>(pre[q].y));
      *reinterpret_cast<double2*>(dst + 2) = make_double2(static_cast<double>(pre[q].z), static_cast<double>(pre[q].w));
    }
    if (j0 + kStep < nb) prefetch(j0 + kStep);
    __syncthreads();
    if constexpr (R == 8) {
      // 8 rows x 8 key blocks per warp as an fp64 tensor-core product (m8n8k4, 16 steps over the 64 columns): the
      // integer products and sums stay below 2^53, so the result is the exact dot product whatever the order.  A
      // lane holds A[g][t] = q row g, column 4 s + t (kept in registers for the whole kernel) and loads
      // B[t][g] = key block g of the warp's eight, column 4 s + t; it ends with the scores of row g against key
      // blocks 2 t and 2 t + 1.
      const int g = lane >> 2, t4 = lane & 3;
      const double* kr = s_k + (warp * 8 + g) * kPitch + t4;
      double c[2][2] = {{0.0, 0.0}, {0.0, 0.0}};  // two accumulation chains (even / odd steps) hide the MMA latency
      double bv[kHeadDim / 4];
#pragma unroll
      for (int st = 0; st < kHeadDim / 4; ++st) bv[st] = kr[4 * st];
#pragma unroll
      for (int st = 0; st < kHeadDim / 4; ++st) {
        asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0, %1}, {%2}, {%3}, {%0, %1};"
                     : "+d"(c[st & 1][0]), "+d"(c[st & 1][1])
                     : "d"(q_frag[st]), "d"(bv[st]));
      }
      const double cc[2] = {c[0][0] + c[1][0], c[0][1] + c[1][1]};
#pragma unroll
      for (int x = 0; x < 2; ++x) {
        const int j = j0 + warp * 8 + 2 * t4 + x;
        if (j < nb) {
          const int valid = min(block, tokens - j * block);
          const double tt = cc[x] * static_cast<double>(k_scales[bh_rows + j]) / static_cast<double>(valid) + 0.0;
          s_key[static_cast<size_t>(g) * pitch + j] = order_key(tt);
        }
      }
    } else if (jj < nj) {
      const double2* kr = reinterpret_cast<const double2*>(s_k + jj * kPitch);
      const double2* qr = reinterpret_cast<const double2*>(s_q + rg * kRowsPerLane * kPitch);
      double acc[kRowsPerLane];
#pragma unroll
      for (int x = 0; x < kRowsPerLane; ++x) acc[x] = 0.0;
#pragma unroll 8
      for (int d2 = 0; d2 < kHeadDim / 2; ++d2) {
        const double2 kv = kr[d2];
#pragma unroll
        for (int x = 0; x < kRowsPerLane; ++x) {
          const double2 qv = qr[x * (kPitch / 2) + d2];
          acc[x] = fma(qv.x, kv.x, acc[x]);
          acc[x] = fma(qv.y, kv.y, acc[x]);
        }
      }
      const int j = j0 + jj;
      const int valid = min(block, tokens - j * block);
      const double ks = static_cast<double>(k_scales[bh_rows + j]);
      const double n_valid = static_cast<double>(valid);
#pragma unroll
      for (int x = 0; x < kRowsPerLane; ++x) {
        const double t = acc[x] * ks / n_valid + 0.0;
        s_key[static_cast<size_t>(rg * kRowsPerLane + x) * pitch + j] = order_key(t);
      }
    }
  }
  __syncthreads();
  const int i = i0 + warp;
  if (i >= nb) return;

  // Phase B
  const unsigned long long* keys = s_key + static_cast<size_t>(warp) * pitch;
  unsigned int* hist = s_hist + warp * 256;
  const Selection sc = select_top(keys, nb, k_crit, hist, lane);
  const Selection sm = select_top(keys, nb, nb - k_neg, hist, lane);

  // Phase C
  const size_t row = bh_rows + i;
  signed char* out_cls = cls + row * nb;
  int n_crit = 0, n_marg = 0, tie_c = 0, tie_m = 0;
  const unsigned below = (1u << lane) - 1u;
  for (int j0 = 0; j0 < nb; j0 += 32) {
    const int j = j0 + lane;
    const bool in = j < nb;
    const unsigned long long key = in ? keys[j] : 0ull;
    const unsigned long long kc = key & sc.mask, km = key & sm.mask;
    const bool eq_c = in && kc == sc.prefix, eq_m = in && km == sm.prefix;
    const unsigned b_eq_c = __ballot_sync(0xFFFFFFFFu, eq_c), b_eq_m = __ballot_sync(0xFFFFFFFFu, eq_m);
    const bool sel_c = in && (kc > sc.prefix || (eq_c && tie_c + __popc(b_eq_c & below) < sc.take));
    const bool sel_m = in && (km > sm.prefix || (eq_m && tie_m + __popc(b_eq_m & below) < sm.take));
    tie_c += __popc(b_eq_c);
    tie_m += __popc(b_eq_m);
    const int c = !in ? -1 : (sel_c ? 2 : (sel_m ? 1 : 0));
    if (in) out_cls[j] = static_cast<signed char>(c);
    const unsigned m_crit = __ballot_sync(0xFFFFFFFFu, c == 2);
    const unsigned m_marg = __ballot_sync(0xFFFFFFFFu, c == 1);
    if (c == 2) crit_idx[row * k_crit + n_crit + __popc(m_crit & below)] = j;
    if (c == 1 && marg_idx != nullptr) marg_idx[row * k_marg + n_marg + __popc(m_marg & below)] = j;
    n_crit += __popc(m_crit);
    n_marg += __popc(m_marg);
  }
}

size_t plan_smem_bytes(int nb, int rows) {
  return static_cast<size_t>(rows) * ((nb + 1) & ~1) * 8 + static_cast<size_t>(rows) * kPitch * 8 +
         static_cast<size_t>(kChunk) * kPitch * 8 + static_cast<size_t>(rows) * 256 * 4;
}

template <int R>
lite3r_status launch_rows(const lite3r_fp8& q, const lite3r_fp8& k, const lite3r_shape& s, const Counts& c,
                          const lite3r_plan& plan, int nb, cudaStream_t stream) {
  const size_t smem = plan_smem_bytes(nb, R);
  lite3r_status st = record_cuda(
      cudaFuncSetAttribute(plan_kernel<R>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
  if (st != LITE3R_OK) return st;
  const int row_tiles = ceil_div(nb, R);
  plan_kernel<R><<<s.batch * s.heads * row_tiles, R * 32, smem, stream>>>(q.colsum, k.colsum, k.scales, s.tokens,
                                                                           s.block, nb, c.k_crit, c.k_marg, c.k_neg,
                                                                           plan.cls, plan.crit_idx, plan.marg_idx);
  return after_launch();
}

}  // namespace

lite3r_status launch_plan(const lite3r_fp8& q, const lite3r_fp8& k, const lite3r_shape& s, const Counts& c,
                          const lite3r_plan& plan, cudaStream_t stream) {
  const int nb = ceil_div(s.tokens, s.block);
  constexpr size_t kLimit = 227 * 1024;
  // As many rows per CTA as the row keys allow: the staged key blocks are then shared by more rows.
  if (plan_smem_bytes(nb, 8) <= kLimit) return launch_rows<8>(q, k, s, c, plan, nb, stream);
  if (plan_smem_bytes(nb, 4) <= kLimit) return launch_rows<4>(q, k, s, c, plan, nb, stream);
  if (plan_smem_bytes(nb, 2) <= kLimit) return launch_rows<2>(q, k, s, c, plan, nb, stream);
  if (plan_smem_bytes(nb, 1) <= kLimit) return launch_rows<1>(q, k, s, c, plan, nb, stream);
  return LITE3R_ERR_UNSUPPORTED;  // more than ~24000 blocks per sequence
}

}  // namespace lite3r
