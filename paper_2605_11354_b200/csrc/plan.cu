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
//     over the 64-bit keys (8-bit digits, per-warp histogram in shared memory): it yields a key prefix such that
//     every entry above it is selected, and of the entries equal to it the first `take` in index order are.  That
//     is exactly the total order (score descending, index ascending), at O(Nb) work per row.  Two selections
//     give the classes: the best k_crit are critical, the best Nb - k_neg are critical-or-marginal.
//   Phase C (same warp): class row and ascending index lists, written with ballot prefix sums.
#include "common.cuh"

namespace lite3r {

namespace {

constexpr int kChunk = 64;          // key blocks staged per pass (upper bound; the used part is keys_per_warp * R)
constexpr int kPitch = kHeadDim + 2;  // staged row pitch in doubles: 16-byte aligned rows, conflict-free 16-byte reads

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
  for (int shift = 56; shift >= 0; shift -= 8) {
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
    prefix |= static_cast<unsigned long long>(digit) << shift;
    mask |= 0xFFull << shift;
    __syncwarp();
    if (bin == remaining) break;  // the whole bin is selected: lower digits cannot matter
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
  double* s_q = reinterpret_cast<double*>(s_key + static_cast<size_t>(R) * pitch);    // [R][64]
  double* s_k = s_q + R * kHeadDim;                                                   // [kChunk][kPitch]
  unsigned int* s_hist = reinterpret_cast<unsigned int*>(s_k + kChunk * kPitch);      // [R][256]

  const int row_tiles = (nb + R - 1) / R;
  const int bh = blockIdx.x / row_tiles;
  const int i0 = (blockIdx.x % row_tiles) * R;
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const size_t bh_rows = static_cast<size_t>(bh) * nb;

  for (int t = threadIdx.x; t < R * kHeadDim; t += kThreads) {
    const int r = t / kHeadDim;
    s_q[t] = (i0 + r < nb) ? static_cast<double>(q_colsum[(bh_rows + i0 + r) * kHeadDim + (t % kHeadDim)]) : 0.0;
  }

  // Phase A
  const int kl = lane % kKeysPerWarp, rg = lane / kKeysPerWarp;
  const int jj = warp * kKeysPerWarp + kl;
  for (int j0 = 0; j0 < nb; j0 += kStep) {
    __syncthreads();
    const int nj = min(kStep, nb - j0);
    for (int t = threadIdx.x; t < nj * kHeadDim; t += kThreads)
      s_k[(t / kHeadDim) * kPitch + (t % kHeadDim)] = static_cast<double>(k_colsum[(bh_rows + j0) * kHeadDim + t]);
    __syncthreads();
    if (jj < nj) {
      const double2* kr = reinterpret_cast<const double2*>(s_k + jj * kPitch);
      const double2* qr = reinterpret_cast<const double2*>(s_q + rg * kRowsPerLane * kHeadDim);
      double acc[kRowsPerLane];
#pragma unroll
      for (int x = 0; x < kRowsPerLane; ++x) acc[x] = 0.0;
#pragma unroll 8
      for (int d2 = 0; d2 < kHeadDim / 2; ++d2) {
        const double2 kv = kr[d2];
#pragma unroll
        for (int x = 0; x < kRowsPerLane; ++x) {
          const double2 qv = qr[x * (kHeadDim / 2) + d2];
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
  return static_cast<size_t>(rows) * ((nb + 1) & ~1) * 8 + static_cast<size_t>(rows) * kHeadDim * 8 +
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
