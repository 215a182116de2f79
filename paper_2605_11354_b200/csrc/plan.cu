// K2: pooled scores and row-wise top-k block classification (Algorithm 1 lines 2-3 on block means).
//
// The pooled mean of block i is colsum_i * 2^-9 * scale_i / valid_i with colsum an exact integer vector, so
//   s_ij = (colsum^Q_i . colsum^K_j) * [scale^K_j / valid_j] * [scale^Q_i / (valid_i * 8 * 2^18)].
// The last bracket is a positive constant of row i and cannot change the ranking inside the row, so the
// kernel ranks t_ij = (integer dot product, exact in fp64 below 2^53) * scale^K_j / valid_j.  Two fp64
// roundings separate t_ij from the exact value; the ranking is therefore the exact one except between
// scores that agree to ~1e-15 relative.  Ranking order: score descending, then key-block index ascending.
//
// One CTA of R warps handles R consecutive query blocks of one (b, h): warp r owns row r.  Scores of the R rows
// live in shared memory as order-preserving 64-bit keys; the rank of every entry is found by counting the
// entries that precede it, which needs no sort and gives the total order directly.
#include "common.cuh"

namespace lite3r {

namespace {

constexpr int kRows = 4;           // query blocks (rows) per CTA, one warp each
constexpr int kThreads = kRows * 32;
constexpr int kChunk = 64;         // key blocks staged per pass
constexpr int kPad = kHeadDim + 1; // padded row of the staged chunk: conflict-free column walks

// Maps a double to an unsigned key with the same order (larger double -> larger key).
__device__ __forceinline__ unsigned long long order_key(double v) {
  const unsigned long long u = static_cast<unsigned long long>(__double_as_longlong(v));
  return (u >> 63) ? ~u : (u | 0x8000000000000000ull);
}

__global__ void __launch_bounds__(kThreads) plan_kernel(const int* __restrict__ q_colsum,
                                                        const int* __restrict__ k_colsum,
                                                        const float* __restrict__ k_scales, int tokens, int block,
                                                        int nb, int k_crit, int k_marg, int k_neg,
                                                        signed char* __restrict__ cls, int* __restrict__ crit_idx,
                                                        int* __restrict__ marg_idx) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  unsigned long long* s_key = reinterpret_cast<unsigned long long*>(smem_raw);      // [kRows][nb]
  double* s_q = reinterpret_cast<double*>(s_key + static_cast<size_t>(kRows) * nb); // [kRows][64]
  double* s_k = s_q + kRows * kHeadDim;                                             // [kChunk][kPad]
  signed char* s_cls = reinterpret_cast<signed char*>(s_k + kChunk * kPad);         // [kRows][nb]

  const int row_tiles = (nb + kRows - 1) / kRows;
  const int bh = blockIdx.x / row_tiles;
  const int i0 = (blockIdx.x % row_tiles) * kRows;
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int i = i0 + warp;
  const bool row_ok = i < nb;
  const size_t bh_rows = static_cast<size_t>(bh) * nb;

  for (int t = threadIdx.x; t < kRows * kHeadDim; t += kThreads) {
    const int r = t / kHeadDim;
    s_q[t] = (i0 + r < nb) ? static_cast<double>(q_colsum[(bh_rows + i0 + r) * kHeadDim + (t % kHeadDim)]) : 0.0;
  }

  // Phase A: scores of R rows against all key blocks, kChunk key blocks at a time.
  for (int j0 = 0; j0 < nb; j0 += kChunk) {
    __syncthreads();
    const int nj = min(kChunk, nb - j0);
    for (int t = threadIdx.x; t < nj * kHeadDim; t += kThreads) {
      s_k[(t / kHeadDim) * kPad + (t % kHeadDim)] = static_cast<double>(k_colsum[(bh_rows + j0) * kHeadDim + t]);
    }
    __syncthreads();
    if (row_ok) {
#pragma unroll
      for (int half = 0; half < kChunk / 32; ++half) {
        const int jj = lane + half * 32;
        if (jj < nj) {
          const double* kr = s_k + jj * kPad;
          const double* qr = s_q + warp * kHeadDim;
          double dot = 0.0;
#pragma unroll 16
          for (int d = 0; d < kHeadDim; ++d) dot = fma(qr[d], kr[d], dot);
          const int j = j0 + jj;
          const int valid = min(block, tokens - j * block);
          const double t = dot * static_cast<double>(k_scales[bh_rows + j]) / static_cast<double>(valid) + 0.0;
          s_key[static_cast<size_t>(warp) * nb + j] = order_key(t);
        }
      }
    }
  }
  __syncwarp();
  if (!row_ok) return;

  // Phase B: rank by counting predecessors in (score desc, index asc) order; class from the rank.
  const unsigned long long* keys = s_key + static_cast<size_t>(warp) * nb;
  signed char* my_cls = s_cls + static_cast<size_t>(warp) * nb;
  for (int j = lane; j < nb; j += 64) {
    const int ja = j, jb = j + 32;  // two entries per lane share every shared-memory read
    const unsigned long long ka = keys[ja];
    const unsigned long long kb = jb < nb ? keys[jb] : 0ull;
    int ra = 0, rb = 0;
    for (int o = 0; o < nb; ++o) {
      const unsigned long long ko = keys[o];
      ra += (ko > ka) || (ko == ka && o < ja);
      rb += (ko > kb) || (ko == kb && o < jb);
    }
    my_cls[ja] = ra < k_crit ? 2 : (ra >= nb - k_neg ? 0 : 1);
    if (jb < nb) my_cls[jb] = rb < k_crit ? 2 : (rb >= nb - k_neg ? 0 : 1);
  }
  __syncwarp();

  // Phase C: write the class row and the ascending index lists.
  const size_t row = bh_rows + i;
  signed char* out_cls = cls + row * nb;
  int n_crit = 0, n_marg = 0;
  for (int j0 = 0; j0 < nb; j0 += 32) {
    const int j = j0 + lane;
    const int c = j < nb ? my_cls[j] : -1;
    if (j < nb) out_cls[j] = static_cast<signed char>(c);
    const unsigned m_crit = __ballot_sync(0xFFFFFFFFu, c == 2);
    const unsigned m_marg = __ballot_sync(0xFFFFFFFFu, c == 1);
    const unsigned below = (1u << lane) - 1u;
    if (c == 2) crit_idx[row * k_crit + n_crit + __popc(m_crit & below)] = j;
    if (c == 1 && marg_idx != nullptr) marg_idx[row * k_marg + n_marg + __popc(m_marg & below)] = j;
    n_crit += __popc(m_crit);
    n_marg += __popc(m_marg);
  }
}

size_t plan_smem_bytes(int nb) {
  return static_cast<size_t>(kRows) * nb * 8 + (kRows * kHeadDim + kChunk * kPad) * 8 + static_cast<size_t>(kRows) * nb;
}

}  // namespace

lite3r_status launch_plan(const lite3r_fp8& q, const lite3r_fp8& k, const lite3r_shape& s, const Counts& c,
                          const lite3r_plan& plan, cudaStream_t stream) {
  const int nb = ceil_div(s.tokens, s.block);
  const size_t smem = plan_smem_bytes(nb);
  if (smem > 227 * 1024) return LITE3R_ERR_UNSUPPORTED;  // more than ~5900 blocks per sequence
  lite3r_status st = record_cuda(
      cudaFuncSetAttribute(plan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
  if (st != LITE3R_OK) return st;
  const int row_tiles = ceil_div(nb, kRows);
  plan_kernel<<<s.batch * s.heads * row_tiles, kThreads, smem, stream>>>(q.colsum, k.colsum, k.scales, s.tokens,
                                                                          s.block, nb, c.k_crit, c.k_marg, c.k_neg,
                                                                          plan.cls, plan.crit_idx, plan.marg_idx);
  return after_launch();
}

}  // namespace lite3r
