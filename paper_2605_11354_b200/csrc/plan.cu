// K2: pooled scores and row-wise top-k block classification (the score and TopKMask steps of Algorithm 1 on block means).
//
// The pooled mean of block i is colsum_i * 2^-9 * scale_i / valid_i with colsum an exact integer vector, so
//   s_ij = (colsum^Q_i . colsum^K_j) * [scale^K_j / valid_j] * [scale^Q_i / (valid_i * 8 * 2^18)].
// The last bracket is a positive constant of row i and cannot change the ranking inside the row, so the
// kernel ranks t_ij = (integer dot product, exact in fp64 below 2^53) * scale^K_j / valid_j.  Two fp64
// roundings separate t_ij from the exact value; the ranking is therefore the exact one except between
// scores that agree to ~1e-15 relative.  Ranking order: score descending, then key-block index ascending.
//
// One CTA of R warps handles R consecutive query blocks (rows) of one (b, h); R = 8 unless the row keys of a very
// long sequence do not fit in shared memory.
//   Phase A (whole CTA): the scores of the R rows against all key blocks, kept in shared memory as order-preserving
//     64-bit keys.  R = 8: fp64 tensor-core products (m8n8k4) fed with the int32 column sums straight from global
//     memory, no staging and no barrier.  R < 8: 64 key blocks at a time staged in shared memory as doubles; a lane
//     owns one key block and R/4 rows, so every staged value feeds several fp64 FMAs.
//   Phase B (one warp per row): "the k best of the row".  A histogram over 256 buckets that are linear in the score
//     places the k-th best in a bucket of usually a handful of keys; those are listed by index and a
//     most-significant-digit-first radix select over their 64-bit keys (8-bit digits placed at the highest bit on
//     which the remaining candidates differ, per-warp histogram in shared memory) decides between them: it yields a
//     key prefix such that every entry above it is selected, and of the entries equal to it the first `take` in
//     index order are.  That is exactly the total order (score descending, index ascending), at O(Nb) work per
//     row.  Two selections give the classes: the best k_crit are critical, the best Nb - k_neg are
//     critical-or-marginal.
//   Phase C (same warp): class row and ascending index lists, written with ballot prefix sums.
#include <atomic>

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
  // An entry is selected when its bucket is above `bucket`; inside that bucket when (key & mask) > prefix, and of the
  // entries with (key & mask) == prefix the first `take` in index order.
  unsigned long long prefix, mask;
  int take, bucket;
};

constexpr int kBuckets = 256;
constexpr int kMaxListed = 128;  // candidates of a threshold bucket kept as an index list; fuller buckets are re-scanned

// Position of rank `remaining` (1-based, counted from the top bin down) in a 256-bin histogram: the bin holding it, the
// entries in the bins above and the size of that bin.  Warp-collective; lane L owns bins 255-8L .. 248-8L.
struct Located {
  int bin, above, size;
};
__device__ __forceinline__ Located locate(const unsigned int* hist, int remaining, int lane) {
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
  Located r = {0, 0, 0};
  if (mine) {
    int run = excl;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      if (r.size == 0 && run + cnt[i] >= remaining) {
        r.bin = 255 - 8 * lane - i;
        r.above = run;
        r.size = cnt[i];
      }
      run += cnt[i];
    }
  }
  const int src = __ffs(__ballot_sync(0xFFFFFFFFu, mine)) - 1;
  r.bin = __shfl_sync(0xFFFFFFFFu, r.bin, src);
  r.above = __shfl_sync(0xFFFFFFFFu, r.above, src);
  r.size = __shfl_sync(0xFFFFFFFFu, r.size, src);
  return r;
}

// The k best (largest key, then lowest position) of the m candidates cand(0) .. cand(m - 1), 0 < k < m as far as the
// valid ones go: cand(c, key) says whether candidate c takes part and gives its key.  Most-significant-digit-first
// radix select over the 64-bit keys, 8-bit digits placed at the highest bit on which the remaining candidates still
// differ (keys of one row share their sign and leading exponent bits, so fixed digit positions would spend whole
// passes on digits that are equal for everyone).  Warp-collective; hist is this warp's 256 counters.
template <class Cand>
__device__ void radix_select(Cand cand, int m, int k, unsigned int* hist, int lane, Selection& s) {
  unsigned long long prefix = 0ull, mask = 0ull;
  int remaining = k;
  while (true) {
    unsigned long long all_and = ~0ull, all_or = 0ull;
    for (int c = lane; c < m; c += 32) {
      unsigned long long key;
      if (cand(c, key) && (key & mask) == prefix) {
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
    for (int c = lane; c < m; c += 32) {
      unsigned long long key;
      if (cand(c, key) && (key & mask) == prefix) atomicAdd(&hist[static_cast<unsigned int>(key >> shift) & 255u], 1u);
    }
    __syncwarp();
    const Located at = locate(hist, remaining, lane);
    remaining -= at.above;
    const unsigned long long field = 0xFFull << shift;
    prefix = (prefix & ~field) | (static_cast<unsigned long long>(at.bin) << shift);
    mask |= field;
    __syncwarp();
    if (at.size == remaining || shift == 0) break;  // the whole bin is selected, or every bit has been decided
  }
  s.prefix = prefix;
  s.mask = mask;
  s.take = remaining;
}

// The k best (largest key, then lowest index) of keys[0..n).  First a histogram over 256 buckets that are linear in
// the score (bucket(j), any monotone map of the score to 0..255, computed from a single-precision copy): it places
// the k-th best in one bucket with usually a handful of entries, listed by index (idx, at most kMaxListed) for the
// radix select that decides between them.  hist must hold the bucket counts of the row on entry.  Warp-collective.
template <class Bucket>
__device__ Selection select_top(const unsigned long long* keys, Bucket bucket, int n, int k, unsigned int* hist,
                                const unsigned int* bucket_hist, unsigned short* idx, int lane) {
  Selection s;
  s.prefix = 0ull;
  s.mask = 0ull;
  s.take = 0;
  if (k <= 0) {  // nothing selected
    s.bucket = kBuckets;
    return s;
  }
  if (k >= n) {  // everything selected
    s.bucket = -1;
    return s;
  }
  const Located at = locate(bucket_hist, k, lane);
  s.bucket = at.bin;
  const int remaining = k - at.above;
  if (remaining == at.size) {  // the whole bucket is selected
    s.take = at.size;
    return s;
  }
  if (at.size <= kMaxListed) {
    const unsigned below = (1u << lane) - 1u;
    int listed = 0;
    for (int j0 = 0; j0 < n; j0 += 32) {
      const int j = j0 + lane;
      const bool is = j < n && bucket(j) == at.bin;
      const unsigned b = __ballot_sync(0xFFFFFFFFu, is);
      if (is) idx[listed + __popc(b & below)] = static_cast<unsigned short>(j);
      listed += __popc(b);
    }
    __syncwarp();
    radix_select([&](int c, unsigned long long& key) {
      key = keys[idx[c]];
      return true;
    }, at.size, remaining, hist, lane, s);
  } else {
    radix_select([&](int c, unsigned long long& key) {
      key = keys[c];
      return bucket(c) == at.bin;
    }, n, remaining, hist, lane, s);
  }
  return s;
}

template <int R>
__global__ void __launch_bounds__(R * 32) plan_kernel(const int* __restrict__ q_colsum, const int* __restrict__ k_colsum,
                                                       const float* __restrict__ k_scales, int tokens, int block,
                                                       int nb, int k_crit, int k_marg, int k_neg,
                                                       signed char* __restrict__ cls, int* __restrict__ crit_idx,
                                                       int* __restrict__ marg_idx) {
  constexpr int kThreads = R * 32;
  constexpr bool kDirect = R >= 8;                // column sums straight from global memory into the fp64 MMA
  constexpr int kTiles = kDirect ? R / 8 : 1;     // 8-row MMA tiles per warp
  constexpr int kGroups = R >= 4 ? 4 : R;        // (staged path) row groups inside a warp
  constexpr int kRowsPerLane = R / kGroups;       // (staged path) rows whose score one lane accumulates
  constexpr int kKeysPerWarp = 32 / kGroups;
  constexpr int kStep = kKeysPerWarp * R;         // (staged path) key blocks per staged pass (<= kChunk)
  static_assert(kDirect || kStep <= kChunk, "staging buffer too small");

  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int pitch = (nb + 1) & ~1;  // key-row pitch: keeps everything behind the keys 16-byte aligned
  unsigned long long* s_key = reinterpret_cast<unsigned long long*>(smem_raw);        // [R][pitch]
  unsigned int* s_hist = reinterpret_cast<unsigned int*>(s_key + static_cast<size_t>(R) * pitch);  // [R][2][256]
  unsigned short* s_idx = reinterpret_cast<unsigned short*>(s_hist + R * 2 * kBuckets);            // [R][2][kMaxListed]
  float2* s_range = reinterpret_cast<float2*>(s_idx + R * 2 * kMaxListed);                         // [R][R]     (direct)
  unsigned char* s_bkt = reinterpret_cast<unsigned char*>(s_range + R * R);                        // [R][pitch] (direct)

  const int row_tiles = (nb + R - 1) / R;
  const int bh = blockIdx.x / row_tiles;
  const int i0 = (blockIdx.x % row_tiles) * R;
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const size_t bh_rows = static_cast<size_t>(bh) * nb;

  if constexpr (kDirect) {
    // Phase A, R rows x 8 key blocks per warp and step as fp64 tensor-core products (m8n8k4, 16 k-steps over the 64
    // columns, one 8-row tile after the other against the same B values): the integer products and sums stay below
    // 2^53, so the result is the exact dot product whatever the order.  The product does not care which column sits
    // at which k index as long as A and B agree, so lane (g, t) supplies columns 16 t .. 16 t + 15 of its row (q
    // row g of each tile for A, key block g of the warp's eight for B): 64 contiguous bytes of the int32 column
    // sums, read straight from global memory (L2) one step ahead, with no staging and no barrier.  Every CTA
    // streams all column sums of its (b, h) once, which is what bounds this phase: hence as many rows per CTA as
    // shared memory allows.  int32 -> fp64 is exact and takes one xor and one subtraction: the double with high
    // word 0x43300000 and low word v ^ 2^31 is 2^52 + 2^31 + v.
    const int g = lane >> 2, t4 = lane & 3;
    auto widen = [](int v) {
      return __hiloint2double(0x43300000, v ^ static_cast<int>(0x80000000u)) - 4503601774854144.0;
    };
    // `local` is a block index inside the (b, h); past the end the last block is read instead (its products land
    // in rows or columns that are never stored), which keeps the loads free of predicates and zero fills
    auto load16 = [&](const int* base, int local, int4 dst[4]) {
      const int4* src = reinterpret_cast<const int4*>(base + (bh_rows + min(local, nb - 1)) * kHeadDim + 16 * t4);
#pragma unroll
      for (int q = 0; q < 4; ++q) dst[q] = __ldg(src + q);
    };
    double q_frag[kTiles][16];
#pragma unroll
    for (int m = 0; m < kTiles; ++m) {
      int4 qv[4];
      load16(q_colsum, i0 + 8 * m + g, qv);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        q_frag[m][4 * q] = widen(qv[q].x);
        q_frag[m][4 * q + 1] = widen(qv[q].y);
        q_frag[m][4 * q + 2] = widen(qv[q].z);
        q_frag[m][4 * q + 3] = widen(qv[q].w);
      }
    }
    // the scales of the two key blocks whose scores the lane ends up with travel with the column sums
    auto load_scales = [&](int j, float dst[2]) {
#pragma unroll
      for (int x = 0; x < 2; ++x) dst[x] = __ldg(k_scales + bh_rows + min(j + x, nb - 1));
    };
    int4 nxt[4];
    float nxt_ks[2];
    load16(k_colsum, warp * 8 + g, nxt);
    load_scales(warp * 8 + 2 * t4, nxt_ks);
    float lo[kTiles], hi[kTiles];  // range of the scores of row 8 m + g, as far as this lane sees them
#pragma unroll
    for (int m = 0; m < kTiles; ++m) {
      lo[m] = INFINITY;
      hi[m] = -INFINITY;
    }
    const bool block_pow2 = (block & (block - 1)) == 0;
    const double inv_block = 1.0 / static_cast<double>(block);
    for (int j0 = warp * 8; j0 < nb; j0 += 8 * R) {
      int4 cur[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) cur[q] = nxt[q];
      const float cur_ks[2] = {nxt_ks[0], nxt_ks[1]};
      if (j0 + 8 * R < nb) {
        load16(k_colsum, j0 + 8 * R + g, nxt);
        load_scales(j0 + 8 * R + 2 * t4, nxt_ks);
      }
      // per tile two accumulation chains (even / odd k-steps), which hide the MMA latency; four were slower
      constexpr int kChains = 2;
      double c[kTiles][kChains][2];
#pragma unroll
      for (int m = 0; m < kTiles; ++m) {
#pragma unroll
        for (int n = 0; n < kChains; ++n) c[m][n][0] = c[m][n][1] = 0.0;
      }
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int vals[4] = {cur[q].x, cur[q].y, cur[q].z, cur[q].w};
#pragma unroll
        for (int y = 0; y < 4; ++y) {
          const int st = 4 * q + y;
          const double bv = widen(vals[y]);
#pragma unroll
          for (int m = 0; m < kTiles; ++m) {
            asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0, %1}, {%2}, {%3}, {%0, %1};"
                         : "+d"(c[m][st % kChains][0]), "+d"(c[m][st % kChains][1])
                         : "d"(q_frag[m][st]), "d"(bv));
          }
        }
      }
      // the lane ends with the scores of rows 8 m + g against key blocks 2 t and 2 t + 1 of the warp's eight
#pragma unroll
      for (int x = 0; x < 2; ++x) {
        const int j = j0 + 2 * t4 + x;
        if (j < nb) {
          const int valid = min(block, tokens - j * block);
          const double ks = static_cast<double>(cur_ks[x]);
          const bool full = valid == block && block_pow2;
#pragma unroll
          for (int m = 0; m < kTiles; ++m) {
            // a full block of 2^n tokens divides exactly by a multiplication; only the last block can be shorter
            const double num = (c[m][0][x] + c[m][1][x]) * ks;
            const double tt = (full ? num * inv_block : num / static_cast<double>(valid)) + 0.0;
            s_key[static_cast<size_t>(8 * m + g) * pitch + j] = order_key(tt);
            // range of the row in single precision, for the bucket histogram of the selection
            const float tf = static_cast<float>(tt);
            lo[m] = fminf(lo[m], tf);
            hi[m] = fmaxf(hi[m], tf);
          }
        }
      }
    }
#pragma unroll
    for (int m = 0; m < kTiles; ++m) {
#pragma unroll
      for (int o = 1; o <= 2; o <<= 1) {
        lo[m] = fminf(lo[m], __shfl_xor_sync(0xFFFFFFFFu, lo[m], o));
        hi[m] = fmaxf(hi[m], __shfl_xor_sync(0xFFFFFFFFu, hi[m], o));
      }
      if (t4 == 0) s_range[warp * R + 8 * m + g] = make_float2(lo[m], hi[m]);
    }
  } else {
    // Phase A for sequences too long for eight rows of keys per CTA: the column sums of kStep key blocks at a time
    // are staged in shared memory as doubles (fetched with 16-byte loads one pass ahead); a lane owns one key block
    // and R / 4 rows, so every staged value feeds several fp64 FMAs.  Both staged arrays use a row pitch of 68
    // doubles, which keeps the 16-byte reads of the key rows and of the row groups of a warp on different banks.
    double* s_q = reinterpret_cast<double*>(s_idx + R * 2 * kMaxListed);  // [R][kPitch]
    double* s_k = s_q + R * kPitch;                             // [kChunk][kPitch]
    for (int t = threadIdx.x; t < R * kHeadDim; t += kThreads) {
      const int r = t / kHeadDim, d = t % kHeadDim;
      s_q[r * kPitch + d] = (i0 + r < nb) ? static_cast<double>(q_colsum[(bh_rows + i0 + r) * kHeadDim + d]) : 0.0;
    }
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
      if (jj < nj) {
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
  }
  __syncthreads();
  const int i = i0 + warp;
  if (i >= nb) return;

  // Phase B
  const unsigned long long* keys = s_key + static_cast<size_t>(warp) * pitch;
  unsigned int* hist = s_hist + warp * 2 * kBuckets;  // radix digits; the second half holds the bucket counts
  unsigned int* bucket_hist = hist + kBuckets;
  // Buckets linear in the score between the row's extremes; with fewer than eight rows per CTA (very long
  // sequences) there is no single-precision copy and every key falls into bucket 0, which leaves the whole
  // selection to the radix select.
  float lo = 0.f, scale = 0.f;
  unsigned char* bkt = s_bkt + static_cast<size_t>(warp) * pitch;
  if constexpr (kDirect) {
    float2 range = lane < R ? s_range[lane * R + warp] : make_float2(INFINITY, -INFINITY);
#pragma unroll
    for (int o = 1; o < R; o <<= 1) {
      range.x = fminf(range.x, __shfl_xor_sync(0xFFFFFFFFu, range.x, o));
      range.y = fmaxf(range.y, __shfl_xor_sync(0xFFFFFFFFu, range.y, o));
    }
    range.x = __shfl_sync(0xFFFFFFFFu, range.x, 0);
    range.y = __shfl_sync(0xFFFFFFFFu, range.y, 0);
    lo = range.x;
    scale = range.y > range.x ? 255.5f / (range.y - range.x) : 0.f;
  }
  auto bucket = [&](int j) -> int {
    if constexpr (!kDirect) return 0;
    return bkt[j];
  };
#pragma unroll
  for (int b = 0; b < 8; ++b) bucket_hist[lane + 32 * b] = 0u;
  __syncwarp();
  for (int j = lane; j < nb; j += 32) {
    int b = 0;
    if constexpr (kDirect) {
      // key -> double -> float: every step keeps the order (weakly), which is all the buckets need
      const unsigned long long key = keys[j];
      const unsigned long long u = (key >> 63) ? (key & 0x7FFFFFFFFFFFFFFFull) : ~key;
      const float tf = static_cast<float>(__longlong_as_double(static_cast<long long>(u)));
      b = min(kBuckets - 1, max(0, __float2int_rz((tf - lo) * scale)));
      bkt[j] = static_cast<unsigned char>(b);
    }
    atomicAdd(&bucket_hist[b], 1u);
  }
  __syncwarp();
  unsigned short* idx = s_idx + warp * 2 * kMaxListed;
  const Selection sc = select_top(keys, bucket, nb, k_crit, hist, bucket_hist, idx, lane);
  const Selection sm = select_top(keys, bucket, nb, nb - k_neg, hist, bucket_hist, idx + kMaxListed, lane);

  // Phase C
  const size_t row = bh_rows + i;
  signed char* out_cls = cls + row * nb;
  int n_crit = 0, n_marg = 0, tie_c = 0, tie_m = 0;
  const unsigned below = (1u << lane) - 1u;
#pragma unroll 2
  for (int j0 = 0; j0 < nb; j0 += 32) {
    const int j = j0 + lane;
    const bool in = j < nb;
    const int bk = in ? bucket(j) : -2;
    bool sel_c = in && bk > sc.bucket, sel_m = in && bk > sm.bucket;
    // the 64-bit keys only matter for entries inside one of the two threshold buckets: most groups of 32 have none
    if (__any_sync(0xFFFFFFFFu, bk == sc.bucket || bk == sm.bucket)) {
      const unsigned long long key = in ? keys[j] : 0ull;
      const unsigned long long kc = key & sc.mask, km = key & sm.mask;
      const bool eq_c = bk == sc.bucket && kc == sc.prefix, eq_m = bk == sm.bucket && km == sm.prefix;
      const unsigned b_eq_c = __ballot_sync(0xFFFFFFFFu, eq_c), b_eq_m = __ballot_sync(0xFFFFFFFFu, eq_m);
      sel_c = sel_c || (bk == sc.bucket && kc > sc.prefix) || (eq_c && tie_c + __popc(b_eq_c & below) < sc.take);
      sel_m = sel_m || (bk == sm.bucket && km > sm.prefix) || (eq_m && tie_m + __popc(b_eq_m & below) < sm.take);
      tie_c += __popc(b_eq_c);
      tie_m += __popc(b_eq_m);
    }
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

// The same plan with the scores kept in shared memory as single-precision values (4 bytes per key instead of an
// 8-byte ordered key), for long rows: sixteen rows per CTA then fit where eight did, so the column sums of a (b, h)
// are streamed half as often and twice as many warps hide the latencies of the selection and of the class pass.
// The ranking stays the exact one.  The single-precision copy is a monotone (weakly order-preserving) image of the
// exact score and only places a key in one of the 256 buckets; the few keys of a threshold bucket are decided by
// their exact 64-bit keys, which are recomputed for them from the integer column sums (an int64 dot product, equal
// to the tensor-core result as long as that is exact, i.e. below 2^53).
// Warp w of the R = 8 or 16 warps: in phase A row tile w % (R / 8) (eight rows) against every (R / 8)-th group of
// eight key blocks; in phases B and C row w.
template <int R>
__global__ void __launch_bounds__(R * 32) plan_compact_kernel(const int* __restrict__ q_colsum, const int* __restrict__ k_colsum,
                                                               const float* __restrict__ k_scales, int tokens, int block,
                                                               int nb, int k_crit, int k_marg, int k_neg,
                                                               signed char* __restrict__ cls, int* __restrict__ crit_idx,
                                                               int* __restrict__ marg_idx) {
  constexpr int kRowTiles = R / 8;
  constexpr int kGroups = R / kRowTiles;  // warps that share a row tile (= 8)
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int pitch = (nb + 3) & ~3;
  float* s_val = reinterpret_cast<float*>(smem_raw);                                              // [R][pitch]
  unsigned int* s_hist = reinterpret_cast<unsigned int*>(s_val + static_cast<size_t>(R) * pitch);  // [R][2][256]
  unsigned long long* s_ckey = reinterpret_cast<unsigned long long*>(s_hist + R * 2 * kBuckets);   // [R][2][kMaxListed]
  int* s_q = reinterpret_cast<int*>(s_ckey + R * 2 * kMaxListed);                                  // [R][64]
  float2* s_range = reinterpret_cast<float2*>(s_q + R * kHeadDim);                                 // [kGroups][R]
  unsigned short* s_idx = reinterpret_cast<unsigned short*>(s_range + kGroups * R);                // [R][2][kMaxListed]

  const int row_tiles = (nb + R - 1) / R;
  const int bh = blockIdx.x / row_tiles;
  const int i0 = (blockIdx.x % row_tiles) * R;
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const size_t bh_rows = static_cast<size_t>(bh) * nb;
  const bool block_pow2 = (block & (block - 1)) == 0;
  const double inv_block = 1.0 / static_cast<double>(block);

  // the ranking score from an exact dot product (same expression in phase A and for the recomputed keys)
  auto ranking_score = [&](double dot, float ks, int j) {
    const int valid = min(block, tokens - j * block);
    const double num = dot * static_cast<double>(ks);
    return ((valid == block && block_pow2) ? num * inv_block : num / static_cast<double>(valid)) + 0.0;
  };

  {
    // Phase A: fp64 tensor-core products of the exactly widened int32 column sums (see plan_kernel).
    const int tile = warp % kRowTiles, grp = warp / kRowTiles;
    const int g = lane >> 2, t4 = lane & 3;
    auto widen = [](int v) { return __int2double_rn(v); };  // exact; one instruction
    // `local` is a block index inside the (b, h); past the end the last block is read instead (its products land
    // in rows or columns that are never stored), which keeps the loads free of predicates and zero fills
    auto load16 = [&](const int* base, int local, int4 dst[4]) {
      const int4* src = reinterpret_cast<const int4*>(base + (bh_rows + min(local, nb - 1)) * kHeadDim + 16 * t4);
#pragma unroll
      for (int q = 0; q < 4; ++q) dst[q] = __ldg(src + q);
    };
    double q_frag[16];
    {
      int4 qv[4];
      load16(q_colsum, i0 + 8 * tile + g, qv);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        q_frag[4 * q] = widen(qv[q].x);
        q_frag[4 * q + 1] = widen(qv[q].y);
        q_frag[4 * q + 2] = widen(qv[q].z);
        q_frag[4 * q + 3] = widen(qv[q].w);
      }
    }
    auto load_scales = [&](int j, float dst[2]) {
#pragma unroll
      for (int x = 0; x < 2; ++x) dst[x] = __ldg(k_scales + bh_rows + min(j + x, nb - 1));
    };
    int4 nxt[4];
    float nxt_ks[2];
    load16(k_colsum, grp * 8 + g, nxt);
    load_scales(grp * 8 + 2 * t4, nxt_ks);
    float lo = INFINITY, hi = -INFINITY;
    float* const my_val = s_val + static_cast<size_t>(8 * tile + g) * pitch;
    // key blocks in whole blocks of a power-of-two size divide by a multiplication that is exact, so the scale and
    // the division fold into one factor per key block; only the last key block of a sequence can be shorter
    const int last_full = (tokens % block == 0 && block_pow2) ? nb : (block_pow2 ? nb - 1 : 0);  // key blocks below this are whole
#pragma unroll 2
    for (int j0 = grp * 8; j0 < nb; j0 += 8 * kGroups) {
      int4 cur[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) cur[q] = nxt[q];
      const float cur_ks[2] = {nxt_ks[0], nxt_ks[1]};
      if (j0 + 8 * kGroups < nb) {
        load16(k_colsum, j0 + 8 * kGroups + g, nxt);
        load_scales(j0 + 8 * kGroups + 2 * t4, nxt_ks);
      }
      double c[2][2] = {{0.0, 0.0}, {0.0, 0.0}};
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int vals[4] = {cur[q].x, cur[q].y, cur[q].z, cur[q].w};
#pragma unroll
        for (int y = 0; y < 4; ++y) {
          const int st = 4 * q + y;
          const double bv = widen(vals[y]);
          asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0, %1}, {%2}, {%3}, {%0, %1};"
                       : "+d"(c[st & 1][0]), "+d"(c[st & 1][1])
                       : "d"(q_frag[st]), "d"(bv));
        }
      }
      if (j0 + 8 <= last_full) {  // all eight key blocks of the step exist and are whole (warp-uniform)
        float tf[2];
#pragma unroll
        for (int x = 0; x < 2; ++x) {
          tf[x] = static_cast<float>((c[0][x] + c[1][x]) * (static_cast<double>(cur_ks[x]) * inv_block) + 0.0);
          lo = fminf(lo, tf[x]);
          hi = fmaxf(hi, tf[x]);
        }
        *reinterpret_cast<float2*>(my_val + j0 + 2 * t4) = make_float2(tf[0], tf[1]);
      } else {
#pragma unroll
        for (int x = 0; x < 2; ++x) {
          const int j = j0 + 2 * t4 + x;
          if (j < nb) {
            const float tf = static_cast<float>(ranking_score(c[0][x] + c[1][x], cur_ks[x], j));
            my_val[j] = tf;
            lo = fminf(lo, tf);
            hi = fmaxf(hi, tf);
          }
        }
      }
    }
#pragma unroll
    for (int o = 1; o <= 2; o <<= 1) {
      lo = fminf(lo, __shfl_xor_sync(0xFFFFFFFFu, lo, o));
      hi = fmaxf(hi, __shfl_xor_sync(0xFFFFFFFFu, hi, o));
    }
    if (t4 == 0) s_range[grp * R + 8 * tile + g] = make_float2(lo, hi);
  }
  __syncthreads();
  const int i = i0 + warp;
  if (i >= nb) return;

  // Phase B
  const float* vals = s_val + static_cast<size_t>(warp) * pitch;
  unsigned int* hist = s_hist + warp * 2 * kBuckets;
  unsigned int* bucket_hist = hist + kBuckets;
  float2 range = lane < kGroups ? s_range[lane * R + warp] : make_float2(INFINITY, -INFINITY);
#pragma unroll
  for (int o = 1; o < kGroups; o <<= 1) {
    range.x = fminf(range.x, __shfl_xor_sync(0xFFFFFFFFu, range.x, o));
    range.y = fmaxf(range.y, __shfl_xor_sync(0xFFFFFFFFu, range.y, o));
  }
  const float lo = __shfl_sync(0xFFFFFFFFu, range.x, 0), hi = __shfl_sync(0xFFFFFFFFu, range.y, 0);
  // A key's place between the row's extremes on a 16-bit scale; its upper eight bits are the bucket of the first
  // histogram, the lower eight refine a bucket that turns out too full to list.  Both are monotone in the score.
  const float scale = hi > lo ? 65535.5f / (hi - lo) : 0.f;
  // computed once, in the histogram pass, and left in place of the score (which nothing needs after that)
  int* const places = reinterpret_cast<int*>(s_val + static_cast<size_t>(warp) * pitch);
  auto fine = [&](int j) -> int { return places[j]; };
  // exact 64-bit key of entry j of this row (the row's own column sums wait in shared memory)
  int* const q_row = s_q + warp * kHeadDim;
  q_row[lane] = __ldg(q_colsum + (bh_rows + i) * kHeadDim + lane);
  q_row[lane + 32] = __ldg(q_colsum + (bh_rows + i) * kHeadDim + lane + 32);
  const int4* const q4 = reinterpret_cast<const int4*>(q_row);
  auto exact_key = [&](int j) -> unsigned long long {
    const int4* const k4 = reinterpret_cast<const int4*>(k_colsum + (bh_rows + j) * kHeadDim);
    long long dot = 0;
#pragma unroll
    for (int d = 0; d < kHeadDim / 4; ++d) {
      const int4 a = q4[d], b = __ldg(k4 + d);
      dot += static_cast<long long>(a.x) * b.x + static_cast<long long>(a.y) * b.y + static_cast<long long>(a.z) * b.z +
             static_cast<long long>(a.w) * b.w;
    }
    return order_key(ranking_score(static_cast<double>(dot), __ldg(k_scales + bh_rows + j), j));
  };
#pragma unroll
  for (int b = 0; b < 8; ++b) bucket_hist[lane + 32 * b] = 0u;
  __syncwarp();
  for (int j = lane; j < nb; j += 32) {
    const int f = min(65535, max(0, __float2int_rz((vals[j] - lo) * scale)));
    places[j] = f;
    atomicAdd(&bucket_hist[f >> 8], 1u);
  }
  __syncwarp();

  // A selection: entries whose place is above t_hi are selected, those inside [t_lo, t_hi] are decided by their exact
  // keys (prefix / mask / take as in Selection), the rest are not.  Each selection leaves the entries of its
  // threshold range (ascending index) and their exact keys behind for the class pass: keys_from 0 = no key needed
  // (the whole range goes one way), 1 = listed, 2 = recompute (still too many to list after the refinement).
  // The two selections of a row go through their stages together, so that the refinement and the listing each take
  // one pass over the row for both.
  struct Chosen {
    Selection s;
    int t_lo, t_hi, keys_from, remaining, size;
    bool refine, list;
  };
  auto begin = [&](int k) -> Chosen {
    Chosen r;
    r.keys_from = 0;
    r.s.prefix = 0ull;
    r.s.mask = 0ull;
    r.s.take = 0;
    r.s.bucket = 0;
    r.remaining = r.size = 0;
    r.refine = r.list = false;
    if (k <= 0) {
      r.t_lo = r.t_hi = 65536;
      return r;
    }
    if (k >= nb) {
      r.t_lo = r.t_hi = -1;
      return r;
    }
    const Located at = locate(bucket_hist, k, lane);
    r.t_lo = at.bin << 8;
    r.t_hi = r.t_lo + 255;
    r.remaining = k - at.above;
    r.size = at.size;
    if (r.remaining == r.size)
      r.s.take = r.size;
    else if (r.size > kMaxListed)
      r.refine = true;
    else
      r.list = true;
    return r;
  };
  Chosen cc = begin(k_crit), cm = begin(nb - k_neg);
  if (cc.refine || cm.refine) {  // histograms of the lower eight bits inside the two threshold buckets
#pragma unroll
    for (int b = 0; b < 8; ++b) {
      hist[lane + 32 * b] = 0u;
      bucket_hist[lane + 32 * b] = 0u;  // the first histogram has served both selections
    }
    __syncwarp();
    const int bin_c = cc.refine ? cc.t_lo >> 8 : -1, bin_m = cm.refine ? cm.t_lo >> 8 : -1;
    for (int j = lane; j < nb; j += 32) {
      const int f = fine(j);
      if ((f >> 8) == bin_c) atomicAdd(&hist[f & 255], 1u);
      if ((f >> 8) == bin_m) atomicAdd(&bucket_hist[f & 255], 1u);
    }
    __syncwarp();
    auto refined = [&](Chosen& r, const unsigned int* h) {
      if (!r.refine) return;
      const Located at2 = locate(h, r.remaining, lane);
      r.t_lo = r.t_hi = (r.t_lo & ~255) | at2.bin;
      r.remaining -= at2.above;
      r.size = at2.size;
      if (r.remaining == r.size)
        r.s.take = r.size;
      else if (r.size <= kMaxListed)
        r.list = true;
      else
        r.keys_from = 2;  // more than kMaxListed entries in one of 65536 places (near-equal scores)
    };
    refined(cc, hist);
    refined(cm, bucket_hist);
    __syncwarp();
  }
  unsigned long long* const ckey_c = s_ckey + warp * 2 * kMaxListed;
  unsigned long long* const ckey_m = ckey_c + kMaxListed;
  unsigned short* const idx_c = s_idx + warp * 2 * kMaxListed;
  unsigned short* const idx_m = idx_c + kMaxListed;
  if (cc.list || cm.list) {  // positions of the entries inside the two threshold ranges, ascending
    const unsigned below = (1u << lane) - 1u;
    int listed_c = 0, listed_m = 0;
    for (int j0 = 0; j0 < nb; j0 += 32) {
      const int j = j0 + lane;
      const int f = j < nb ? fine(j) : -1;
      const bool is_c = cc.list && f >= cc.t_lo && f <= cc.t_hi, is_m = cm.list && f >= cm.t_lo && f <= cm.t_hi;
      const unsigned b_c = __ballot_sync(0xFFFFFFFFu, is_c), b_m = __ballot_sync(0xFFFFFFFFu, is_m);
      if (is_c) idx_c[listed_c + __popc(b_c & below)] = static_cast<unsigned short>(j);
      if (is_m) idx_m[listed_m + __popc(b_m & below)] = static_cast<unsigned short>(j);
      listed_c += __popc(b_c);
      listed_m += __popc(b_m);
    }
    __syncwarp();
    if (cc.list)
      for (int c = lane; c < cc.size; c += 32) ckey_c[c] = exact_key(idx_c[c]);
    if (cm.list)
      for (int c = lane; c < cm.size; c += 32) ckey_m[c] = exact_key(idx_m[c]);
    __syncwarp();
  }
  auto finish = [&](Chosen& r, const unsigned long long* ckey) {
    if (r.list) {
      r.keys_from = 1;
      radix_select([&](int c, unsigned long long& key) {
        key = ckey[c];
        return true;
      }, r.size, r.remaining, hist, lane, r.s);
    } else if (r.keys_from == 2) {  // every pass recomputes the keys it looks at
      const int t_lo = r.t_lo, t_hi = r.t_hi;
      radix_select([&](int c, unsigned long long& key) {
        const int f = fine(c);
        if (f < t_lo || f > t_hi) return false;
        key = exact_key(c);
        return true;
      }, nb, r.remaining, hist, lane, r.s);
    }
  };
  finish(cc, ckey_c);
  finish(cm, ckey_m);
  const Selection sc = cc.s, sm = cm.s;
  const int from_c = cc.keys_from, from_m = cm.keys_from;

  // Phase C
  const size_t row = bh_rows + i;
  signed char* out_cls = cls + row * nb;
  int n_crit = 0, n_marg = 0, tie_c = 0, tie_m = 0, seen_c = 0, seen_m = 0;
  const unsigned below = (1u << lane) - 1u;
#pragma unroll 2
  for (int j0 = 0; j0 < nb; j0 += 32) {
    const int j = j0 + lane;
    const bool in = j < nb;
    const int f = in ? fine(j) : -2;
    bool sel_c = in && f > cc.t_hi, sel_m = in && f > cm.t_hi;
    const bool at_c = f >= cc.t_lo && f <= cc.t_hi, at_m = f >= cm.t_lo && f <= cm.t_hi;
    if (__any_sync(0xFFFFFFFFu, at_c || at_m)) {
      // the entries of a threshold bucket come by in the order in which the selection listed them
      const unsigned b_at_c = __ballot_sync(0xFFFFFFFFu, at_c), b_at_m = __ballot_sync(0xFFFFFFFFu, at_m);
      unsigned long long kc = 0ull, km = 0ull;
      if (at_c && from_c != 0) kc = (from_c == 1 ? ckey_c[seen_c + __popc(b_at_c & below)] : exact_key(j)) & sc.mask;
      if (at_m && from_m != 0) km = (from_m == 1 ? ckey_m[seen_m + __popc(b_at_m & below)] : exact_key(j)) & sm.mask;
      seen_c += __popc(b_at_c);
      seen_m += __popc(b_at_m);
      const bool eq_c = at_c && kc == sc.prefix, eq_m = at_m && km == sm.prefix;
      const unsigned b_eq_c = __ballot_sync(0xFFFFFFFFu, eq_c), b_eq_m = __ballot_sync(0xFFFFFFFFu, eq_m);
      sel_c = sel_c || (at_c && kc > sc.prefix) || (eq_c && tie_c + __popc(b_eq_c & below) < sc.take);
      sel_m = sel_m || (at_m && km > sm.prefix) || (eq_m && tie_m + __popc(b_eq_m & below) < sm.take);
      tie_c += __popc(b_eq_c);
      tie_m += __popc(b_eq_m);
    }
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

size_t plan_compact_smem_bytes(int nb, int rows) {
  const size_t pitch = static_cast<size_t>((nb + 3) & ~3);
  return rows * pitch * 4 + static_cast<size_t>(rows) * 2 * kBuckets * 4 + static_cast<size_t>(rows) * 2 * kMaxListed * 8 +
         static_cast<size_t>(rows) * kHeadDim * 4 + static_cast<size_t>(8) * rows * sizeof(float2) +
         static_cast<size_t>(rows) * 2 * kMaxListed * 2;
}

template <int R>
lite3r_status launch_compact(const lite3r_fp8& q, const lite3r_fp8& k, const lite3r_shape& s, const Counts& c,
                             const lite3r_plan& plan, int nb, cudaStream_t stream) {
  const size_t smem = plan_compact_smem_bytes(nb, R);
  lite3r_status st = ensure_dynamic_smem(plan_compact_kernel<R>, static_cast<int>(smem));
  if (st != LITE3R_OK) return st;
  const int row_tiles = ceil_div(nb, R);
  plan_compact_kernel<R><<<s.batch * s.heads * row_tiles, R * 32, smem, stream>>>(q.colsum, k.colsum, k.scales, s.tokens,
                                                                                   s.block, nb, c.k_crit, c.k_marg, c.k_neg,
                                                                                   plan.cls, plan.crit_idx, plan.marg_idx);
  return after_launch();
}

size_t plan_smem_bytes(int nb, int rows) {
  const size_t pitch = static_cast<size_t>((nb + 1) & ~1);
  const size_t common = rows * pitch * 8 + static_cast<size_t>(rows) * 2 * kBuckets * 4 +
                        static_cast<size_t>(rows) * 2 * kMaxListed * 2;  // keys, two histograms, two index lists
  // eight rows or more: score ranges and one bucket byte per key (the column sums come straight from global memory);
  // fewer rows: the staged column sums as doubles
  if (rows >= 8) return common + static_cast<size_t>(rows) * rows * sizeof(float2) + rows * pitch;
  return common + static_cast<size_t>(rows) * kPitch * 8 + static_cast<size_t>(kChunk) * kPitch * 8;
}

template <int R>
lite3r_status launch_rows(const lite3r_fp8& q, const lite3r_fp8& k, const lite3r_shape& s, const Counts& c,
                          const lite3r_plan& plan, int nb, cudaStream_t stream) {
  const size_t smem = plan_smem_bytes(nb, R);
  lite3r_status st = ensure_dynamic_smem(plan_kernel<R>, static_cast<int>(smem));
  if (st != LITE3R_OK) return st;
  const int row_tiles = ceil_div(nb, R);
  plan_kernel<R><<<s.batch * s.heads * row_tiles, R * 32, smem, stream>>>(q.colsum, k.colsum, k.scales, s.tokens,
                                                                           s.block, nb, c.k_crit, c.k_marg, c.k_neg,
                                                                           plan.cls, plan.crit_idx, plan.marg_idx);
  return after_launch();
}

}  // namespace

// Test hook: which kernel launch_plan takes (0 = by size, as described there).
static std::atomic<int> g_plan_variant{0};
void set_plan_variant(int variant) { g_plan_variant.store(variant, std::memory_order_relaxed); }

lite3r_status launch_plan(const lite3r_fp8& q, const lite3r_fp8& k, const lite3r_shape& s, const Counts& c,
                          const lite3r_plan& plan, cudaStream_t stream) {
  const int nb = ceil_div(s.tokens, s.block);
  constexpr size_t kLimit = 227 * 1024;
  switch (g_plan_variant.load(std::memory_order_relaxed)) {  // forced by a test; sizes that do not fit are refused
    case 1: return plan_smem_bytes(nb, 8) <= kLimit ? launch_rows<8>(q, k, s, c, plan, nb, stream) : LITE3R_ERR_UNSUPPORTED;
    case 2: return plan_compact_smem_bytes(nb, 8) <= kLimit && nb <= 65536 ? launch_compact<8>(q, k, s, c, plan, nb, stream) : LITE3R_ERR_UNSUPPORTED;
    case 3: return plan_compact_smem_bytes(nb, 16) <= kLimit && nb <= 65536 ? launch_compact<16>(q, k, s, c, plan, nb, stream) : LITE3R_ERR_UNSUPPORTED;
    case 4: return plan_smem_bytes(nb, 4) <= kLimit ? launch_rows<4>(q, k, s, c, plan, nb, stream) : LITE3R_ERR_UNSUPPORTED;
    default: break;
  }
  // Long rows (where the 8-byte keys of eight rows would leave room for a single CTA per SM): single-precision scores in
  // shared memory, sixteen rows per CTA when that still leaves every SM several CTAs to work on, else eight (index
  // lists hold 16-bit positions: rows of up to 65536 blocks).
  int sms = 0;
  lite3r_status st = sm_count(&sms);
  if (st != LITE3R_OK) return st;
  if (plan_smem_bytes(nb, 8) > kLimit / 2 && nb <= 65536) {
    const long long ctas16 = static_cast<long long>(s.batch) * s.heads * ceil_div(nb, 16);
    if (ctas16 >= 4ll * sms && plan_compact_smem_bytes(nb, 16) <= kLimit) return launch_compact<16>(q, k, s, c, plan, nb, stream);
    if (plan_compact_smem_bytes(nb, 8) <= kLimit) return launch_compact<8>(q, k, s, c, plan, nb, stream);
  }
  // As many rows per CTA as the row keys allow: the staged key blocks are then shared by more rows.
  if (plan_smem_bytes(nb, 8) <= kLimit) return launch_rows<8>(q, k, s, c, plan, nb, stream);
  if (plan_smem_bytes(nb, 4) <= kLimit) return launch_rows<4>(q, k, s, c, plan, nb, stream);
  if (plan_smem_bytes(nb, 2) <= kLimit) return launch_rows<2>(q, k, s, c, plan, nb, stream);
  if (plan_smem_bytes(nb, 1) <= kLimit) return launch_rows<1>(q, k, s, c, plan, nb, stream);
  return LITE3R_ERR_UNSUPPORTED;  // more than ~24000 blocks per sequence
}

}  // namespace lite3r
