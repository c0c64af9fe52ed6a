// Algorithm 1 ("Context Allocation") on the device, as ONE cooperative kernel whose CTAs
// meet at grid barriers between the phases:
//
//   A  A^C[t] = exp2(max_r log2 p_rt) from the scores pass' encoded maxima (Eq. 5);
//   B  MaxPooling(size = stride = m), once per distinct m, then the stride-1 window pooling
//      (average or max) of every (m, n) combination, and a histogram of the top 11 bits of
//      the 64-bit key (pooled value, then lower cell index first);
//   C  every CTA finds, for the combinations it scans, the histogram bin that holds the
//      K_m-th largest key;
//   D  one scan gathers the candidates: cells above that bin, the bin's cells too when all of
//      them are wanted; otherwise the bin's cells (at most kPendCap) are set aside and one CTA
//      per combination picks the wanted number of highest keys among them with a radix select
//      over the remaining 53 bits in shared memory.  Only a plateau of more than kPendCap
//      cells in the bin (exactly equal pooled values, mostly) takes the long way: two more
//      histogram passes over the array, then the ties in cell order (the tiles are in cell
//      order, so a count of the holders per tile plus an ordered rank inside the tile settle
//      which cells win);
//   E  ranking (value descending, cell ascending) by counting, spread over the grid;
//   F  one CTA walks the combinations in loop order: maps cells back to tokens, skips tokens
//      already allocated, stops each combination at its quota B_c, then writes the allocated
//      positions in ascending order.
//
// Work of phases B-D is cut into tiles of kSelTile cells of one combination; every CTA owns a
// contiguous run of tiles, the same in every phase.
#include "select_kernels.cuh"
#include "sm100_ptx.cuh"

namespace ilre {

__device__ __forceinline__ unsigned long long make_key(float w, uint32_t cell) {
  return (static_cast<unsigned long long>(float_to_ordered(w)) << 32) | (0xFFFFFFFFu - cell);
}

__device__ __forceinline__ void pass_bits(int pass, int& shift, int& bits) {
  const int sh[kSelectPasses] = {53, 42, 32};
  const int bt[kSelectPasses] = {11, 11, 10};
  shift = sh[pass];
  bits = bt[pass];
}

struct SelShared {
  uint32_t hist[kHistBins];
  uint32_t scan[33];
  int flag;
  unsigned long long prefix[kMaxCombos];   // per combination: radix prefix found so far
  uint32_t state[kMaxCombos];              // per combination: threshold settled / candidate count
  uint32_t krem[kMaxCombos];               // per combination: keys still wanted inside the prefix
  uint8_t mode[kMaxCombos];                // per combination, after the first pass: 0 settled,
                                           // 1 threshold bin handed to one CTA, 2 full-scan passes
  uint32_t tot[2][32];                     // warp totals of the one-barrier block scan
};

// Grid-wide barrier (all CTAs are co-resident: cooperative launch).  The arrival counter is
// zero when the kernel starts and only grows: the k-th barrier completes when it reaches
// k * gridDim.x.  One thread per CTA arrives with a release at device scope (cumulative over the
// CTA's writes, which the block barrier before it orders) and polls with acquire loads; no
// value comes back from the arrival, so a barrier costs one trip to the L2 instead of two.
// The wait is bounded; a CTA that gives up records it and leaves the kernel.
// kCluster: the whole grid is one thread-block cluster (short contexts): the hardware cluster
// barrier takes the place of the counter, with release / acquire ordering at cluster scope.
template <bool kCluster>
__device__ __forceinline__ bool grid_sync(const SelectParams& p, SelShared* sh, uint32_t& epoch) {
  if constexpr (kCluster) {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
    return true;
  }
  ++epoch;
  __syncthreads();
  if (threadIdx.x == 0) {
    int ok = 1;
    const uint32_t target = epoch * (gridDim.x + static_cast<uint32_t>(p.barrier_extra));
    asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(p.barrier) : "memory");
    const long long t0 = clock64();
    for (uint32_t it = 1;; ++it) {
      uint32_t arrived;
      asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(arrived) : "l"(p.barrier) : "memory");
      if (arrived >= target) break;
      if ((it & 0xFF) == 0 && clock64() - t0 > p.wait_limit) {
        atomicCAS(p.status, 0, kDevGridBarrier);
        ok = 0;
        break;
      }
    }
    sh->flag = ok;
  }
  __syncthreads();
  return sh->flag != 0;
}

// Exclusive prefix sum over the block of kSelThreads threads; *total receives the block sum.
__device__ __forceinline__ uint32_t block_exclusive_scan(uint32_t v, uint32_t* sh_warp,
                                                         uint32_t* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
    if (lane >= o) incl += t;
  }
  __syncthreads();                       // protects sh_warp from the previous call's readers
  if (lane == 31) sh_warp[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    uint32_t w = sh_warp[lane];
    uint32_t wi = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, wi, o);
      if (lane >= o) wi += t;
    }
    sh_warp[lane] = wi - w;              // exclusive warp offsets
    if (lane == 31) sh_warp[32] = wi;    // grand total
  }
  __syncthreads();
  *total = sh_warp[32];
  return sh_warp[warp] + incl - v;
}

// Adds one digit per thread (0xFFFFFFFF = none) to the shared histogram, one atomic per
// distinct digit of the warp: plateaus of equal pooled values are the common case.
__device__ __forceinline__ void hist_add(uint32_t* hist, uint32_t digit) {
  if (!__any_sync(0xFFFFFFFFu, digit != 0xFFFFFFFFu)) return;
  const uint32_t peers = __match_any_sync(0xFFFFFFFFu, digit);
  if (digit != 0xFFFFFFFFu && (threadIdx.x & 31) == __ffs(peers) - 1)
    atomicAdd(&hist[digit], __popc(peers));
}

__device__ __forceinline__ void hist_flush(uint32_t* sh_hist, uint32_t* gh) {
  __syncthreads();
  for (int b = threadIdx.x; b < kHistBins; b += kSelThreads) {
    const uint32_t v = sh_hist[b];
    if (v) { atomicAdd(&gh[b], v); sh_hist[b] = 0u; }
  }
  __syncthreads();
}

// Combination that owns `tile`.  Tiles are visited in increasing order, so the search resumes
// from the previous answer (`cur`, 0 at first).
__device__ __forceinline__ int combo_of_tile(const ComboTable& tbl, int tile, int& cur) {
  while (cur + 1 < tbl.n_comb && tile >= tbl.tile_begin[cur + 1]) ++cur;
  return cur;
}

static constexpr int kTilePer = kSelTile / kSelThreads;
static constexpr int kMaxWalkWarps = kSelThreads / 32;
static constexpr int kScanGroup = 4;      // tiles whose loads are issued together

// Pooled values of one tile, kTilePer per thread, all loads in flight together.
__device__ __forceinline__ void fetch_tile(const ComboTable& tbl, const SelectParams& p, int tile,
                                           int& cur, const uint32_t* skip, float (&wv)[kTilePer]) {
  const int combo = combo_of_tile(tbl, tile, cur);
  if (skip && skip[combo]) return;
  const float* w = p.pooled + static_cast<long long>(combo) * p.pooled_stride;
  const int c0 = (tile - tbl.tile_begin[combo]) * kSelTile;
  const int c1 = min(tbl.len[combo], c0 + kSelTile);
#pragma unroll
  for (int k = 0; k < kTilePer; ++k) {
    const int c = c0 + k * kSelThreads + threadIdx.x;
    wv[k] = (c < c1) ? __ldcg(&w[c]) : 0.f;
  }
}

// Phase B1 for one tile of source `src`: cells of MaxPooling(size = stride = m), a shorter
// last cell where m does not divide the length.  The tokens are read coalesced into `buf`
// (kSrcTileTokens floats), all loads in flight together.
__device__ __forceinline__ void maxpool_tile(const ComboTable& tbl, const SelectParams& p, int src,
                                             int tile_in_src, float* buf) {
  const int m = tbl.src_m[src], len = tbl.src_len[src];
  const long long Lp = p.L - p.n_sink;
  const float* a = p.scores + p.n_sink;
  const int cells_per_tile = kSrcTileTokens / m;
  const int c0 = tile_in_src * cells_per_tile;
  const int n_cells = min(cells_per_tile, len - c0);
  const long long t0 = static_cast<long long>(c0) * m;
  const int n_tok = static_cast<int>(min(static_cast<long long>(n_cells) * m, Lp - t0));
  constexpr int kLd = kSrcTileTokens / kSelThreads;
  float v[kLd];
#pragma unroll
  for (int k = 0; k < kLd; ++k) {
    const int i = k * kSelThreads + threadIdx.x;
    v[k] = (i < n_tok) ? __ldcg(a + t0 + i) : -INFINITY;
  }
#pragma unroll
  for (int k = 0; k < kLd; ++k) buf[k * kSelThreads + threadIdx.x] = v[k];
  __syncthreads();
  float* out = p.maxpooled + static_cast<long long>(src) * p.maxpooled_stride;
  for (int c = threadIdx.x; c < n_cells; c += kSelThreads) {
    float acc = buf[c * m];
    for (int j = 1; j < m; ++j) acc = fmaxf(acc, buf[c * m + j]);
    out[c0 + c] = acc;
  }
  __syncthreads();
}

// Phase B2 for one tile: pooled cells [c0, c0 + n_out) of `combo` from its max-pooled source
// (the scores themselves for m = 1), written to p.pooled; the first-pass radix digit of every
// cell goes to the shared histogram.  `buf0`/`buf1` hold kSelTile + kMaxWin floats each.
__device__ __forceinline__ void pool_tile(const ComboTable& tbl, const SelectParams& p, int combo,
                                          int c0, float* buf0, float* buf1, uint32_t* sh_hist) {
  const int n = tbl.n[combo], len = tbl.len[combo];
  const int source = tbl.src[combo];
  const float* a = (source < 0)
      ? p.scores + p.n_sink
      : p.maxpooled + static_cast<long long>(source) * p.maxpooled_stride;
  const int lo = c0 - n / 2;
  const int n_out = min(kSelTile, len - c0);
  const int span = n_out + n - 1;
  const float pad = (p.win_op == 0) ? 0.f : -INFINITY;
  {
    constexpr int kLd = (kSelTile + kMaxWin + kSelThreads - 1) / kSelThreads;
    float v[kLd];
#pragma unroll
    for (int k = 0; k < kLd; ++k) {
      const int idx = k * kSelThreads + threadIdx.x, u = lo + idx;
      v[k] = (idx < span && u >= 0 && u < len) ? __ldcg(a + u) : pad;
    }
#pragma unroll
    for (int k = 0; k < kLd; ++k) {
      const int idx = k * kSelThreads + threadIdx.x;
      if (idx < span) buf0[idx] = v[k];
    }
  }
  __syncthreads();
  // Window maximum by doubling: after the step of width w, src[i] = max of cells [i, i + w);
  // a window of n cells is then the maximum of two overlapping runs of width w <= n < 2w.
  float* src = buf0;
  int w = 1;
  if (p.win_op != 0) {
    float* dst = buf1;
    while (2 * w <= n) {
      const int cnt = span - 2 * w + 1;
      for (int i = threadIdx.x; i < cnt; i += kSelThreads) dst[i] = fmaxf(src[i], src[i + w]);
      __syncthreads();
      float* t = src; src = dst; dst = t;
      w *= 2;
    }
  }
  float* out = p.pooled + static_cast<long long>(combo) * p.pooled_stride;
  for (int base = 0; base < n_out; base += kSelThreads) {
    const int i = base + threadIdx.x;
    uint32_t digit = 0xFFFFFFFFu;
    if (i < n_out) {
      float acc;
      if (p.win_op == 0) {
        acc = 0.f;
        for (int j = 0; j < n; ++j) acc += src[i + j];       // left to right, as the definition
        acc = acc / static_cast<float>(n);
      } else {
        acc = fmaxf(src[i], src[i + n - w]);
      }
      out[c0 + i] = acc;
      digit = static_cast<uint32_t>(make_key(acc, static_cast<uint32_t>(c0 + i)) >> 53);
    }
    hist_add(sh_hist, digit);
  }
  __syncthreads();
}

// Locates the bin of pass `pass` that holds the k-th largest key of `combo` among those that
// match the prefix so far and extends the prefix.  Every CTA does this for the combinations
// whose tiles it scans, from the same global histogram, so all of them reach the same answer.
// The state lives in shared memory.  A combination is settled (state = 1) when every key of
// the chosen bin is wanted: then "key >= prefix" selects exactly K_m keys.
__device__ __forceinline__ void bin_search(const SelectParams& p, int n_comb, int combo, int pass,
                                           SelShared* sh) {
  int shift, bits;
  pass_bits(pass, shift, bits);
  const uint32_t* gh = p.hist + (static_cast<long long>(pass) * n_comb + combo) * kHistBins;
  const unsigned long long prefix = sh->prefix[combo];
  const uint32_t k_rem = sh->krem[combo];
  constexpr int kPer = kHistBins / kSelThreads;
  uint32_t h[kPer];
  uint32_t total = 0;
#pragma unroll
  for (int j = 0; j < kPer; ++j) {
    h[j] = __ldcg(&gh[kHistBins - 1 - (kPer * threadIdx.x + j)]);   // bins in descending order
    total += h[j];
  }
  uint32_t grand;
  const uint32_t excl = block_exclusive_scan(total, sh->scan, &grand);   // ends with a barrier
  if (excl < k_rem && k_rem <= excl + total) {
    uint32_t cum = excl;
#pragma unroll
    for (int j = 0; j < kPer; ++j) {
      if (k_rem > cum && k_rem <= cum + h[j]) {
        const uint32_t bin = kHistBins - 1 - (kPer * threadIdx.x + j);
        const uint32_t new_k = k_rem - cum;
        sh->prefix[combo] = prefix | (static_cast<unsigned long long>(bin) << shift);
        sh->krem[combo] = new_k;
        sh->state[combo] = (h[j] == new_k) ? 1u : 0u;
        if (pass == 0 && h[j] != new_k) {
          // The threshold bin holds more cells than are wanted from it.  Few enough: they are
          // set aside during the gather and one CTA picks the new_k highest of them; too many
          // (a plateau across the bin): the remaining passes scan the whole array.
          if (h[j] <= static_cast<uint32_t>(kPendCap)) {
            sh->mode[combo] = 1;
            p.cand_count[2 * kMaxCombos + combo] = new_k;
          } else {
            sh->mode[combo] = 2;
            p.cand_count[3 * kMaxCombos] = 1u;
          }
        }
      }
      cum += h[j];
    }
  }
  if (threadIdx.x == 0 && (k_rem > grand || k_rem == 0))
    sh->state[combo] = 1u;                                 // fewer keys than asked: take all
  __syncthreads();
}

// Phase E: ranks the candidates [lo, hi) of `combo` among all of its n candidates by counting
// the keys above each (keys are distinct).
//
// Lists of kRankBucketMin..kRankChunk keys are first split into kRankBuckets value ranges, so
// that a candidate is compared with its own range only: kRankSamples keys taken at even
// strides are ranked among themselves, every fourth of them becomes a splitter, every key of
// the list goes to the bucket "number of splitters above it" (bucket 0 holds the largest
// keys) and is stored bucket by bucket in shared memory.  rank = keys in the buckets before
// + keys above inside the bucket.  The result does not depend on which keys were sampled,
// only the work per candidate does; every CTA samples for itself.
//
// Other lists take the plain form: the keys are staged in shared memory (at most kRankChunk
// at a time), a thread owns one candidate and one slice of the keys, the threads of a warp
// share the slice, so every key is one broadcast read for 32 comparisons; the slices' counts
// meet in shared-memory counters.
static constexpr int kRankChunk = 8192;
static constexpr int kRankSamples = 128;
static constexpr int kRankBuckets = 32;
static constexpr int kRankBucketMin = 1024;

struct RankScratch {
  unsigned long long samp[kRankSamples];
  unsigned long long spl[kRankBuckets];    // splitters, descending; the last entry is unused
  uint32_t srank[kRankSamples];
  uint32_t count[kRankBuckets];
  uint32_t start[kRankBuckets + 1];
};

// Number of splitters above `key`.
__device__ __forceinline__ int rank_bucket(const unsigned long long* spl, unsigned long long key) {
  int b = 0;
#pragma unroll
  for (int step = kRankBuckets / 2; step >= 1; step >>= 1)
    if (spl[b + step - 1] > key) b += step;
  return b;
}

__device__ __forceinline__ void rank_range_bucketed(const unsigned long long* cand, int* ranked, int n,
                                                    int lo, int hi, unsigned long long* grouped,
                                                    RankScratch* rs) {
  constexpr int kLd = kRankChunk / kSelThreads;
  const int tid = threadIdx.x;
  unsigned long long v[kLd];
#pragma unroll
  for (int k = 0; k < kLd; ++k) {
    const int i = k * kSelThreads + tid;
    v[k] = (i < n) ? __ldcg(&cand[i]) : 0ull;
  }
  __syncthreads();                                          // previous users of rs / grouped
  if (tid < kRankSamples) {
    rs->samp[tid] = __ldcg(&cand[static_cast<int>((static_cast<long long>(tid) * n) / kRankSamples)]);
    rs->srank[tid] = 0;
  }
  if (tid < kRankBuckets) rs->count[tid] = 0;
  __syncthreads();
  {                                                         // rank the samples among themselves
    constexpr int kPer = kRankSamples / (kSelThreads / kRankSamples);
    const int si = tid % kRankSamples, j0 = (tid / kRankSamples) * kPer;
    const unsigned long long mine = rs->samp[si];
    uint32_t above = 0;
#pragma unroll
    for (int j = 0; j < kPer; ++j) above += (rs->samp[j0 + j] > mine) ? 1u : 0u;
    if (above) atomicAdd(&rs->srank[si], above);
  }
  __syncthreads();
  if (tid < kRankSamples) {
    const uint32_t r = rs->srank[tid];
    if ((r & 3u) == 3u) rs->spl[r >> 2] = rs->samp[tid];
  }
  __syncthreads();
  uint32_t where[kLd];                                      // bucket << 16 | slot inside the bucket
#pragma unroll
  for (int k = 0; k < kLd; ++k) {
    const int i = k * kSelThreads + tid;
    if (i < n) {
      const int b = rank_bucket(rs->spl, v[k]);
      where[k] = (static_cast<uint32_t>(b) << 16) | atomicAdd(&rs->count[b], 1u);
    }
  }
  __syncthreads();
  if (tid < 32) {
    const uint32_t c = rs->count[tid];
    uint32_t incl = c;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const uint32_t o = __shfl_up_sync(0xFFFFFFFFu, incl, d);
      if (tid >= d) incl += o;
    }
    rs->start[tid] = incl - c;
    if (tid == 31) rs->start[32] = incl;
  }
  __syncthreads();
#pragma unroll
  for (int k = 0; k < kLd; ++k) {
    const int i = k * kSelThreads + tid;
    if (i < n) grouped[rs->start[where[k] >> 16] + (where[k] & 0xFFFFu)] = v[k];
  }
  __syncthreads();
  for (int c0 = lo; c0 < hi; c0 += kSelThreads) {
    const int nc = min(kSelThreads, hi - c0);
    int g = 1;                                              // threads per candidate
    while (g < 32 && 2 * g * nc <= kSelThreads) g <<= 1;
    const int local = tid / g, sub = tid % g;
    const bool active = local < nc;
    const unsigned long long key = active ? __ldcg(&cand[c0 + local]) : ~0ull;
    int j = 0, j1 = 0, first = 0;
    if (active) {
      const int b = rank_bucket(rs->spl, key);
      first = static_cast<int>(rs->start[b]);
      j = first + sub;
      j1 = static_cast<int>(rs->start[b + 1]);
    }
    int above = 0;
    for (; j < j1; j += g) above += (grouped[j] > key) ? 1 : 0;
    for (int d = 1; d < g; d <<= 1) above += __shfl_xor_sync(0xFFFFFFFFu, above, d);
    if (active && sub == 0)
      ranked[first + above] = static_cast<int>(0xFFFFFFFFu - static_cast<uint32_t>(key & 0xFFFFFFFFull));
  }
}

__device__ __forceinline__ void rank_range(const SelectParams& p, int combo, int n, int lo, int hi,
                                           unsigned long long* chunk, int* count_s, RankScratch* rs) {
  const unsigned long long* cand = p.cand + static_cast<long long>(combo) * p.cand_stride;
  int* ranked = p.ranked + static_cast<long long>(combo) * p.cand_stride;
  if (n >= kRankBucketMin && n <= kRankChunk) {
    rank_range_bucketed(cand, ranked, n, lo, hi, chunk, rs);
    return;
  }
  for (int c0 = lo; c0 < hi; c0 += kSelThreads) {
    const int nc = min(kSelThreads, hi - c0);               // candidates of this round
    const int cpad = (nc + 31) & ~31;
    const int n_slices = kSelThreads / cpad;                // >= 1; whole warps per slice
    const int local = threadIdx.x % cpad, slice = threadIdx.x / cpad;
    const bool active = slice < n_slices && local < nc;
    const unsigned long long key = active ? __ldcg(&cand[c0 + local]) : ~0ull;
    __syncthreads();                                        // previous users of count_s / chunk
    if (threadIdx.x < cpad) count_s[threadIdx.x] = 0;
    int above = 0;
    for (int base = 0; base < n; base += kRankChunk) {
      const int cnt = min(kRankChunk, n - base);
      if (base > 0) __syncthreads();
      constexpr int kLd = kRankChunk / kSelThreads;         // all loads in flight together
      unsigned long long v[kLd];
#pragma unroll
      for (int k = 0; k < kLd; ++k) {
        const int i = k * kSelThreads + threadIdx.x;
        v[k] = (i < cnt) ? __ldcg(&cand[base + i]) : 0ull;
      }
#pragma unroll
      for (int k = 0; k < kLd; ++k) {
        const int i = k * kSelThreads + threadIdx.x;
        if (i < cnt) chunk[i] = v[k];
      }
      __syncthreads();
      const int per = (cnt + n_slices - 1) / n_slices;
      const int j0 = min(cnt, slice * per), j1 = min(cnt, j0 + per);
      if (slice < n_slices) {                               // warp-uniform
        int j = j0;
        for (; j + 4 <= j1; j += 4) {
          above += (chunk[j] > key) ? 1 : 0;
          above += (chunk[j + 1] > key) ? 1 : 0;
          above += (chunk[j + 2] > key) ? 1 : 0;
          above += (chunk[j + 3] > key) ? 1 : 0;
        }
        for (; j < j1; ++j) above += (chunk[j] > key) ? 1 : 0;
      }
    }
    if (active && above) atomicAdd(&count_s[local], above);
    __syncthreads();
    if (threadIdx.x < nc)                                   // slice 0 holds candidate c0 + threadIdx.x
      ranked[count_s[threadIdx.x]] = static_cast<int>(0xFFFFFFFFu - static_cast<uint32_t>(key & 0xFFFFFFFFull));
  }
}

// One CTA picks the `wanted` highest of the n_p keys that the gather set aside for `combo`
// (all of them share the top 11 bits) and appends them to the combination's candidates.
// Radix select over the remaining 53 bits, 11/10/11/11/10 per pass, histograms in shared memory.
__device__ __forceinline__ void resolve_pending(const SelectParams& p, const ComboTable& tbl,
                                                int combo, int n_p, SelShared* sh) {
  constexpr int kPer = kPendCap / kSelThreads;
  const unsigned long long* pend = p.pending + static_cast<long long>(combo) * kPendCap;
  unsigned long long* cand = p.cand + static_cast<long long>(combo) * p.cand_stride;
  const uint32_t wanted = __ldcg(&p.cand_count[2 * kMaxCombos + combo]);
  const uint32_t base = __ldcg(&p.cand_count[combo]);
  __shared__ unsigned long long s_prefix;
  __shared__ uint32_t s_krem, s_slot;
  __shared__ int s_done;
  unsigned long long key[kPer];
#pragma unroll
  for (int j = 0; j < kPer; ++j) {
    const int i = j * kSelThreads + threadIdx.x;
    key[j] = (i < n_p) ? __ldcg(&pend[i]) : 0ull;
  }
  __syncthreads();                                         // earlier users of the shared words are done
  if (threadIdx.x == 0) {
    s_prefix = (key[0] >> 53) << 53;                       // thread 0 holds key 0 (n_p >= 1)
    s_krem = wanted;
    s_done = (wanted >= static_cast<uint32_t>(n_p)) || wanted == 0u;
    s_slot = 0u;
  }
  for (int b = threadIdx.x; b < kHistBins; b += kSelThreads) sh->hist[b] = 0u;
  __syncthreads();
  const int shifts[5] = {42, 32, 21, 10, 0};
  const int widths[5] = {11, 10, 11, 11, 10};
  for (int pass = 0; pass < 5; ++pass) {
    if (s_done) break;                                     // uniform: read after a barrier
    const int shift = shifts[pass], bits = widths[pass];
    const unsigned long long prefix = s_prefix;
    const uint32_t k_rem = s_krem;
#pragma unroll
    for (int j = 0; j < kPer; ++j) {
      if (j * kSelThreads >= n_p) break;                   // uniform
      const int i = j * kSelThreads + threadIdx.x;
      uint32_t digit = 0xFFFFFFFFu;
      if (i < n_p && ((key[j] ^ prefix) >> (shift + bits)) == 0ull)
        digit = static_cast<uint32_t>(key[j] >> shift) & ((1u << bits) - 1u);
      hist_add(sh->hist, digit);
    }
    __syncthreads();
    const uint32_t h0 = sh->hist[kHistBins - 1 - 2 * threadIdx.x];   // bins in descending order
    const uint32_t h1 = sh->hist[kHistBins - 2 - 2 * threadIdx.x];
    uint32_t total;
    const uint32_t excl = block_exclusive_scan(h0 + h1, sh->scan, &total);
    sh->hist[kHistBins - 1 - 2 * threadIdx.x] = 0u;
    sh->hist[kHistBins - 2 - 2 * threadIdx.x] = 0u;
    if (k_rem > excl && k_rem <= excl + h0 + h1) {
      const bool first = k_rem <= excl + h0;
      const uint32_t bin = first ? kHistBins - 1 - 2 * threadIdx.x : kHistBins - 2 - 2 * threadIdx.x;
      const uint32_t above = first ? excl : excl + h0;
      const uint32_t cnt = first ? h0 : h1;
      s_prefix = prefix | (static_cast<unsigned long long>(bin) << shift);
      s_krem = k_rem - above;
      s_done = (cnt == k_rem - above) || pass == 4;
    }
    __syncthreads();
  }
  // every key at or above the threshold is wanted: exactly `wanted` of them (keys are distinct)
  const unsigned long long threshold = (wanted >= static_cast<uint32_t>(n_p)) ? 0ull : s_prefix;
  const int lane = threadIdx.x & 31;
#pragma unroll
  for (int j = 0; j < kPer; ++j) {
    if (j * kSelThreads >= n_p) break;                     // uniform
    const int i = j * kSelThreads + threadIdx.x;
    const bool take = wanted != 0u && i < n_p && key[j] >= threshold;
    const uint32_t votes = __ballot_sync(0xFFFFFFFFu, take);
    if (votes) {
      uint32_t slot = 0;
      if (lane == __ffs(votes) - 1) slot = atomicAdd(&s_slot, __popc(votes));
      slot = base + __shfl_sync(0xFFFFFFFFu, slot, __ffs(votes) - 1) + __popc(votes & ((1u << lane) - 1u));
      if (take && slot < static_cast<uint32_t>(tbl.k_m[combo])) cand[slot] = key[j];
    }
  }
  __syncthreads();
  if (threadIdx.x == 0) p.cand_count[combo] = base + s_slot;
  __syncthreads();
}

// Bitmap word access of the quota walk.  The bitmap lives in shared memory on the common path;
// naming the address space spares the generic-address forms.
template <bool kSmem>
__device__ __forceinline__ uint32_t bitmap_word(const uint32_t* bm, int w) {
  if constexpr (kSmem) {
    uint32_t v;
    asm volatile("ld.volatile.shared.u32 %0, [%1];" : "=r"(v) : "r"(smem_u32(bm + w)) : "memory");
    return v;
  } else {
    return *reinterpret_cast<const volatile uint32_t*>(bm + w);
  }
}
template <bool kSmem>
__device__ __forceinline__ void bitmap_set(uint32_t* bm, int w, uint32_t bits) {
  if constexpr (kSmem) {
    asm volatile("red.shared.or.b32 [%0], %1;" ::"r"(smem_u32(bm + w)), "r"(bits) : "memory");
  } else {
    atomicOr(bm + w, bits);
  }
}

// Tokens of cell `cell` (size m) that are not allocated yet, as a bit mask (bit j = token j).
// Positions fit 32 bits (L < 2^31).
template <bool kSmem>
__device__ __forceinline__ unsigned long long fresh_tokens(const uint32_t* bm, int cell, int m,
                                                           int Lp, int n_sink) {
  if (m == 1) {
    const int pos = n_sink + cell;
    return ((bitmap_word<kSmem>(bm, pos >> 5) >> (pos & 31)) & 1u) ^ 1u;
  }
  const int t0 = cell * m;
  const int cnt = min(m, Lp - t0);
  const int pos0 = n_sink + t0;
  const int w0 = pos0 >> 5, sh = pos0 & 31;
  if (m <= 32) {
    // at most 32 consecutive bits: two bitmap words, one funnel shift (the bitmap has
    // ceil(L / 32) words; a word past its end is not read)
    const uint32_t lo = bitmap_word<kSmem>(bm, w0);
    const uint32_t hi = (sh + cnt > 32) ? bitmap_word<kSmem>(bm, w0 + 1) : 0u;
    const uint32_t taken32 = __funnelshift_r(lo, hi, sh);
    const uint32_t mask32 = (cnt >= 32) ? 0xFFFFFFFFu : ((1u << cnt) - 1u);
    return static_cast<unsigned long long>(~taken32 & mask32);
  }
  // up to 64 consecutive bits sit in at most three bitmap words
  const int last_w = (pos0 + cnt - 1) >> 5;
  unsigned long long taken = bitmap_word<kSmem>(bm, w0);
  if (last_w > w0) taken |= static_cast<unsigned long long>(bitmap_word<kSmem>(bm, w0 + 1)) << 32;
  taken >>= sh;
  if (last_w > w0 + 1)                                    // only with sh > 0 and cnt > 64 - sh
    taken |= static_cast<unsigned long long>(bitmap_word<kSmem>(bm, w0 + 2)) << (64 - sh);
  const unsigned long long mask = (cnt >= 64) ? ~0ull : ((1ull << cnt) - 1ull);
  return ~taken & mask;
}

// Exclusive prefix sum over the block with a single barrier: every warp scans the 32 warp
// totals itself.  `slot` alternates between calls (two buffers), which keeps a call's readers
// apart from the next call's writers.
__device__ __forceinline__ uint32_t block_exclusive_scan_1(uint32_t v, uint32_t (*tot)[32],
                                                           int slot, uint32_t* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
    if (lane >= o) incl += t;
  }
  if (lane == 31) tot[slot][warp] = incl;
  __syncthreads();
  const uint32_t w = tot[slot][lane];
  uint32_t wi = w;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, wi, o);
    if (lane >= o) wi += t;
  }
  *total = __shfl_sync(0xFFFFFFFFu, wi, 31);
  return __shfl_sync(0xFFFFFFFFu, wi - w, warp) + incl - v;
}

// Phase F (one CTA): quota walk over the ranked cells of every combination, then the
// ascending list of allocated positions.  The bitmap lives in shared memory when it fits,
// else in global memory.  Every thread owns a run of consecutive ranks; the cells of one combination are disjoint, so the new-token counts of all its cells
// can be taken before any of them is marked.
template <bool kBitmapInSmem>
__device__ __forceinline__ void allocate(const ComboTable& tbl, const SelectParams& p,
                                         uint8_t* dyn_smem, SelShared* sh) {
  // Two instantiations, so that the compiler knows the bitmap's address space on the common
  // path (shared memory) instead of going through generic loads and atomics.
  uint32_t* bm;
  int* staged;
  if constexpr (kBitmapInSmem) {
    bm = reinterpret_cast<uint32_t*>(dyn_smem);
    staged = reinterpret_cast<int*>(dyn_smem + ((((p.L + 31) / 32) * 4 + 15) & ~15ll));
  } else {
    bm = p.bitmap;
    staged = reinterpret_cast<int*>(dyn_smem);
  }
  __shared__ uint32_t warp_totals[2][kMaxWalkWarps];
  const int n_walk = p.walk_threads;                       // multiple of 32, <= kSelThreads
  const int Lp = static_cast<int>(p.L - p.n_sink);
  for (int combo = threadIdx.x; combo < tbl.n_comb; combo += kSelThreads)
    sh->state[combo] = __ldcg(&p.cand_count[combo]);
  __syncthreads();
  // The walk is a chain of short dependent steps per combination, so what it costs is the
  // number of warps that have to issue them: walk_threads threads walk (about two ranked
  // cells each for the longest list, at least 256), the others wait for the output pass.  The ranked cells of a combination reach shared memory by 16-byte
  // asynchronous copies, one combination ahead when two staging buffers fit.
  if (static_cast<int>(threadIdx.x) < n_walk) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    auto walk_barrier = [&] { asm volatile("bar.sync 1, %0;" ::"r"(n_walk) : "memory"); };
    auto candidates = [&](int combo) {
      return min(static_cast<int>(min(sh->state[combo], static_cast<uint32_t>(kMaxKm))),
                 tbl.k_m[combo]);
    };
    const bool two = p.stage_double != 0;
    auto issue_copy = [&](int combo) {
      const int K = candidates(combo);
      const int* ranked = p.ranked + static_cast<long long>(combo) * p.cand_stride;
      int* dst = staged + ((two && (combo & 1)) ? p.stage_capacity : 0);
      for (int r = 4 * threadIdx.x; r < K; r += 4 * n_walk)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(dst + r)),
                     "l"(ranked + r) : "memory");
      asm volatile("cp.async.commit_group;" ::: "memory");
    };
    if (tbl.n_comb > 0) issue_copy(0);
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    walk_barrier();
    for (int combo = 0; combo < tbl.n_comb; ++combo) {
      const int m = tbl.m[combo];
      const uint32_t quota = static_cast<uint32_t>(tbl.quota[combo]);
      const int K = candidates(combo);
      const int* cells = staged + ((two && (combo & 1)) ? p.stage_capacity : 0);
      // the other buffer last served combination combo - 1, which every thread has left
      if (two && combo + 1 < tbl.n_comb) issue_copy(combo + 1);
      // thread t owns the ranks [t * per, (t + 1) * per)
      const int per = (K + n_walk - 1) / n_walk;
      const int r0 = min(K, static_cast<int>(threadIdx.x) * per), r1 = min(K, r0 + per);
      uint32_t mine = 0;
      int r = r0;
      for (; r + 4 <= r1; r += 4) {                            // four cells' loads in flight together
        const int c0 = cells[r], c1 = cells[r + 1], c2 = cells[r + 2], c3 = cells[r + 3];
        const unsigned long long f0 = fresh_tokens<kBitmapInSmem>(bm, c0, m, Lp, p.n_sink);
        const unsigned long long f1 = fresh_tokens<kBitmapInSmem>(bm, c1, m, Lp, p.n_sink);
        const unsigned long long f2 = fresh_tokens<kBitmapInSmem>(bm, c2, m, Lp, p.n_sink);
        const unsigned long long f3 = fresh_tokens<kBitmapInSmem>(bm, c3, m, Lp, p.n_sink);
        mine += __popcll(f0) + __popcll(f1) + __popcll(f2) + __popcll(f3);
      }
      for (; r < r1; ++r)
        mine += __popcll(fresh_tokens<kBitmapInSmem>(bm, cells[r], m, Lp, p.n_sink));
      // exclusive prefix over the walking threads: tokens that higher-ranked cells bring
      uint32_t incl = mine;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += t;
      }
      if (lane == 31) warp_totals[combo & 1][warp] = incl;
      walk_barrier();
      const uint32_t wt = (lane < n_walk / 32) ? warp_totals[combo & 1][lane] : 0u;
      uint32_t wi = wt;
#pragma unroll
      for (int o = 1; o < kMaxWalkWarps; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, wi, o);
        if (lane >= o) wi += t;
      }
      const uint32_t total = __shfl_sync(0xFFFFFFFFu, wi, 31);
      uint32_t ord = __shfl_sync(0xFFFFFFFFu, wi - wt, warp) + incl - mine;
      // accept in rank order while the quota lasts; inside a cell in ascending position; the
      // tokens of a cell are marked with one atomic per bitmap word (at most three words)
      for (r = r0; r < r1 && ord < quota; ++r) {
        const int cell = cells[r];
        unsigned long long f = fresh_tokens<kBitmapInSmem>(bm, cell, m, Lp, p.n_sink);
        if (f == 0ull) continue;
        uint32_t n_new = __popcll(f);
        if (ord + n_new > quota) {                             // the quota ends inside this cell
          unsigned long long kept = 0ull;
          for (uint32_t k = quota - ord; k > 0; --k) {
            const unsigned long long lowest = f & (0ull - f);
            kept |= lowest;
            f ^= lowest;
          }
          f = kept;
          n_new = quota - ord;
        }
        ord += n_new;
        const int pos0 = p.n_sink + cell * m;
        const int w0 = pos0 >> 5, sft = pos0 & 31;
        const unsigned long long shifted = f << sft;
        const uint32_t b0 = static_cast<uint32_t>(shifted), b1 = static_cast<uint32_t>(shifted >> 32);
        const uint32_t b2 = sft ? static_cast<uint32_t>(f >> (64 - sft)) : 0u;
        if (b0) bitmap_set<kBitmapInSmem>(bm, w0, b0);
        if (b1) bitmap_set<kBitmapInSmem>(bm, w0 + 1, b1);
        if (b2) bitmap_set<kBitmapInSmem>(bm, w0 + 2, b2);
      }
      if (total < quota && threadIdx.x == 0) atomicCAS(p.status, 0, kDevQuota);
      if (!two) {                                              // one buffer: copy only once it is free
        walk_barrier();
        if (combo + 1 < tbl.n_comb) issue_copy(combo + 1);
      }
      asm volatile("cp.async.wait_group 0;" ::: "memory");
      walk_barrier();                                          // bitmap updates and the next cells visible
    }
  }
  __syncthreads();

  // Ascending output.  One SM does this, so what counts is the number of instructions it has
  // to issue.  Up to kSelThreads bitmap words (32K positions) a thread takes one word.  Longer
  // contexts: the sink part is the identity; for the rest the bitmap is read four words per
  // lane and load (a warp owns a contiguous run of words), twice: to count the words that hold
  // an allocated position outside the sink part, then to list them in ascending order in
  // shared memory (where the staged cells were; they are done with).  There are at most
  // `budget` such words, usually a few hundred: the threads share them out evenly, take the
  // prefix of their position counts and write the positions.
  const long long n_words = (p.L + 31) / 32;
  const uint32_t cap = static_cast<uint32_t>(p.n_sink + p.budget);
  if (n_words <= kSelThreads) {
    // short context: a thread per bitmap word (sink bits included), one prefix sum
    uint32_t bits = (static_cast<long long>(threadIdx.x) < n_words)
                        ? bitmap_word<kBitmapInSmem>(bm, static_cast<int>(threadIdx.x)) : 0u;
    uint32_t total;
    uint32_t at = block_exclusive_scan(__popc(bits), sh->scan, &total);
    while (bits) {
      const int b = __ffs(bits) - 1;
      bits &= bits - 1;
      if (at < cap) p.out_idx[at] = static_cast<int>(threadIdx.x) * 32 + b;
      ++at;
    }
    if (threadIdx.x == 0 && total != cap) atomicCAS(p.status, 0, kDevQuota);
    return;
  }
  const int n_w = static_cast<int>(n_words);                // L < 2^31: word and quad numbers fit an int
  const int n_quads = (n_w + 3) / 4;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rounds = (n_quads + kSelThreads - 1) / kSelThreads;      // per warp
  const int q_begin = warp * rounds * 32;
  int* list = staged;
  // bits of word w that stand for allocated positions outside the sink part
  const int sink_words = p.n_sink >> 5;                     // words that lie in the sink part entirely
  const uint32_t sink_tail = ~((1u << (p.n_sink & 31)) - 1u);         // the word after them: its bits outside
  auto outside_sink = [&](uint32_t bits, int w) -> uint32_t {
    return (w > sink_words) ? bits : ((w < sink_words) ? 0u : (bits & sink_tail));
  };
  const int plain_from = sink_words / 4 + 1, plain_to = n_w / 4;      // quads that need no fixing
  auto load_quad = [&](int q) -> uint4 {
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (q >= n_quads) return v;
    if constexpr (kBitmapInSmem) {
      asm volatile("ld.volatile.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                   : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(smem_u32(bm) + 16u * q) : "memory");
    } else {
      v = __ldcg(reinterpret_cast<const uint4*>(bm) + q);
    }
    if (q >= plain_from && q < plain_to) return v;
    const int w0 = 4 * q;
    if (w0 + 1 >= n_w) v.y = 0u;                            // words past the end hold nothing
    if (w0 + 2 >= n_w) v.z = 0u;
    if (w0 + 3 >= n_w) v.w = 0u;
    v.x = outside_sink(v.x, w0); v.y = outside_sink(v.y, w0 + 1);
    v.z = outside_sink(v.z, w0 + 2); v.w = outside_sink(v.w, w0 + 3);
    return v;
  };
  for (int j = threadIdx.x; j < p.n_sink; j += kSelThreads) p.out_idx[j] = j;
  uint32_t n_mine = 0;
  for (int k = 0; k < rounds; ++k) {
    const uint4 v = load_quad(q_begin + k * 32 + lane);
    n_mine += (v.x != 0u) + (v.y != 0u) + (v.z != 0u) + (v.w != 0u);
  }
  uint32_t n_entries;
  uint32_t running = block_exclusive_scan(n_mine, sh->scan, &n_entries);
  running = __shfl_sync(0xFFFFFFFFu, running, 0);            // entries of the warps before this one
  const uint32_t lt = (1u << lane) - 1u;
  for (int k = 0; k < rounds; ++k) {
    const int q = q_begin + k * 32 + lane;
    const uint4 v = load_quad(q);
    if (__ballot_sync(0xFFFFFFFFu, (v.x | v.y | v.z | v.w) != 0u) == 0u) continue;
    const uint32_t b0 = __ballot_sync(0xFFFFFFFFu, v.x != 0u), b1 = __ballot_sync(0xFFFFFFFFu, v.y != 0u);
    const uint32_t b2 = __ballot_sync(0xFFFFFFFFu, v.z != 0u), b3 = __ballot_sync(0xFFFFFFFFu, v.w != 0u);
    uint32_t at = running + __popc(b0 & lt) + __popc(b1 & lt) + __popc(b2 & lt) + __popc(b3 & lt);
    const uint32_t room = static_cast<uint32_t>(p.budget);  // the list's size; never short unless a quota was overrun
    if (v.x) { if (at < room) list[at] = 4 * q; ++at; }
    if (v.y) { if (at < room) list[at] = 4 * q + 1; ++at; }
    if (v.z) { if (at < room) list[at] = 4 * q + 2; ++at; }
    if (v.w) { if (at < room) list[at] = 4 * q + 3; ++at; }
    running += __popc(b0) + __popc(b1) + __popc(b2) + __popc(b3);
  }
  __syncthreads();
  n_entries = min(n_entries, static_cast<uint32_t>(p.budget));
  const int per = static_cast<int>((n_entries + kSelThreads - 1) / kSelThreads);
  const int e_begin = min(static_cast<int>(n_entries), static_cast<int>(threadIdx.x) * per);
  const int e_end = min(static_cast<int>(n_entries), e_begin + per);
  uint32_t mine = 0;
  for (int e = e_begin; e < e_end; ++e) {
    const int w = list[e];
    mine += __popc(outside_sink(bitmap_word<kBitmapInSmem>(bm, w), w));
  }
  uint32_t total;
  uint32_t at = static_cast<uint32_t>(p.n_sink) + block_exclusive_scan(mine, sh->scan, &total);
  for (int e = e_begin; e < e_end; ++e) {
    const int w = list[e];
    uint32_t bits = outside_sink(bitmap_word<kBitmapInSmem>(bm, w), w);
    while (bits) {
      const int b = __ffs(bits) - 1;
      bits &= bits - 1;
      if (at < cap) p.out_idx[at] = w * 32 + b;
      ++at;
    }
  }
  if (threadIdx.x == 0 && total != static_cast<uint32_t>(p.budget)) atomicCAS(p.status, 0, kDevQuota);
}

template <bool kCluster>
__global__ void __launch_bounds__(kSelThreads, 1)
select_kernel(const ComboTable tbl, const SelectParams p) {
  extern __shared__ __align__(16) uint8_t dyn_smem[];
  __shared__ SelShared sh;
  const int n_tiles = tbl.tile_begin[tbl.n_comb];
  const int t_begin = static_cast<int>(static_cast<long long>(blockIdx.x) * n_tiles / gridDim.x);
  const int t_end = static_cast<int>(static_cast<long long>(blockIdx.x + 1) * n_tiles / gridDim.x);
  for (int b = threadIdx.x; b < kHistBins; b += kSelThreads) sh.hist[b] = 0u;
  uint32_t epoch = 0;
  grid_dep_wait();       // the kernel before this one (scores, state cleared for this run) is done

  // ---- A: scores from the encoded maxima, one exp per position ----
  if (!p.scores_given) {
    const long long stride = static_cast<long long>(gridDim.x) * kSelThreads;
    for (long long t = static_cast<long long>(blockIdx.x) * kSelThreads + threadIdx.x; t < p.L;
         t += stride) {
      const float a = exp2f(ordered_to_float(__ldcg(&p.enc[t])));
      p.scores[t] = a;
      if (p.user_scores) p.user_scores[t] = a;
    }
  }
  if (!grid_sync<kCluster>(p, &sh, epoch)) return;

  // ---- B1: strided max-pool arrays, one per distinct m > 1 ----
  if (tbl.n_src > 0) {
    float* buf = reinterpret_cast<float*>(dyn_smem);
    const int n_st = tbl.src_tile_begin[tbl.n_src];
    const int s_begin = static_cast<int>(static_cast<long long>(blockIdx.x) * n_st / gridDim.x);
    const int s_end = static_cast<int>(static_cast<long long>(blockIdx.x + 1) * n_st / gridDim.x);
    int src = 0;
    for (int tile = s_begin; tile < s_end; ++tile) {
      while (src + 1 < tbl.n_src && tile >= tbl.src_tile_begin[src + 1]) ++src;
      maxpool_tile(tbl, p, src, tile - tbl.src_tile_begin[src], buf);
    }
    if (!grid_sync<kCluster>(p, &sh, epoch)) return;
  }

  // ---- B2: window pooling of every combination + first histogram ----
  {
    float* buf0 = reinterpret_cast<float*>(dyn_smem);
    float* buf1 = buf0 + (kSelTile + kMaxWin);
    int cur = -1, cursor = 0;
    for (int tile = t_begin; tile < t_end; ++tile) {
      const int combo = combo_of_tile(tbl, tile, cursor);
      if (combo != cur && cur >= 0)
        hist_flush(sh.hist, p.hist + static_cast<long long>(cur) * kHistBins);
      cur = combo;
      pool_tile(tbl, p, combo, (tile - tbl.tile_begin[combo]) * kSelTile, buf0, buf1, sh.hist);
    }
    if (cur >= 0) hist_flush(sh.hist, p.hist + static_cast<long long>(cur) * kHistBins);
  }
  if (!grid_sync<kCluster>(p, &sh, epoch)) return;

  // ---- C: radix select of the K_m-th largest value ----
  // combinations whose tiles this CTA scans
  int c_lo = 0, c_hi = -1;
  if (t_begin < t_end) {
    int cursor = 0;
    c_lo = combo_of_tile(tbl, t_begin, cursor);
    c_hi = combo_of_tile(tbl, t_end - 1, cursor);
  }
  for (int combo = c_lo + threadIdx.x; combo <= c_hi; combo += kSelThreads) {
    sh.prefix[combo] = 0ull;
    sh.krem[combo] = static_cast<uint32_t>(tbl.k_m[combo]);
    sh.state[combo] = 0u;
    sh.mode[combo] = 0;
  }
  __syncthreads();
  for (int combo = c_lo; combo <= c_hi; ++combo) bin_search(p, tbl.n_comb, combo, 0, &sh);

  // ---- D: the gather.  After the first pass a combination knows the bin (top 11 bits of the
  // key) that holds its K_m-th value.  One scan settles almost everything: cells above that
  // bin are candidates; where every cell of the bin is wanted too (or few cells exist), the
  // bin's cells are candidates as well; otherwise the bin's cells are set aside (at most
  // kPendCap of them) and one CTA picks the wanted number of highest keys among them.
  {
    const int lane = threadIdx.x & 31;
    int load_cursor = 0, cursor = 0;
    for (int t0 = t_begin; t0 < t_end; t0 += kScanGroup) {
      float wv[kScanGroup][kTilePer];
#pragma unroll
      for (int g = 0; g < kScanGroup; ++g)
        if (t0 + g < t_end) fetch_tile(tbl, p, t0 + g, load_cursor, nullptr, wv[g]);
#pragma unroll
      for (int g = 0; g < kScanGroup; ++g) {
        const int tile = t0 + g;
        if (tile >= t_end) break;
        const int combo = combo_of_tile(tbl, tile, cursor);
        const int mode = sh.mode[combo];
        if (mode == 2) continue;                             // left to the full-scan passes
        const unsigned long long threshold = sh.prefix[combo];
        const uint32_t bin = static_cast<uint32_t>(threshold >> 53);
        unsigned long long* cand = p.cand + static_cast<long long>(combo) * p.cand_stride;
        unsigned long long* pend = p.pending + static_cast<long long>(combo) * kPendCap;
        const int c0 = (tile - tbl.tile_begin[combo]) * kSelTile;
        const int c1 = min(tbl.len[combo], c0 + kSelTile);
#pragma unroll
        for (int k = 0; k < kTilePer; ++k) {
          const int c = c0 + k * kSelThreads + threadIdx.x;
          unsigned long long key = 0ull;
          bool take = false, aside = false;
          if (c < c1) {
            key = make_key(wv[g][k], static_cast<uint32_t>(c));
            if (mode == 0) {
              take = key >= threshold;
            } else {
              const uint32_t digit = static_cast<uint32_t>(key >> 53);
              take = digit > bin;
              aside = digit == bin;
            }
          }
          const uint32_t votes = __ballot_sync(0xFFFFFFFFu, take);
          if (votes) {
            uint32_t slot = 0;
            if (lane == __ffs(votes) - 1) slot = atomicAdd(&p.cand_count[combo], __popc(votes));
            slot = __shfl_sync(0xFFFFFFFFu, slot, __ffs(votes) - 1) +
                   __popc(votes & ((1u << lane) - 1u));
            if (take && slot < static_cast<uint32_t>(tbl.k_m[combo])) cand[slot] = key;
          }
          const uint32_t held = __ballot_sync(0xFFFFFFFFu, aside);
          if (held) {
            uint32_t slot = 0;
            if (lane == __ffs(held) - 1)
              slot = atomicAdd(&p.cand_count[kMaxCombos + combo], __popc(held));
            slot = __shfl_sync(0xFFFFFFFFu, slot, __ffs(held) - 1) +
                   __popc(held & ((1u << lane) - 1u));
            if (aside && slot < static_cast<uint32_t>(kPendCap)) pend[slot] = key;
          }
        }
      }
    }
  }
  if (!grid_sync<kCluster>(p, &sh, epoch)) return;

  // The cells set aside: one CTA per combination selects the highest `wanted` keys among them
  // (radix select over the remaining 53 bits of the key in shared memory) and appends them.
  for (int combo = blockIdx.x; combo < tbl.n_comb; combo += gridDim.x) {
    const int n_p = static_cast<int>(min(__ldcg(&p.cand_count[kMaxCombos + combo]),
                                         static_cast<uint32_t>(kPendCap)));
    if (n_p == 0) continue;                                  // uniform
    resolve_pending(p, tbl, combo, n_p, &sh);
  }

  // A plateau across a whole bin (more than kPendCap equal-digit cells): the remaining passes
  // over the array, for those combinations only.  The flag is the same for every CTA.
  if (__ldcg(&p.cand_count[3 * kMaxCombos]) != 0u) {
    for (int combo = c_lo + threadIdx.x; combo <= c_hi; combo += kSelThreads)
      if (sh.mode[combo] != 2) sh.state[combo] = 1u;         // nothing left to do for these
    __syncthreads();
    for (int pass = 1; pass < kSelectPasses; ++pass) {
      int shift, bits;
      pass_bits(pass, shift, bits);
      const uint32_t mask = (1u << bits) - 1u;
      uint32_t* hist_pass = p.hist + static_cast<long long>(pass) * tbl.n_comb * kHistBins;
      int cur = -1, load_cursor = 0, cursor = 0;
      for (int t0 = t_begin; t0 < t_end; t0 += kScanGroup) {
        float wv[kScanGroup][kTilePer];
#pragma unroll
        for (int g = 0; g < kScanGroup; ++g)
          if (t0 + g < t_end) fetch_tile(tbl, p, t0 + g, load_cursor, sh.state, wv[g]);
#pragma unroll
        for (int g = 0; g < kScanGroup; ++g) {
          const int tile = t0 + g;
          if (tile >= t_end) break;
          const int combo = combo_of_tile(tbl, tile, cursor);
          if (sh.state[combo]) continue;
          if (combo != cur && cur >= 0)
            hist_flush(sh.hist, hist_pass + static_cast<long long>(cur) * kHistBins);
          cur = combo;
          const unsigned long long prefix = sh.prefix[combo];
          const int c0 = (tile - tbl.tile_begin[combo]) * kSelTile;
          const int c1 = min(tbl.len[combo], c0 + kSelTile);
#pragma unroll
          for (int k = 0; k < kTilePer; ++k) {
            const int c = c0 + k * kSelThreads + threadIdx.x;
            uint32_t digit = 0xFFFFFFFFu;                    // sentinel: does not take part
            if (c < c1) {
              const unsigned long long key = make_key(wv[g][k], static_cast<uint32_t>(c));
              if (((key ^ prefix) >> (shift + bits)) == 0ull)
                digit = static_cast<uint32_t>(key >> shift) & mask;
            }
            hist_add(sh.hist, digit);
          }
        }
      }
      if (cur >= 0) hist_flush(sh.hist, hist_pass + static_cast<long long>(cur) * kHistBins);
      if (!grid_sync<kCluster>(p, &sh, epoch)) return;
      for (int combo = c_lo; combo <= c_hi; ++combo)
        if (sh.state[combo] == 0u) bin_search(p, tbl.n_comb, combo, pass, &sh);
    }

    // ---- D: ties at the K_m-th value, then the gather ----
    // A combination that is not settled by now has its K_m-th value v (upper half of the
    // prefix) and wants krem of the cells that hold exactly v: the ones with the lowest index.
    {
      int load_cursor = 0, cursor = 0;
      for (int t0 = t_begin; t0 < t_end; t0 += kScanGroup) {
        float wv[kScanGroup][kTilePer];
#pragma unroll
        for (int g = 0; g < kScanGroup; ++g)
          if (t0 + g < t_end) fetch_tile(tbl, p, t0 + g, load_cursor, sh.state, wv[g]);
#pragma unroll
        for (int g = 0; g < kScanGroup; ++g) {
          const int tile = t0 + g;
          if (tile >= t_end) break;
          const int combo = combo_of_tile(tbl, tile, cursor);
          if (sh.state[combo]) continue;
          const uint32_t v_star = static_cast<uint32_t>(sh.prefix[combo] >> 32);
          const int c0 = (tile - tbl.tile_begin[combo]) * kSelTile;
          const int c1 = min(tbl.len[combo], c0 + kSelTile);
          int mine = 0;
#pragma unroll
          for (int k = 0; k < kTilePer; ++k) {
            const int c = c0 + k * kSelThreads + threadIdx.x;
            mine += (c < c1 && float_to_ordered(wv[g][k]) == v_star) ? 1 : 0;
          }
          const int holders = __syncthreads_count(mine & 1) + 2 * __syncthreads_count(mine & 2) +
                              4 * __syncthreads_count(mine & 4);
          if (threadIdx.x == 0) p.tile_ties[tile] = holders;
        }
      }
    }
    if (!grid_sync<kCluster>(p, &sh, epoch)) return;
    {
      const int lane = threadIdx.x & 31;
      int load_cursor = 0, cursor = 0;
      for (int t0 = t_begin; t0 < t_end; t0 += kScanGroup) {
        float wv[kScanGroup][kTilePer];
#pragma unroll
        for (int g = 0; g < kScanGroup; ++g)
          if (t0 + g < t_end) fetch_tile(tbl, p, t0 + g, load_cursor, nullptr, wv[g]);
#pragma unroll
        for (int g = 0; g < kScanGroup; ++g) {
          const int tile = t0 + g;
          if (tile >= t_end) break;
          const int combo = combo_of_tile(tbl, tile, cursor);
          if (sh.mode[combo] != 2) continue;                   // gathered in the first scan
          const bool settled = sh.state[combo] != 0u;
          const unsigned long long threshold = sh.prefix[combo];
          const uint32_t v_star = static_cast<uint32_t>(threshold >> 32);
          const uint32_t wanted = sh.krem[combo];
          unsigned long long* cand = p.cand + static_cast<long long>(combo) * p.cand_stride;
          const int c0 = (tile - tbl.tile_begin[combo]) * kSelTile;
          const int c1 = min(tbl.len[combo], c0 + kSelTile);
          // holders of v in the earlier tiles of this combination (tiles are in cell order)
          uint32_t before = 0;
          bool ties_here = false;
          if (!settled) {
            ties_here = __ldcg(&p.tile_ties[tile]) > 0;      // uniform
            if (ties_here) {
              uint32_t part = 0;
              for (int t = tbl.tile_begin[combo] + threadIdx.x; t < tile; t += kSelThreads)
                part += static_cast<uint32_t>(__ldcg(&p.tile_ties[t]));
              block_exclusive_scan_1(part, sh.tot, 0, &before);
              __syncthreads();
            }
          }
#pragma unroll
          for (int k = 0; k < kTilePer; ++k) {
            const int c = c0 + k * kSelThreads + threadIdx.x;
            unsigned long long key = 0ull;
            bool take = false, holder = false;
            if (c < c1) {
              key = make_key(wv[g][k], static_cast<uint32_t>(c));
              const uint32_t v = static_cast<uint32_t>(key >> 32);
              if (settled) take = key >= threshold;
              else { take = v > v_star; holder = v == v_star; }
            }
            if (ties_here) {                                 // uniform
              uint32_t in_row;
              const uint32_t rank = before + block_exclusive_scan_1(holder ? 1u : 0u, sh.tot, 1, &in_row);
              __syncthreads();
              if (holder && rank < wanted) take = true;
              before += in_row;
            }
            const uint32_t votes = __ballot_sync(0xFFFFFFFFu, take);
            if (votes) {
              uint32_t slot = 0;
              if (lane == __ffs(votes) - 1) slot = atomicAdd(&p.cand_count[combo], __popc(votes));
              slot = __shfl_sync(0xFFFFFFFFu, slot, __ffs(votes) - 1) +
                     __popc(votes & ((1u << lane) - 1u));
              if (take && slot < static_cast<uint32_t>(tbl.k_m[combo])) cand[slot] = key;
            }
          }
        }
      }
    }
  }
  if (!grid_sync<kCluster>(p, &sh, epoch)) return;

  // ---- E: ranking ----
  {
    unsigned long long* chunk = reinterpret_cast<unsigned long long*>(dyn_smem);
    __shared__ int rank_count[kSelThreads];
    __shared__ RankScratch rank_scratch;
    for (int combo = threadIdx.x; combo < tbl.n_comb; combo += kSelThreads)
      sh.state[combo] = min(min(__ldcg(&p.cand_count[combo]), static_cast<uint32_t>(kMaxKm)),
                            static_cast<uint32_t>(tbl.k_m[combo]));
    __syncthreads();
    const int grid = static_cast<int>(gridDim.x), bid = static_cast<int>(blockIdx.x);
    if (tbl.rank_by_list) {
      // Enough CTAs: each serves one combination only (a CTA that met two would stage and
      // split both lists, and the whole grid would wait for it).  The host has dealt the CTAs
      // out: combination c has [rank_cta_begin[c], rank_cta_begin[c + 1]).
      for (int combo = 0; combo < tbl.n_comb; ++combo) {
        const int b0 = tbl.rank_cta_begin[combo], b1 = tbl.rank_cta_begin[combo + 1];
        if (bid < b0 || bid >= b1) continue;
        const uint32_t n = sh.state[combo], share = b1 - b0, k = bid - b0;
        const int lo = static_cast<int>(n * k / share), hi = static_cast<int>(n * (k + 1) / share);
        if (lo < hi) rank_range(p, combo, static_cast<int>(n), lo, hi, chunk, rank_count, &rank_scratch);
      }
    } else {
      // fewer CTAs than lists: every CTA takes a contiguous run of all candidates
      long long n_cand = 0;
      for (int combo = 0; combo < tbl.n_comb; ++combo) n_cand += sh.state[combo];
      const int i_begin = static_cast<int>(static_cast<long long>(bid) * n_cand / grid);
      const int i_end = static_cast<int>(static_cast<long long>(bid + 1) * n_cand / grid);
      int first = 0;
      for (int combo = 0; combo < tbl.n_comb; ++combo) {
        const int n = static_cast<int>(sh.state[combo]);
        const int lo = max(i_begin, first) - first, hi = min(i_end, first + n) - first;
        if (lo < hi) rank_range(p, combo, n, lo, hi, chunk, rank_count, &rank_scratch);
        first += n;
      }
    }
  }
  if (!grid_sync<kCluster>(p, &sh, epoch)) return;

  // ---- F: allocation and ascending output (one CTA) ----
  if (blockIdx.x != 0) return;
  if (p.bitmap_in_smem) {
    uint32_t* bm = reinterpret_cast<uint32_t*>(dyn_smem);
    const long long n_words = (p.L + 31) / 32;
    for (long long w = threadIdx.x; w < n_words; w += kSelThreads) {
      const long long lo = w * 32;
      uint32_t bits = 0;
      if (p.n_sink > lo) bits = (p.n_sink - lo >= 32) ? 0xFFFFFFFFu : ((1u << (p.n_sink - lo)) - 1u);
      bm[w] = bits;
    }
    __syncthreads();
    allocate<true>(tbl, p, dyn_smem, &sh);
  } else {
    allocate<false>(tbl, p, dyn_smem, &sh);
  }
}

// ---------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------
size_t select_smem_bytes(long long L, int max_km, int budget, SelectParams* p) {
  size_t bytes = 2 * static_cast<size_t>(kSelTile + kMaxWin) * sizeof(float);  // pooling tiles
  if (kSrcTileTokens * sizeof(float) > bytes) bytes = kSrcTileTokens * sizeof(float);
  if (kRankChunk * sizeof(unsigned long long) > bytes) bytes = kRankChunk * sizeof(unsigned long long);
  // quota walk: bitmap (when it fits) + one or two staging buffers of max_km cell ids
  const size_t cap = (static_cast<size_t>(max_km < 1 ? 1 : max_km) + 3) & ~size_t(3);
  const size_t bm_bytes = (static_cast<size_t>((L + 31) / 32) * sizeof(uint32_t) + 15) & ~size_t(15);
  p->bitmap_in_smem = bm_bytes <= static_cast<size_t>(kSelBitmapSmemBytes) ? 1 : 0;
  const size_t base = p->bitmap_in_smem ? bm_bytes : 0;
  int walkers = ((max_km + 1) / 2 + 31) & ~31;               // about two ranked cells per thread
  p->walk_threads = walkers < 256 ? 256 : (walkers > kSelThreads ? kSelThreads : walkers);
  p->stage_capacity = static_cast<int>(cap);
  p->stage_double = (base + 2 * cap * sizeof(int) <= static_cast<size_t>(kSelMaxDynSmemBytes)) ? 1 : 0;
  size_t after_bitmap = (p->stage_double ? 2 : 1) * cap * sizeof(int);
  // the output pass lists the bitmap words that hold allocated positions (at most `budget`)
  // where the staged cells were
  size_t list_bytes = static_cast<size_t>((L + 31) / 32);
  if (list_bytes > static_cast<size_t>(budget < 0 ? 0 : budget)) list_bytes = budget < 0 ? 0 : budget;
  list_bytes *= sizeof(int);
  if (list_bytes > after_bitmap) after_bitmap = list_bytes;
  const size_t alloc_bytes = base + after_bitmap;
  if (alloc_bytes > bytes) bytes = alloc_bytes;
  return bytes;
}

cudaError_t select_max_grid(int n_sm, int* max_grid) {
  cudaError_t e = cudaFuncSetAttribute(select_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       kSelMaxDynSmemBytes);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(select_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           kSelMaxDynSmemBytes);
  if (e != cudaSuccess) return e;
  int per_sm = 0;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, select_kernel<false>, kSelThreads,
                                                    kSelMaxDynSmemBytes);
  if (e != cudaSuccess) return e;
  if (per_sm < 1) return cudaErrorLaunchOutOfResources;
  *max_grid = n_sm;                      // one CTA per SM is plenty for these phases
  return cudaSuccess;
}

// Deals the CTAs of the grid out to the combinations for the ranking phase: each list gets
// its share of the grid by candidates, at least one CTA, never past what the lists after it
// still need.  With fewer CTAs than lists the kernel splits the candidates evenly instead.
static void assign_ranking(ComboTable* t, int grid) {
  long long n_cand = 0;
  int n_lists = 0;
  for (int c = 0; c < t->n_comb; ++c) {
    n_cand += t->k_m[c];
    n_lists += t->k_m[c] > 0 ? 1 : 0;
  }
  t->rank_by_list = (n_lists > 0 && grid >= n_lists) ? 1 : 0;
  long long before = 0;
  int b0 = 0, lists_left = n_lists;
  for (int c = 0; c < t->n_comb; ++c) {
    t->rank_cta_begin[c] = b0;
    if (!t->rank_by_list || t->k_m[c] <= 0) continue;
    --lists_left;
    before += t->k_m[c];
    int b1 = static_cast<int>((before * grid + n_cand / 2) / n_cand);
    if (b1 < b0 + 1) b1 = b0 + 1;
    if (b1 > grid - lists_left) b1 = grid - lists_left;
    if (lists_left == 0) b1 = grid;
    b0 = b1;
  }
  t->rank_cta_begin[t->n_comb] = b0;
}

cudaError_t launch_select(const ComboTable& table, const SelectParams& p, int grid, size_t smem,
                          cudaStream_t st) {
  ComboTable tbl = table;
  assign_ranking(&tbl, grid);
  // Short contexts need few CTAs: up to kSelClusterMax of them run as one thread-block cluster,
  // whose hardware barrier costs a fraction of a trip to the L2 (not with the self test's
  // barrier that cannot complete: that one is the counter's).  Longer ones: a cooperative
  // launch (every CTA resident: they wait on one another).  Either way the launch may overlap
  // the end of the kernel before it in the stream; the kernel waits before it reads anything.
  const bool cluster = grid <= kSelClusterMax && p.barrier_extra == 0;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(kSelThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  if (cluster) {
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = grid;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
  } else {
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
  }
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  return cluster ? cudaLaunchKernelEx(&cfg, select_kernel<true>, tbl, p)
                 : cudaLaunchKernelEx(&cfg, select_kernel<false>, tbl, p);
}

}  // namespace ilre
