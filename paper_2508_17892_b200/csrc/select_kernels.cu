// Algorithm 1 ("Context Allocation") on the device.
//
//   pool_kernel        MaxPooling(size = stride = m) fused with the stride-1 window pooling
//                      (average or max) of every (m, n) combination;
//   select_pass_kernel radix select of the K_m largest 64-bit keys (pooled value, then lower
//                      cell index first), 11/11/10 bits per pass, all combinations at once;
//   gather_kernel      collects the selected keys;
//   rank_sort_kernel   orders them (value descending, cell ascending);
//   allocate_kernel    walks the combinations in loop order: maps cells back to tokens, skips
//                      tokens already allocated, stops each combination at its quota B_c, then
//                      writes the allocated positions in ascending order.
#include "select_kernels.cuh"
#include "sm100_ptx.cuh"

namespace ilre {

__device__ __forceinline__ unsigned long long make_key(float w, uint32_t cell) {
  return (static_cast<unsigned long long>(float_to_ordered(w)) << 32) | (0xFFFFFFFFu - cell);
}

// ---------------------------------------------------------------------------------------
// pooling
// ---------------------------------------------------------------------------------------
static constexpr int kPoolTile = 1024;
static constexpr int kPoolThreads = 256;

__global__ void __launch_bounds__(kPoolThreads)
pool_kernel(const ComboTable tbl, const SelectParams p) {
  __shared__ float cells[kPoolTile + kMaxWin];
  const int combo = blockIdx.y;
  const int m = tbl.m[combo], n = tbl.n[combo], len = tbl.len[combo];
  const int c0 = blockIdx.x * kPoolTile;
  if (c0 >= len) return;
  const long long Lp = p.L - p.n_sink;                     // scores without the sink part
  const float* a = p.scores + p.n_sink;
  const int lo = c0 - n / 2;
  const int span = min(kPoolTile, len - c0) + n - 1;
  const float pad = (p.win_op == 0) ? 0.f : -INFINITY;
  for (int idx = threadIdx.x; idx < span; idx += kPoolThreads) {
    const int u = lo + idx;
    float v = pad;
    if (u >= 0 && u < len) {
      const long long t0 = static_cast<long long>(u) * m;
      const long long t1 = min(t0 + m, Lp);
      v = a[t0];
      for (long long t = t0 + 1; t < t1; ++t) v = fmaxf(v, a[t]);
    }
    cells[idx] = v;
  }
  __syncthreads();
  float* out = p.pooled + static_cast<long long>(combo) * p.pooled_stride;
  const int n_out = min(kPoolTile, len - c0);
  for (int i = threadIdx.x; i < n_out; i += kPoolThreads) {
    float acc;
    if (p.win_op == 0) {
      acc = 0.f;
      for (int j = 0; j < n; ++j) acc += cells[i + j];
      acc = acc / static_cast<float>(n);
    } else {
      acc = cells[i];
      for (int j = 1; j < n; ++j) acc = fmaxf(acc, cells[i + j]);
    }
    out[c0 + i] = acc;
  }
}

// ---------------------------------------------------------------------------------------
// radix select
// ---------------------------------------------------------------------------------------
static constexpr int kSelThreads = 512;
static constexpr int kSelItemsPerThread = 16;

__device__ __forceinline__ void pass_bits(int pass, int& shift, int& bits) {
  const int sh[kSelectPasses] = {53, 42, 32, 21, 10, 0};
  const int bt[kSelectPasses] = {11, 11, 10, 11, 11, 10};
  shift = sh[pass];
  bits = bt[pass];
}

__global__ void __launch_bounds__(kSelThreads)
select_pass_kernel(const ComboTable tbl, const SelectParams p, const int pass) {
  __shared__ uint32_t sh_hist[kHistBins];
  __shared__ uint32_t sh_warp[kSelThreads / 32];
  __shared__ int sh_last;
  const int combo = blockIdx.y;
  if (p.sel_done[combo]) return;
  const int len = tbl.len[combo];
  int shift, bits;
  pass_bits(pass, shift, bits);
  const unsigned long long prefix = p.sel_prefix[combo];
  const uint32_t mask = (1u << bits) - 1u;
  for (int b = threadIdx.x; b < kHistBins; b += kSelThreads) sh_hist[b] = 0u;
  __syncthreads();

  const float* w = p.pooled + static_cast<long long>(combo) * p.pooled_stride;
  const int per_block = (len + gridDim.x - 1) / gridDim.x;
  const int begin = blockIdx.x * per_block;
  const int end = min(len, begin + per_block);
  const int lane = threadIdx.x & 31;
  for (int base = begin; base < end; base += kSelThreads) {
    const int c = base + threadIdx.x;
    uint32_t digit = 0xFFFFFFFFu;                          // sentinel: does not take part
    if (c < end) {
      const unsigned long long key = make_key(w[c], static_cast<uint32_t>(c));
      if (pass == 0 || ((key ^ prefix) >> (shift + bits)) == 0ull)
        digit = static_cast<uint32_t>(key >> shift) & mask;
    }
    const uint32_t peers = __match_any_sync(0xFFFFFFFFu, digit);
    if (digit != 0xFFFFFFFFu && lane == __ffs(peers) - 1) atomicAdd(&sh_hist[digit], __popc(peers));
  }
  __syncthreads();
  uint32_t* gh = p.hist + static_cast<long long>(combo) * kHistBins;
  for (int b = threadIdx.x; b < kHistBins; b += kSelThreads)
    if (sh_hist[b]) atomicAdd(&gh[b], sh_hist[b]);
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const uint32_t t = atomicAdd(&p.sel_ticket[combo], 1u);
    sh_last = (t == gridDim.x - 1);
  }
  __syncthreads();
  if (!sh_last) return;
  __threadfence();

  // Last block of this combination: locate the bin that holds the k-th largest key.
  const uint32_t k_rem = p.sel_krem[combo];
  uint32_t h[4];
  uint32_t total = 0;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    h[j] = __ldcg(&gh[kHistBins - 1 - (4 * threadIdx.x + j)]);   // bins in descending order
    total += h[j];
  }
  uint32_t incl = total;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t v = __shfl_up_sync(0xFFFFFFFFu, incl, o);
    if (lane >= o) incl += v;
  }
  const int warp = threadIdx.x >> 5;
  if (lane == 31) sh_warp[warp] = incl;
  __syncthreads();
  uint32_t warp_off = 0;
  for (int wv = 0; wv < warp; ++wv) warp_off += sh_warp[wv];
  const uint32_t excl = warp_off + incl - total;
  if (excl < k_rem && k_rem <= excl + total) {
    uint32_t cum = excl;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      if (k_rem > cum && k_rem <= cum + h[j]) {
        const uint32_t bin = kHistBins - 1 - (4 * threadIdx.x + j);
        const uint32_t new_k = k_rem - cum;
        p.sel_prefix[combo] = prefix | (static_cast<unsigned long long>(bin) << shift);
        p.sel_krem[combo] = new_k;
        p.sel_done[combo] = (h[j] == new_k || pass == kSelectPasses - 1) ? 1u : 0u;
      }
      cum += h[j];
    }
  }
  uint32_t grand = 0;
  for (int wv = 0; wv < kSelThreads / 32; ++wv) grand += sh_warp[wv];
  if (threadIdx.x == 0) {
    if (k_rem > grand || k_rem == 0) p.sel_done[combo] = 1u;   // fewer keys than asked: take all
    p.sel_ticket[combo] = 0u;
  }
  for (int b = threadIdx.x; b < kHistBins; b += kSelThreads) gh[b] = 0u;
}

__global__ void __launch_bounds__(kSelThreads)
gather_kernel(const ComboTable tbl, const SelectParams p) {
  const int combo = blockIdx.y;
  const int len = tbl.len[combo];
  const unsigned long long threshold = p.sel_prefix[combo];
  const float* w = p.pooled + static_cast<long long>(combo) * p.pooled_stride;
  unsigned long long* cand = p.cand + static_cast<long long>(combo) * p.cand_stride;
  const int per_block = (len + gridDim.x - 1) / gridDim.x;
  const int begin = blockIdx.x * per_block;
  const int end = min(len, begin + per_block);
  for (int c = begin + threadIdx.x; c < end; c += kSelThreads) {
    const unsigned long long key = make_key(w[c], static_cast<uint32_t>(c));
    if (key >= threshold) {
      const uint32_t pos = atomicAdd(&p.cand_count[combo], 1u);
      if (pos < static_cast<uint32_t>(tbl.k_m[combo])) cand[pos] = key;
    }
  }
}

// ---------------------------------------------------------------------------------------
// ranking: bitonic sort of <= kMaxKm keys, descending
// ---------------------------------------------------------------------------------------
static constexpr int kSortThreads = 1024;

__global__ void __launch_bounds__(kSortThreads)
rank_sort_kernel(const ComboTable tbl, const SelectParams p, const int pow2) {
  extern __shared__ unsigned long long keys[];
  const int combo = blockIdx.x;
  const int n = min(static_cast<int>(min(p.cand_count[combo], static_cast<uint32_t>(kMaxKm))),
                    tbl.k_m[combo]);
  const unsigned long long* cand = p.cand + static_cast<long long>(combo) * p.cand_stride;
  for (int i = threadIdx.x; i < pow2; i += kSortThreads) keys[i] = (i < n) ? cand[i] : 0ull;
  __syncthreads();
  for (int k = 2; k <= pow2; k <<= 1) {
    for (int j = k >> 1; j > 0; j >>= 1) {
      for (int i = threadIdx.x; i < pow2; i += kSortThreads) {
        const int x = i ^ j;
        if (x > i) {
          const unsigned long long a = keys[i], b = keys[x];
          const bool descending_block = ((i & k) == 0);
          if (descending_block ? (a < b) : (a > b)) { keys[i] = b; keys[x] = a; }
        }
      }
      __syncthreads();
    }
  }
  int* ranked = p.ranked + static_cast<long long>(combo) * p.cand_stride;
  for (int i = threadIdx.x; i < n; i += kSortThreads)
    ranked[i] = static_cast<int>(0xFFFFFFFFu - static_cast<uint32_t>(keys[i] & 0xFFFFFFFFull));
}

// ---------------------------------------------------------------------------------------
// allocation
// ---------------------------------------------------------------------------------------
static constexpr int kAllocThreads = 1024;

// Exclusive prefix sum over the block; *total receives the block sum.
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

__global__ void __launch_bounds__(kAllocThreads)
allocate_kernel(const ComboTable tbl, const SelectParams p) {
  __shared__ uint32_t sh_warp[33];
  const long long Lp = p.L - p.n_sink;
  for (int combo = 0; combo < tbl.n_comb; ++combo) {
    const int m = tbl.m[combo];
    const int quota = tbl.quota[combo];
    const int K = min(static_cast<int>(min(p.cand_count[combo], static_cast<uint32_t>(kMaxKm))),
                      tbl.k_m[combo]);
    const int* ranked = p.ranked + static_cast<long long>(combo) * p.cand_stride;
    int taken = 0;                                            // uniform across the block
    for (int base = 0; base < K && taken < quota; base += kAllocThreads) {
      const int r = base + threadIdx.x;
      unsigned long long fresh = 0ull;                        // bit j: token j of the cell is new
      long long t0 = 0;
      if (r < K) {
        t0 = static_cast<long long>(ranked[r]) * m;
        for (int j = 0; j < m; ++j) {
          const long long t = t0 + j;
          if (t < Lp) {
            const long long pos = p.n_sink + t;
            const uint32_t word = __ldcg(&p.bitmap[pos >> 5]);
            if (!((word >> (pos & 31)) & 1u)) fresh |= (1ull << j);
          }
        }
      }
      uint32_t total;
      const uint32_t before = block_exclusive_scan(__popcll(fresh), sh_warp, &total);
      const int room = quota - taken;
      uint32_t ord = before;
      while (fresh && ord < static_cast<uint32_t>(room)) {    // ascending position inside the cell
        const int j = __ffsll(static_cast<long long>(fresh)) - 1;
        fresh &= fresh - 1;
        const long long pos = p.n_sink + t0 + j;
        atomicOr(&p.bitmap[pos >> 5], 1u << (pos & 31));
        ++ord;
      }
      taken += min(static_cast<int>(total), room);
      __syncthreads();                                        // bitmap updates visible to the block
    }
    if (taken < quota && threadIdx.x == 0) atomicCAS(p.status, 0, kDevQuota);
    __syncthreads();
  }

  // Ascending output: every thread owns a contiguous run of bitmap words.
  const long long n_words = (p.L + 31) / 32;
  const long long per_thread = (n_words + kAllocThreads - 1) / kAllocThreads;
  const long long w0 = min(n_words, static_cast<long long>(threadIdx.x) * per_thread);
  const long long w1 = min(n_words, w0 + per_thread);
  uint32_t count = 0;
  for (long long w = w0; w < w1; ++w) count += __popc(__ldcg(&p.bitmap[w]));
  uint32_t total;
  uint32_t off = block_exclusive_scan(count, sh_warp, &total);
  const uint32_t cap = static_cast<uint32_t>(p.n_sink + p.budget);
  for (long long w = w0; w < w1; ++w) {
    uint32_t bits = __ldcg(&p.bitmap[w]);
    while (bits) {
      const int b = __ffs(bits) - 1;
      bits &= bits - 1;
      if (off < cap) p.out_idx[off] = static_cast<int>(w * 32 + b);
      ++off;
    }
  }
  if (threadIdx.x == 0 && total != cap) atomicCAS(p.status, 0, kDevQuota);
}

// ---------------------------------------------------------------------------------------
// launchers
// ---------------------------------------------------------------------------------------
static int select_blocks(int max_len) {
  int nb = (max_len + kSelThreads * kSelItemsPerThread - 1) / (kSelThreads * kSelItemsPerThread);
  if (nb < 1) nb = 1;
  if (nb > 256) nb = 256;
  return nb;
}

cudaError_t launch_pool(const ComboTable& tbl, const SelectParams& p, int max_len,
                        cudaStream_t st) {
  dim3 grid((max_len + kPoolTile - 1) / kPoolTile, tbl.n_comb);
  pool_kernel<<<grid, kPoolThreads, 0, st>>>(tbl, p);
  return cudaGetLastError();
}

cudaError_t launch_select_pass(const ComboTable& tbl, const SelectParams& p, int max_len, int pass,
                               cudaStream_t st) {
  dim3 grid(select_blocks(max_len), tbl.n_comb);
  select_pass_kernel<<<grid, kSelThreads, 0, st>>>(tbl, p, pass);
  return cudaGetLastError();
}

cudaError_t launch_gather(const ComboTable& tbl, const SelectParams& p, int max_len,
                          cudaStream_t st) {
  dim3 grid(select_blocks(max_len), tbl.n_comb);
  gather_kernel<<<grid, kSelThreads, 0, st>>>(tbl, p);
  return cudaGetLastError();
}

cudaError_t launch_rank_sort(const ComboTable& tbl, const SelectParams& p, int max_km,
                             cudaStream_t st) {
  int pow2 = 2;
  while (pow2 < max_km) pow2 <<= 1;
  const size_t smem = static_cast<size_t>(pow2) * sizeof(unsigned long long);
  cudaError_t e = cudaFuncSetAttribute(rank_sort_kernel,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  rank_sort_kernel<<<tbl.n_comb, kSortThreads, smem, st>>>(tbl, p, pow2);
  return cudaGetLastError();
}

cudaError_t launch_allocate(const ComboTable& tbl, const SelectParams& p, cudaStream_t st) {
  allocate_kernel<<<1, kAllocThreads, 0, st>>>(tbl, p);
  return cudaGetLastError();
}

}  // namespace ilre
