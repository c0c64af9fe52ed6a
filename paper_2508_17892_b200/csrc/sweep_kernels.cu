// Offline choice of the retrieval layer (Section 3.3, first paragraph; Appendix A.1).
#include "sweep_kernels.cuh"

namespace ilre {

namespace {

// first i in [0, n) with a[i] >= v (a ascending)
__device__ __forceinline__ int lower_bound(const int32_t* __restrict__ a, int n, long long v) {
  int lo = 0, hi = n;
  while (lo < hi) {
    const int mid = (lo + hi) >> 1;
    if (a[mid] < v) lo = mid + 1; else hi = mid;
  }
  return lo;
}

// One CTA.  A phrase is a contiguous position range and every index list is ascending without
// repeats, so the recalled positions inside a phrase are the list entries between two binary
// searches.
__global__ void __launch_bounds__(1024)
layer_recall_kernel(const int32_t* __restrict__ idx, int n_layers, int n_idx,
                    const int32_t* __restrict__ span_begin, const int32_t* __restrict__ span_len,
                    int n_spans, int32_t* __restrict__ hits, int32_t* __restrict__ full,
                    int32_t* __restrict__ layer) {
  __shared__ int s_full[kMaxSweepLayers];
  for (int l = threadIdx.x; l < n_layers; l += blockDim.x) s_full[l] = 0;
  __syncthreads();
  const long long pairs = static_cast<long long>(n_layers) * n_spans;
  for (long long e = threadIdx.x; e < pairs; e += blockDim.x) {
    const int l = static_cast<int>(e / n_spans), s = static_cast<int>(e % n_spans);
    const int32_t* row = idx + static_cast<long long>(l) * n_idx;
    const long long b = span_begin[s], n = span_len[s];
    const int h = lower_bound(row, n_idx, b + n) - lower_bound(row, n_idx, b);
    if (hits) hits[e] = h;
    if (h == n) atomicAdd(&s_full[l], 1);
  }
  __syncthreads();
  for (int l = threadIdx.x; l < n_layers; l += blockDim.x) full[l] = s_full[l];
  if (threadIdx.x == 0) {
    int best = 0;
    for (int l = 1; l < n_layers; ++l)
      if (s_full[l] > s_full[best]) best = l;      // strict: the smallest index keeps a tie
    *layer = best;
  }
}

}  // namespace

cudaError_t launch_layer_recall(const int32_t* idx, int n_layers, int n_idx,
                                const int32_t* span_begin, const int32_t* span_len, int n_spans,
                                int32_t* hits, int32_t* full, int32_t* layer, cudaStream_t st) {
  layer_recall_kernel<<<1, 1024, 0, st>>>(idx, n_layers, n_idx, span_begin, span_len, n_spans,
                                          hits, full, layer);
  return cudaGetLastError();
}

}  // namespace ilre
