// ilre_topk_positions_noalloc: plain top-k of a score array with ascending output, for callers
// that must not allocate device memory.
//
// Some users of this library run in places where cudaMalloc is off limits: inside a serving
// loop whose memory is owned by a framework pool with a fixed budget, in a latency-critical
// thread where the implicit device synchronisation of cudaMalloc/cudaFree is not acceptable,
// or in a plug-in that is only handed buffers and a stream.  The regular entry points need a
// handle whose workspace is allocated by ilre_recall_create().  This one needs no handle: its
// only scratch (a bitmap of the chosen positions) lives in a fixed, file-scope __device__ array
// that every GPU which loads the library carries until the process exits.
//
// It is the one-combination case of the allocation step (one max kernel of size 1, one window
// of size 1, no sink): the k highest scores, equal scores ranked by lower position, returned as
// ascending positions.  One CTA does the whole job (radix select in shared memory, bitmap in the
// static scratch, compaction), so it is meant for occasional use, not for the hot path.
#include <cuda_runtime.h>

#include <cstdint>
#include <mutex>

#include "../../include/ilre_recall.h"
#include "sm100_ptx.cuh"

namespace {

constexpr int kThreads = 1024;
constexpr int kBins = 2048;
constexpr long long kMaxL = ILRE_NOALLOC_MAX_L;
constexpr int kScratchWords = static_cast<int>(kMaxL / 32);
constexpr int kMaxDevices = 64;

// The scratch itself.  In host code this name is only a handle for the runtime, not a device
// address: the address a kernel may use comes from cudaGetSymbolAddress (see scratch_for()).
static __device__ __align__(256) uint32_t g_topk_bitmap[kScratchWords];

std::mutex g_setup_mutex;
uint32_t* g_bitmap_addr[kMaxDevices] = {nullptr};

// Device address of the scratch on `device`, which must be the current device.  Looked up once
// per device; the first lookup may load the module, so it should happen outside stream capture.
cudaError_t scratch_for(int device, uint32_t** out) {
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_bitmap_addr[device]) {
    void* p = nullptr;
    const cudaError_t e = cudaGetSymbolAddress(&p, g_topk_bitmap);
    if (e != cudaSuccess) return e;
    g_bitmap_addr[device] = static_cast<uint32_t*>(p);
  }
  *out = g_bitmap_addr[device];
  return cudaSuccess;
}

// Sort key of one score: value first, then lower position.  Adding +0.0 turns -0.0 into +0.0,
// so that the two zeros tie like any other pair of equal scores.
__device__ __forceinline__ unsigned long long key_of(float v, uint32_t pos) {
  return (static_cast<unsigned long long>(ilre::float_to_ordered(v + 0.0f)) << 32) |
         (0xFFFFFFFFu - pos);
}

// Exclusive block scan over 1024 threads; *total = block sum.
__device__ __forceinline__ uint32_t scan_excl(uint32_t v, uint32_t* sh, uint32_t* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
    if (lane >= o) incl += t;
  }
  __syncthreads();
  if (lane == 31) sh[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    const uint32_t w = sh[lane];
    uint32_t wi = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, wi, o);
      if (lane >= o) wi += t;
    }
    sh[lane] = wi - w;
    if (lane == 31) sh[32] = wi;
  }
  __syncthreads();
  *total = sh[32];
  return sh[warp] + incl - v;
}

__global__ void __launch_bounds__(kThreads)
topk_positions_kernel(const float* __restrict__ scores, const int n, const int k,
                      int* __restrict__ out_idx, uint32_t* __restrict__ bitmap) {
  __shared__ uint32_t hist[kBins];
  __shared__ uint32_t sh_scan[33];
  __shared__ unsigned long long sh_prefix;
  __shared__ uint32_t sh_krem;
  __shared__ int sh_done;
  const int n_words = (n + 31) / 32;
  // the scratch keeps the previous call's bits: clear the part this call uses
  for (int w = threadIdx.x; w < n_words; w += kThreads) bitmap[w] = 0u;
  if (threadIdx.x == 0) { sh_prefix = 0ull; sh_krem = static_cast<uint32_t>(k); sh_done = (k == 0); }
  __syncthreads();

  const int shifts[6] = {53, 42, 32, 21, 10, 0};
  const int widths[6] = {11, 11, 10, 11, 11, 10};
  const int lane = threadIdx.x & 31;
  for (int pass = 0; pass < 6; ++pass) {
    if (sh_done) break;                                   // uniform: read after a barrier
    const int shift = shifts[pass], bits = widths[pass];
    const unsigned long long prefix = sh_prefix;
    const uint32_t k_rem = sh_krem;
    for (int b = threadIdx.x; b < kBins; b += kThreads) hist[b] = 0u;
    __syncthreads();
    for (int base = 0; base < n; base += kThreads) {
      const int i = base + threadIdx.x;
      uint32_t digit = 0xFFFFFFFFu;
      if (i < n) {
        const unsigned long long key = key_of(scores[i], static_cast<uint32_t>(i));
        if (pass == 0 || ((key ^ prefix) >> (shift + bits)) == 0ull)
          digit = static_cast<uint32_t>(key >> shift) & ((1u << bits) - 1u);
      }
      const uint32_t peers = __match_any_sync(0xFFFFFFFFu, digit);
      if (digit != 0xFFFFFFFFu && lane == __ffs(peers) - 1) atomicAdd(&hist[digit], __popc(peers));
    }
    __syncthreads();
    // bins in descending order, two per thread
    const uint32_t h0 = hist[kBins - 1 - 2 * threadIdx.x];
    const uint32_t h1 = hist[kBins - 2 - 2 * threadIdx.x];
    uint32_t total;
    const uint32_t excl = scan_excl(h0 + h1, sh_scan, &total);
    if (k_rem > excl && k_rem <= excl + h0 + h1) {
      const bool first = k_rem <= excl + h0;
      const uint32_t bin = first ? kBins - 1 - 2 * threadIdx.x : kBins - 2 - 2 * threadIdx.x;
      const uint32_t above = first ? excl : excl + h0;
      const uint32_t cnt = first ? h0 : h1;
      sh_prefix = prefix | (static_cast<unsigned long long>(bin) << shift);
      sh_krem = k_rem - above;
      sh_done = (cnt == k_rem - above) || pass == 5;
    }
    __syncthreads();
  }
  // every key >= the threshold is selected: exactly k of them
  const unsigned long long threshold = sh_prefix;
  if (k > 0) {
    for (int i = threadIdx.x; i < n; i += kThreads)
      if (key_of(scores[i], static_cast<uint32_t>(i)) >= threshold)
        atomicOr(&bitmap[i >> 5], 1u << (i & 31));
  }
  __threadfence_block();
  __syncthreads();
  // ascending output
  const int per_thread = (n_words + kThreads - 1) / kThreads;
  const int w0 = min(n_words, static_cast<int>(threadIdx.x) * per_thread);
  const int w1 = min(n_words, w0 + per_thread);
  uint32_t count = 0;
  for (int w = w0; w < w1; ++w) count += __popc(__ldcg(&bitmap[w]));
  uint32_t total;
  uint32_t off = scan_excl(count, sh_scan, &total);
  for (int w = w0; w < w1; ++w) {
    uint32_t word = __ldcg(&bitmap[w]);
    while (word) {
      const int b = __ffs(word) - 1;
      word &= word - 1;
      if (off < static_cast<uint32_t>(k)) out_idx[off] = w * 32 + b;
      ++off;
    }
  }
}

}  // namespace

extern "C" int ilre_topk_positions_noalloc(const float* scores_dev, int64_t L, int32_t k,
                                           int32_t* out_idx_dev, void* cuda_stream) {
  if (!scores_dev || L < 1 || k < 0 || (k > 0 && !out_idx_dev)) return ILRE_ERR_INVALID_ARG;
  if (L > kMaxL) return ILRE_ERR_CAPACITY;             // the static scratch holds kMaxL bits
  if (k > L) return ILRE_ERR_BUDGET;
  int device = -1;
  if (cudaGetDevice(&device) != cudaSuccess) return ILRE_ERR_CUDA;
  if (device < 0 || device >= kMaxDevices) return ILRE_ERR_UNSUPPORTED;
  uint32_t* bitmap = nullptr;
  if (scratch_for(device, &bitmap) != cudaSuccess) return ILRE_ERR_CUDA;
  topk_positions_kernel<<<1, kThreads, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      scores_dev, static_cast<int>(L), k, out_idx_dev, bitmap);
  return cudaGetLastError() == cudaSuccess ? ILRE_OK : ILRE_ERR_CUDA;
}
