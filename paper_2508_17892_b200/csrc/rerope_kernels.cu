// Eq. 7: K~^{C_i} = R(D_i) K^{C_i} for the chunks i < N_C - 1 of the retrieval layer's key
// cache, D_i = (N_C - 1 - i) * chunk positions, so that every cached key sits within two
// chunks of the query.  A streaming kernel bound by HBM: every byte of the rotated part of
// the cache is read once and written once.  The file also holds the small gather that turns
// the recalled positions into the compressed prompt.
#include <cuda_bf16.h>

#include "rerope_kernels.cuh"

namespace ilre {

__global__ void rope_table_kernel(float2* __restrict__ table, int n_rows, int chunk, double theta) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= n_rows * kRopeHalfDim) return;
  const int row = idx / kRopeHalfDim, c = idx % kRopeHalfDim;
  const double dist = static_cast<double>(row + 1) * static_cast<double>(chunk);
  const double ang = dist * pow(theta, -2.0 * static_cast<double>(c) / (2.0 * kRopeHalfDim));
  double sn, cs;
  sincos(ang, &sn, &cs);
  table[idx] = make_float2(static_cast<float>(cs), static_cast<float>(sn));
}

// Rotates the eight channel pairs held by `lo` (channels 8s .. 8s+7) and `hi` (channels
// 64+8s .. 64+8s+7): lo' = lo cos - hi sin, hi' = lo sin + hi cos, in fp32, rounded to bf16
// (nearest even).
__device__ __forceinline__ void rotate8(uint4& lo, uint4& hi, const float2* __restrict__ cs) {
  uint32_t* l = reinterpret_cast<uint32_t*>(&lo);
  uint32_t* h = reinterpret_cast<uint32_t*>(&hi);
  const float4* cs4 = reinterpret_cast<const float4*>(cs);
#pragma unroll
  for (int w = 0; w < 4; ++w) {
    const float4 t = __ldg(cs4 + w);                       // (cos, sin) of two channel pairs
    const float l0 = __uint_as_float(l[w] << 16), l1 = __uint_as_float(l[w] & 0xFFFF0000u);
    const float h0 = __uint_as_float(h[w] << 16), h1 = __uint_as_float(h[w] & 0xFFFF0000u);
    const float nl0 = fmaf(l0, t.x, -h0 * t.y), nh0 = fmaf(l0, t.y, h0 * t.x);
    const float nl1 = fmaf(l1, t.z, -h1 * t.w), nh1 = fmaf(l1, t.w, h1 * t.z);
    const __nv_bfloat162 pl = __floats2bfloat162_rn(nl0, nl1);
    const __nv_bfloat162 ph = __floats2bfloat162_rn(nh0, nh1);
    l[w] = *reinterpret_cast<const uint32_t*>(&pl);
    h[w] = *reinterpret_cast<const uint32_t*>(&ph);
  }
}

static constexpr int kReropeThreads = 256;
static constexpr int kReropeUnroll = 1;        // (row, segment) items per thread in flight
static constexpr int kReropeCtasPerSm = 4;

__global__ void __launch_bounds__(kReropeThreads)
rerope_kernel(const ReropeParams p) {
  // One item = one 16-byte segment pair (low half, high half) of one (position, kv head) row;
  // eight consecutive threads cover a row, a warp four rows = 1 KB of contiguous cache.
  const long long n_items = p.L * p.n_kv * 8;
  const bool copy_tail = p.k_out != p.k_in;
  const long long rot_end = (p.n_chunks >= 2)                // first position of chunk N_C - 1
      ? static_cast<long long>(p.n_sink) + (p.n_chunks - 2) * p.chunk : 0;
  const long long stride = static_cast<long long>(gridDim.x) * kReropeThreads;
  const long long limit = copy_tail ? n_items : rot_end * p.n_kv * 8;
  for (long long base = static_cast<long long>(blockIdx.x) * kReropeThreads + threadIdx.x;
       base < limit; base += stride * kReropeUnroll) {
    uint4 lo[kReropeUnroll], hi[kReropeUnroll];
#pragma unroll
    for (int u = 0; u < kReropeUnroll; ++u) {
      const long long item = base + u * stride;
      if (item < limit) {
        const long long row = item >> 3;
        const int seg = static_cast<int>(item & 7);
        lo[u] = p.k_in[row * 16 + seg];
        hi[u] = p.k_in[row * 16 + 8 + seg];
      }
    }
#pragma unroll
    for (int u = 0; u < kReropeUnroll; ++u) {
      const long long item = base + u * stride;
      if (item < limit) {
        const long long row = item >> 3;
        const int seg = static_cast<int>(item & 7);
        const long long t = row / p.n_kv;
        if (t < rot_end) {
          const long long i = (t < p.n_sink) ? 1 : 1 + (t - p.n_sink) / p.chunk;   // 1-based chunk
          const long long dist_row = p.n_chunks - 1 - i - 1;                       // D / chunk - 1
          rotate8(lo[u], hi[u], p.table + dist_row * kRopeHalfDim + seg * 8);
        }
        p.k_out[row * 16 + seg] = lo[u];
        p.k_out[row * 16 + 8 + seg] = hi[u];
      }
    }
  }
}

// Eq. 6: K^{S,i} = R^{i-2}(D_C) K^S, the sink keys of a layer before the retrieval layer as
// chunk i > 2 sees them.  The power of the rotation is one rotation by (i - 2) * D_C, taken
// from the cached (never re-rotated) sink keys, so the keys are rounded once however large i is.
// `cs` is the table row of that distance.  A few KB: one item per thread.
__global__ void rotate_rows_kernel(const uint4* __restrict__ k_in, uint4* __restrict__ k_out,
                                   long long n_items, const float2* __restrict__ cs) {
  const long long item = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (item >= n_items) return;
  const long long row = item >> 3;
  const int seg = static_cast<int>(item & 7);
  uint4 lo = k_in[row * 16 + seg], hi = k_in[row * 16 + 8 + seg];
  if (cs) rotate8(lo, hi, cs + seg * 8);
  k_out[row * 16 + seg] = lo;
  k_out[row * 16 + 8 + seg] = hi;
}

cudaError_t launch_rotate_rows(const uint4* k_in, uint4* k_out, long long n_rows,
                               const float2* table_row, cudaStream_t st) {
  const long long n_items = n_rows * 8;
  if (n_items < 1) return cudaSuccess;
  rotate_rows_kernel<<<static_cast<unsigned>((n_items + 255) / 256), 256, 0, st>>>(k_in, k_out, n_items,
                                                                                  table_row);
  return cudaGetLastError();
}

// Algorithm 1's last step and the hand-over to the inference engine: the compressed prompt is
// the input ids at the chosen positions followed by the ids of the query part.
__global__ void gather_ids_kernel(const int32_t* __restrict__ ids, long long L,
                                  const int32_t* __restrict__ idx, int n_idx,
                                  const int32_t* __restrict__ query_ids, int n_query,
                                  int32_t* __restrict__ out) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n_idx) {
    const int pos = idx[i];
    out[i] = (pos >= 0 && pos < L) ? ids[pos] : -1;      // -1 marks a position outside the context
  } else if (i < n_idx + n_query) {
    out[i] = query_ids[i - n_idx];
  }
}

cudaError_t launch_gather_ids(const int32_t* ids, long long L, const int32_t* idx, int n_idx,
                              const int32_t* query_ids, int n_query, int32_t* out,
                              cudaStream_t st) {
  const int n = n_idx + n_query;
  if (n < 1) return cudaSuccess;
  gather_ids_kernel<<<(n + 255) / 256, 256, 0, st>>>(ids, L, idx, n_idx, query_ids, n_query, out);
  return cudaGetLastError();
}

cudaError_t launch_rope_table(float2* table, int n_rows, int chunk, double theta,
                              cudaStream_t st) {
  if (n_rows < 1) return cudaSuccess;
  const int n = n_rows * kRopeHalfDim;
  rope_table_kernel<<<(n + 255) / 256, 256, 0, st>>>(table, n_rows, chunk, theta);
  return cudaGetLastError();
}

cudaError_t launch_rerope(const ReropeParams& p, int n_sm, cudaStream_t st) {
  // Four CTAs of 256 threads per SM, all resident, one item per thread in flight: measured
  // fastest (0.70 ms for a 2 GiB cache; 8 CTAs or 2-8 items in flight: 0.72-1.17 ms).
  rerope_kernel<<<n_sm * kReropeCtasPerSm, kReropeThreads, 0, st>>>(p);
  return cudaGetLastError();
}

}  // namespace ilre
