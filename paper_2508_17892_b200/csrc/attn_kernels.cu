// Streaming chunked prefill attention of one chunk:
//   O[j, h, :] = sum_k softmax_k(q[j,h] . K[k, kv(h)] / sqrt(d)) V[k, kv(h), :],   k <= n_prefix + j,
// where the first n_prefix rows of K/V are the cached sink and sliding-window tokens (visible
// to every query of the chunk) and the remaining c rows the chunk's own (visible causally).
//
// One CTA per (128 query tokens, query head).  Both contractions run on the tensor cores:
// S = Q K^T into tensor memory, and O += P V with P written to shared memory as bf16 by the
// softmax warps.  Two sweeps over the (at most a dozen) key tiles: the first takes the row
// statistics, the second forms normalised probabilities, so that O accumulates in tensor memory
// without rescaling.  Key/value tiles come through one TMA ring.
#include <cuda_bf16.h>

#include "attn_kernels.cuh"
#include "sm100_ptx.cuh"

namespace ilre {

static constexpr int kAttnStages = 4;
static constexpr int kAttnTileBytes = 128 * 128 * 2;       // one 128 x 128 bf16 tile
static constexpr int kAttnTailBytes = 256;
static constexpr int kAttnSoftmaxWarps = 4;

struct AttnTail {
  uint64_t q_full;
  uint64_t kv_full[kAttnStages];
  uint64_t kv_empty[kAttnStages];
  uint64_t s_full[2];
  uint64_t s_empty[2];
  uint64_t p_full;
  uint64_t p_empty;
  uint64_t o_full;
  uint32_t tmem_base;
  int abort_flag;
};
static_assert(sizeof(AttnTail) <= kAttnTailBytes, "tail too large");

// Shared-memory matrix descriptor of an operand whose contiguous dimension is M or N (here: the
// value tile, head channels contiguous), 128-byte swizzle: 64-channel x 8-row atoms of 1024 bytes;
// `lbo` = byte distance of the next 64 channels, `sbo` = byte distance of the next 8 rows.
__device__ __forceinline__ uint64_t umma_desc_sw128_mn(uint32_t addr, uint32_t lbo, uint32_t sbo) {
  const uint32_t lo = ((addr >> 4) & 0x3FFFu) | (((lbo >> 4) & 0x3FFFu) << 16);
  const uint32_t hi = ((sbo >> 4) & 0x3FFFu) | (1u << 14) | (2u << 29);
  return (static_cast<uint64_t>(hi) << 32) | lo;
}

__global__ void __launch_bounds__(kAttnThreads, 1)
chunk_attention_kernel(const __grid_constant__ CUtensorMap map_q,
                       const __grid_constant__ CUtensorMap map_k,
                       const __grid_constant__ CUtensorMap map_v, const AttnParams p) {
  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t smem_base = smem_u32(smem);
  const uint32_t q_s = smem_base;
  const uint32_t ring_s = q_s + kAttnTileBytes;
  const uint32_t p_s = ring_s + kAttnStages * kAttnTileBytes;
  uint8_t* p_ptr = smem + (1 + kAttnStages) * kAttnTileBytes;
  AttnTail* tail = reinterpret_cast<AttnTail*>(smem + (2 + kAttnStages) * kAttnTileBytes);
  volatile int* abort_flag = &tail->abort_flag;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  const int j0 = blockIdx.x * 128;                      // first query token of this CTA
  const int h = blockIdx.y, g = h / (p.n_q / p.n_kv);
  const int last_q = min(j0 + 128, p.c) - 1;
  const int n_tiles = (p.n_prefix + last_q) / 128 + 1;   // key tiles that hold a visible key

  if (threadIdx.x == 0) {
    tail->abort_flag = 0;
    if (smem_base & 1023u) {
      tail->abort_flag = 1;
      atomicCAS(p.status, 0, kDevSmemAlign);
    }
    mbar_init(smem_u32(&tail->q_full), 1);
    for (int s = 0; s < kAttnStages; ++s) {
      mbar_init(smem_u32(&tail->kv_full[s]), 1);
      mbar_init(smem_u32(&tail->kv_empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&tail->s_full[b]), 1);
      mbar_init(smem_u32(&tail->s_empty[b]), kAttnSoftmaxWarps);
    }
    mbar_init(smem_u32(&tail->p_full), kAttnSoftmaxWarps);
    mbar_init(smem_u32(&tail->p_empty), 1);
    mbar_init(smem_u32(&tail->o_full), 1);
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&tail->tmem_base), 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tail->tmem_base;
  const uint32_t tmem_o = tmem_base + 256;
  const bool run = (*abort_flag == 0);

  // Ring items: sweep 1 = K_0 .. K_{T-1}; sweep 2 = K_0, V_0, K_1, V_1, ...
  if (warp == 0) {
    if (lane == 0 && run) {
      const uint32_t qf = smem_u32(&tail->q_full);
      mbar_arrive_expect_tx(qf, kAttnTileBytes);
      tma_load_2d(q_s, &map_q, h * 128, j0, qf);
      tma_load_2d(q_s + 16384, &map_q, h * 128 + 64, j0, qf);
      const int n_items = 3 * n_tiles;
      for (int it = 0; it < n_items; ++it) {
        const int s = it % kAttnStages;
        const uint32_t use = static_cast<uint32_t>(it / kAttnStages);
        if (!mbar_wait(smem_u32(&tail->kv_empty[s]), (use & 1u) ^ 1u, abort_flag, p.status,
                       kDevWaitKEmpty))
          break;
        const bool is_v = it >= n_tiles && ((it - n_tiles) & 1);
        const int t = it < n_tiles ? it : (it - n_tiles) >> 1;
        const CUtensorMap* map = is_v ? &map_v : &map_k;
        const uint32_t bar = smem_u32(&tail->kv_full[s]);
        mbar_arrive_expect_tx(bar, kAttnTileBytes);
        tma_load_2d(ring_s + s * kAttnTileBytes, map, g * 128, t * 128, bar);
        tma_load_2d(ring_s + s * kAttnTileBytes + 16384, map, g * 128 + 64, t * 128, bar);
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && run) {
      constexpr uint32_t idesc_s = umma_idesc_bf16(128, 128);
      constexpr uint32_t idesc_o = umma_idesc_bf16(128, 128) | (1u << 16);   // B = V: channels contiguous
      bool ok = mbar_wait(smem_u32(&tail->q_full), 0, abort_flag, p.status, kDevWaitQFull);
      tc_fence_after();
      uint32_t u = 0;                                     // S accumulators issued so far
      auto issue_s = [&](int item) -> bool {
        const uint32_t b = u & 1u, use = u >> 1;
        if (!mbar_wait(smem_u32(&tail->s_empty[b]), (use & 1u) ^ 1u, abort_flag, p.status,
                       kDevWaitAccEmpty))
          return false;
        const int s = item % kAttnStages;
        if (!mbar_wait(smem_u32(&tail->kv_full[s]), static_cast<uint32_t>(item / kAttnStages) & 1u,
                       abort_flag, p.status, kDevWaitKFull))
          return false;
        tc_fence_after();
        const uint32_t k_s = ring_s + s * kAttnTileBytes;
#pragma unroll
        for (int kb = 0; kb < 2; ++kb)
#pragma unroll
          for (int ks = 0; ks < 4; ++ks)
            umma_bf16(tmem_base + b * 128, umma_desc_sw128(q_s + kb * 16384 + ks * 32),
                      umma_desc_sw128(k_s + kb * 16384 + ks * 32), idesc_s, (kb | ks) != 0);
        umma_commit(smem_u32(&tail->kv_empty[s]));
        umma_commit(smem_u32(&tail->s_full[b]));
        ++u;
        return true;
      };
      for (int t = 0; t < n_tiles && ok; ++t) ok = issue_s(t);                 // sweep 1
      if (ok) ok = issue_s(n_tiles);                                           // S of tile 0, sweep 2
      for (int t = 0; t < n_tiles && ok; ++t) {
        if (t + 1 < n_tiles) ok = issue_s(n_tiles + 2 * (t + 1));
        if (!ok) break;
        const int item = n_tiles + 2 * t + 1;                                  // V_t
        const int s = item % kAttnStages;
        ok = mbar_wait(smem_u32(&tail->p_full), static_cast<uint32_t>(t) & 1u, abort_flag, p.status,
                       kDevWaitAccFull) &&
             mbar_wait(smem_u32(&tail->kv_full[s]), static_cast<uint32_t>(item / kAttnStages) & 1u,
                       abort_flag, p.status, kDevWaitKFull);
        if (!ok) break;
        tc_fence_after();
        const uint32_t v_s = ring_s + s * kAttnTileBytes;
#pragma unroll
        for (int kb = 0; kb < 2; ++kb)
#pragma unroll
          for (int ks = 0; ks < 4; ++ks)
            umma_bf16(tmem_o, umma_desc_sw128(p_s + kb * 16384 + ks * 32),
                      umma_desc_sw128_mn(v_s + (kb * 64 + ks * 16) * 128, 16384, 1024), idesc_o,
                      (t | kb | ks) != 0);
        umma_commit(smem_u32(&tail->kv_empty[s]));
        umma_commit(smem_u32(&tail->p_empty));
      }
      if (ok) umma_commit(smem_u32(&tail->o_full));
    }
  } else {
    const int quad = warp & 3;
    const int row = quad * 32 + lane;
    const int qj = j0 + row;
    const int limit = p.n_prefix + qj;                   // last visible key row of this query
    const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(quad * 32) << 16);
    const float c2 = p.c2;
    bool ok = run;
    uint32_t u = 0;
    // ---- sweep 1: row maximum and sum of exponentials ----
    float m = -1e30f, z = 0.f;
    for (int t = 0; t < n_tiles && ok; ++t, ++u) {
      const uint32_t b = u & 1u, use = u >> 1;
      ok = mbar_wait(smem_u32(&tail->s_full[b]), use & 1u, abort_flag, p.status, kDevWaitAccFull);
      if (!ok) break;
      tc_fence_after();
#pragma unroll 1
      for (int q4 = 0; q4 < 4; ++q4) {
        float v[32];
        tmem_ld32(lane_base + b * 128 + q4 * 32, v);
        tmem_ld_wait();
        const int k0 = t * 128 + q4 * 32;
        float cm = -INFINITY;
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          if (k0 + i > limit) v[i] = -INFINITY;
          cm = fmaxf(cm, v[i]);
        }
        const float m_new = fmaxf(m, cm);
        const float nm = -m_new * c2;
        float sum = 0.f;
#pragma unroll
        for (int i = 0; i < 32; ++i) sum += ex2_approx(fmaf(v[i], c2, nm));
        z = fmaf(z, ex2_approx((m - m_new) * c2), sum);
        m = m_new;
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&tail->s_empty[b]));
    }
    const float nl = -(m * c2 + log2f(z));               // -lse in log2 units
    // ---- sweep 2: normalised probabilities as the bf16 A operand of O += P V ----
    for (int t = 0; t < n_tiles && ok; ++t, ++u) {
      const uint32_t b = u & 1u, use = u >> 1;
      ok = mbar_wait(smem_u32(&tail->s_full[b]), use & 1u, abort_flag, p.status, kDevWaitAccFull);
      if (!ok) break;
      tc_fence_after();
      uint32_t packed[64];
#pragma unroll
      for (int q4 = 0; q4 < 4; ++q4) {
        float v[32];
        tmem_ld32(lane_base + b * 128 + q4 * 32, v);
        tmem_ld_wait();
        const int k0 = t * 128 + q4 * 32;
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
          const float p0 = (k0 + i <= limit) ? ex2_approx(fmaf(v[i], c2, nl)) : 0.f;
          const float p1 = (k0 + i + 1 <= limit) ? ex2_approx(fmaf(v[i + 1], c2, nl)) : 0.f;
          const __nv_bfloat162 pr = __floats2bfloat162_rn(p0, p1);
          packed[q4 * 16 + (i >> 1)] = *reinterpret_cast<const uint32_t*>(&pr);
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&tail->s_empty[b]));
      // the previous tile's P must have been consumed by its MMAs
      ok = mbar_wait(smem_u32(&tail->p_empty), (static_cast<uint32_t>(t) & 1u) ^ 1u, abort_flag,
                     p.status, kDevWaitAccEmpty);
      if (!ok) break;
      // P[row][key]: two halves of 64 keys, rows of 128 bytes, 16-byte groups XOR-swizzled by
      // the row index (the layout TMA's 128-byte swizzle produces for the other operands)
#pragma unroll
      for (int grp = 0; grp < 16; ++grp) {
        const int half = grp >> 3, c16 = grp & 7;
        uint4* dst = reinterpret_cast<uint4*>(p_ptr + half * 16384 + row * 128 +
                                              ((c16 ^ (row & 7)) << 4));
        *dst = make_uint4(packed[grp * 4], packed[grp * 4 + 1], packed[grp * 4 + 2],
                          packed[grp * 4 + 3]);
      }
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&tail->p_full));
    }
    // ---- output ----
    if (ok) ok = mbar_wait(smem_u32(&tail->o_full), 0, abort_flag, p.status, kDevWaitAccFull);
    if (ok) {
      tc_fence_after();
      uint16_t* dst = p.out + (static_cast<size_t>(qj) * p.n_q + h) * 128;
#pragma unroll 1
      for (int q4 = 0; q4 < 4; ++q4) {
        float v[32];
        tmem_ld32(lane_base + 256 + q4 * 32, v);
        tmem_ld_wait();
        if (qj < p.c) {
          uint32_t w[16];
#pragma unroll
          for (int i = 0; i < 32; i += 2) {
            const __nv_bfloat162 pr = __floats2bfloat162_rn(v[i], v[i + 1]);
            w[i >> 1] = *reinterpret_cast<const uint32_t*>(&pr);
          }
          uint4* d4 = reinterpret_cast<uint4*>(dst + q4 * 32);
#pragma unroll
          for (int q = 0; q < 4; ++q) d4[q] = make_uint4(w[4 * q], w[4 * q + 1], w[4 * q + 2], w[4 * q + 3]);
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

size_t attn_smem_bytes() {
  return static_cast<size_t>(2 + kAttnStages) * kAttnTileBytes + kAttnTailBytes;
}

cudaError_t launch_chunk_attention(const CUtensorMap& map_q, const CUtensorMap& map_k,
                                   const CUtensorMap& map_v, const AttnParams& p, cudaStream_t st) {
  const size_t smem = attn_smem_bytes();
  cudaError_t e = cudaFuncSetAttribute(chunk_attention_kernel,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       static_cast<int>(smem));
  if (e != cudaSuccess) return e;
  dim3 grid((p.c + 127) / 128, p.n_q);
  chunk_attention_kernel<<<grid, kAttnThreads, smem, st>>>(map_q, map_k, map_v, p);
  return cudaGetLastError();
}

}  // namespace ilre
