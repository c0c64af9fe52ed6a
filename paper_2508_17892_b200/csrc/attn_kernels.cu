// Streaming chunked prefill attention of one chunk:
//   O[j, h, :] = sum_k softmax_k(q[j,h] . K[k, kv(h)] / sqrt(d)) V[k, kv(h), :],   k <= n_prefix + j,
// where the first n_prefix rows of K/V are the cached sink and sliding-window tokens (visible
// to every query of the chunk) and the remaining c rows the chunk's own (visible causally).
//
// One CTA per (128 query tokens, pair of query heads that share a kv head).  Both contractions
// run on the tensor cores: S = Q K^T into tensor memory, and O += P V with P written to shared
// memory as bf16 by the softmax warps (four per head, one thread per query row).  The two heads
// are two independent streams over the same key/value tiles (one TMA ring feeds both): while
// the softmax warps of one stream work on their S tile, the tensor cores serve the other
// stream.  Two threads issue the MMAs, one every S and one every O += P V, because an issuing
// thread is held until the tensor pipe takes its instruction.  One sweep over the key tiles
// with an online softmax: probabilities are taken against a per-row reference maximum, O
// accumulates in tensor memory and is rescaled there only when a row's maximum has run ahead
// of its reference by more than 2^8 (rare after the first tiles); the row sums divide the
// output at the end.  Heavier CTAs (later query tiles see more keys) are launched first.
#include <cuda_bf16.h>

#include "attn_kernels.cuh"
#include "sm100_ptx.cuh"

namespace ilre {

static constexpr int kAttnStages = 3;
static constexpr int kAttnTileBytes = 128 * 128 * 2;       // one 128 x 128 bf16 tile
static constexpr int kAttnTailBytes = 256;
static constexpr int kAttnPolyPairs = 2;                   // of every 16 pairs of exponentials
static constexpr int kAttnSoftmaxWarps = 4;                // per stream: one per TMEM lane quadrant

struct AttnTail {
  uint64_t q_full;
  uint64_t kv_full[kAttnStages];
  uint64_t kv_empty[kAttnStages];
  uint64_t s_full[2];          // per stream
  uint64_t s_empty[2];
  uint64_t p_full[2];
  uint64_t p_empty[2];
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
  const uint32_t q_s = smem_base;                                        // 2 tiles
  const uint32_t ring_s = q_s + 2 * kAttnTileBytes;
  const uint32_t p_s = ring_s + kAttnStages * kAttnTileBytes;           // 2 tiles
  uint8_t* p_ptr = smem + (2 + kAttnStages) * kAttnTileBytes;
  AttnTail* tail = reinterpret_cast<AttnTail*>(smem + (4 + kAttnStages) * kAttnTileBytes);
  volatile int* abort_flag = &tail->abort_flag;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // Work items in launch order, heaviest first (later query tiles see more keys): the query
  // tiles from split_from on with one CTA per head, then the others with one CTA per head pair.
  int qt, h0, n_streams;
  {
    const int n_single = p.pair ? (p.n_qt - p.split_from) * p.n_q : p.n_qt * p.n_q;
    const int b = blockIdx.x;
    if (b < n_single) {
      qt = p.n_qt - 1 - b / p.n_q;
      h0 = b % p.n_q;
      n_streams = 1;
    } else {
      const int n_pairs = p.n_q / 2, r = b - n_single;
      qt = p.split_from - 1 - r / n_pairs;
      h0 = 2 * (r % n_pairs);                            // head of stream 0; stream 1 = h0 + 1
      n_streams = 2;
    }
  }
  const int j0 = qt * 128;                               // first query token
  const int g = h0 / (p.n_q / p.n_kv);
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
    for (int x = 0; x < 2; ++x) {
      mbar_init(smem_u32(&tail->s_full[x]), 1);
      mbar_init(smem_u32(&tail->s_empty[x]), kAttnSoftmaxWarps);
      mbar_init(smem_u32(&tail->p_full[x]), kAttnSoftmaxWarps);
      mbar_init(smem_u32(&tail->p_empty[x]), 1);
    }
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
  const bool run = (*abort_flag == 0);

  // TMEM columns: S of stream x at 128 x, O of stream x at 256 + 128 x.
  // Ring items (key and value tiles) are each used by both streams.
  if (warp == 0) {
    if (lane == 0 && run) {
      const uint32_t qf = smem_u32(&tail->q_full);
      mbar_arrive_expect_tx(qf, n_streams * kAttnTileBytes);
      for (int x = 0; x < n_streams; ++x) {
        tma_load_2d(q_s + x * kAttnTileBytes, &map_q, (h0 + x) * 128, j0, qf);
        tma_load_2d(q_s + x * kAttnTileBytes + 16384, &map_q, (h0 + x) * 128 + 64, j0, qf);
      }
      // Ring order K_0, K_1, V_0, K_2, V_1, ..., K_{n-1}, V_{n-2}, V_{n-1}: the key tile runs
      // one tile ahead of the value tile, because S of the next tile is issued while the
      // softmax of the current one is still running (see the MMA warp).
      const int n_items = 2 * n_tiles;
      for (int it = 0; it < n_items; ++it) {
        const int s = it % kAttnStages;
        const uint32_t use = static_cast<uint32_t>(it / kAttnStages);
        if (!mbar_wait(smem_u32(&tail->kv_empty[s]), (use & 1u) ^ 1u, abort_flag, p.status,
                       kDevWaitKEmpty))
          break;
        const bool is_k = (it == 0) || ((it & 1) && it != n_items - 1);
        const int t = (it == 0) ? 0 : (it == n_items - 1) ? n_tiles - 1 : is_k ? (it + 1) / 2 : it / 2 - 1;
        const CUtensorMap* map = is_k ? &map_k : &map_v;
        const uint32_t bar = smem_u32(&tail->kv_full[s]);
        mbar_arrive_expect_tx(bar, kAttnTileBytes);
        tma_load_2d(ring_s + s * kAttnTileBytes, map, g * 128, t * 128, bar);
        tma_load_2d(ring_s + s * kAttnTileBytes + 16384, map, g * 128 + 64, t * 128, bar);
      }
    }
  } else if (warp == 1 || warp == 2) {
    // Two MMA-issuing threads.  tcgen05.mma holds its issuing thread until the tensor pipe
    // takes the instruction, so one thread alone leaves the pipe idle whenever it tests
    // barriers or commits.  Warp 1 issues every S = Q K^T (both streams), warp 2 every
    // O += P V; each polls its two streams' barriers without blocking and issues whichever is
    // ready, and the bookkeeping of one overlaps the MMAs of the other.  A key tile's ring
    // slot is released by the S issuer, a value tile's by the PV issuer, once both streams
    // have issued the MMAs that read it.
    if (lane == 0 && run) {
      constexpr uint32_t idesc_s = umma_idesc_bf16(128, 128);
      constexpr uint32_t idesc_o = umma_idesc_bf16(128, 128) | (1u << 16);   // B = V: channels contiguous
      const bool s_role = (warp == 1);
      auto k_item = [&](int t) -> int { return t == 0 ? 0 : 2 * t - 1; };
      auto v_item = [&](int t) -> int { return t < n_tiles - 1 ? 2 * t + 2 : 2 * n_tiles - 1; };
      auto ring_ready = [&](int item) -> bool {
        return mbar_test_wait(smem_u32(&tail->kv_full[item % kAttnStages]),
                              static_cast<uint32_t>(item / kAttnStages) & 1u);
      };
      bool ok = true;
      if (s_role) {
        ok = mbar_wait(smem_u32(&tail->q_full), 0, abort_flag, p.status, kDevWaitQFull);
        tc_fence_after();
      }
      int next[2] = {0, 0};                               // per stream: next tile to issue
      if (n_streams == 1) next[1] = n_tiles;
      int released = 0;
      long long t_idle = 0;
      uint32_t spins = 0;
      while (ok && (next[0] < n_tiles || next[1] < n_tiles)) {
        bool progress = false;
#pragma unroll
        for (int x = 0; x < 2; ++x) {
          const int t = next[x];
          if (t >= n_tiles) continue;
          if (s_role) {
            // S_x(t): needs the key tile and, after the first, S_x(t-1) read out of tensor memory
            if (ring_ready(k_item(t)) &&
                (t == 0 || mbar_test_wait(smem_u32(&tail->s_empty[x]), static_cast<uint32_t>(t - 1) & 1u))) {
              tc_fence_after();
              const uint32_t k_s = ring_s + (k_item(t) % kAttnStages) * kAttnTileBytes;
              const uint32_t qx = q_s + x * kAttnTileBytes;
#pragma unroll
              for (int kb = 0; kb < 2; ++kb)
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)
                  umma_bf16(tmem_base + x * 128, umma_desc_sw128(qx + kb * 16384 + ks * 32),
                            umma_desc_sw128(k_s + kb * 16384 + ks * 32), idesc_s, (kb | ks) != 0);
              umma_commit(smem_u32(&tail->s_full[x]));
              next[x] = t + 1;
              progress = true;
              while (released < min(next[0], next[1])) {
                umma_commit(smem_u32(&tail->kv_empty[k_item(released) % kAttnStages]));
                ++released;
              }
            }
          } else {
            // O_x += P_x(t) V_t: needs P written and the value tile
            if (mbar_test_wait(smem_u32(&tail->p_full[x]), static_cast<uint32_t>(t) & 1u) &&
                ring_ready(v_item(t))) {
              tc_fence_after();
              const uint32_t v_s = ring_s + (v_item(t) % kAttnStages) * kAttnTileBytes;
              const uint32_t px = p_s + x * kAttnTileBytes;
#pragma unroll
              for (int kb = 0; kb < 2; ++kb)
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)
                  umma_bf16(tmem_base + 256 + x * 128, umma_desc_sw128(px + kb * 16384 + ks * 32),
                            umma_desc_sw128_mn(v_s + (kb * 64 + ks * 16) * 128, 16384, 1024), idesc_o,
                            (t | kb | ks) != 0);
              umma_commit(smem_u32(&tail->p_empty[x]));
              next[x] = t + 1;
              progress = true;
              while (released < min(next[0], next[1])) {
                umma_commit(smem_u32(&tail->kv_empty[v_item(released) % kAttnStages]));
                ++released;
              }
            }
          }
        }
        // bounded: give up when nothing became ready for kWaitCycleLimit cycles
        if (progress) {
          spins = 0;
        } else {
          if (spins == 0) t_idle = clock64();
          if ((++spins & 0x3FF) == 0) {
            if (*abort_flag) {
              ok = false;
            } else if (clock64() - t_idle > kWaitCycleLimit) {
              *abort_flag = 1;
              atomicCAS(p.status, 0, kDevWaitAccFull);
              ok = false;
            }
          }
        }
      }
      if (ok && !s_role) umma_commit(smem_u32(&tail->o_full));
    }
  } else if (warp >= 3 && (warp - 3) / kAttnSoftmaxWarps < n_streams) {
    // Softmax warps of stream x: warp w reads TMEM lane quadrant w % 4, so a thread owns one
    // query row: its 128 logits of the tile, its running reference and sum, its row of P and
    // of O.  No thread ever needs another's values.
    const int x = (warp - 3) / kAttnSoftmaxWarps;
    const int quad = warp & 3;
    const int row = quad * 32 + lane;
    const int qj = j0 + row;
    const int h = h0 + x;
    const int limit = p.n_prefix + qj;                   // last visible key row of this query
    const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(quad * 32) << 16);
    const uint32_t s_tm = lane_base + x * 128, o_tm = lane_base + 256 + x * 128;
    uint8_t* p_mine = p_ptr + x * kAttnTileBytes;
    const float c2 = p.c2;
    bool ok = run;
    // Online softmax: `ref` is the row's reference maximum (raw logits), `l` the sum of
    // 2^((s - ref) c2) over the keys seen so far.
    constexpr float kRefSlack = 8.f;                     // log2 units
    float ref = -INFINITY, l = 0.f;
    for (int t = 0; t < n_tiles && ok; ++t) {
      ok = mbar_wait(smem_u32(&tail->s_full[x]), static_cast<uint32_t>(t) & 1u, abort_flag,
                     p.status, kDevWaitAccFull);
      if (!ok) break;
      // The row's 128 logits stay in registers for both the maximum and the exponentials, so
      // S leaves tensor memory once and the tensor cores get it back for the next tile right
      // away.  Only the tiles on the causal diagonal need the mask; there the hidden logits
      // become -inf, which the code below turns into probability 0.
      float vv[4][32];
#define V(i) vv[(i) >> 5][(i) & 31]
      tc_fence_after();
      tmem_ld32(s_tm, vv[0]);
      tmem_ld32(s_tm + 32, vv[1]);
      tmem_ld32(s_tm + 64, vv[2]);
      tmem_ld32(s_tm + 96, vv[3]);
      tmem_ld_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&tail->s_empty[x]));
      const int k0 = t * 128;
      if (k0 + 127 > p.n_prefix + j0) {
#pragma unroll
        for (int i = 0; i < 128; ++i) V(i) = (k0 + i <= limit) ? V(i) : -INFINITY;
      }
      float m0 = fmax3(V(0), V(1), V(2)), m1 = fmax3(V(3), V(4), V(5));
#pragma unroll
      for (int i = 6; i < 126; i += 4) {
        m0 = fmax3(m0, V(i), V(i + 1));
        m1 = fmax3(m1, V(i + 2), V(i + 3));
      }
      const float cm = fmax3(m0, m1, fmaxf(V(126), V(127)));
      // move the reference only when the maximum has run ahead of it
      float scale = 1.f;
      if ((cm - ref) * c2 > kRefSlack || ref == -INFINITY) {
        scale = (ref == -INFINITY) ? 0.f : ex2_approx((ref - cm) * c2);
        ref = (cm == -INFINITY) ? ref : cm;
      }
      const float nr = (ref == -INFINITY) ? 0.f : -ref * c2;
      // the previous tile's P must have been consumed (and O updated) by its MMAs
      ok = mbar_wait(smem_u32(&tail->p_empty[x]), (static_cast<uint32_t>(t) & 1u) ^ 1u, abort_flag,
                     p.status, kDevWaitAccEmpty);
      if (!ok) break;
      // Exponentials in groups of 32 keys; each group's bf16 pairs go straight to P[row][key]
      // (two halves of 64 keys, rows of 128 bytes, 16-byte groups XOR-swizzled by the row index:
      // the layout TMA's 128-byte swizzle produces for the other operands), so the stores
      // drain while the next group is computed.
      float2 sum2 = make_float2(0.f, 0.f);
#pragma unroll
      for (int g32 = 0; g32 < 4; ++g32) {
        uint32_t w[16];
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
          const float2 a = ffma2(make_float2(V(g32 * 32 + i), V(g32 * 32 + i + 1)), make_float2(c2, c2),
                                 make_float2(nr, nr));
          // kAttnPolyPairs of every 16 pairs take 2^x from the FMA-pipe polynomial: the two
          // streams share each scheduler's special-function unit, which is the busiest pipe
          const int pr16 = i >> 1;
          const bool poly = ((pr16 + 1) * kAttnPolyPairs) / 16 > (pr16 * kAttnPolyPairs) / 16;
          const float2 pp = poly ? exp2_poly2(a) : make_float2(ex2_approx(a.x), ex2_approx(a.y));
          sum2 = fadd2(sum2, pp);
          const __nv_bfloat162 pr = __floats2bfloat162_rn(pp.x, pp.y);
          w[i >> 1] = *reinterpret_cast<const uint32_t*>(&pr);
        }
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const int c16 = g32 * 4 + c;
          uint4* dst = reinterpret_cast<uint4*>(p_mine + (c16 >> 3) * 16384 + row * 128 +
                                                (((c16 & 7) ^ (row & 7)) << 4));
          *dst = make_uint4(w[c * 4], w[c * 4 + 1], w[c * 4 + 2], w[c * 4 + 3]);
        }
      }
      l = fmaf(l, scale, sum2.x + sum2.y);
      if (t > 0 && __any_sync(0xFFFFFFFFu, scale != 1.f)) {
        // rescale this warp's 32 rows of O to the new references
        tc_fence_after();
#pragma unroll 1
        for (int q4 = 0; q4 < 4; ++q4) {
          float o[32];
          tmem_ld32(o_tm + q4 * 32, o);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 32; ++i) o[i] *= scale;
          tmem_st32(o_tm + q4 * 32, o);
        }
        tmem_st_wait();
        tc_fence_before();
      }
#undef V
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&tail->p_full[x]));
    }
    // ---- output: O / sum, this thread's row ----
    const float inv_l = 1.f / l;
    if (ok) ok = mbar_wait(smem_u32(&tail->o_full), 0, abort_flag, p.status, kDevWaitAccFull);
    if (ok) {
      tc_fence_after();
      uint16_t* dst = p.out + (static_cast<size_t>(qj) * p.n_q + h) * 128;
#pragma unroll 1
      for (int q4 = 0; q4 < 4; ++q4) {
        float v[32];
        tmem_ld32(o_tm + q4 * 32, v);
        tmem_ld_wait();
        if (qj < p.c) {
          uint32_t w[16];
#pragma unroll
          for (int i = 0; i < 32; i += 2) {
            const __nv_bfloat162 pr = __floats2bfloat162_rn(v[i] * inv_l, v[i + 1] * inv_l);
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
  return static_cast<size_t>(4 + kAttnStages) * kAttnTileBytes + kAttnTailBytes;
}

cudaError_t launch_chunk_attention(const CUtensorMap& map_q, const CUtensorMap& map_k,
                                   const CUtensorMap& map_v, AttnParams p, int n_sm, cudaStream_t st) {
  const size_t smem = attn_smem_bytes();
  cudaError_t e = cudaFuncSetAttribute(chunk_attention_kernel,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       static_cast<int>(smem));
  if (e != cudaSuccess) return e;
  p.n_qt = (p.c + 127) / 128;
  p.split_from = p.n_qt;
  long long n_cta = static_cast<long long>(p.n_qt) * (p.pair ? p.n_q / 2 : p.n_q);
  if (p.pair) {
    // A short chunk leaves SMs idle while the wave lasts as long as its heaviest CTA: give the
    // heaviest query tiles one CTA per head for as long as everything still fits one wave.
    while (p.split_from > 0 && n_cta + p.n_q / 2 <= n_sm) {
      --p.split_from;
      n_cta += p.n_q / 2;
    }
  }
  chunk_attention_kernel<<<static_cast<unsigned>(n_cta), kAttnThreads, smem, st>>>(map_q, map_k, map_v, p);
  return cudaGetLastError();
}

}  // namespace ilre
