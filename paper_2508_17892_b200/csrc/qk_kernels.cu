// Query-context attention kernels of the recall path (Eq. 4 and Eq. 5 of the paper).
//
// The [heads, q_len, L] probability tensor is never written to memory.  Two passes over the
// key cache, both TMA -> shared memory -> tcgen05.mma -> tensor memory:
//   row statistics: D[row, key] tiles, one thread per query row keeps an online (max, sum-exp);
//   scores:         D[key, row] tiles (operands swapped), one thread per context position keeps
//                   max over rows of (logit - lse_row); exp is monotone, so one exp per position
//                   is taken afterwards.
#include "qk_kernels.cuh"
#include <utility>
#include "sm100_ptx.cuh"

namespace ilre {

// ---------------------------------------------------------------------------------------
// shared-memory tail layout (after the Q block and the K stages)
// ---------------------------------------------------------------------------------------
struct SmemTail {
  uint64_t q_full;
  uint64_t k_full[kMaxStages];
  uint64_t k_empty[kMaxStages];
  uint64_t acc_full[4];
  uint64_t acc_empty[4];
  uint32_t tmem_base;
  int abort_flag;
  long long stamp_cycles;            // start of the optional clock stamp (kept out of registers)
  unsigned long long stamp_ns;
};
static_assert(sizeof(SmemTail) <= kSmemTailBytes, "tail too large");

struct CtaItem {
  int chunk, group, g;
  int tile_begin, n_tiles;
};

__device__ __forceinline__ CtaItem decode_item(const QkParams& p) {
  CtaItem it;
  it.chunk = blockIdx.x / p.n_groups;
  it.group = blockIdx.x % p.n_groups;
  it.g = it.group / p.n_rb;
  const long long t0 = static_cast<long long>(it.chunk) * p.n_tiles / p.cpg;
  const long long t1 = static_cast<long long>(it.chunk + 1) * p.n_tiles / p.cpg;
  it.tile_begin = static_cast<int>(t0);
  it.n_tiles = static_cast<int>(t1 - t0);
  return it;
}

// Common prologue: barrier init, TMEM allocation.  Returns the TMEM base address.
__device__ __forceinline__ uint32_t cta_setup(SmemTail* tail, uint32_t smem_base, int stages,
                                              int n_acc, int acc_readers, int* status,
                                              int k_releasers = 1) {
  const int warp = threadIdx.x >> 5;
  if (threadIdx.x == 0) {
    tail->abort_flag = 0;
    if (smem_base & 1023u) {                       // swizzled tiles need 1024-byte alignment
      tail->abort_flag = 1;
      atomicCAS(status, 0, kDevSmemAlign);
    }
    mbar_init(smem_u32(&tail->q_full), 1);
    for (int s = 0; s < stages; ++s) {
      mbar_init(smem_u32(&tail->k_full[s]), 1);
      mbar_init(smem_u32(&tail->k_empty[s]), k_releasers);
    }
    for (int b = 0; b < n_acc; ++b) {
      mbar_init(smem_u32(&tail->acc_full[b]), 1);
      mbar_init(smem_u32(&tail->acc_empty[b]), acc_readers);
    }
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&tail->tmem_base), 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  return tail->tmem_base;
}

__device__ __forceinline__ void cta_teardown(uint32_t tmem_base) {
  tc_fence_before();
  __syncthreads();
  if ((threadIdx.x >> 5) == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

// TMA producer: the resident Q block once, then the K tiles of this CTA's key range.
__device__ __forceinline__ void producer_loop(const CUtensorMap* tmapK, const CUtensorMap* tmapQ,
                                              const QkParams& p, const CtaItem& it,
                                              SmemTail* tail, uint32_t q_s, uint32_t k_s,
                                              int skip_tiles = 0) {
  volatile int* abort_flag = &tail->abort_flag;
  const uint32_t qf = smem_u32(&tail->q_full);
  mbar_arrive_expect_tx(qf, static_cast<uint32_t>(p.rb_rows) * 256u);
  for (int kb = 0; kb < 2; ++kb)
    for (int mt = 0; mt < p.rb_rows / 128; ++mt)
      tma_load_2d(q_s + kb * p.rb_rows * 128 + mt * 16384, tmapQ, kb * 64,
                  it.group * p.rb_rows + mt * 128, qf);
  // ring position as (stage, phase) counters: no division by the run-time stage count
  int s = 0;
  uint32_t phase = 0;
  for (int i = 0; i < it.n_tiles - skip_tiles; ++i) {
    if (!mbar_wait(smem_u32(&tail->k_empty[s]), phase ^ 1u, abort_flag, p.status, kDevWaitKEmpty))
      break;
    const uint32_t kf = smem_u32(&tail->k_full[s]);
    mbar_arrive_expect_tx(kf, kStageBytes);
    const int row = (it.tile_begin + i) * kTileKeys;
    tma_load_2d(k_s + s * kStageBytes, tmapK, it.g * 128, row, kf);
    tma_load_2d(k_s + s * kStageBytes + 16384, tmapK, it.g * 128 + 64, row, kf);
    if (++s == p.stages) { s = 0; phase ^= 1u; }
  }
}

// Sum over 32 logits of 2^(v * c2 + nm).  Of every 16 pairs, NPOLY take the polynomial on the
// FMA pipe and the rest the special-function unit, so that both pipes work in parallel.
template <int NPOLY>
__device__ __forceinline__ float chunk_sum_exp2(const float (&v)[32], float c2, float nm) {
  const float2 c2v = make_float2(c2, c2), nmv = make_float2(nm, nm);
  float2 acc0 = make_float2(0.f, 0.f), acc1 = make_float2(0.f, 0.f);
#pragma unroll
  for (int pr = 0; pr < 16; ++pr) {
    const float2 x = ffma2(make_float2(v[2 * pr], v[2 * pr + 1]), c2v, nmv);
    float2 e;
    if (((pr + 1) * NPOLY) / 16 > (pr * NPOLY) / 16) {
      e = exp2_poly2(x);
    } else {
      e.x = ex2_approx(x.x);
      e.y = ex2_approx(x.y);
    }
    if (pr & 1) acc1 = fadd2(acc1, e); else acc0 = fadd2(acc0, e);
  }
  return (acc0.x + acc0.y) + (acc1.x + acc1.y);
}

// Online (max, sum-exp) update of one query row with 32 more logits of the key tile.  Keys
// past L (ragged last tile) become -inf: the special-function path maps them to 0 and the
// polynomial's clamp to 2^-125, which vanishes against the row's sum (>= 1).
template <int NPOLY>
__device__ __forceinline__ void row_chunk_update(float (&v)[32], int col0, int valid, float c2,
                                                 float& m, float& z) {
  if (valid < kTileKeys) {
#pragma unroll
    for (int j = 0; j < 32; ++j)
      if (col0 + j >= valid) v[j] = -INFINITY;
  }
  float cm0 = fmax3(v[0], v[1], v[2]), cm1 = fmax3(v[3], v[4], v[5]);
#pragma unroll
  for (int j = 6; j < 30; j += 4) {
    cm0 = fmax3(cm0, v[j], v[j + 1]);
    cm1 = fmax3(cm1, v[j + 2], v[j + 3]);
  }
  const float m_new = fmaxf(fmax3(m, cm0, cm1), fmaxf(v[30], v[31]));
  const float nm = -m_new * c2;
  const float sum = chunk_sum_exp2<NPOLY>(v, c2, nm);
  if (m_new > m) {                         // rare once the first tiles have been seen
    z *= ex2_approx((m - m_new) * c2);
    m = m_new;
  }
  z += sum;
}

// ---------------------------------------------------------------------------------------
// Pass A: row statistics.  MT = number of 128-row tiles of the resident Q block.
// ---------------------------------------------------------------------------------------
template <int MT, int NPOLY>
__global__ void __launch_bounds__(kStatsThreads, 1)
row_stats_kernel(const __grid_constant__ CUtensorMap tmapK,
                 const __grid_constant__ CUtensorMap tmapQ, const QkParams p) {
  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t smem_base = smem_u32(smem);
  const uint32_t q_s = smem_base;
  const uint32_t k_s = smem_base + MT * 128 * 256;
  SmemTail* tail = reinterpret_cast<SmemTail*>(smem + MT * 128 * 256 + p.stages * kStageBytes);
  volatile int* abort_flag = &tail->abort_flag;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const CtaItem it = decode_item(p);

  const uint32_t tmem_base = cta_setup(tail, smem_base, p.stages, 4, 4, p.status);
  const bool run = (it.n_tiles > 0) && (*abort_flag == 0);
  const bool stamp = (p.clk != nullptr) && blockIdx.x == 0 && threadIdx.x == 0;
  if (stamp) {
    unsigned long long ns0;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(ns0));
    tail->stamp_cycles = clock64();
    tail->stamp_ns = ns0;
  }

  if (warp == 0) {
    if (lane == 0 && run) {
      // The packed query comes from the kernel before this one, which may still be running.
      // After that the next kernel's CTAs may come in as SMs fall free.
      grid_dep_wait();
      grid_dep_launch();
      producer_loop(&tmapK, &tmapQ, p, it, tail, q_s, k_s, p.skip_tiles);
    }
  } else if (warp == 1) {
    if (lane == 0 && run) {
      constexpr uint32_t idesc = umma_idesc_bf16(128, kTileKeys);
      bool ok = mbar_wait(smem_u32(&tail->q_full), 0, abort_flag, p.status, kDevWaitQFull, p.wait_limit);
      tc_fence_after();
      uint32_t u = 0;
      int s = 0;
      uint32_t kphase = 0;
      for (int i = 0; i < it.n_tiles && ok; ++i) {
        ok = mbar_wait(smem_u32(&tail->k_full[s]), kphase, abort_flag, p.status, kDevWaitKFull, p.wait_limit);
        if (!ok) break;
        tc_fence_after();
        for (int mt = 0; mt < MT; ++mt, ++u) {
          const uint32_t b = u & 3u, use = u >> 2;
          ok = mbar_wait(smem_u32(&tail->acc_empty[b]), (use & 1u) ^ 1u, abort_flag, p.status,
                         kDevWaitAccEmpty, p.wait_limit);
          if (!ok) break;
          tc_fence_after();
#pragma unroll
          for (int kb = 0; kb < 2; ++kb)
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
              const uint64_t a = umma_desc_sw128(q_s + kb * (MT * 128 * 128) + mt * 16384 + ks * 32);
              const uint64_t bd = umma_desc_sw128(k_s + s * kStageBytes + kb * 16384 + ks * 32);
              umma_bf16(tmem_base + b * 128, a, bd, idesc, (kb | ks) != 0);
            }
          umma_commit(smem_u32(&tail->acc_full[b]));
        }
        umma_commit(smem_u32(&tail->k_empty[s]));
        if (++s == p.stages) { s = 0; kphase ^= 1u; }
      }
    }
  } else if (warp >= 2) {
    // Consumer warpgroups take the accumulator buffers in turn, so that they sit in different
    // phases (waiting, loading, taking maxima, exponentials) and keep the special-function
    // and FMA pipes fed.  Each thread owns one query row of the buffer and walks its 128
    // columns in chunks of 32, loading the next chunk from tensor memory while it works on
    // the current one.
    const int wg = (warp - 2) >> 2;
    const int quad = warp & 3;               // TMEM lane quadrant this warp may read
    // Accumulator u belongs to warpgroup u % 4 and holds row tile u % MT.  With 1, 2 or 4 row
    // tiles a warpgroup therefore always meets the same row tile (wg % MT) and a thread keeps
    // one (max, sum) pair; only with 3 row tiles does it meet all of them in turn.
    constexpr int kStates = (MT == 3) ? 3 : 1;
    float m[kStates], z[kStates];
#pragma unroll
    for (int j = 0; j < kStates; ++j) { m[j] = -1e30f; z[j] = 0.f; }
    const float c2 = p.c2;
    const uint32_t n_acc = run ? static_cast<uint32_t>(it.n_tiles) * MT : 0u;
    // One copy of the loop body serves every (key tile, row tile): the warpgroups run at
    // different places of the loop, and a body unrolled over the row tiles would not fit the
    // instruction cache between them.
#pragma unroll 1
    for (uint32_t u = wg; u < n_acc; u += kStatsWarpgroups) {
      const int i = static_cast<int>(u / MT), mt = static_cast<int>(u % MT);
      const long long key0 = static_cast<long long>(it.tile_begin + i) * kTileKeys;
      const int valid = static_cast<int>(min(static_cast<long long>(kTileKeys), p.L - key0));
      const uint32_t b = u & 3u, use = u >> 2;
      if (!mbar_wait(smem_u32(&tail->acc_full[b]), use & 1u, abort_flag, p.status,
                     kDevWaitAccFull, p.wait_limit))
        break;
      tc_fence_after();
      float mr = m[0], zr = z[0];
      if (kStates > 1) {
#pragma unroll
        for (int j = 1; j < kStates; ++j)
          if (j == mt) { mr = m[j]; zr = z[j]; }
      }
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + b * 128;
      float va[32], vb[32];
      tmem_ld32(taddr, va);
      tmem_ld_wait();
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        tmem_ld32(taddr + 64 * h + 32, vb);
        row_chunk_update<NPOLY>(va, 64 * h, valid, c2, mr, zr);
        tmem_ld_wait();
        if (h == 0) {
          tmem_ld32(taddr + 64, va);
        } else {
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(smem_u32(&tail->acc_empty[b]));
        }
        row_chunk_update<NPOLY>(vb, 64 * h + 32, valid, c2, mr, zr);
        if (h == 0) tmem_ld_wait();
      }
      if (kStates > 1) {
#pragma unroll
        for (int j = 0; j < kStates; ++j)
          if (j == mt) { m[j] = mr; z[j] = zr; }
      } else {
        m[0] = mr; z[0] = zr;
      }
    }
    // Merge the warpgroups' statistics through shared memory and write this CTA's partial
    // statistics: (max in log2 units, sum).  Every warpgroup stores a pair for every row tile
    // (a neutral one for the row tiles it never met); warpgroup 0 merges.  The scratch aliases
    // the first K stage, which is idle once every warpgroup has read its last accumulator
    // (every MMA, hence every TMA load, has completed by then).
    float2* scratch = reinterpret_cast<float2*>(smem + MT * 128 * 256);
    const int row_in_tile = quad * 32 + lane;
    asm volatile("bar.sync 1, %0;" ::"r"(kStatsConsumerWarps * 32) : "memory");
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
      float2 mine = make_float2(-1e30f, 0.f);
      if (kStates > 1) {
#pragma unroll
        for (int j = 0; j < kStates; ++j)
          if (j == mt) mine = make_float2(m[j], z[j]);
      } else if (mt == wg % MT) {
        mine = make_float2(m[0], z[0]);
      }
      scratch[(wg * MT + mt) * 128 + row_in_tile] = mine;
    }
    asm volatile("bar.sync 1, %0;" ::"r"(kStatsConsumerWarps * 32) : "memory");
    if (wg == 0) {
      float2* out = reinterpret_cast<float2*>(p.partial) +
                    (static_cast<size_t>(it.group) * p.cpg + it.chunk) * (MT * 128);
#pragma unroll
      for (int mt = 0; mt < MT; ++mt) {
        float mm = -1e30f;
#pragma unroll
        for (int w = 0; w < kStatsWarpgroups; ++w)
          mm = fmaxf(mm, scratch[(w * MT + mt) * 128 + row_in_tile].x);
        float zz = 0.f;
#pragma unroll
        for (int w = 0; w < kStatsWarpgroups; ++w) {
          const float2 o = scratch[(w * MT + mt) * 128 + row_in_tile];
          zz += o.y * exp2f((o.x - mm) * c2);
        }
        out[mt * 128 + row_in_tile] = make_float2(mm * c2, zz);
      }
    }
  }
  if (stamp) {
    unsigned long long ns1;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(ns1));
    p.clk[0] = static_cast<unsigned long long>(clock64() - tail->stamp_cycles);
    p.clk[1] = ns1 - tail->stamp_ns;
  }
  cta_teardown(tmem_base);
}

// Combines the partial statistics of one row (per key chunk of this launch, or per key shard)
// into (max in log2 units, sum); -lse in log2 units for the scores pass (-inf marks a padding
// row); `publish` also stores the user-visible natural-log lse.
__device__ __forceinline__ float2 merged_stats(const MergeParams& p, int group, int within,
                                               int* user_row) {
  const int g = group / p.n_rb, rb = group % p.n_rb;
  const int rg = rb * p.rb_rows + within;
  *user_row = -1;
  if (rg >= p.group_size * p.q_len) return make_float2(-INFINITY, 0.f);
  const int i = rg / p.group_size, j = rg % p.group_size;
  *user_row = i * p.n_q + g * p.group_size + j;
  const float2* part;
  size_t stride;
  int n;
  if (p.n_ext > 0) {                     // one entry per key shard
    part = p.ext_stats + *user_row;
    stride = static_cast<size_t>(p.q_len) * p.n_q;
    n = p.n_ext;
  } else {                               // one entry per key chunk of this launch
    part = reinterpret_cast<const float2*>(p.partial) +
           static_cast<size_t>(group) * p.cpg * p.rb_rows + within;
    stride = p.rb_rows;
    n = p.cpg;
  }
  float mm = -INFINITY;
  for (int c = 0; c < n; ++c) mm = fmaxf(mm, __ldcg(&part[c * stride]).x);
  float zz = 0.f;
  for (int c = 0; c < n; ++c) {
    const float2 v = __ldcg(&part[c * stride]);
    zz += v.y * exp2f(v.x - mm);
  }
  return make_float2(mm, zz);
}

__device__ __forceinline__ float merged_neg_lse2(const MergeParams& p, int group, int within,
                                                 bool publish) {
  int user_row;
  const float2 st = merged_stats(p, group, within, &user_row);
  if (user_row < 0) return -INFINITY;
  const float lse2 = st.x + log2f(st.y);
  if (publish) p.row_lse[user_row] = lse2 * 0.69314718055994530942f;
  return -lse2;
}

__global__ void export_stats_kernel(MergeParams p, float2* __restrict__ out) {
  const int prow = blockIdx.x * blockDim.x + threadIdx.x;
  if (prow >= p.n_groups * p.rb_rows) return;
  int user_row;
  const float2 st = merged_stats(p, prow / p.rb_rows, prow % p.rb_rows, &user_row);
  if (user_row >= 0) out[user_row] = st;
}

__global__ void decode_scores_kernel(const uint32_t* __restrict__ enc, float* __restrict__ out,
                                     long long L) {
  const long long t = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (t < L) out[t] = exp2f(ordered_to_float(enc[t]));
}

// ---------------------------------------------------------------------------------------
// Pass B: scores.  D[key, row]; per context position max over rows of log2-probability.
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kQkThreads, 1)
scores_kernel(const __grid_constant__ CUtensorMap tmapK,
              const __grid_constant__ CUtensorMap tmapQ, const QkParams p, const MergeParams mp) {
  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t smem_base = smem_u32(smem);
  const uint32_t q_s = smem_base;
  const uint32_t k_s = smem_base + p.rb_rows * 256;
  SmemTail* tail = reinterpret_cast<SmemTail*>(smem + p.rb_rows * 256 + p.stages * kStageBytes);
  float* nl = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(tail) + kSmemTailBytes);
  volatile int* abort_flag = &tail->abort_flag;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const CtaItem it = decode_item(p);
  const int n_nh = (p.rb_rows + 255) / 256;

  // Two MMA-issuing threads (warps 1 and 2), one per accumulator buffer: tcgen05.mma holds its
  // issuing thread until the tensor pipe takes the instruction, so the waits and commits of
  // one thread overlap the MMAs of the other.  With two row halves per key tile each thread
  // issues one half of every tile and both release the tile's stage; with one, the threads
  // take the tiles in turn.
  const int k_releasers = (n_nh >= 2) ? 2 : 1;
  const uint32_t tmem_base = cta_setup(tail, smem_base, p.stages, 2, kConsumerWarps, p.status,
                                       k_releasers);
  const bool run = (it.n_tiles > 0) && (*abort_flag == 0);

  if (warp == 0) {
    if (lane == 0 && run) {
      grid_dep_wait();                   // the kernel before this one (it packed the query or made the statistics) is done
      grid_dep_launch();                 // the next kernel's CTAs may come in as SMs fall free
      producer_loop(&tmapK, &tmapQ, p, it, tail, q_s, k_s);
    }
  } else if (warp == 1 || warp == 2) {
    if (lane == 0 && run) {
      const uint32_t mine = static_cast<uint32_t>(warp - 1);          // accumulator buffer
      bool ok = mbar_wait(smem_u32(&tail->q_full), 0, abort_flag, p.status, kDevWaitQFull);
      tc_fence_after();
      uint32_t u = 0;
      int s = -1;
      uint32_t kphase = 1;
      for (int i = 0; i < it.n_tiles && ok; ++i) {
        if (++s == p.stages) s = 0;                      // stage and phase of key tile i
        if (s == 0) kphase ^= 1u;
        if (n_nh == 1 && ((static_cast<uint32_t>(i) & 1u) != mine)) { ++u; continue; }
        ok = mbar_wait(smem_u32(&tail->k_full[s]), kphase, abort_flag, p.status, kDevWaitKFull);
        if (!ok) break;
        tc_fence_after();
        for (int nh = 0; nh < n_nh; ++nh, ++u) {
          if ((u & 1u) != mine) continue;
          const int N = min(256, p.rb_rows - nh * 256);
          const uint32_t idesc = umma_idesc_bf16(128, N);
          const uint32_t b = u & 1u, use = u >> 1;
          ok = mbar_wait(smem_u32(&tail->acc_empty[b]), (use & 1u) ^ 1u, abort_flag, p.status,
                         kDevWaitAccEmpty);
          if (!ok) break;
          tc_fence_after();
#pragma unroll
          for (int kb = 0; kb < 2; ++kb)
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
              const uint64_t a = umma_desc_sw128(k_s + s * kStageBytes + kb * 16384 + ks * 32);
              const uint64_t bd =
                  umma_desc_sw128(q_s + kb * (p.rb_rows * 128) + nh * (256 * 128) + ks * 32);
              umma_bf16(tmem_base + b * 256, a, bd, idesc, (kb | ks) != 0);
            }
          umma_commit(smem_u32(&tail->acc_full[b]));
        }
        umma_commit(smem_u32(&tail->k_empty[s]));
      }
    }
  } else if (warp >= 4) {
    // The consumer warps merge the per-key-chunk statistics of the CTA's rows (a few KB from
    // L2; the CTAs of the first key chunk also publish the natural-log lse).  The statistics
    // come from the kernel before this one, which may still be running when this CTA starts
    // (the set-up above does not wait for it).
    grid_dep_wait();
    for (int i = threadIdx.x - 128; i < p.rb_rows; i += kConsumerWarps * 32)
      nl[i] = merged_neg_lse2(mp, it.group, i, it.chunk == 0);
    asm volatile("bar.sync 2, %0;" ::"r"(kConsumerWarps * 32) : "memory");
    const int wg = (warp - 4) >> 2;
    const int quad = warp & 3;
    const float c2 = p.c2;
    bool ok = run;
    uint32_t u = 0;
    for (int i = 0; i < it.n_tiles && ok; ++i) {
      float best = -INFINITY;
      for (int nh = 0; nh < n_nh && ok; ++nh) {
        const int N = min(256, p.rb_rows - nh * 256);
        const int half = N >> 1;
        const uint32_t b = u & 1u, use = u >> 1;
        ++u;
        ok = mbar_wait(smem_u32(&tail->acc_full[b]), use & 1u, abort_flag, p.status,
                       kDevWaitAccFull);
        if (!ok) break;
        tc_fence_after();
        const int col0 = wg * half;
        const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + b * 256 + col0;
        const float4* nl4 = reinterpret_cast<const float4*>(nl + nh * 256 + col0);
        float b0 = -INFINITY, b1 = -INFINITY, b2 = -INFINITY, b3 = -INFINITY;
        for (int c = 0; c < half; c += 32) {
          float v[32];
          tmem_ld32(taddr + c, v);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 32; j += 4) {
            const float4 n4 = nl4[(c + j) >> 2];
            b0 = fmaxf(b0, fmaf(v[j], c2, n4.x));
            b1 = fmaxf(b1, fmaf(v[j + 1], c2, n4.y));
            b2 = fmaxf(b2, fmaf(v[j + 2], c2, n4.z));
            b3 = fmaxf(b3, fmaf(v[j + 3], c2, n4.w));
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&tail->acc_empty[b]));
        best = fmaxf(best, fmaxf(fmaxf(b0, b1), fmaxf(b2, b3)));
      }
      const long long t = static_cast<long long>(it.tile_begin + i) * kTileKeys + quad * 32 + lane;
      if (ok && t < p.L) atomicMax(p.enc + t, float_to_ordered(best));
    }
  }
  cta_teardown(tmem_base);
}

// ---------------------------------------------------------------------------------------
// small kernels around the two passes
// ---------------------------------------------------------------------------------------

// Packs the query rows of every (kv head, row block) contiguously, zero-padded to rb_rows,
// and clears the per-run state (encoded scores, bitmap with the sink bits set, selection
// state).
__global__ void prepare_kernel(const uint4* __restrict__ q, uint4* __restrict__ qp, PrepParams p) {
  grid_dep_launch();                     // the statistics kernel sets itself up meanwhile
  const long long tid = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  const long long nthreads = static_cast<long long>(gridDim.x) * blockDim.x;
  // packed query: 16 x uint4 per 128-element row
  const long long n_pack = static_cast<long long>(p.n_kv) * p.n_rb * p.rb_rows * 16;
  for (long long e = tid; e < n_pack; e += nthreads) {
    const int part = static_cast<int>(e & 15);
    const long long prow = e >> 4;
    const int within = static_cast<int>(prow % p.rb_rows);
    const int group = static_cast<int>(prow / p.rb_rows);
    const int g = group / p.n_rb, rb = group % p.n_rb;
    const int rg = rb * p.rb_rows + within;               // row inside the kv head's group
    uint4 val = make_uint4(0, 0, 0, 0);
    if (rg < p.group_size * p.q_len) {
      const int i = rg / p.group_size, j = rg % p.group_size;
      val = q[(static_cast<long long>(i) * p.n_q + g * p.group_size + j) * 16 + part];
    }
    qp[e] = val;
  }
  for (long long t = tid; t < p.L; t += nthreads) p.enc[t] = 0u;
  const long long n_words = (p.L + 31) / 32;
  for (long long w = tid; w < n_words; w += nthreads) {
    const long long lo = w * 32;
    uint32_t bits = 0;
    if (p.n_sink > lo) bits = (p.n_sink - lo >= 32) ? 0xFFFFFFFFu : ((1u << (p.n_sink - lo)) - 1u);
    p.bitmap[w] = bits;
  }
  for (long long e = tid; e < p.hist_words; e += nthreads) p.hist[e] = 0u;
  if (tid == 0) *p.grid_barrier = 0u;
  for (long long c = tid; c < p.sel_state_words; c += nthreads) p.cand_count[c] = 0u;
}

// ---------------------------------------------------------------------------------------
// host-side launchers
// ---------------------------------------------------------------------------------------
// Launch that may overlap the end of the kernel before it in the stream (programmatic
// dependent launch): the kernel itself waits (grid_dep_wait) before it touches that kernel's output.
template <typename... Params, typename... Args>
static cudaError_t launch_after_previous(void (*kernel)(Params...), int grid, int block, size_t smem,
                                         cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(block);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

size_t row_stats_smem_bytes(int rb_rows, int stages) {
  return static_cast<size_t>(rb_rows) * 256 + static_cast<size_t>(stages) * kStageBytes +
         kSmemTailBytes;
}
size_t scores_smem_bytes(int rb_rows, int stages) {
  return row_stats_smem_bytes(rb_rows, stages) + static_cast<size_t>(rb_rows) * sizeof(float);
}

template <int MT>
static cudaError_t launch_row_stats_mt(const CUtensorMap& tk, const CUtensorMap& tq,
                                       const QkParams& p, cudaStream_t st) {
  const size_t smem = row_stats_smem_bytes(MT * 128, p.stages);
  cudaError_t e = cudaFuncSetAttribute(row_stats_kernel<MT, kRowStatsPolyPairs>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  return launch_after_previous(row_stats_kernel<MT, kRowStatsPolyPairs>, p.n_groups * p.cpg,
                               kStatsThreads, smem, st, tk, tq, p);
}

cudaError_t launch_row_stats(const CUtensorMap& tk, const CUtensorMap& tq, const QkParams& p,
                             cudaStream_t st) {
  switch (p.rb_rows / 128) {
    case 1: return launch_row_stats_mt<1>(tk, tq, p, st);
    case 2: return launch_row_stats_mt<2>(tk, tq, p, st);
    case 3: return launch_row_stats_mt<3>(tk, tq, p, st);
    case 4: return launch_row_stats_mt<4>(tk, tq, p, st);
    default: return cudaErrorInvalidValue;
  }
}

cudaError_t launch_export_stats(const MergeParams& p, float2* out, cudaStream_t st) {
  const int n = p.n_groups * p.rb_rows;
  export_stats_kernel<<<(n + 127) / 128, 128, 0, st>>>(p, out);
  return cudaGetLastError();
}

cudaError_t launch_decode_scores(const uint32_t* enc, float* out, long long L, cudaStream_t st) {
  decode_scores_kernel<<<static_cast<unsigned>((L + 255) / 256), 256, 0, st>>>(enc, out, L);
  return cudaGetLastError();
}

cudaError_t launch_scores(const CUtensorMap& tk, const CUtensorMap& tq, const QkParams& p,
                          const MergeParams& mp, cudaStream_t st) {
  const size_t smem = scores_smem_bytes(p.rb_rows, p.stages);
  cudaError_t e = cudaFuncSetAttribute(scores_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)smem);
  if (e != cudaSuccess) return e;
  return launch_after_previous(scores_kernel, p.n_groups * p.cpg, kQkThreads, smem, st, tk, tq, p, mp);
}

cudaError_t launch_prepare(const void* q, void* qp, const PrepParams& p, int n_sm,
                           cudaStream_t st) {
  prepare_kernel<<<n_sm * 4, 256, 0, st>>>(static_cast<const uint4*>(q), static_cast<uint4*>(qp), p);
  return cudaGetLastError();
}

}  // namespace ilre
