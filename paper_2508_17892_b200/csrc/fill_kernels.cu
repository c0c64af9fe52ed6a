// Key projection of the retrieval layer fused with RoPE and the write into the key cache:
//   K[pos, g, :] = R(pos) (X[pos, :] W_K[g*128:(g+1)*128, :]^T + b)      (Eq. 1, Eq. 3)
// A dense contraction, so it runs on the tensor cores: TMA -> shared memory (128-byte
// swizzle) -> tcgen05.mma with the accumulator in tensor memory -> epilogue warps that read
// the accumulator one token per thread, rotate the channel pairs (c, c + 64) of each head,
// round to bf16 and store the cache rows.  Persistent CTAs walk the output tiles
// (128 tokens x 1 or 2 heads); tiles of one token block are neighbours in that order, so the
// block's activations are read from HBM once and served from L2 to the other heads.
#include <cuda_bf16.h>

#include "fill_kernels.cuh"
#include "sm100_ptx.cuh"

namespace ilre {

static constexpr int kFillMaxStages = 8;
static constexpr int kFillEpilogueWarps = 4;
static constexpr int kFillMaxDynSmem = 232448;
static constexpr int kFillTailBytes = 256;

struct FillTail {
  uint64_t full[kFillMaxStages];
  uint64_t empty[kFillMaxStages];
  uint64_t acc_full[2];
  uint64_t acc_empty[2];
  uint32_t tmem_base;
  int abort_flag;
};
static_assert(sizeof(FillTail) <= kFillTailBytes, "tail too large");

__global__ void rope_pos_table_kernel(float2* __restrict__ lo, float2* __restrict__ hi, int hi_rows,
                                      double theta) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  const int n_lo = kRopeLoRows * 64;
  if (idx >= n_lo + hi_rows * 64) return;
  const bool is_lo = idx < n_lo;
  const int e = is_lo ? idx : idx - n_lo;
  const int row = e / 64, c = e % 64;
  const double pos = is_lo ? static_cast<double>(row)
                           : static_cast<double>(row) * static_cast<double>(kRopeLoRows);
  const double ang = pos * pow(theta, -2.0 * static_cast<double>(c) / 128.0);
  double sn, cs;
  sincos(ang, &sn, &cs);
  (is_lo ? lo : hi)[e] = make_float2(static_cast<float>(cs), static_cast<float>(sn));
}

template <int NT>
__global__ void __launch_bounds__(kFillThreads, 1)
fill_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
            const FillParams p) {
  constexpr int kStageBytesA = kFillTileM * kFillBlockK * 2;           // 16 KB
  constexpr int kStageBytesB = NT * kFillBlockK * 2;
  constexpr int kStageBytes = kStageBytesA + kStageBytesB;
  constexpr int kHeadsPerTile = NT / 128;
  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t smem_base = smem_u32(smem);
  FillTail* tail = reinterpret_cast<FillTail*>(smem + p.stages * kStageBytes);
  volatile int* abort_flag = &tail->abort_flag;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  const int n_ntiles = p.n_kv * 128 / NT;
  const long long m_tiles = (p.n_tok + kFillTileM - 1) / kFillTileM;
  const long long n_tiles = m_tiles * n_ntiles;
  const int k_blocks = p.d_model / kFillBlockK;

  if (threadIdx.x == 0) {
    tail->abort_flag = 0;
    if (smem_base & 1023u) {
      tail->abort_flag = 1;
      atomicCAS(p.status, 0, kDevSmemAlign);
    }
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(smem_u32(&tail->full[s]), 1);
      mbar_init(smem_u32(&tail->empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&tail->acc_full[b]), 1);
      mbar_init(smem_u32(&tail->acc_empty[b]), kFillEpilogueWarps);
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
  const uint32_t tmem_base = tail->tmem_base;
  const bool run = (*abort_flag == 0);

  if (warp == 0) {
    if (lane == 0 && run) {
      // ring position kept as (stage, phase) counters: a division by the run-time stage count
      // per 64-channel block would cost this thread more than the block's TMA issue
      int s = 0;
      uint32_t phase = 0;
      for (long long tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
        const int m0 = static_cast<int>(tile / n_ntiles) * kFillTileM;
        const int n0 = static_cast<int>(tile % n_ntiles) * NT;
        bool ok = true;
        for (int kb = 0; kb < k_blocks && ok; ++kb) {
          ok = mbar_wait(smem_u32(&tail->empty[s]), phase ^ 1u, abort_flag, p.status,
                         kDevWaitKEmpty);
          if (!ok) break;
          const uint32_t bar = smem_u32(&tail->full[s]);
          mbar_arrive_expect_tx(bar, kStageBytes);
          const uint32_t dst = smem_base + s * kStageBytes;
          tma_load_2d(dst, &map_x, kb * kFillBlockK, m0, bar);
          tma_load_2d(dst + kStageBytesA, &map_w, kb * kFillBlockK, n0, bar);
          if (++s == p.stages) { s = 0; phase ^= 1u; }
        }
        if (!ok) break;
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && run) {
      constexpr uint32_t idesc = umma_idesc_bf16(kFillTileM, NT);
      // (stage, phase) counters instead of a division per block: the tensor pipe idles while
      // this thread does anything but issue
      uint32_t local = 0;
      int s = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (long long tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++local) {
        const uint32_t buf = local & 1u, use = local >> 1;
        ok = mbar_wait(smem_u32(&tail->acc_empty[buf]), (use & 1u) ^ 1u, abort_flag, p.status,
                       kDevWaitAccEmpty);
        if (!ok) break;
        tc_fence_after();
        for (int kb = 0; kb < k_blocks; ++kb) {
          ok = mbar_wait(smem_u32(&tail->full[s]), phase, abort_flag, p.status, kDevWaitKFull);
          if (!ok) break;
          tc_fence_after();
          const uint32_t a0 = smem_base + s * kStageBytes;
#pragma unroll
          for (int ks = 0; ks < 4; ++ks)
            umma_bf16(tmem_base + buf * NT, umma_desc_sw128(a0 + ks * 32),
                      umma_desc_sw128(a0 + kStageBytesA + ks * 32), idesc, (kb | ks) != 0);
          umma_commit(smem_u32(&tail->empty[s]));
          if (++s == p.stages) { s = 0; phase ^= 1u; }
        }
        if (ok) umma_commit(smem_u32(&tail->acc_full[buf]));
      }
    }
  } else {
    // Epilogue: thread = token row of the tile (TMEM lane), warp = lane quadrant.
    const int quad = warp & 3;
    uint32_t local = 0;
    bool ok = run;
    for (long long tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++local) {
      const long long m0 = (tile / n_ntiles) * kFillTileM;
      const int n_tile = static_cast<int>(tile % n_ntiles);
      const uint32_t buf = local & 1u, use = local >> 1;
      ok = mbar_wait(smem_u32(&tail->acc_full[buf]), use & 1u, abort_flag, p.status,
                     kDevWaitAccFull);
      if (!ok) break;
      tc_fence_after();
      const long long token = m0 + quad * 32 + lane;
      const bool live = token < p.n_tok;
      const long long pos = p.pos0 + (live ? token : 0);
      const float4* t_lo = reinterpret_cast<const float4*>(p.rope_lo + (pos % kRopeLoRows) * 64);
      const float4* t_hi = reinterpret_cast<const float4*>(p.rope_hi + (pos / kRopeLoRows) * 64);
      const uint32_t trow = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + buf * NT;
#pragma unroll 1
      for (int part = 0; part < kHeadsPerTile * 2; ++part) {
        const int hh = part >> 1, c0 = (part & 1) * 32;
        float v_lo[32], v_hi[32];
        tmem_ld32(trow + hh * 128 + c0, v_lo);
        tmem_ld32(trow + hh * 128 + 64 + c0, v_hi);
        tmem_ld_wait();
        if (part == kHeadsPerTile * 2 - 1) {               // accumulator fully read
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(smem_u32(&tail->acc_empty[buf]));
        }
        const int head = n_tile * kHeadsPerTile + hh;
        uint32_t out_lo[16], out_hi[16];
#pragma unroll
        for (int j = 0; j < 32; j += 2) {
          // (cos, sin) of pos * theta_c by angle addition of the two table entries
          const float4 a = __ldg(t_lo + ((c0 + j) >> 1)), b = __ldg(t_hi + ((c0 + j) >> 1));
          const float cs0 = fmaf(a.x, b.x, -a.y * b.y), sn0 = fmaf(a.y, b.x, a.x * b.y);
          const float cs1 = fmaf(a.z, b.z, -a.w * b.w), sn1 = fmaf(a.w, b.z, a.z * b.w);
          float l0 = v_lo[j], l1 = v_lo[j + 1], h0 = v_hi[j], h1 = v_hi[j + 1];
          if (p.bias) {
            const uint16_t* bp = p.bias + head * 128 + c0 + j;
            l0 += __uint_as_float(static_cast<uint32_t>(__ldg(bp)) << 16);
            l1 += __uint_as_float(static_cast<uint32_t>(__ldg(bp + 1)) << 16);
            h0 += __uint_as_float(static_cast<uint32_t>(__ldg(bp + 64)) << 16);
            h1 += __uint_as_float(static_cast<uint32_t>(__ldg(bp + 65)) << 16);
          }
          const __nv_bfloat162 pl = __floats2bfloat162_rn(fmaf(l0, cs0, -h0 * sn0),
                                                          fmaf(l1, cs1, -h1 * sn1));
          const __nv_bfloat162 ph = __floats2bfloat162_rn(fmaf(l0, sn0, h0 * cs0),
                                                          fmaf(l1, sn1, h1 * cs1));
          out_lo[j >> 1] = *reinterpret_cast<const uint32_t*>(&pl);
          out_hi[j >> 1] = *reinterpret_cast<const uint32_t*>(&ph);
        }
        if (live) {
          uint16_t* row = p.k_cache + ((p.pos0 + token) * p.n_kv + head) * 128;
          uint4* dst_lo = reinterpret_cast<uint4*>(row + c0);
          uint4* dst_hi = reinterpret_cast<uint4*>(row + 64 + c0);
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            dst_lo[q] = make_uint4(out_lo[4 * q], out_lo[4 * q + 1], out_lo[4 * q + 2], out_lo[4 * q + 3]);
            dst_hi[q] = make_uint4(out_hi[4 * q], out_hi[4 * q + 1], out_hi[4 * q + 2], out_hi[4 * q + 3]);
          }
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

size_t fill_smem_bytes(int tile_n, int stages) {
  return static_cast<size_t>(stages) * (kFillTileM * kFillBlockK * 2 + tile_n * kFillBlockK * 2) +
         kFillTailBytes;
}

int fill_max_stages(int tile_n) {
  int s = (kFillMaxDynSmem - kFillTailBytes) / (kFillTileM * kFillBlockK * 2 + tile_n * kFillBlockK * 2);
  return s > kFillMaxStages ? kFillMaxStages : s;
}

cudaError_t launch_rope_pos_tables(float2* lo, float2* hi, int hi_rows, double theta,
                                   cudaStream_t st) {
  const int n = (kRopeLoRows + hi_rows) * 64;
  rope_pos_table_kernel<<<(n + 255) / 256, 256, 0, st>>>(lo, hi, hi_rows, theta);
  return cudaGetLastError();
}

template <int NT>
static cudaError_t launch_fill_nt(const CUtensorMap& mx, const CUtensorMap& mw, const FillParams& p,
                                  int grid, cudaStream_t st) {
  const size_t smem = fill_smem_bytes(NT, p.stages);
  cudaError_t e = cudaFuncSetAttribute(fill_kernel<NT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       static_cast<int>(smem));
  if (e != cudaSuccess) return e;
  fill_kernel<NT><<<grid, kFillThreads, smem, st>>>(mx, mw, p);
  return cudaGetLastError();
}

cudaError_t launch_fill(const CUtensorMap& map_x, const CUtensorMap& map_w, const FillParams& p,
                        int tile_n, int grid, cudaStream_t st) {
  if (tile_n == 256) return launch_fill_nt<256>(map_x, map_w, p, grid, st);
  if (tile_n == 128) return launch_fill_nt<128>(map_x, map_w, p, grid, st);
  return cudaErrorInvalidValue;
}

}  // namespace ilre
