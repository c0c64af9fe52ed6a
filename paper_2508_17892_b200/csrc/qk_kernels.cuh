// Parameters and launchers of the query-context attention kernels (Eq. 4, Eq. 5).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace ilre {

static constexpr int kHeadDim = 128;
static constexpr int kTileKeys = 128;              // keys per K tile (one TMA stage)
static constexpr int kStageBytes = kTileKeys * kHeadDim * 2;
static constexpr int kMaxStages = 6;
static constexpr int kMaxRbRows = 512;             // query rows resident in shared memory
static constexpr int kQkThreads = 384;             // scores: warp 0 TMA, warps 1-2 MMA, warps 4..11 consumers
static constexpr int kConsumerWarps = 8;
// Row statistics: warp 0 TMA, warp 1 MMA, then kStatsWarpgroups consumer warpgroups of four
// warps (one per TMEM lane quadrant); accumulator buffer u belongs to warpgroup u % kStatsWarpgroups.
static constexpr int kStatsWarpgroups = 4;
// A warpgroup's first accumulator must be one of the first four (the number of TMEM buffers):
// a parity wait on a buffer that has not completed its first phase yet would pass at once.
static_assert(kStatsWarpgroups >= 1 && kStatsWarpgroups <= 4, "at most one warpgroup per TMEM buffer");
static constexpr int kStatsConsumerWarps = 4 * kStatsWarpgroups;
static constexpr int kStatsThreads = 64 + 32 * kStatsConsumerWarps;
static constexpr int kSmemTailBytes = 256;
static constexpr int kMaxDynSmem = 232448;         // 227 KB per CTA on sm_100

// Row statistics: how many of every 16 logit pairs take 2^x from the FMA-pipe polynomial
// instead of the special-function unit (0 = none).  Balances the two pipes.
static constexpr int kRowStatsPolyPairs = 4;

// Geometry of one recall, shared by both passes.
struct QkParams {
  long long L;
  int n_tiles;       // ceil(L / kTileKeys)
  int n_groups;      // n_kv_heads * n_rb
  int n_rb;          // row blocks per kv head
  int rb_rows;       // rows per block, multiple of 128, <= kMaxRbRows
  int cpg;           // key chunks (CTAs) per group
  int stages;
  float c2;          // log2(e) / sqrt(d)
  float* partial;    // [n_groups][cpg][rb_rows][2]: (max * c2, sum-exp) per key chunk
  uint32_t* enc;     // [L]: order-preserving uint of max_r log2 p_rt
  int* status;
  // When non-null, CTA 0 of the row-statistics kernel stores how long it ran in SM cycles and
  // in nanoseconds of the global timer: their ratio is the SM clock the kernel really ran at
  // (under the power cap it is well below what the driver reports).
  unsigned long long* clk;
  // Failure-detection self test (see ilre_recall_selftest_wait): spin budget of the
  // row-statistics kernel's waits in SM cycles, and how many of its last key tiles the
  // producer leaves out (0 in normal operation).
  long long wait_limit;
  int skip_tiles;
};

struct PrepParams {
  int n_kv, n_q, group_size, q_len, n_rb, rb_rows;
  long long L;
  int n_sink;
  uint32_t* enc;
  uint32_t* bitmap;
  uint32_t* hist;
  long long hist_words;     // words of the radix histograms to clear
  int n_comb;
  uint32_t* cand_count;     // per-run state words of the selection kernel, cleared here
  int sel_state_words;
  uint32_t* grid_barrier;   // arrival counter of the selection kernel's grid barrier
};

struct MergeParams {
  int n_groups, n_rb, rb_rows, cpg, group_size, q_len, n_q;
  const float* partial;
  float* row_lse;    // [q_len][n_q] natural-log lse
  // Key-range sharding: when n_ext > 0 the statistics come from ext_stats
  // [n_ext][q_len * n_q] (max in log2 units, sum) -- one entry per shard, rows in the
  // caller's order i * n_q + h -- instead of this launch's own partials.
  const float2* ext_stats;
  int n_ext;
};

size_t row_stats_smem_bytes(int rb_rows, int stages);
size_t scores_smem_bytes(int rb_rows, int stages);

cudaError_t launch_prepare(const void* q, void* qp, const PrepParams& p, int n_sm, cudaStream_t st);
cudaError_t launch_row_stats(const CUtensorMap& tk, const CUtensorMap& tq, const QkParams& p,
                             cudaStream_t st);
// (max in log2 units, sum of exponentials) of every query row over the keys of this launch,
// rows in the caller's order i * n_q + h.
cudaError_t launch_export_stats(const MergeParams& p, float2* out, cudaStream_t st);
// out[t] = exp2 of the encoded maxima (the scores of Eq. 5 for a key shard)
cudaError_t launch_decode_scores(const uint32_t* enc, float* out, long long L, cudaStream_t st);
cudaError_t launch_scores(const CUtensorMap& tk, const CUtensorMap& tq, const QkParams& p,
                          const MergeParams& mp, cudaStream_t st);

}  // namespace ilre
