// Parameters and launcher of the Algorithm 1 kernel: pooling, ranked top-K_m per combination,
// quota allocation with de-duplication, ascending output.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace ilre {

static constexpr int kMaxCombos = 64;
static constexpr int kHistBins = 2048;
static constexpr int kMaxWin = 1024;        // largest stride-1 window size
static constexpr int kMaxMaxSize = 64;      // largest strided max-pool size
static constexpr int kMaxKm = 16384;        // largest K_m (bounds the candidate lists)
static constexpr int kSelectPasses = 3;     // 32 value bits of the key in 11/11/10-bit digits
static constexpr int kSelThreads = 1024;    // threads per CTA of the selection kernel
static constexpr int kSelTile = 4096;       // cells of one combination per work tile
static constexpr int kSrcTileTokens = 8192; // tokens per work tile of the strided max-pool
static constexpr int kSelClusterMax = 8;     // grids up to this size run as one thread-block cluster
static constexpr int kPendCap = 8192;        // cells of the threshold bin resolved by one CTA (else: more passes)
static constexpr int kSelBitmapSmemBytes = 136 * 1024;   // bitmap kept in shared memory up to this
static constexpr int kSelMaxDynSmemBytes = kSelBitmapSmemBytes + kMaxKm * 4;

// One entry per (m_i, n_j) combination, in Algorithm 1's loop order.
struct ComboTable {
  int n_comb;
  int m[kMaxCombos];       // strided max-pool size
  int n[kMaxCombos];       // window size
  int len[kMaxCombos];     // number of cells = ceil((L - n_sink) / m)
  int k_m[kMaxCombos];     // candidates ranked for this combination
  int quota[kMaxCombos];   // B_c
  int tile_begin[kMaxCombos + 1];   // first work tile of each combination (prefix sums)
  // Distinct strided max-pool sizes m > 1 ("sources"): their pooled arrays are computed once
  // and shared by every window size.  src[c] = source of combination c, -1 = the scores.
  int n_src;
  int src[kMaxCombos];
  int src_m[kMaxCombos];
  int src_len[kMaxCombos];
  int src_tile_begin[kMaxCombos + 1];   // tiles of kSrcTileTokens / m cells each
  // Ranking phase (filled in by launch_select): with rank_by_list, combination c is ranked by
  // the CTAs [rank_cta_begin[c], rank_cta_begin[c + 1]).
  int rank_by_list;
  int rank_cta_begin[kMaxCombos + 1];
};

struct SelectParams {
  const uint32_t* enc;     // [L] order-preserving uint of max_r log2 p_rt (scores pass output)
  float* scores;           // A^C [L]
  float* user_scores;      // optional copy of A^C for the caller, or null
  int scores_given;        // 1: `scores` already holds A^C (phase A is skipped)
  long long L;
  int n_sink;
  int win_op;              // 0 average, 1 max
  float* maxpooled;        // [n_src][maxpooled_stride] strided max-pool of the scores
  long long maxpooled_stride;
  float* pooled;           // [n_comb][pooled_stride]
  long long pooled_stride;
  uint32_t* hist;          // [kSelectPasses][n_comb][kHistBins], zero on entry
  int* tile_ties;          // [work tiles]: cells of a tile that hold the K_m-th value
  unsigned long long* cand;   // [n_comb][cand_stride] selected 64-bit keys
  int cand_stride;
  uint32_t* cand_count;    // [4 * kMaxCombos]: candidates gathered per combination; then, at
                           // kMaxCombos, 2 kMaxCombos and 3 kMaxCombos: cells pending in the
                           // threshold bin, keys still wanted from it, and one flag word
                           // (some combination needs the full-scan passes); zero on entry
  unsigned long long* pending;   // [n_comb][kPendCap] keys of the threshold bin
  int* ranked;             // [n_comb][cand_stride] cell ids in rank order (cand_stride: multiple of 4)
  uint32_t* bitmap;        // [ceil(L/32)] in global memory, used when it does not fit shared memory
  int bitmap_in_smem;
  int stage_capacity;      // cell ids per staging buffer of the quota walk (>= largest K_m, multiple of 4)
  int stage_double;        // two staging buffers fit shared memory
  int walk_threads;        // threads that walk the combinations in the allocation phase
  int* out_idx;            // [n_sink + budget]
  int budget;
  uint32_t* barrier;       // grid barrier arrival counter, zero when the kernel starts
  int* status;
  // Failure-detection self test (see ilre_recall_selftest_wait): spin budget of a grid
  // barrier in SM cycles, and how many CTAs more than the grid has the barrier waits for
  // (0 in normal operation).
  long long wait_limit;
  int barrier_extra;
};

// Dynamic shared memory the kernel needs for a context of L positions and a budget.
// Also fills p->bitmap_in_smem, p->stage_capacity, p->stage_double and p->walk_threads.
size_t select_smem_bytes(long long L, int max_km, int budget, SelectParams* p);
// Largest grid that is co-resident on the device (the kernel's CTAs wait on one another).
cudaError_t select_max_grid(int n_sm, int* max_grid);
// One cooperative launch: A^C from the encoded maxima, then all of Algorithm 1.
cudaError_t launch_select(const ComboTable& tbl, const SelectParams& p, int grid, size_t smem,
                          cudaStream_t st);

}  // namespace ilre
