// Parameters and launchers of the Algorithm 1 kernels: pooling, ranked top-K_m per
// combination, quota allocation with de-duplication, ascending output.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace ilre {

static constexpr int kMaxCombos = 64;
static constexpr int kHistBins = 2048;
static constexpr int kMaxWin = 1024;        // largest stride-1 window size
static constexpr int kMaxMaxSize = 64;      // largest strided max-pool size
static constexpr int kMaxKm = 16384;        // largest K_m the in-block ranking sort holds
static constexpr int kSelectPasses = 6;     // 64-bit (value, index) key, 11/11/10 bits twice

// One entry per (m_i, n_j) combination, in Algorithm 1's loop order.
struct ComboTable {
  int n_comb;
  int m[kMaxCombos];       // strided max-pool size
  int n[kMaxCombos];       // window size
  int len[kMaxCombos];     // number of cells = ceil((L - n_sink) / m)
  int k_m[kMaxCombos];     // candidates ranked for this combination
  int quota[kMaxCombos];   // B_c
};

struct SelectParams {
  const float* scores;     // A^C [L]
  long long L;
  int n_sink;
  int win_op;              // 0 average, 1 max
  float* pooled;           // [n_comb][pooled_stride]
  long long pooled_stride;
  uint32_t* hist;          // [n_comb][kHistBins]
  unsigned long long* sel_prefix;
  uint32_t* sel_krem;
  uint32_t* sel_done;
  uint32_t* sel_ticket;
  unsigned long long* cand;   // [n_comb][cand_stride] selected 64-bit keys
  int cand_stride;
  uint32_t* cand_count;
  int* ranked;             // [n_comb][cand_stride] cell ids in rank order
  uint32_t* bitmap;        // [ceil(L/32)]
  int* out_idx;            // [n_sink + budget]
  int budget;
  int* status;
};

cudaError_t launch_pool(const ComboTable& tbl, const SelectParams& p, int max_len, cudaStream_t st);
cudaError_t launch_select_pass(const ComboTable& tbl, const SelectParams& p, int max_len, int pass,
                               cudaStream_t st);
cudaError_t launch_gather(const ComboTable& tbl, const SelectParams& p, int max_len,
                          cudaStream_t st);
cudaError_t launch_rank_sort(const ComboTable& tbl, const SelectParams& p, int max_km,
                             cudaStream_t st);
cudaError_t launch_allocate(const ComboTable& tbl, const SelectParams& p, cudaStream_t st);

}  // namespace ilre
