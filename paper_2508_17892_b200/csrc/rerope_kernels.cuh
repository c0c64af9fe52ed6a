// Re-rotation of the retrieval layer's cached keys under Dual Chunk Attention (Eq. 7).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace ilre {

static constexpr int kRopeTableRows = 8192;     // distinct chunk distances the table can hold
static constexpr int kRopeHalfDim = 64;         // head_dim / 2

struct ReropeParams {
  const uint4* k_in;      // bf16 [L][n_kv][128] as 16 x uint4 per (position, kv head)
  uint4* k_out;           // may alias k_in
  long long L;
  int n_kv;
  int chunk;
  int n_sink;
  long long n_chunks;     // N_C = ceil((L - n_sink) / chunk)
  const float2* table;    // [n_chunks - 2][64]: (cos, sin) of D * theta^(-2c/d), D = (row+1)*chunk
};

// (cos, sin) of every (chunk distance, channel pair) in double precision, stored as fp32.
cudaError_t launch_rope_table(float2* table, int n_rows, int chunk, double theta,
                              cudaStream_t st);
// K~ = R(D_i) K for the chunks before the last two; the last two are copied when out != in.
cudaError_t launch_rerope(const ReropeParams& p, int n_sm, cudaStream_t st);

// Every (row, kv head) vector of k_in [n_rows][128] turned by the distance of `table_row`
// ([64] (cos, sin)); a null row copies.  k_out may alias k_in.
cudaError_t launch_rotate_rows(const uint4* k_in, uint4* k_out, long long n_rows,
                               const float2* table_row, cudaStream_t st);

// out = ids[idx[0..n_idx)] followed by query_ids[0..n_query)
cudaError_t launch_gather_ids(const int32_t* ids, long long L, const int32_t* idx, int n_idx,
                              const int32_t* query_ids, int n_query, int32_t* out,
                              cudaStream_t st);

}  // namespace ilre
