// Key-cache fill of the retrieval layer: K = PE(X W_K^T + b) written into the cache (Eq. 1 with
// the RoPE of Eq. 3; Section 3.3, the step at the retrieval layer).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace ilre {

static constexpr int kFillBlockK = 64;          // model channels per pipeline stage (128 B rows)
static constexpr int kFillTileM = 128;          // tokens per output tile
static constexpr int kFillThreads = 192;        // warp 0 TMA, warp 1 MMA, warps 2..5 epilogue
static constexpr int kRopeLoRows = 1024;        // position = hi * kRopeLoRows + lo

struct FillParams {
  long long n_tok;        // tokens of this call
  int d_model;            // multiple of kFillBlockK
  int n_kv;               // kv heads; W has n_kv * 128 rows
  long long pos0;         // position of the first token
  const uint16_t* bias;   // optional bf16 [n_kv * 128], or null
  const float2* rope_lo;  // [kRopeLoRows][64]: (cos, sin) of lo * theta^(-2c/128)
  const float2* rope_hi;  // [..][64]: (cos, sin) of hi * kRopeLoRows * theta^(-2c/128)
  uint16_t* k_cache;      // bf16 [L][n_kv][128]
  int stages;
  int* status;
};

size_t fill_smem_bytes(int tile_n, int stages);
int fill_max_stages(int tile_n);
cudaError_t launch_rope_pos_tables(float2* lo, float2* hi, int hi_rows, double theta,
                                   cudaStream_t st);
// tile_n = 128 (one head per tile) or 256 (two heads per tile)
cudaError_t launch_fill(const CUtensorMap& map_x, const CUtensorMap& map_w, const FillParams& p,
                        int tile_n, int grid, cudaStream_t st);

}  // namespace ilre
