// Streaming chunked prefill attention of one chunk (Eq. 2 with the Lambda-shaped mask): the
// layers before the retrieval layer attend to the cached sink + sliding-window keys/values and,
// causally, to the chunk's own.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace ilre {

static constexpr int kAttnThreads = 352;     // warp 0 TMA, warp 1 S MMAs, warp 2 PV MMAs, warps 3..6 / 7..10 softmax

struct AttnParams {
  int c;             // query tokens of the chunk
  int n_prefix;      // rows of K/V visible to every query (sink + sliding window)
  int n_q, n_kv;     // query heads, kv heads
  int pair;          // 1: a CTA serves two query heads of one kv head; 0: one head
  int n_qt;          // query tiles of 128 tokens
  int split_from;    // query tiles >= split_from get one CTA per head (pair mode only; n_qt = none)
  float c2;          // log2(e) / sqrt(d)
  uint16_t* out;     // bf16 [c][n_q][128]
  int* status;
};

size_t attn_smem_bytes();
// One CTA per (query tile, head pair) -- or per head, for the query tiles from split_from on;
// fills p.n_qt and p.split_from (n_sm: SMs of the device).
cudaError_t launch_chunk_attention(const CUtensorMap& map_q, const CUtensorMap& map_k,
                                   const CUtensorMap& map_v, AttnParams p, int n_sm, cudaStream_t st);

}  // namespace ilre
