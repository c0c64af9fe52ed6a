// Offline choice of the retrieval layer from the recalled index lists of the candidate layers
// (Section 3.3, first paragraph; retrieval task of Appendix A.1).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace ilre {

static constexpr int kMaxSweepLayers = 1024;

// hits[l][s] = recalled positions of layer l inside phrase s; full[l] = phrases recalled
// completely; *layer = smallest l with the largest full[l].  idx rows must be ascending.
cudaError_t launch_layer_recall(const int32_t* idx, int n_layers, int n_idx,
                                const int32_t* span_begin, const int32_t* span_len, int n_spans,
                                int32_t* hits, int32_t* full, int32_t* layer, cudaStream_t st);

}  // namespace ilre
