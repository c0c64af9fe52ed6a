// C ABI of the recall library: handle, argument validation, workspace, launch sequence.
#include <cuda.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstdint>
#include <cstdlib>
#include <cstring>
#include <new>

#include <nvtx3/nvToolsExt.h>

#include "../../include/ilre_recall.h"
#include "attn_kernels.cuh"
#include "fill_kernels.cuh"
#include "qk_kernels.cuh"
#include "rerope_kernels.cuh"
#include "sweep_kernels.cuh"
#include "select_kernels.cuh"
#include "sm100_ptx.cuh"

using namespace ilre;

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

constexpr int kNumStages = 4;            // timed stages (see ilre_recall_stage_times)
constexpr int kProfRing = 32;            // runs whose stage events are kept for averaging
constexpr int kMaxSinkStaging = 65536;
static constexpr int kHostPieces = 16;              // most pieces of a pipelined host upload
static constexpr long long kHostPieceMinKeys = 65536;   // no piece shorter than this (128-key multiple)

struct Geometry {
  int group_size, n_rb, rb_rows, n_groups, cpg, n_tiles, stages;
};

}  // namespace

static constexpr int kGuardBytes = 256;       // written once behind every workspace buffer
static constexpr int kGuardByte = 0xA5;
static constexpr int kMaxGuards = 48;

struct ilre_recall {
  ilre_recall_config_t cfg;
  int n_sm;
  EncodeTiledFn encode;
  const uint8_t* guard[kMaxGuards];           // the guard zones, for ilre_recall_check_guards
  int n_guards;
  // workspace (device)
  void* qp;
  float* partial;
  float* row_lse;
  uint32_t* enc;
  float* scores;
  float* pooled;
  float* maxpooled;
  uint32_t* hist;
  int* tile_ties;
  uint32_t* grid_barrier;
  float2* rope_table;                   // (cos, sin) per (chunk distance, channel pair)
  int rope_rows, rope_chunk;            // what the table currently holds
  double rope_theta;
  cudaEvent_t rope_ready;               // recorded after the table's build, on rope_stream
  cudaStream_t rope_stream;
  float2* pos_lo;                       // RoPE angle tables of the key-cache fill
  float2* pos_hi;
  int pos_hi_rows;
  double pos_theta;                     // theta the tables were built for (0 = none)
  cudaEvent_t pos_ready;                // recorded after their build, on pos_stream
  cudaStream_t pos_stream;
  unsigned long long* cand;
  uint32_t* cand_count;
  unsigned long long* pending;
  int* ranked;
  uint32_t* bitmap;
  int* status;
  unsigned long long* clk;              // (cycles, ns) of the last profiled row-statistics launch
  // optional staging for the host entry point
  void* stage_k;
  void* stage_q;
  int* stage_idx;
  // pipelined upload of the host entry point: the key cache is copied in pieces on a stream
  // of its own while the row statistics of the pieces already on the device are computed
  cudaStream_t copy_stream;
  cudaEvent_t copy_begin;
  cudaEvent_t piece_done[kHostPieces];
  float2* piece_stats;                  // [kHostPieces][max_q_len * n_q_heads]
  // bookkeeping
  cudaEvent_t ev[kProfRing][kNumStages + 1];
  int profiling;
  long long prof_runs;                  // runs recorded since profiling was switched on
  int last_launches;
  int last_q_len;
  cudaStream_t last_stream;
  int cand_stride;
  int select_max_grid;                  // co-resident CTAs of the selection kernel
  long long wait_limit;                 // spin budget of the device waits, SM cycles
  int inject;                           // failure-detection self test: which wait cannot complete
};

namespace {

// A named range on the host time line for tracing tools that read NVTX (a no-op without one).
struct TraceRange {
  explicit TraceRange(const char* name) { nvtxRangePushA(name); }
  ~TraceRange() { nvtxRangePop(); }
  TraceRange(const TraceRange&) = delete;
  TraceRange& operator=(const TraceRange&) = delete;
};

// True while `st` is being captured into a CUDA graph.
bool capturing(cudaStream_t st) {
  cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
  return cudaStreamIsCapturing(st, &cs) == cudaSuccess && cs != cudaStreamCaptureStatusNone;
}

// Makes `st` wait for the table build that `ev` marks, issued on another stream.  A stream
// under capture may not wait for an event recorded outside the capture: there the caller
// orders the graph's launch behind the build (the build itself is refused under capture).
cudaError_t wait_for_tables(cudaStream_t st, cudaEvent_t ev) {
  if (capturing(st)) return cudaSuccess;
  return cudaStreamWaitEvent(st, ev, 0);
}

struct DeviceGuard {
  int prev;
  bool ok;
  explicit DeviceGuard(int dev) : prev(-1), ok(false) {
    if (cudaGetDevice(&prev) != cudaSuccess) return;
    ok = (prev == dev) || (cudaSetDevice(dev) == cudaSuccess);
  }
  ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

int rows_padded_bound(int group_size, int q_len) {
  const long long rg = static_cast<long long>(group_size) * q_len;
  const long long n_rb = (rg + kMaxRbRows - 1) / kMaxRbRows;
  return static_cast<int>(rg + 128 * (n_rb + 1));
}

Geometry make_geometry(const ilre_recall_config_t& c, int n_sm, long long L, int q_len) {
  Geometry g;
  g.group_size = c.n_q_heads / c.n_kv_heads;
  const int rg = g.group_size * q_len;
  g.n_rb = (rg + kMaxRbRows - 1) / kMaxRbRows;
  const int per = (rg + g.n_rb - 1) / g.n_rb;
  g.rb_rows = ((per + 127) / 128) * 128;
  g.n_groups = c.n_kv_heads * g.n_rb;
  g.n_tiles = static_cast<int>((L + kTileKeys - 1) / kTileKeys);
  g.cpg = n_sm / g.n_groups;
  if (g.cpg < 1) g.cpg = 1;
  if (g.cpg > g.n_tiles) g.cpg = g.n_tiles;
  const long long fixed = static_cast<long long>(g.rb_rows) * 256 + kSmemTailBytes +
                          static_cast<long long>(g.rb_rows) * 4;
  g.stages = static_cast<int>((kMaxDynSmem - fixed) / kStageBytes);
  if (g.stages > kMaxStages) g.stages = kMaxStages;
  return g;
}

// One workspace buffer of the handle, followed by a guard zone of kGuardBytes that nothing may
// write to (checked by ilre_recall_check_guards).
template <class T>
bool dev_alloc(ilre_recall* h, T** p, size_t count) {
  *p = nullptr;
  const size_t bytes = ((count ? count : 1) * sizeof(T) + 15) & ~static_cast<size_t>(15);
  if (h->n_guards >= kMaxGuards) return false;
  if (cudaMalloc(reinterpret_cast<void**>(p), bytes + kGuardBytes) != cudaSuccess) return false;
  uint8_t* zone = reinterpret_cast<uint8_t*>(*p) + bytes;
  if (cudaMemset(zone, kGuardByte, kGuardBytes) != cudaSuccess) return false;
  h->guard[h->n_guards++] = zone;
  return true;
}

void free_all(ilre_recall* h) {
  cudaFree(h->qp); cudaFree(h->partial); cudaFree(h->row_lse);
  cudaFree(h->enc); cudaFree(h->scores); cudaFree(h->pooled); cudaFree(h->maxpooled); cudaFree(h->hist);
  cudaFree(h->tile_ties); cudaFree(h->grid_barrier); cudaFree(h->rope_table); cudaFree(h->pos_lo); cudaFree(h->pos_hi);
  cudaFree(h->cand); cudaFree(h->cand_count); cudaFree(h->pending); cudaFree(h->ranked); cudaFree(h->bitmap);
  cudaFree(h->status); cudaFree(h->clk); cudaFree(h->stage_k); cudaFree(h->stage_q); cudaFree(h->stage_idx);
  cudaFree(h->piece_stats);
  if (h->copy_stream) cudaStreamDestroy(h->copy_stream);
  if (h->copy_begin) cudaEventDestroy(h->copy_begin);
  if (h->rope_ready) cudaEventDestroy(h->rope_ready);
  if (h->pos_ready) cudaEventDestroy(h->pos_ready);
  for (int i = 0; i < kHostPieces; ++i)
    if (h->piece_done[i]) cudaEventDestroy(h->piece_done[i]);
  for (int r = 0; r < kProfRing; ++r)
    for (int i = 0; i <= kNumStages; ++i)
      if (h->ev[r][i]) cudaEventDestroy(h->ev[r][i]);
}

bool encode_2d(EncodeTiledFn fn, CUtensorMap* map, const void* base, uint64_t inner, uint64_t rows,
               uint64_t row_pitch_bytes, uint32_t box_rows = kTileKeys) {
  const cuuint64_t gdim[2] = {inner, rows};
  const cuuint64_t gstride[1] = {row_pitch_bytes};
  const cuuint32_t box[2] = {64, static_cast<cuuint32_t>(box_rows)};
  const cuuint32_t estride[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstride, box,
            estride, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// with_qk: the call reads a key cache and a query; with_select: it runs Algorithm 1.
int validate_run(const ilre_recall* h, const void* k, long long L, const void* q, int q_len,
                 int budget, const ilre_pool_spec_t* spec, const void* out_idx, bool with_qk,
                 bool with_select) {
  if (!h || !spec) return ILRE_ERR_INVALID_ARG;
  if (with_qk && (!k || !q)) return ILRE_ERR_INVALID_ARG;
  if (L < 1 || q_len < 1 || budget < 0) return ILRE_ERR_INVALID_ARG;
  // an empty result (no budget, no sink part) needs no output buffer
  if (with_select && !out_idx && (budget > 0 || spec->n_sink > 0)) return ILRE_ERR_INVALID_ARG;
  if (spec->n_max < 1 || spec->n_win < 1 || !spec->max_sizes || !spec->win_sizes)
    return ILRE_ERR_INVALID_ARG;
  if (spec->n_sink < 0 || spec->win_op < 0 || spec->win_op > 1) return ILRE_ERR_INVALID_ARG;
  if (spec->reduce_op != 0) return ILRE_ERR_UNSUPPORTED;
  for (int i = 0; i < spec->n_max; ++i) {
    if (spec->max_sizes[i] < 1) return ILRE_ERR_INVALID_ARG;
    if (spec->max_sizes[i] > kMaxMaxSize) return ILRE_ERR_UNSUPPORTED;
  }
  for (int j = 0; j < spec->n_win; ++j) {
    if (spec->win_sizes[j] < 1) return ILRE_ERR_INVALID_ARG;
    if (spec->win_sizes[j] > kMaxWin) return ILRE_ERR_UNSUPPORTED;
  }
  const long long n_comb = static_cast<long long>(spec->n_max) * spec->n_win;
  if (L > h->cfg.max_L || q_len > h->cfg.max_q_len || budget > h->cfg.max_budget ||
      n_comb > h->cfg.max_combinations)
    return ILRE_ERR_CAPACITY;
  if (spec->n_sink > L || budget > L - spec->n_sink) return ILRE_ERR_BUDGET;
  if (with_qk && ((reinterpret_cast<uintptr_t>(k) & 15u) || (reinterpret_cast<uintptr_t>(q) & 15u)))
    return ILRE_ERR_ALIGNMENT;
  return ILRE_OK;
}

#define ILRE_CUDA(expr)                                   \
  do {                                                    \
    if ((expr) != cudaSuccess) return ILRE_ERR_CUDA;      \
  } while (0)

}  // namespace

extern "C" {

int ilre_recall_create(const ilre_recall_config_t* cfg, ilre_recall_t** out) {
  if (!cfg || !out) return ILRE_ERR_INVALID_ARG;
  if (cfg->n_kv_heads < 1 || cfg->n_q_heads < 1 || cfg->max_L < 1 || cfg->max_q_len < 1 ||
      cfg->max_budget < 0 || cfg->max_combinations < 1 || cfg->device < 0)
    return ILRE_ERR_INVALID_ARG;
  if (cfg->head_dim != kHeadDim || cfg->n_q_heads % cfg->n_kv_heads != 0)
    return ILRE_ERR_UNSUPPORTED;
  if (cfg->max_L > 2147483647LL - 256 || cfg->max_budget > kMaxKm - 2 ||
      cfg->max_combinations > kMaxCombos)
    return ILRE_ERR_CAPACITY;
  if (static_cast<long long>(cfg->n_q_heads / cfg->n_kv_heads) * cfg->max_q_len > (1 << 24))
    return ILRE_ERR_CAPACITY;

  int n_dev = 0;
  if (cudaGetDeviceCount(&n_dev) != cudaSuccess || cfg->device >= n_dev) return ILRE_ERR_CUDA;
  DeviceGuard guard(cfg->device);
  if (!guard.ok) return ILRE_ERR_CUDA;
  cudaDeviceProp prop;
  ILRE_CUDA(cudaGetDeviceProperties(&prop, cfg->device));
  if (prop.major != 10) return ILRE_ERR_UNSUPPORTED;       // tcgen05 / TMEM kernels: sm_100 only

  ilre_recall* h = new (std::nothrow) ilre_recall();
  if (!h) return ILRE_ERR_NOMEM;
  std::memset(h, 0, sizeof(*h));
  h->cfg = *cfg;
  h->n_sm = prop.multiProcessorCount;
  h->wait_limit = kWaitCycleLimit;

  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) !=
          cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn) {
    delete h;
    return ILRE_ERR_CUDA;
  }
  h->encode = reinterpret_cast<EncodeTiledFn>(fn);

  const int group_size = cfg->n_q_heads / cfg->n_kv_heads;
  const size_t rows_pad = static_cast<size_t>(rows_padded_bound(group_size, cfg->max_q_len));
  const size_t max_groups = static_cast<size_t>(cfg->n_kv_heads) *
      ((static_cast<size_t>(group_size) * cfg->max_q_len + kMaxRbRows - 1) / kMaxRbRows);
  const size_t max_items = max_groups > static_cast<size_t>(h->n_sm) ? max_groups : h->n_sm;
  const size_t maxL = static_cast<size_t>(cfg->max_L);
  const size_t ncomb = static_cast<size_t>(cfg->max_combinations);
  h->cand_stride = (cfg->max_budget + 2 + 3) & ~3;    // rows of the ranked lists start 16-byte aligned

  bool ok = true;
  ok = ok && dev_alloc(h, reinterpret_cast<uint8_t**>(&h->qp), cfg->n_kv_heads * rows_pad * 256);
  ok = ok && dev_alloc(h, &h->partial, max_items * kMaxRbRows * 2);
  ok = ok && dev_alloc(h, &h->row_lse, static_cast<size_t>(cfg->max_q_len) * cfg->n_q_heads);
  ok = ok && dev_alloc(h, &h->enc, maxL);
  ok = ok && dev_alloc(h, &h->scores, maxL);
  ok = ok && dev_alloc(h, &h->pooled, ncomb * maxL);
  ok = ok && dev_alloc(h, &h->maxpooled, ncomb * (maxL / 2 + 1));   // one array per distinct m > 1
  ok = ok && dev_alloc(h, &h->hist, static_cast<size_t>(kSelectPasses) * kMaxCombos * kHistBins);
  ok = ok && dev_alloc(h, &h->tile_ties, ncomb * (maxL / kSelTile + 1));
  ok = ok && dev_alloc(h, &h->grid_barrier, 1);
  ok = ok && dev_alloc(h, &h->rope_table, static_cast<size_t>(kRopeTableRows) * kRopeHalfDim);
  h->pos_hi_rows = static_cast<int>(cfg->max_L / kRopeLoRows + 2);
  ok = ok && dev_alloc(h, &h->pos_lo, static_cast<size_t>(kRopeLoRows) * 64);
  ok = ok && dev_alloc(h, &h->pos_hi, static_cast<size_t>(h->pos_hi_rows) * 64);
  ok = ok && dev_alloc(h, &h->cand, ncomb * h->cand_stride);
  ok = ok && dev_alloc(h, &h->cand_count, 4 * static_cast<size_t>(kMaxCombos));
  ok = ok && dev_alloc(h, &h->pending, ncomb * kPendCap);
  ok = ok && dev_alloc(h, &h->ranked, ncomb * h->cand_stride);
  ok = ok && dev_alloc(h, &h->bitmap, (maxL + 31) / 32 + 4);    // read four words at a time
  ok = ok && dev_alloc(h, &h->status, 1);
  ok = ok && dev_alloc(h, &h->clk, 2);
  if (ok && cfg->host_staging) {
    ok = ok && dev_alloc(h, reinterpret_cast<uint8_t**>(&h->stage_k), maxL * cfg->n_kv_heads * 256);
    ok = ok && dev_alloc(h, reinterpret_cast<uint8_t**>(&h->stage_q),
                         static_cast<size_t>(cfg->max_q_len) * cfg->n_q_heads * 256);
    ok = ok && dev_alloc(h, &h->stage_idx, static_cast<size_t>(cfg->max_budget) + kMaxSinkStaging);
    ok = ok && dev_alloc(h, &h->piece_stats, static_cast<size_t>(kHostPieces) * cfg->max_q_len * cfg->n_q_heads);
    ok = ok && (cudaStreamCreateWithFlags(&h->copy_stream, cudaStreamNonBlocking) == cudaSuccess);
    ok = ok && (cudaEventCreateWithFlags(&h->copy_begin, cudaEventDisableTiming) == cudaSuccess);
    for (int i = 0; ok && i < kHostPieces; ++i)
      ok = (cudaEventCreateWithFlags(&h->piece_done[i], cudaEventDisableTiming) == cudaSuccess);
  }
  for (int r = 0; ok && r < kProfRing; ++r)
    for (int i = 0; ok && i <= kNumStages; ++i)
      ok = (cudaEventCreate(&h->ev[r][i]) == cudaSuccess);
  ok = ok && (cudaEventCreateWithFlags(&h->rope_ready, cudaEventDisableTiming) == cudaSuccess);
  ok = ok && (cudaEventCreateWithFlags(&h->pos_ready, cudaEventDisableTiming) == cudaSuccess);
  if (ok) ok = (cudaMemset(h->status, 0, sizeof(int)) == cudaSuccess);
  if (ok) ok = (cudaMemset(h->clk, 0, 2 * sizeof(unsigned long long)) == cudaSuccess);
  if (ok) ok = (cudaMemset(h->grid_barrier, 0, sizeof(uint32_t)) == cudaSuccess);
  if (ok) ok = (select_max_grid(h->n_sm, &h->select_max_grid) == cudaSuccess);
  if (ok) ok = (cudaDeviceSynchronize() == cudaSuccess);
  if (!ok) {
    cudaGetLastError();
    free_all(h);
    delete h;
    return ILRE_ERR_NOMEM;
  }
  *out = h;
  return ILRE_OK;
}

}  // extern "C"

namespace {

enum : int { kStageStats = 1, kStageScores = 2, kStageSelect = 4 };

// What one call computes: any of the three stages of the recall, with the hand-over points of
// a key-range sharded run (statistics out / in, scores out / in).
struct RunIo {
  int stages;
  float2* stats_out;            // kStageStats alone: per-row (max in log2 units, sum) of this shard
  const float2* ext_stats;      // kStageScores alone: the shards' statistics [n_ext][q_len * n_q]
  int n_ext;
  float* shard_scores_out;      // kStageScores alone: A^C of this shard's positions
  const float* scores_in;       // kStageSelect alone: A^C of the whole context
};

int recall_impl(ilre_recall_t* h, const void* k_cache_dev, int64_t L, const void* query_dev,
                int32_t q_len, int32_t budget, const ilre_pool_spec_t* spec,
                int32_t* out_idx_dev, float* out_scores_dev, void* cuda_stream, const RunIo& io) {
  static const int32_t kOne = 1;
  static const ilre_pool_spec_t kNoPooling = {1, &kOne, 1, &kOne, 0, 0, 0};
  const bool with_qk = (io.stages & (kStageStats | kStageScores)) != 0;
  const bool with_select = (io.stages & kStageSelect) != 0;
  if (!h) return ILRE_ERR_INVALID_ARG;
  if (!with_select) { spec = &kNoPooling; budget = 0; }
  if (!with_qk) q_len = 1;
  const int v = validate_run(h, k_cache_dev, L, query_dev, q_len, budget, spec, out_idx_dev,
                             with_qk, with_select);
  if (v != ILRE_OK) return v;
  DeviceGuard guard(h->cfg.device);
  if (!guard.ok) return ILRE_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const Geometry g = make_geometry(h->cfg, h->n_sm, L, q_len);
  if (g.stages < 2) return ILRE_ERR_UNSUPPORTED;

  // combination table (Algorithm 1 loop order: max sizes outer, window sizes inner)
  ComboTable tbl;
  std::memset(&tbl, 0, sizeof(tbl));
  const long long Lp = L - spec->n_sink;
  tbl.n_comb = (budget > 0) ? spec->n_max * spec->n_win : 0;
  long long allocated_before = 0;
  for (int i = 0, c = 0; i < spec->n_max && tbl.n_comb; ++i)
    for (int j = 0; j < spec->n_win; ++j, ++c) {
      const int m = spec->max_sizes[i];
      const long long len = (Lp + m - 1) / m;
      long long km = budget / m + 1 + ((Lp % m) != 0 ? 1 : 0);
      if (km > len) km = len;
      tbl.m[c] = m;
      tbl.n[c] = spec->win_sizes[j];
      tbl.len[c] = static_cast<int>(len);
      tbl.quota[c] = budget / tbl.n_comb + (c < budget % tbl.n_comb ? 1 : 0);
      // Algorithm 1 ranks K_m cells, but the quota walk of this combination cannot go further
      // than quota cells that bring a new token plus the cells made up entirely of tokens the
      // earlier combinations took (at most allocated / m full cells and the partial tail
      // cell).  Ranking only that many gives the same walk and, for all but the last
      // combinations, far fewer candidates to select and order.
      long long reach = tbl.quota[c] + allocated_before / m + ((Lp % m) != 0 ? 1 : 0);
      if (reach < 1) reach = 1;
      if (km > reach) km = reach;
      tbl.k_m[c] = static_cast<int>(km);
      allocated_before += tbl.quota[c];
      tbl.tile_begin[c + 1] = tbl.tile_begin[c] + static_cast<int>((len + kSelTile - 1) / kSelTile);
      // the strided max-pool of size m is shared by all window sizes
      tbl.src[c] = -1;
      if (m > 1) {
        int s = 0;
        while (s < tbl.n_src && tbl.src_m[s] != m) ++s;
        if (s == tbl.n_src) {
          const int cells_per_tile = kSrcTileTokens / m;
          tbl.src_m[s] = m;
          tbl.src_len[s] = static_cast<int>(len);
          tbl.src_tile_begin[s + 1] =
              tbl.src_tile_begin[s] + static_cast<int>((len + cells_per_tile - 1) / cells_per_tile);
          ++tbl.n_src;
        }
        tbl.src[c] = s;
      }
    }

  CUtensorMap map_k, map_q;
  std::memset(&map_k, 0, sizeof(map_k));
  std::memset(&map_q, 0, sizeof(map_q));
  if (with_qk &&
      (!encode_2d(h->encode, &map_k, k_cache_dev, static_cast<uint64_t>(h->cfg.n_kv_heads) * 128,
                  static_cast<uint64_t>(L), static_cast<uint64_t>(h->cfg.n_kv_heads) * 256) ||
       !encode_2d(h->encode, &map_q, h->qp, 128, static_cast<uint64_t>(g.n_groups) * g.rb_rows, 256)))
    return ILRE_ERR_CUDA;

  QkParams qk;
  qk.L = L; qk.n_tiles = g.n_tiles; qk.n_groups = g.n_groups; qk.n_rb = g.n_rb;
  qk.rb_rows = g.rb_rows; qk.cpg = g.cpg; qk.stages = g.stages;
  qk.c2 = static_cast<float>(1.4426950408889634 / std::sqrt(static_cast<double>(kHeadDim)));
  qk.partial = h->partial; qk.enc = h->enc; qk.status = h->status;
  qk.clk = h->profiling ? h->clk : nullptr;
  qk.wait_limit = h->wait_limit;
  qk.skip_tiles = (h->inject == ILRE_SELFTEST_MISSING_KEY_TILE) ? 1 : 0;

  PrepParams pp;
  std::memset(&pp, 0, sizeof(pp));
  pp.n_kv = h->cfg.n_kv_heads; pp.n_q = h->cfg.n_q_heads; pp.group_size = g.group_size;
  pp.q_len = q_len; pp.n_rb = g.n_rb; pp.rb_rows = g.rb_rows; pp.L = L; pp.n_sink = spec->n_sink;
  pp.enc = h->enc; pp.bitmap = h->bitmap; pp.hist = h->hist;
  pp.n_comb = tbl.n_comb;
  pp.hist_words = static_cast<long long>(kSelectPasses) * tbl.n_comb * kHistBins;
  pp.cand_count = h->cand_count; pp.grid_barrier = h->grid_barrier;
  pp.sel_state_words = 4 * kMaxCombos;

  MergeParams mp;
  mp.n_groups = g.n_groups; mp.n_rb = g.n_rb; mp.rb_rows = g.rb_rows; mp.cpg = g.cpg;
  mp.group_size = g.group_size; mp.q_len = q_len; mp.n_q = h->cfg.n_q_heads;
  mp.partial = h->partial; mp.row_lse = h->row_lse;

  SelectParams sp;
  std::memset(&sp, 0, sizeof(sp));
  sp.enc = h->enc; sp.scores = h->scores; sp.user_scores = out_scores_dev;
  sp.L = L; sp.n_sink = spec->n_sink; sp.win_op = spec->win_op;
  sp.pooled = h->pooled; sp.pooled_stride = h->cfg.max_L; sp.hist = h->hist;
  sp.maxpooled = h->maxpooled; sp.maxpooled_stride = h->cfg.max_L / 2 + 1;
  sp.tile_ties = h->tile_ties;
  sp.cand = h->cand; sp.cand_stride = h->cand_stride;
  sp.cand_count = h->cand_count; sp.pending = h->pending; sp.ranked = h->ranked; sp.bitmap = h->bitmap;
  sp.out_idx = out_idx_dev; sp.budget = budget; sp.barrier = h->grid_barrier;
  sp.status = h->status;
  sp.wait_limit = h->wait_limit;
  sp.barrier_extra = (h->inject == ILRE_SELFTEST_GRID_BARRIER) ? 1 : 0;
  int max_km = 1;
  for (int c = 0; c < tbl.n_comb; ++c) max_km = tbl.k_m[c] > max_km ? tbl.k_m[c] : max_km;
  const size_t select_smem = select_smem_bytes(L, max_km, budget, &sp);
  // Grid of the selection kernel: enough CTAs for the scan tiles and for the ranking (about a
  // hundred candidates per CTA), but no more, since every grid barrier pays for them.
  long long want_grid = tbl.tile_begin[tbl.n_comb];
  long long n_cand = 0;
  for (int c = 0; c < tbl.n_comb; ++c) n_cand += tbl.k_m[c];
  if (n_cand / 96 > want_grid) want_grid = n_cand / 96;
  if (want_grid < 1) want_grid = 1;
  // a grid just above the cluster size: the cluster barrier is worth more than the extra CTAs
  if (want_grid > kSelClusterMax && want_grid <= 2 * kSelClusterMax) want_grid = kSelClusterMax;
  if (want_grid > h->select_max_grid) want_grid = h->select_max_grid;
  const int select_grid = static_cast<int>(want_grid);

  const bool prof = h->profiling != 0;
  int launches = 0;
  h->last_stream = st;
  h->last_q_len = q_len;
  cudaEvent_t* ev = h->ev[h->prof_runs % kProfRing];
#define ILRE_MARK(i) do { if (prof) ILRE_CUDA(cudaEventRecord(ev[i], st)); } while (0)

  if (!with_qk) pp.n_rb = 0;                             // no query to pack
  mp.ext_stats = io.ext_stats; mp.n_ext = io.n_ext;
  if (io.scores_in) { sp.scores = const_cast<float*>(io.scores_in); sp.scores_given = 1; }
  ILRE_MARK(0);
  {
    TraceRange r("ilre: prepare");
    ILRE_CUDA(launch_prepare(query_dev, h->qp, pp, h->n_sm, st)); ++launches;
  }
  ILRE_MARK(1);
  if (io.stages & kStageStats) {
    TraceRange r("ilre: row statistics (Eq. 4)");
    ILRE_CUDA(launch_row_stats(map_k, map_q, qk, st)); ++launches;
    if (io.stats_out) { ILRE_CUDA(launch_export_stats(mp, io.stats_out, st)); ++launches; }
  }
  ILRE_MARK(2);
  if (io.stages & kStageScores) {
    TraceRange r("ilre: scores (Eq. 5)");
    ILRE_CUDA(launch_scores(map_k, map_q, qk, mp, st)); ++launches;
    if (io.shard_scores_out) {
      ILRE_CUDA(launch_decode_scores(h->enc, io.shard_scores_out, L, st)); ++launches;
    }
  }
  ILRE_MARK(3);
  if (with_select) {
    TraceRange r("ilre: selection (Algorithm 1)");
    ILRE_CUDA(launch_select(tbl, sp, select_grid, select_smem, st)); ++launches;
  }
  ILRE_MARK(4);
#undef ILRE_MARK
  h->last_launches = launches;
  if (prof) ++h->prof_runs;
  return ILRE_OK;
}

}  // namespace

extern "C" {

int ilre_recall_run(ilre_recall_t* h, const void* k_cache_dev, int64_t L, const void* query_dev,
                    int32_t q_len, int32_t budget, const ilre_pool_spec_t* spec,
                    int32_t* out_idx_dev, float* out_scores_dev, void* cuda_stream) {
  const RunIo io = {kStageStats | kStageScores | kStageSelect, nullptr, nullptr, 0, nullptr, nullptr};
  return recall_impl(h, k_cache_dev, L, query_dev, q_len, budget, spec, out_idx_dev, out_scores_dev,
                     cuda_stream, io);
}

int ilre_recall_shard_stats(ilre_recall_t* h, const void* k_shard_dev, int64_t L_shard,
                            const void* query_dev, int32_t q_len, float* stats_out_dev,
                            void* cuda_stream) {
  if (!stats_out_dev) return ILRE_ERR_INVALID_ARG;
  const RunIo io = {kStageStats, reinterpret_cast<float2*>(stats_out_dev), nullptr, 0, nullptr, nullptr};
  return recall_impl(h, k_shard_dev, L_shard, query_dev, q_len, 0, nullptr, nullptr, nullptr,
                     cuda_stream, io);
}

int ilre_recall_shard_scores(ilre_recall_t* h, const void* k_shard_dev, int64_t L_shard,
                             const void* query_dev, int32_t q_len, const float* stats_all_dev,
                             int32_t n_shards, float* scores_out_dev, void* cuda_stream) {
  if (!stats_all_dev || n_shards < 1 || !scores_out_dev) return ILRE_ERR_INVALID_ARG;
  const RunIo io = {kStageScores, nullptr, reinterpret_cast<const float2*>(stats_all_dev), n_shards,
                    scores_out_dev, nullptr};
  return recall_impl(h, k_shard_dev, L_shard, query_dev, q_len, 0, nullptr, nullptr, nullptr,
                     cuda_stream, io);
}

int ilre_recall_allocate(ilre_recall_t* h, const float* scores_dev, int64_t L, int32_t budget,
                         const ilre_pool_spec_t* spec, int32_t* out_idx_dev, void* cuda_stream) {
  if (!scores_dev) return ILRE_ERR_INVALID_ARG;
  const RunIo io = {kStageSelect, nullptr, nullptr, 0, nullptr, scores_dev};
  return recall_impl(h, nullptr, L, nullptr, 1, budget, spec, out_idx_dev, nullptr, cuda_stream, io);
}

int ilre_recall_run_host(ilre_recall_t* h, const void* k_cache_host, int64_t L,
                         const void* query_host, int32_t q_len, int32_t budget,
                         const ilre_pool_spec_t* spec, int32_t* out_idx_host,
                         float* out_scores_host, void* cuda_stream) {
  TraceRange trace("ilre: recall from host memory");
  if (!h || !h->stage_k) return ILRE_ERR_INVALID_ARG;
  const int v = validate_run(h, k_cache_host, L, query_host, q_len, budget, spec, out_idx_host,
                             true, true);
  if (v != ILRE_OK && v != ILRE_ERR_ALIGNMENT) return v;
  if (spec->n_sink > kMaxSinkStaging) return ILRE_ERR_CAPACITY;
  DeviceGuard guard(h->cfg.device);
  if (!guard.ok) return ILRE_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const size_t k_bytes = static_cast<size_t>(L) * h->cfg.n_kv_heads * 256;
  const size_t q_bytes = static_cast<size_t>(q_len) * h->cfg.n_q_heads * 256;
  ILRE_CUDA(cudaMemcpyAsync(h->stage_q, query_host, q_bytes, cudaMemcpyHostToDevice, st));
  // Long contexts: the upload takes ten times longer than the kernels, so the cache goes up in
  // pieces on the copy stream and the row statistics of every piece (Eq. 4's max and sum over
  // its keys) are computed as soon as it has landed; what is left after the last piece is its
  // statistics, the scores pass (which merges the pieces' statistics like those of key
  // shards) and Algorithm 1.
  long long piece_keys = ((L + kHostPieces - 1) / kHostPieces + 127) / 128 * 128;
  if (piece_keys < kHostPieceMinKeys) piece_keys = kHostPieceMinKeys;
  const int n_pieces = static_cast<int>((L + piece_keys - 1) / piece_keys);
  int rc;
  if (n_pieces < 2) {
    ILRE_CUDA(cudaMemcpyAsync(h->stage_k, k_cache_host, k_bytes, cudaMemcpyHostToDevice, st));
    rc = ilre_recall_run(h, h->stage_k, L, h->stage_q, q_len, budget, spec, h->stage_idx, nullptr,
                         st);
  } else {
    const size_t row_bytes = static_cast<size_t>(h->cfg.n_kv_heads) * 256;
    const size_t n_rows = static_cast<size_t>(q_len) * h->cfg.n_q_heads;
    ILRE_CUDA(cudaEventRecord(h->copy_begin, st));            // the staging buffer is free again
    ILRE_CUDA(cudaStreamWaitEvent(h->copy_stream, h->copy_begin, 0));
    rc = ILRE_OK;
    for (int i = 0; i < n_pieces && rc == ILRE_OK; ++i) {
      const long long lo = i * piece_keys;
      const long long hi = (lo + piece_keys < L) ? lo + piece_keys : static_cast<long long>(L);
      uint8_t* dst = static_cast<uint8_t*>(h->stage_k) + lo * row_bytes;
      ILRE_CUDA(cudaMemcpyAsync(dst, static_cast<const uint8_t*>(k_cache_host) + lo * row_bytes,
                                (hi - lo) * row_bytes, cudaMemcpyHostToDevice, h->copy_stream));
      ILRE_CUDA(cudaEventRecord(h->piece_done[i], h->copy_stream));
      ILRE_CUDA(cudaStreamWaitEvent(st, h->piece_done[i], 0));
      const RunIo io = {kStageStats, h->piece_stats + i * n_rows, nullptr, 0, nullptr, nullptr};
      rc = recall_impl(h, dst, hi - lo, h->stage_q, q_len, 0, nullptr, nullptr, nullptr, st, io);
    }
    if (rc == ILRE_OK) {
      const RunIo io = {kStageScores | kStageSelect, nullptr, h->piece_stats, n_pieces, nullptr,
                        nullptr};
      rc = recall_impl(h, h->stage_k, L, h->stage_q, q_len, budget, spec, h->stage_idx, nullptr, st,
                       io);
    }
    if (rc != ILRE_OK) cudaStreamSynchronize(h->copy_stream);   // nothing in flight on return
  }
  if (rc != ILRE_OK) return rc;
  ILRE_CUDA(cudaMemcpyAsync(out_idx_host, h->stage_idx,
                            static_cast<size_t>(spec->n_sink + budget) * sizeof(int32_t),
                            cudaMemcpyDeviceToHost, st));
  if (out_scores_host)
    ILRE_CUDA(cudaMemcpyAsync(out_scores_host, h->scores, static_cast<size_t>(L) * sizeof(float),
                              cudaMemcpyDeviceToHost, st));
  ILRE_CUDA(cudaStreamSynchronize(st));
  return ILRE_OK;
}

int ilre_recall_chunk_attention(ilre_recall_t* h, const void* q_dev, const void* k_dev,
                                const void* v_dev, int32_t chunk_len, int32_t n_prefix,
                                void* out_dev, void* cuda_stream) {
  TraceRange trace("ilre: chunk attention (Eq. 2)");
  if (!h || !q_dev || !k_dev || !v_dev || !out_dev || chunk_len < 1 || n_prefix < 0)
    return ILRE_ERR_INVALID_ARG;
  if (static_cast<long long>(chunk_len) + n_prefix > 2147483647LL - 256) return ILRE_ERR_CAPACITY;
  if ((reinterpret_cast<uintptr_t>(q_dev) & 15u) || (reinterpret_cast<uintptr_t>(k_dev) & 15u) ||
      (reinterpret_cast<uintptr_t>(v_dev) & 15u) || (reinterpret_cast<uintptr_t>(out_dev) & 15u))
    return ILRE_ERR_ALIGNMENT;
  DeviceGuard guard(h->cfg.device);
  if (!guard.ok) return ILRE_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  h->last_stream = st;
  const uint64_t n_rows = static_cast<uint64_t>(n_prefix) + chunk_len;
  const uint64_t q_inner = static_cast<uint64_t>(h->cfg.n_q_heads) * kHeadDim;
  const uint64_t kv_inner = static_cast<uint64_t>(h->cfg.n_kv_heads) * kHeadDim;
  CUtensorMap map_q, map_k, map_v;
  if (!encode_2d(h->encode, &map_q, q_dev, q_inner, chunk_len, q_inner * 2, 128) ||
      !encode_2d(h->encode, &map_k, k_dev, kv_inner, n_rows, kv_inner * 2, 128) ||
      !encode_2d(h->encode, &map_v, v_dev, kv_inner, n_rows, kv_inner * 2, 128))
    return ILRE_ERR_CUDA;
  AttnParams ap;
  ap.c = chunk_len; ap.n_prefix = n_prefix; ap.n_q = h->cfg.n_q_heads; ap.n_kv = h->cfg.n_kv_heads;
  ap.pair = ((h->cfg.n_q_heads / h->cfg.n_kv_heads) % 2 == 0) ? 1 : 0;   // two heads of one kv head per CTA
  ap.c2 = static_cast<float>(1.4426950408889634 / std::sqrt(static_cast<double>(kHeadDim)));
  ap.out = static_cast<uint16_t*>(out_dev); ap.status = h->status;
  ILRE_CUDA(launch_chunk_attention(map_q, map_k, map_v, ap, h->n_sm, st));
  h->last_launches = 1;
  return ILRE_OK;
}

int ilre_recall_fill_keys(ilre_recall_t* h, const void* x_dev, int64_t n_tok, int32_t d_model,
                          const void* w_k_dev, const void* bias_dev, int64_t pos0,
                          double rope_theta, void* k_cache_dev, int64_t L, void* cuda_stream) {
  TraceRange trace("ilre: key fill (Eq. 1, Eq. 3)");
  if (!h || !x_dev || !w_k_dev || !k_cache_dev || n_tok < 0 || d_model < 1 || pos0 < 0 || L < 1 ||
      !(rope_theta > 1.0))
    return ILRE_ERR_INVALID_ARG;
  if (d_model % kFillBlockK != 0) return ILRE_ERR_UNSUPPORTED;
  if (L > h->cfg.max_L || pos0 + n_tok > L || n_tok > 2147483647LL - 256) return ILRE_ERR_CAPACITY;
  if ((reinterpret_cast<uintptr_t>(x_dev) & 15u) || (reinterpret_cast<uintptr_t>(w_k_dev) & 15u) ||
      (reinterpret_cast<uintptr_t>(k_cache_dev) & 15u))
    return ILRE_ERR_ALIGNMENT;
  if (n_tok == 0) return ILRE_OK;
  DeviceGuard guard(h->cfg.device);
  if (!guard.ok) return ILRE_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  h->last_stream = st;
  int launches = 0;
  if (h->pos_theta != rope_theta) {                    // tables depend on theta only
    if (capturing(st)) return ILRE_ERR_UNSUPPORTED;    // a replay would not know they are stale
    ILRE_CUDA(launch_rope_pos_tables(h->pos_lo, h->pos_hi, h->pos_hi_rows, rope_theta, st));
    ILRE_CUDA(cudaEventRecord(h->pos_ready, st));
    h->pos_theta = rope_theta;
    h->pos_stream = st;
    ++launches;
  } else if (st != h->pos_stream) {                    // built on another stream: wait for it
    ILRE_CUDA(wait_for_tables(st, h->pos_ready));
  }
  const int n_out = h->cfg.n_kv_heads * kHeadDim;
  const long long m_tiles = (n_tok + kFillTileM - 1) / kFillTileM;
  // two heads per tile when that still gives every SM a tile, one head per tile otherwise
  const int tile_n = (n_out % 256 == 0 && m_tiles * (n_out / 256) >= h->n_sm) ? 256 : 128;
  const long long n_tiles = m_tiles * (n_out / tile_n);
  CUtensorMap map_x, map_w;
  if (!encode_2d(h->encode, &map_x, x_dev, static_cast<uint64_t>(d_model),
                 static_cast<uint64_t>(n_tok), static_cast<uint64_t>(d_model) * 2, kFillTileM))
    return ILRE_ERR_CUDA;
  if (!encode_2d(h->encode, &map_w, w_k_dev, static_cast<uint64_t>(d_model),
                 static_cast<uint64_t>(n_out), static_cast<uint64_t>(d_model) * 2, tile_n))
    return ILRE_ERR_CUDA;
  FillParams fp;
  fp.n_tok = n_tok; fp.d_model = d_model; fp.n_kv = h->cfg.n_kv_heads; fp.pos0 = pos0;
  fp.bias = static_cast<const uint16_t*>(bias_dev);
  fp.rope_lo = h->pos_lo; fp.rope_hi = h->pos_hi;
  fp.k_cache = static_cast<uint16_t*>(k_cache_dev);
  fp.stages = fill_max_stages(tile_n);
  fp.status = h->status;
  const int grid = static_cast<int>(n_tiles < h->n_sm ? n_tiles : h->n_sm);
  ILRE_CUDA(launch_fill(map_x, map_w, fp, tile_n, grid, st)); ++launches;
  h->last_launches = launches;
  return ILRE_OK;
}

int ilre_recall_rerope_keys(ilre_recall_t* h, const void* k_cache_dev, void* k_out_dev, int64_t L,
                            int32_t chunk_size, int32_t n_sink, double rope_theta,
                            void* cuda_stream) {
  TraceRange trace("ilre: re-rotation (Eq. 7)");
  if (!h || !k_cache_dev || !k_out_dev || L < 1 || chunk_size < 1 || n_sink < 0 || n_sink > L ||
      !(rope_theta > 1.0))
    return ILRE_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(k_cache_dev) & 15u) || (reinterpret_cast<uintptr_t>(k_out_dev) & 15u))
    return ILRE_ERR_ALIGNMENT;
  const long long n_chunks = (L - n_sink + chunk_size - 1) / chunk_size;
  const long long n_rows = n_chunks - 2;               // distinct non-zero distances D_i
  if (n_rows > kRopeTableRows) return ILRE_ERR_CAPACITY;
  if (n_rows < 1 && k_out_dev == k_cache_dev) return ILRE_OK;    // nothing moves
  DeviceGuard guard(h->cfg.device);
  if (!guard.ok) return ILRE_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  h->last_stream = st;
  int launches = 0;
  // The table depends on (chunk, theta) only; rows beyond what an earlier call built are
  // the reason to rebuild.  Rebuilding is stream-ordered before the rotation.
  if (n_rows > 0 && (h->rope_chunk != chunk_size || h->rope_theta != rope_theta ||
                     h->rope_rows < n_rows)) {
    if (capturing(st)) return ILRE_ERR_UNSUPPORTED;    // a replay would not know the table is stale
    ILRE_CUDA(launch_rope_table(h->rope_table, static_cast<int>(n_rows), chunk_size, rope_theta, st));
    ILRE_CUDA(cudaEventRecord(h->rope_ready, st));
    h->rope_chunk = chunk_size; h->rope_theta = rope_theta; h->rope_rows = static_cast<int>(n_rows);
    h->rope_stream = st;
    ++launches;
  } else if (n_rows > 0 && st != h->rope_stream) {     // built on another stream: wait for it
    ILRE_CUDA(wait_for_tables(st, h->rope_ready));
  }
  ReropeParams rp;
  rp.k_in = static_cast<const uint4*>(k_cache_dev);
  rp.k_out = static_cast<uint4*>(k_out_dev);
  rp.L = L; rp.n_kv = h->cfg.n_kv_heads; rp.chunk = chunk_size; rp.n_sink = n_sink;
  rp.n_chunks = n_chunks; rp.table = h->rope_table;
  ILRE_CUDA(launch_rerope(rp, h->n_sm, st)); ++launches;
  h->last_launches = launches;
  return ILRE_OK;
}

int ilre_recall_rerope_sinks(ilre_recall_t* h, const void* k_sink_dev, void* k_out_dev,
                             int32_t n_sink, int32_t chunk_size, int32_t chunk_index,
                             double rope_theta, void* cuda_stream) {
  if (!h || !k_sink_dev || !k_out_dev || n_sink < 0 || chunk_size < 1 || chunk_index < 1 ||
      !(rope_theta > 1.0))
    return ILRE_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(k_sink_dev) & 15u) || (reinterpret_cast<uintptr_t>(k_out_dev) & 15u))
    return ILRE_ERR_ALIGNMENT;
  const long long turns = static_cast<long long>(chunk_index) - 2;     // power of R(D_C)
  if (turns > kRopeTableRows) return ILRE_ERR_CAPACITY;
  if (n_sink == 0 || (turns < 1 && k_out_dev == k_sink_dev)) return ILRE_OK;
  DeviceGuard guard(h->cfg.device);
  if (!guard.ok) return ILRE_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  h->last_stream = st;
  int launches = 0;
  const float2* row = nullptr;
  if (turns >= 1) {
    // Table row r holds the distance (r + 1) * chunk.  Chunks arrive one after another, so
    // the table is built ahead in powers of two rather than one row per call.
    if (h->rope_chunk != chunk_size || h->rope_theta != rope_theta || h->rope_rows < turns) {
      long long want = 64;
      while (want < turns) want *= 2;
      if (want > kRopeTableRows) want = kRopeTableRows;
      if (capturing(st)) return ILRE_ERR_UNSUPPORTED;  // a replay would not know the table is stale
      ILRE_CUDA(launch_rope_table(h->rope_table, static_cast<int>(want), chunk_size, rope_theta, st));
      ILRE_CUDA(cudaEventRecord(h->rope_ready, st));
      h->rope_chunk = chunk_size; h->rope_theta = rope_theta; h->rope_rows = static_cast<int>(want);
      h->rope_stream = st;
      ++launches;
    } else if (st != h->rope_stream) {                 // built on another stream: wait for it
      ILRE_CUDA(wait_for_tables(st, h->rope_ready));
    }
    row = h->rope_table + (turns - 1) * kRopeHalfDim;
  }
  ILRE_CUDA(launch_rotate_rows(static_cast<const uint4*>(k_sink_dev), static_cast<uint4*>(k_out_dev),
                               static_cast<long long>(n_sink) * h->cfg.n_kv_heads, row, st));
  h->last_launches = launches + 1;
  return ILRE_OK;
}

int ilre_gather_input_ids(const int32_t* input_ids_dev, int64_t L, const int32_t* idx_dev,
                          int32_t n_idx, const int32_t* query_ids_dev, int32_t n_query,
                          int32_t* out_ids_dev, void* cuda_stream) {
  if (L < 1 || n_idx < 0 || n_query < 0 || !out_ids_dev || (n_idx > 0 && (!input_ids_dev || !idx_dev)) ||
      (n_query > 0 && !query_ids_dev))
    return ILRE_ERR_INVALID_ARG;
  ILRE_CUDA(launch_gather_ids(input_ids_dev, L, idx_dev, n_idx, query_ids_dev, n_query, out_ids_dev,
                              static_cast<cudaStream_t>(cuda_stream)));
  return ILRE_OK;
}

int ilre_layer_recall(const int32_t* idx_dev, int32_t n_layers, int32_t n_idx,
                      const int32_t* span_begin_dev, const int32_t* span_len_dev, int32_t n_spans,
                      int32_t* hits_out_dev, int32_t* full_out_dev, int32_t* layer_out_dev,
                      void* cuda_stream) {
  if (n_layers < 1 || n_idx < 0 || n_spans < 0 || !full_out_dev || !layer_out_dev ||
      (n_idx > 0 && !idx_dev) || (n_spans > 0 && (!span_begin_dev || !span_len_dev)))
    return ILRE_ERR_INVALID_ARG;
  if (n_layers > kMaxSweepLayers) return ILRE_ERR_CAPACITY;
  ILRE_CUDA(launch_layer_recall(idx_dev, n_layers, n_idx, span_begin_dev, span_len_dev, n_spans,
                                hits_out_dev, full_out_dev, layer_out_dev,
                                static_cast<cudaStream_t>(cuda_stream)));
  return ILRE_OK;
}

int ilre_recall_copy_row_lse(ilre_recall_t* h, float* out_lse_dev, int32_t q_len,
                             void* cuda_stream) {
  if (!h || !out_lse_dev || q_len < 1 || q_len > h->cfg.max_q_len) return ILRE_ERR_INVALID_ARG;
  DeviceGuard guard(h->cfg.device);
  if (!guard.ok) return ILRE_ERR_CUDA;
  ILRE_CUDA(cudaMemcpyAsync(out_lse_dev, h->row_lse,
                            static_cast<size_t>(q_len) * h->cfg.n_q_heads * sizeof(float),
                            cudaMemcpyDeviceToDevice, static_cast<cudaStream_t>(cuda_stream)));
  return ILRE_OK;
}

int ilre_recall_status(ilre_recall_t* h) {
  if (!h) return ILRE_ERR_INVALID_ARG;
  DeviceGuard guard(h->cfg.device);
  if (!guard.ok) return ILRE_ERR_CUDA;
  ILRE_CUDA(cudaStreamSynchronize(h->last_stream));
  int word = 0;
  ILRE_CUDA(cudaMemcpy(&word, h->status, sizeof(int), cudaMemcpyDeviceToHost));
  if (word != 0) ILRE_CUDA(cudaMemset(h->status, 0, sizeof(int)));
  if (word == 0) return ILRE_OK;
  return (word == kDevQuota) ? ILRE_ERR_QUOTA : ILRE_ERR_DEVICE_WAIT;
}

int ilre_recall_sm_clock(ilre_recall_t* h, float* mhz_out_host) {
  if (!h || !mhz_out_host) return ILRE_ERR_INVALID_ARG;
  DeviceGuard guard(h->cfg.device);
  if (!guard.ok) return ILRE_ERR_CUDA;
  ILRE_CUDA(cudaStreamSynchronize(h->last_stream));
  unsigned long long w[2] = {0, 0};
  ILRE_CUDA(cudaMemcpy(w, h->clk, sizeof(w), cudaMemcpyDeviceToHost));
  *mhz_out_host = (w[1] > 0) ? static_cast<float>(1e3 * static_cast<double>(w[0]) / static_cast<double>(w[1])) : 0.f;
  return ILRE_OK;
}

int ilre_recall_selftest_wait(ilre_recall_t* h, int64_t wait_cycle_limit, int32_t what) {
  if (!h || wait_cycle_limit < 0 || what < ILRE_SELFTEST_OFF || what > ILRE_SELFTEST_MISSING_KEY_TILE)
    return ILRE_ERR_INVALID_ARG;
  h->wait_limit = wait_cycle_limit > 0 ? wait_cycle_limit : kWaitCycleLimit;
  h->inject = what;
  return ILRE_OK;
}

int ilre_recall_set_profiling(ilre_recall_t* h, int32_t on) {
  if (!h) return ILRE_ERR_INVALID_ARG;
  h->profiling = on ? 1 : 0;
  h->prof_runs = 0;
  return ILRE_OK;
}

int ilre_recall_stage_times(ilre_recall_t* h, float* ms_host, int32_t n) {
  if (!h || !ms_host || n < 1) return ILRE_ERR_INVALID_ARG;
  if (h->prof_runs < 1) return ILRE_ERR_INVALID_ARG;
  DeviceGuard guard(h->cfg.device);
  if (!guard.ok) return ILRE_ERR_CUDA;
  const int runs = h->prof_runs < kProfRing ? static_cast<int>(h->prof_runs) : kProfRing;
  const int cnt = n < kNumStages ? n : kNumStages;
  for (int i = 0; i < cnt; ++i) ms_host[i] = 0.f;
  for (int r = 0; r < runs; ++r) {
    cudaEvent_t* ev = h->ev[(h->prof_runs - 1 - r) % kProfRing];
    ILRE_CUDA(cudaEventSynchronize(ev[kNumStages]));
    for (int i = 0; i < cnt; ++i) {
      float ms = 0.f;
      ILRE_CUDA(cudaEventElapsedTime(&ms, ev[i], ev[i + 1]));
      ms_host[i] += ms / static_cast<float>(runs);
    }
  }
  return cnt;
}

int ilre_recall_check_guards(ilre_recall_t* h) {
  if (!h) return ILRE_ERR_INVALID_ARG;
  DeviceGuard guard(h->cfg.device);
  if (!guard.ok) return ILRE_ERR_CUDA;
  if (cudaDeviceSynchronize() != cudaSuccess) return ILRE_ERR_CUDA;
  int damaged = 0;
  uint8_t zone[kGuardBytes];
  for (int i = 0; i < h->n_guards; ++i) {
    if (cudaMemcpy(zone, h->guard[i], kGuardBytes, cudaMemcpyDeviceToHost) != cudaSuccess)
      return ILRE_ERR_CUDA;
    bool intact = true;
    for (int b = 0; b < kGuardBytes; ++b) intact = intact && zone[b] == kGuardByte;
    damaged += intact ? 0 : 1;
  }
  return damaged;
}

int ilre_recall_last_launch_count(ilre_recall_t* h) {
  return h ? h->last_launches : ILRE_ERR_INVALID_ARG;
}

int ilre_recall_destroy(ilre_recall_t* h) {
  if (!h) return ILRE_ERR_INVALID_ARG;
  DeviceGuard guard(h->cfg.device);
  if (!guard.ok) return ILRE_ERR_CUDA;
  cudaDeviceSynchronize();
  free_all(h);
  delete h;
  return ILRE_OK;
}

const char* ilre_strerror(int code) {
  switch (code) {
    case ILRE_OK: return "ok";
    case ILRE_ERR_INVALID_ARG: return "invalid argument";
    case ILRE_ERR_UNSUPPORTED: return "unsupported configuration (needs head_dim 128, sm_100)";
    case ILRE_ERR_CAPACITY: return "size exceeds the capacity given at create()";
    case ILRE_ERR_BUDGET: return "budget larger than the context without its sink part";
    case ILRE_ERR_ALIGNMENT: return "key cache / query base address must be 16-byte aligned";
    case ILRE_ERR_CUDA: return "CUDA call failed";
    case ILRE_ERR_DEVICE_WAIT: return "a bounded wait inside a kernel gave up";
    case ILRE_ERR_QUOTA: return "a combination ran out of candidates";
    case ILRE_ERR_NOMEM: return "device allocation failed";
    default: return "unknown status";
  }
}

}  // extern "C"
