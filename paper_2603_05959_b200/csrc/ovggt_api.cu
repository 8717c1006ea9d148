// Host side of the C ABI declared in include/ovggt.h: handle, bookkeeping that needs no device
// read-back (row counts, anchor FIFO, trigger rule), workspace layout and kernel launches.
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <deque>
#include <new>
#include <vector>

#include <nvtx3/nvToolsExt.h>

#include "../../include/ovggt.h"
#include "attn_simt.cuh"
#include "attn_tcgen05.cuh"
#include "common.cuh"
#include "compact_kernels.cuh"
#include "gemm_tcgen05.cuh"
#include "score_kernels.cuh"
#include "select_kernel.cuh"

using namespace ovggt;

namespace {

std::atomic<uint64_t> g_launches{0};
std::atomic<int> g_last_cuda_error{0};

inline int cuda_fail(cudaError_t e) {
  g_last_cuda_error.store((int)e);
  return OVGGT_ERR_CUDA;
}
#define CK(expr)                                  \
  do {                                            \
    cudaError_t e__ = (expr);                     \
    if (e__ != cudaSuccess) return cuda_fail(e__); \
  } while (0)
#define LAUNCHED()                                 \
  do {                                             \
    g_launches.fetch_add(1);                       \
    cudaError_t e__ = cudaGetLastError();          \
    if (e__ != cudaSuccess) return cuda_fail(e__); \
  } while (0)

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

constexpr int kMaxColsumParts = 592;       // 4 CTAs per SM on 148 SMs
constexpr size_t kSmemLimit = 227 * 1024;

int colsum_parts(int rows) { return std::max(1, std::min(kMaxColsumParts, (rows + 15) / 16)); }

// CTAs per cluster of the selection kernels: about 2K candidates per CTA, at most 8 (the portable limit).
int select_cluster_ctas(int N) { return std::max(1, std::min(kSelectMaxCtas, (N + 2047) / 2048)); }

template <typename... KArgs, typename... Args>
cudaError_t launch_cluster(void (*kernel)(KArgs...), dim3 grid, int ncta, size_t smem, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(kSelectThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeClusterDimension;
  attr.val.clusterDim.x = ncta;
  attr.val.clusterDim.y = 1;
  attr.val.clusterDim.z = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, args...);
}

// ------------------------------------------------------------------ single-kernel launchers

int launch_row_norms(const void* x, int rows, int C, int dtype, float* s, cudaStream_t st) {
  if (rows <= 0) return OVGGT_OK;
  const int nvec = C * elem_bytes(dtype) / 16;
  const int grid = (rows + 7) / 8;
  if (dtype == kBF16) k_row_norms<kBF16><<<grid, 256, 0, st>>>((const uint4*)x, rows, nvec, s);
  else                k_row_norms<kF32><<<grid, 256, 0, st>>>((const uint4*)x, rows, nvec, s);
  LAUNCHED();
  return OVGGT_OK;
}

// part: [colsum_parts(rows), C] floats; ksum: [C] floats.
int launch_diversity(const void* K, int rows, int C, int dtype, float* part, float* ksum, float* d,
                     cudaStream_t st) {
  if (rows <= 0) return OVGGT_OK;
  const int nvec = C * elem_bytes(dtype) / 16;
  const int parts = colsum_parts(rows);
  const int rpc = (rows + parts - 1) / parts;
  const int threads = std::min(256, (nvec + 31) / 32 * 32);
  if (dtype == kBF16) k_colsum_partial<kBF16><<<parts, threads, 0, st>>>((const uint4*)K, rows, nvec, rpc, part);
  else                k_colsum_partial<kF32><<<parts, threads, 0, st>>>((const uint4*)K, rows, nvec, rpc, part);
  LAUNCHED();
  k_colsum_final<<<(C + 31) / 32, 1024, 0, st>>>(part, parts, C, ksum);
  LAUNCHED();
  const int grid = std::min((rows + 7) / 8, 148 * 8);
  const size_t smem = (size_t)C * 4;
  if (dtype == kBF16)
    k_diversity<kBF16><<<grid, 256, smem, st>>>((const uint4*)K, rows, nvec, ksum, 1, nullptr, d, grid, nullptr, 0,
                                                nullptr);
  else
    k_diversity<kF32><<<grid, 256, smem, st>>>((const uint4*)K, rows, nvec, ksum, 1, nullptr, d, grid, nullptr, 0,
                                               nullptr);
  LAUNCHED();
  return OVGGT_OK;
}

constexpr int kColsumSlices = 8;

// Diversity from the per-CTA column sums the last compaction left (nparts rows of part): no pass over K for the sums.
// slices: [kColsumSlices, C] floats of scratch, then the column sums [C], then one arrival counter per 32 columns
// (colsum_scratch_bytes(C) in all; the counters zero before the first use).
size_t colsum_scratch_bytes(int C) { return ((size_t)(kColsumSlices + 1) * C * 4 + ((size_t)(C + 31) / 32) * 4 + 255) / 256 * 256; }
// The same launch also computes the residual norms s_raw [resid_rows] of the new frame when resid is given.
int launch_diversity_from_parts(const void* K, int rows, int C, int dtype, const float* part, int nparts, float* slices,
                                float* d, const void* resid, int resid_rows, float* s_raw, cudaStream_t st) {
  if (rows <= 0) return OVGGT_OK;
  const int nvec = C * elem_bytes(dtype) / 16;
  float* ksum = slices + (size_t)kColsumSlices * C;
  int* arrived = reinterpret_cast<int*>(ksum + C);
  k_colsum_final_sliced<<<dim3((C + 31) / 32, kColsumSlices), 1024, 0, st>>>(part, nparts, C, slices, ksum, arrived);
  LAUNCHED();
  const int grid = std::min((rows + 63) / 64, 148 * 8);   // eight rows per warp: the centroid registers are loaded once
  const size_t smem = (size_t)C * 4;
  const int norm_ctas = resid ? (resid_rows + 7) / 8 : 0;
  if (dtype == kBF16)
    k_diversity<kBF16><<<grid + norm_ctas, 256, smem, st>>>((const uint4*)K, rows, nvec, ksum, 1, nullptr, d, grid,
                                                            (const uint4*)resid, resid_rows, s_raw);
  else
    k_diversity<kF32><<<grid + norm_ctas, 256, smem, st>>>((const uint4*)K, rows, nvec, ksum, 1, nullptr, d, grid,
                                                           (const uint4*)resid, resid_rows, s_raw);
  LAUNCHED();
  return OVGGT_OK;
}

// Compaction that also leaves per-CTA column sums of the keys it writes; *nparts = number of partial rows written.
int launch_compact_colsum(const void* ks, const void* vs, const int* surv, int n_keep, int C, int dtype, void* kd,
                          void* vd, float* part, int* nparts, cudaStream_t st, int n_src, int* status) {
  *nparts = 0;
  if (n_keep <= 0) return OVGGT_OK;
  const int nvec = C * elem_bytes(dtype) / 16;
  const int grid = std::min((n_keep + 31) / 32, 148 * 8);   // four survivors (K and V rows) per warp
  if (dtype == kBF16)
    k_compact_colsum<kBF16><<<grid, 256, 0, st>>>((const uint4*)ks, (const uint4*)vs, surv, n_keep, nvec, (uint4*)kd,
                                                  (uint4*)vd, part, n_src, status);
  else
    k_compact_colsum<kF32><<<grid, 256, 0, st>>>((const uint4*)ks, (const uint4*)vs, surv, n_keep, nvec, (uint4*)kd,
                                                 (uint4*)vd, part, n_src, status);
  LAUNCHED();
  *nparts = grid;
  return OVGGT_OK;
}

int launch_compact(const void* ks, const void* vs, const int* surv, int n_keep, int C, int dtype, void* kd,
                   void* vd, cudaStream_t st, int n_src, int* status) {
  if (n_keep <= 0) return OVGGT_OK;
  const int nvec = C * elem_bytes(dtype) / 16;
  const int grid = std::min((2 * n_keep + 7) / 8, 148 * 8);
  k_compact<<<grid, 256, 0, st>>>((const uint4*)ks, (const uint4*)vs, surv, n_keep, nvec, (uint4*)kd, (uint4*)vd, n_src,
                                  status);
  LAUNCHED();
  return OVGGT_OK;
}

// Diversity against sums given as n_slices rows (see k_diversity); the frame's residual norms ride in the same
// launch when resid is given; the folded sums go to ksum_out when it is given.
int launch_diversity_sliced(const void* K, int rows, int C, int dtype, const float* ksum, int n_slices, float* ksum_out,
                            float* d, const void* resid, int resid_rows, float* s_raw, cudaStream_t st) {
  if (rows <= 0) return OVGGT_OK;
  const int nvec = C * elem_bytes(dtype) / 16;
  const int grid = std::min((rows + 63) / 64, 148 * 8);
  const size_t smem = (size_t)C * 4;
  const int norm_ctas = resid ? (resid_rows + 7) / 8 : 0;
  if (dtype == kBF16)
    k_diversity<kBF16><<<grid + norm_ctas, 256, smem, st>>>((const uint4*)K, rows, nvec, ksum, n_slices, ksum_out, d,
                                                            grid, (const uint4*)resid, resid_rows, s_raw);
  else
    k_diversity<kF32><<<grid + norm_ctas, 256, smem, st>>>((const uint4*)K, rows, nvec, ksum, n_slices, ksum_out, d,
                                                           grid, (const uint4*)resid, resid_rows, s_raw);
  LAUNCHED();
  return OVGGT_OK;
}

// Column sums of K [rows, C] into ksum [C] (two kernels; part: [colsum_parts(rows), C] floats of scratch).
int launch_colsum(const void* K, int rows, int C, int dtype, float* part, float* ksum, cudaStream_t st) {
  const int nvec = C * elem_bytes(dtype) / 16;
  const int parts = colsum_parts(rows);
  const int rpc = (rows + parts - 1) / parts;
  const int threads = std::min(256, (nvec + 31) / 32 * 32);
  if (dtype == kBF16) k_colsum_partial<kBF16><<<parts, threads, 0, st>>>((const uint4*)K, rows, nvec, rpc, part);
  else                k_colsum_partial<kF32><<<parts, threads, 0, st>>>((const uint4*)K, rows, nvec, rpc, part);
  LAUNCHED();
  k_colsum_final<<<(C + 31) / 32, 1024, 0, st>>>(part, parts, C, ksum);
  LAUNCHED();
  return OVGGT_OK;
}

// Supp. D, attention-weight criterion: s[j] = mean over the M queries and the heads of the attention key j of the
// frame received, from the log2 denominators the attention left in lse [M, H] (part: [H, M] floats of scratch).
int launch_attention_received(const void* q, const void* k, int M, int C, int n_heads, int dtype, const float* lse,
                              float* part, float* s, cudaStream_t st) {
  (void)C;
  dim3 grid((M + kRecvTile - 1) / kRecvTile, n_heads);
  if (dtype == kBF16) k_attn_received<kBF16><<<grid, 256, 0, st>>>((const uint4*)q, (const uint4*)k, M, n_heads, lse, part);
  else                k_attn_received<kF32><<<grid, 256, 0, st>>>((const uint4*)q, (const uint4*)k, M, n_heads, lse, part);
  LAUNCHED();
  k_fold_heads<<<(M + 255) / 256, 256, 0, st>>>(part, M, n_heads, 1.0f / ((float)M * (float)n_heads), s);
  LAUNCHED();
  return OVGGT_OK;
}

// Supp. D, query-key criterion: s[j] = mean over the M queries and the heads of q_i . k_j / sqrt(d), taken through
// the column sums of Q (qsum [C] after part [colsum_parts(M), C]; three small kernels).
int launch_qk_scores(const void* q, const void* k, int M, int C, int n_heads, int dtype, float* part, float* qsum,
                     float* s, cudaStream_t st) {
  int rc = launch_colsum(q, M, C, dtype, part, qsum, st);
  if (rc) return rc;
  const int nvec = C * elem_bytes(dtype) / 16;
  const float scale = 1.0f / ((float)M * (float)n_heads * sqrtf((float)(C / n_heads)));
  const int grid = (M + 7) / 8;
  if (dtype == kBF16) k_row_dots<kBF16><<<grid, 256, 0, st>>>((const uint4*)k, M, nvec, qsum, scale, s);
  else                k_row_dots<kF32><<<grid, 256, 0, st>>>((const uint4*)k, M, nvec, qsum, scale, s);
  LAUNCHED();
  return OVGGT_OK;
}

// The hole-filling move (and, with delta, what it does to the key column sums).
int launch_fill_holes(void* kc, void* vc, const int* msrc, const int* mdst, const int* mj, const int* n_moves, int max_moves,
                      int C, int dtype, int* slot_meta, float* delta, cudaStream_t st, int rows_cap, int n_meta,
                      int* status) {
  const int nvec = C * elem_bytes(dtype) / 16;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(kFillSlices * kFillClusterCtas);
  cfg.blockDim = dim3(kFillThreads);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = st;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeClusterDimension;
  attr.val.clusterDim.x = kFillClusterCtas;
  attr.val.clusterDim.y = 1;
  attr.val.clusterDim.z = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  cudaError_t e;
  if (dtype == kBF16)
    e = cudaLaunchKernelEx(&cfg, k_fill_holes<kBF16>, (uint4*)kc, (uint4*)vc, msrc, mdst, mj, n_moves, max_moves, nvec,
                           slot_meta, delta, rows_cap, n_meta, status);
  else
    e = cudaLaunchKernelEx(&cfg, k_fill_holes<kF32>, (uint4*)kc, (uint4*)vc, msrc, mdst, mj, n_moves, max_moves, nvec,
                           slot_meta, delta, rows_cap, n_meta, status);
  if (e != cudaSuccess) return cuda_fail(e);
  LAUNCHED();
  return OVGGT_OK;
}

int launch_attention(const void* q, const void* k, const void* v, int M, int N, int H, int dtype, void* out,
                     void* scratch, int* status, cudaStream_t st, AttnKvMaps* maps = nullptr,
                     const float* kmax2 = nullptr, float* lse = nullptr) {
  if (dtype == kBF16) {
    int rc = attn_tcgen05_launch(q, k, v, M, N, H, out, scratch, status, st, maps, 0, kmax2, lse);
    if (rc == OVGGT_OK) g_launches.fetch_add(attn_tcgen05_num_launches(M, N, H));
    if (rc == OVGGT_ERR_CUDA) g_last_cuda_error.store(attn_tcgen05_last_error());
    return rc;
  }
  dim3 grid((M + kSimtRows - 1) / kSimtRows, H);
  k_attn_simt<kF32><<<grid, kSimtRows, 0, st>>>(q, k, v, M, N, H, out, lse);
  LAUNCHED();
  return OVGGT_OK;
}

}  // namespace

// ------------------------------------------------------------------ handle

// Steps between two full recomputations of the key column sums in the hole-filling layout: in between, the sums
// follow the cache by "+ admitted - evicted" corrections, whose fp32 rounding (about 1e-7 relative per step) adds up.
constexpr int kColsumRefreshEvery = 64;

struct LayerState {
  int budget = 0;
  int n = 0;            // rows held between steps
  int cur = 0;          // which of the two meta buffers (ids, flags, stored scores, slots) describes them
  int kv = 0;           // which K/V buffer holds them (always 0 in the hole-filling layout)
  bool pending = false; // a frame was appended and not yet compressed
  int64_t frames_seen = 0, evicted_total = 0, pending_frame = -1;
  int n_prot_init = 0, n_prot_hist = 0;
  int last_N = 0, last_keep = 0;
  // device pointers
  char* kbuf[2];
  char* vbuf[2];
  long long* ids[2];
  uint8_t* flags[2];
  float* stored[2];
  int* slot[2] = {nullptr, nullptr};   // hole-filling layout: physical K/V slot of each logical row
  float *s_raw, *d, *r;
  int* surv;
  int* n_keep_dev;
  float* colsum_part = nullptr;   // stable layout: [148 * 8, C] per-CTA column sums of the keys the last compaction wrote
  int colsum_nparts = 0;          // 0: not available (the next step sums the keys itself)
  // hole-filling layout
  int *move_src = nullptr, *move_dst = nullptr, *move_j = nullptr, *tail_move = nullptr, *n_moves_dev = nullptr;
  bool moves_pending = false;     // the last compress left moves that the next append (or a flush) carries out
  float* moves_delta = nullptr;   // where that move leaves its corrections of the key column sums, or nullptr
  float* ksum[2] = {nullptr, nullptr};   // [1 + kFillSlices, C]: the key column sums a step uses, then the move's corrections
  int kcur = 0;                   // which of the two the next diversity launch reads
  bool ksum_valid = false;        // ksum[kcur] describes the cached keys (else: recompute)
  int since_refresh = 0;
  float* kmax2 = nullptr;         // [n_heads] running upper bound of the squared per-head key norms (bf16 caches)
  AttnKvMaps maps[2];             // tensor maps of the K/V buffers, re-encoded only when the row count changes
  int64_t scores_frame = -1;      // frame whose s_raw and d were already enqueued on the side stream
  size_t kv_bytes = 0;
};

struct ovggt_cache {
  ovggt_config cfg;
  int M = 0, C = 0, Np = 0, elem = 0;
  std::vector<int32_t> budgets;
  std::vector<LayerState> layers;
  // anchors (shared by all layers: the decision of a frame is taken once)
  std::deque<int64_t> anchors;
  int64_t first_frame = -1, last_registration = -1;
  int64_t decided_frame = -1;
  bool decided_register = false;
  int64_t decided_demote = -1;
  // shared scratch
  float *colsum_part = nullptr, *ksum = nullptr;
  float *qk_part = nullptr, *qk_sum = nullptr;       // OVGGT_SCORE_QK: column sums of the frame's queries
  float *attn_lse = nullptr, *attn_part = nullptr;   // OVGGT_SCORE_ATTN: log2 softmax denominators [M, H], per-head sums [H, M]
  void* attn_scratch = nullptr;
  int* status = nullptr;
  // two sets of staging buffers for ovggt_layer_step_host: the copies of one step overlap the kernels of the step before
  char *stage_q[2] = {}, *stage_k[2] = {}, *stage_v[2] = {}, *stage_r[2] = {}, *stage_o[2] = {};
  float* stage_conf[2] = {};
  int stage_next = 0;
  cudaStream_t copy = nullptr;                       // host -> device copies of ovggt_layer_step_host
  cudaEvent_t ev_h2d[2] = {}, ev_done[2] = {};       // set p: inputs have arrived / the step that read them is done
  bool stage_used[2] = {false, false};
  float w_center = 0, w_edge = 0, w_corner = 0;
  cudaStream_t last_stream = nullptr;
  int max_rows = 0;
  // ovggt_layer_step scores the cache (diversity, residual norms) on a second, higher-priority stream while the
  // attention runs: the scores do not depend on the attention.  Host objects only; absent if creation failed.
  cudaStream_t side = nullptr;
  cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
  bool overlap = true;            // ovggt_cache_set_overlap
  bool use_key_bound = true;      // ovggt_cache_set_key_bound
  // optional per-kernel-class timing (host-side CUDA events; no device memory)
  bool prof = false;
  struct ProfRec { int cls; cudaEvent_t a, b; };
  std::vector<ProfRec> prof_recs;
  double prof_ms[OVGGT_PROF_CLASSES] = {0};
  int64_t prof_cnt[OVGGT_PROF_CLASSES] = {0};
};

namespace {
// Records a pair of events around the launches of one kernel class while profiling is on.
struct ProfScope {
  ovggt_cache* h;
  ovggt_cache::ProfRec rec;
  cudaStream_t st;
  bool on;
  ProfScope(ovggt_cache* h_, int cls, cudaStream_t st_) : h(h_), st(st_), on(h_->prof) {
    static const char* const kNames[OVGGT_PROF_CLASSES] = {"ovggt append", "ovggt attention", "ovggt row norms",
                                                           "ovggt diversity", "ovggt select", "ovggt compact"};
    nvtxRangePushA(kNames[cls]);          // a named range around the launches of each class, for timeline tools
    if (!on) return;
    rec.cls = cls;
    if (cudaEventCreate(&rec.a) != cudaSuccess || cudaEventCreate(&rec.b) != cudaSuccess) { on = false; return; }
    cudaEventRecord(rec.a, st);
  }
  ~ProfScope() {
    nvtxRangePop();
    if (!on) return;
    cudaEventRecord(rec.b, st);
    h->prof_recs.push_back(rec);
  }
};
}  // namespace

namespace {

struct Layout {
  size_t total = 0;
  size_t take(size_t bytes, size_t align = 1024) {
    total = align_up(total, align);
    size_t off = total;
    total += bytes;
    return off;
  }
};

bool config_ok(const ovggt_config* c, int* err) {
  *err = OVGGT_ERR_INVALID_ARG;
  if (!c || !c->budget) return false;
  if (c->n_layers < 1 || c->n_heads < 1 || c->head_dim != 64) return false;
  if (c->camera_head != 0 && c->camera_head != 1) return false;
  if (c->camera_head) {   // Supp. C: one camera token per frame and nothing else
    if (c->n_special != 1 || c->grid_h != 0 || c->grid_w != 0 || c->anchor_tokens != 0) return false;
  } else if (c->n_special < 0 || c->grid_h < 1 || c->grid_w < 1) {
    return false;
  }
  if (c->anchor_tokens < 0 || c->anchor_tokens > c->grid_h * c->grid_w) return false;
  if (c->k_max < 0 || c->k_max > OVGGT_MAX_ANCHORS || c->min_anchor_interval < 0) return false;
  if (c->dtype != kF32 && c->dtype != kBF16) return false;
  if (c->score_mode != OVGGT_SCORE_HYBRID && c->score_mode != OVGGT_SCORE_RESIDUAL_STORED &&
      c->score_mode != OVGGT_SCORE_RANDOM && c->score_mode != OVGGT_SCORE_QK && c->score_mode != OVGGT_SCORE_ATTN)
    return false;
  if ((c->score_mode == OVGGT_SCORE_QK || c->score_mode == OVGGT_SCORE_ATTN) && c->camera_head)
    return false;   // the probe concerns the aggregator's caches
  if (c->compaction != OVGGT_COMPACT_FILL_HOLES && c->compaction != OVGGT_COMPACT_STABLE_GATHER) return false;
  if (!(c->alpha >= 0.0f && c->alpha <= 1.0f) || !(c->beta >= 0.0f && c->beta <= 1.0f)) return false;
  const int64_t M = c->n_special + (int64_t)c->grid_h * c->grid_w;
  // Eq. 9; in the camera head's cache an anchor is the frame's one token
  const int64_t pmax = (c->protect_first_frame ? M : 0) + (int64_t)c->k_max * (c->camera_head ? 1 : c->anchor_tokens);
  for (int l = 0; l < c->n_layers; ++l) {
    if (c->budget[l] < M || c->budget[l] < pmax) {
      *err = OVGGT_ERR_BUDGET_TOO_SMALL;
      return false;
    }
    if ((int64_t)c->budget[l] + M > (1 << 30)) return false;
    // the fused selection kernel keeps all B + M candidates of a layer in the shared memory of one cluster
    const int N = c->budget[l] + (int)M, ncta = select_cluster_ctas(N);
    if (compress_smem_bytes((N + ncta - 1) / ncta, c->grid_h * c->grid_w, (int)M) > kSmemLimit) {
      *err = OVGGT_ERR_UNSUPPORTED;
      return false;
    }
  }
  *err = OVGGT_OK;
  return true;
}

// Lays the workspace out; with a handle, also records the pointers.
size_t layout_workspace(const ovggt_config* c, ovggt_cache* h) {
  Layout L;
  const int M = c->n_special + c->grid_h * c->grid_w, C = c->n_heads * c->head_dim;
  const int Np = c->grid_h * c->grid_w;
  const size_t eb = (size_t)elem_bytes(c->dtype);
  char* base = h ? static_cast<char*>(c->workspace) : nullptr;
  int max_rows = 0;
  for (int l = 0; l < c->n_layers; ++l) {
    const size_t R = (size_t)c->budget[l] + M;
    max_rows = std::max(max_rows, (int)R);
    const bool fill = c->compaction == OVGGT_COMPACT_FILL_HOLES;
    const int nkv = fill ? 1 : 2;       // the stable gather writes the other buffer of a pair; hole filling moves in place
    size_t off[32];
    int i = 0;
    for (int b = 0; b < nkv; ++b) off[i++] = L.take(R * C * eb);
    for (int b = 0; b < nkv; ++b) off[i++] = L.take(R * C * eb);
    for (int b = 0; b < 2; ++b) off[i++] = L.take(R * 8);
    for (int b = 0; b < 2; ++b) off[i++] = L.take(R);
    for (int b = 0; b < 2; ++b) off[i++] = L.take(R * 4);
    off[i++] = L.take((size_t)M * 4);   // s_raw
    off[i++] = L.take(R * 4);           // d
    off[i++] = L.take(R * 4);           // r
    off[i++] = L.take(R * 4);           // survivors
    off[i++] = L.take(64);              // n_keep, n_moves
    off[i++] = L.take((size_t)c->n_heads * 4);   // bound of the key norms
    if (fill) {
      for (int b = 0; b < 2; ++b) off[i++] = L.take(R * 4);                                  // slots
      for (int b = 0; b < 4; ++b) off[i++] = L.take((size_t)M * 4);                          // move lists
      for (int b = 0; b < 2; ++b) off[i++] = L.take((size_t)(1 + kFillSlices) * C * 4);      // column sums + corrections
    } else {
      off[i++] = L.take((size_t)148 * 8 * C * 4);   // column-sum partials of the compaction
    }
    if (h) {
      LayerState& S = h->layers[l];
      i = 0;
      S.kbuf[1] = S.vbuf[1] = nullptr;
      for (int b = 0; b < nkv; ++b) S.kbuf[b] = base + off[i++];
      for (int b = 0; b < nkv; ++b) S.vbuf[b] = base + off[i++];
      for (int b = 0; b < 2; ++b) S.ids[b] = reinterpret_cast<long long*>(base + off[i++]);
      for (int b = 0; b < 2; ++b) S.flags[b] = reinterpret_cast<uint8_t*>(base + off[i++]);
      for (int b = 0; b < 2; ++b) S.stored[b] = reinterpret_cast<float*>(base + off[i++]);
      S.s_raw = reinterpret_cast<float*>(base + off[i++]);
      S.d = reinterpret_cast<float*>(base + off[i++]);
      S.r = reinterpret_cast<float*>(base + off[i++]);
      S.surv = reinterpret_cast<int*>(base + off[i++]);
      S.n_keep_dev = reinterpret_cast<int*>(base + off[i++]);
      S.n_moves_dev = S.n_keep_dev + 4;
      S.kmax2 = reinterpret_cast<float*>(base + off[i++]);
      if (fill) {
        for (int b = 0; b < 2; ++b) S.slot[b] = reinterpret_cast<int*>(base + off[i++]);
        S.move_src = reinterpret_cast<int*>(base + off[i++]);
        S.move_dst = reinterpret_cast<int*>(base + off[i++]);
        S.move_j = reinterpret_cast<int*>(base + off[i++]);
        S.tail_move = reinterpret_cast<int*>(base + off[i++]);
        for (int b = 0; b < 2; ++b) S.ksum[b] = reinterpret_cast<float*>(base + off[i++]);
      } else {
        S.colsum_part = reinterpret_cast<float*>(base + off[i++]);
      }
      S.budget = c->budget[l];
      S.kv_bytes = 2 * (size_t)nkv * R * C * eb;
    }
  }
  const size_t o_part = L.take((size_t)kMaxColsumParts * C * 4);
  const size_t o_ksum = L.take(colsum_scratch_bytes(C));
  const size_t o_attn = L.take(ovggt_k_attention_scratch_bytes(M, max_rows, c->n_heads));
  const size_t o_status = L.take(64);
  const bool qk = c->score_mode == OVGGT_SCORE_QK;
  const size_t o_qk = qk ? L.take((size_t)(colsum_parts(M) + 1) * C * 4) : 0;
  const bool aw = c->score_mode == OVGGT_SCORE_ATTN;
  const size_t o_aw = aw ? L.take((size_t)2 * M * c->n_heads * 4) : 0;
  size_t o_stage[2][5], o_conf[2];
  for (int p = 0; p < 2; ++p) {
    for (int i = 0; i < 5; ++i) o_stage[p][i] = L.take((size_t)M * C * eb);
    o_conf[p] = L.take((size_t)Np * 4);
  }
  if (h) {
    h->colsum_part = reinterpret_cast<float*>(base + o_part);
    h->ksum = reinterpret_cast<float*>(base + o_ksum);
    h->attn_scratch = base + o_attn;
    h->status = reinterpret_cast<int*>(base + o_status);
    if (aw) {
      h->attn_lse = reinterpret_cast<float*>(base + o_aw);
      h->attn_part = h->attn_lse + (size_t)M * c->n_heads;
    }
    if (qk) {
      h->qk_part = reinterpret_cast<float*>(base + o_qk);
      h->qk_sum = h->qk_part + (size_t)colsum_parts(M) * C;
    }
    for (int p = 0; p < 2; ++p) {
      h->stage_q[p] = base + o_stage[p][0];
      h->stage_k[p] = base + o_stage[p][1];
      h->stage_v[p] = base + o_stage[p][2];
      h->stage_r[p] = base + o_stage[p][3];
      h->stage_o[p] = base + o_stage[p][4];
      h->stage_conf[p] = reinterpret_cast<float*>(base + o_conf[p]);
    }
    h->max_rows = max_rows;
  }
  return align_up(L.total, 1024);
}

// Score modes whose cached rows are ranked by key diversity (Eq. 7); the query-key probe (Supp. D) differs from the
// hybrid mode only in the criterion of the new frame's rows.
bool ranks_by_diversity(int mode) {
  return mode == OVGGT_SCORE_HYBRID || mode == OVGGT_SCORE_QK || mode == OVGGT_SCORE_ATTN;
}
// Modes whose criterion for the new frame comes out of the attend half (from q and k, or from the attention itself)
// and waits in the layer's s_raw; the compress half then does not read the residual.
bool scored_at_attend(int mode) { return mode == OVGGT_SCORE_QK || mode == OVGGT_SCORE_ATTN; }

int check_layer(ovggt_cache* h, int32_t layer) {
  if (!h) return OVGGT_ERR_INVALID_ARG;
  if (layer < 0 || layer >= (int)h->layers.size()) return OVGGT_ERR_BAD_LAYER;
  return OVGGT_OK;
}

}  // namespace

// ------------------------------------------------------------------ exported API

extern "C" size_t ovggt_workspace_bytes(const ovggt_config* cfg) {
  int err;
  if (!config_ok(cfg, &err)) return 0;
  return layout_workspace(cfg, nullptr);
}

extern "C" int ovggt_cache_create(const ovggt_config* cfg, ovggt_cache** out) {
  if (!out) return OVGGT_ERR_INVALID_ARG;
  *out = nullptr;
  int err;
  if (!config_ok(cfg, &err)) return err;
  if (!cfg->workspace) return OVGGT_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(cfg->workspace) & 1023) return OVGGT_ERR_MISALIGNED;
  if (cfg->workspace_bytes < layout_workspace(cfg, nullptr)) return OVGGT_ERR_WORKSPACE_TOO_SMALL;
  ovggt_cache* h = new (std::nothrow) ovggt_cache();
  if (!h) return OVGGT_ERR_INVALID_ARG;
  h->cfg = *cfg;
  h->budgets.assign(cfg->budget, cfg->budget + cfg->n_layers);
  h->cfg.budget = h->budgets.data();
  h->M = cfg->n_special + cfg->grid_h * cfg->grid_w;
  h->C = cfg->n_heads * cfg->head_dim;
  h->Np = cfg->grid_h * cfg->grid_w;
  h->elem = elem_bytes(cfg->dtype);
  h->layers.resize(cfg->n_layers);
  layout_workspace(&h->cfg, h);
  // Eq. 6: 3x3 Gaussian, sigma = 1, normalised
  const double e1 = std::exp(-0.5), e2 = std::exp(-1.0), z = 1.0 + 4.0 * e1 + 4.0 * e2;
  h->w_center = (float)(1.0 / z);
  h->w_edge = (float)(e1 / z);
  h->w_corner = (float)(e2 / z);
  {
    int lo = 0, hi = 0;
    if (cudaDeviceGetStreamPriorityRange(&lo, &hi) != cudaSuccess ||
        cudaStreamCreateWithPriority(&h->side, cudaStreamNonBlocking, hi) != cudaSuccess ||
        cudaEventCreateWithFlags(&h->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&h->ev_join, cudaEventDisableTiming) != cudaSuccess) {
      if (h->ev_fork) cudaEventDestroy(h->ev_fork);
      if (h->ev_join) cudaEventDestroy(h->ev_join);
      if (h->side) cudaStreamDestroy(h->side);
      h->side = nullptr;
      h->ev_fork = h->ev_join = nullptr;
      (void)cudaGetLastError();
    }
  }
  {
    bool ok = cudaStreamCreateWithFlags(&h->copy, cudaStreamNonBlocking) == cudaSuccess;
    for (int p = 0; p < 2 && ok; ++p)
      ok = cudaEventCreateWithFlags(&h->ev_h2d[p], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&h->ev_done[p], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) {
      for (int p = 0; p < 2; ++p) {
        if (h->ev_h2d[p]) cudaEventDestroy(h->ev_h2d[p]);
        if (h->ev_done[p]) cudaEventDestroy(h->ev_done[p]);
        h->ev_h2d[p] = h->ev_done[p] = nullptr;
      }
      if (h->copy) cudaStreamDestroy(h->copy);
      h->copy = nullptr;
      (void)cudaGetLastError();
    }
  }
  cudaError_t e = cudaMemset(h->status, 0, 64);
  if (e == cudaSuccess) e = cudaMemset(h->ksum, 0, colsum_scratch_bytes(h->C));   // (its arrival counters)
  for (LayerState& S : h->layers)
    if (e == cudaSuccess) e = cudaMemset(S.kmax2, 0, (size_t)cfg->n_heads * 4);

  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  if (e != cudaSuccess) {
    delete h;
    return cuda_fail(e);
  }
  *out = h;
  return OVGGT_OK;
}

extern "C" int ovggt_cache_destroy(ovggt_cache* h) {
  if (!h) return OVGGT_ERR_INVALID_ARG;
  for (auto& r : h->prof_recs) {
    cudaEventDestroy(r.a);
    cudaEventDestroy(r.b);
  }
  if (h->copy) {
    cudaStreamSynchronize(h->copy);
    cudaStreamDestroy(h->copy);
    for (int p = 0; p < 2; ++p) {
      cudaEventDestroy(h->ev_h2d[p]);
      cudaEventDestroy(h->ev_done[p]);
    }
  }
  if (h->side) {
    cudaStreamSynchronize(h->side);
    cudaStreamDestroy(h->side);
    cudaEventDestroy(h->ev_fork);
    cudaEventDestroy(h->ev_join);
  }
  delete h;
  return OVGGT_OK;
}

namespace {
inline bool fill_layout(const ovggt_cache* h) { return h->cfg.compaction == OVGGT_COMPACT_FILL_HOLES; }

// Argument and order checks of the attend half.
int validate_attend(ovggt_cache* h, int32_t layer, const ovggt_frame_io* io) {
  int rc = check_layer(h, layer);
  if (rc) return rc;
  if (!io || !io->q || !io->k || !io->v || !io->out) return OVGGT_ERR_INVALID_ARG;
  if (!aligned16(io->q) || !aligned16(io->k) || !aligned16(io->v) || !aligned16(io->out)) return OVGGT_ERR_MISALIGNED;
  const LayerState& S = h->layers[layer];
  if (S.pending) return OVGGT_ERR_FRAME_ORDER;
  if (S.frames_seen > 0 && io->frame_id <= S.pending_frame) return OVGGT_ERR_FRAME_ORDER;
  if (io->frame_id < 0 || (h->first_frame >= 0 && io->frame_id < h->first_frame)) return OVGGT_ERR_FRAME_ORDER;
  return OVGGT_OK;
}

// The bound of the key norms is kept for bf16 caches whose rows the append kernel holds in one round of loads; the
// attention kernel then takes |q| |k|_max as a fixed softmax reference.  It only grows (evictions do not lower it),
// which keeps it a bound; ovggt_cache_reset clears it, an import recomputes it.
float* key_norm_bound(const ovggt_cache* h, const LayerState& S) {
  return (h->cfg.dtype == kBF16 && h->C * h->elem / 16 <= 128 && h->use_key_bound) ? S.kmax2 : nullptr;
}

// Carry out the moves the layer's last compress left, now, with the stand-alone kernel (for whoever reads the K/V
// buffer or the slots before the next append: export).
int flush_moves(ovggt_cache* h, LayerState& S, cudaStream_t st) {
  if (!S.moves_pending) return OVGGT_OK;
  ProfScope ps(h, OVGGT_PROF_COMPACT, st);
  int rc = launch_fill_holes(S.kbuf[S.kv], S.vbuf[S.kv], S.move_src, S.move_dst, S.move_j, S.n_moves_dev, h->M, h->C,
                             h->cfg.dtype, S.slot[S.cur], S.moves_delta, st, S.budget + h->M, S.budget, h->status);
  if (rc) return rc;
  S.moves_pending = false;
  S.moves_delta = nullptr;
  return OVGGT_OK;
}

// Eq. 2: the append itself; in the hole-filling layout the same launch first carries out the moves the previous
// compress left (they empty exactly the slots the new frame goes into).
int enqueue_append(ovggt_cache* h, int32_t layer, const ovggt_frame_io* io, cudaStream_t st) {
  int rc = validate_attend(h, layer, io);
  if (rc) return rc;
  LayerState& S = h->layers[layer];
  h->last_stream = st;
  const int M = h->M, C = h->C, nvec = C * h->elem / 16, b = S.cur, kb = S.kv;
  ProfScope ps(h, OVGGT_PROF_APPEND, st);
  if (!fill_layout(h)) {
    const int grid = std::min((2 * M + 7) / 8, 148 * 8);
    k_append<<<grid, 256, 0, st>>>((const uint4*)io->k, (const uint4*)io->v, M, nvec, S.n, (long long)io->frame_id,
                                   (uint4*)S.kbuf[kb], (uint4*)S.vbuf[kb], S.ids[b], S.flags[b], S.stored[b], S.slot[b],
                                   key_norm_bound(h, S));
    LAUNCHED();
    return OVGGT_OK;
  }
  AppendFillArgs A;
  A.k_new = (const uint4*)io->k; A.v_new = (const uint4*)io->v;
  A.M = M; A.n = S.n; A.frame_id = (long long)io->frame_id;
  A.k_cache = (uint4*)S.kbuf[kb]; A.v_cache = (uint4*)S.vbuf[kb];
  A.ids = S.ids[b]; A.flags = S.flags[b]; A.stored = S.stored[b]; A.slot = S.slot[b];
  A.kmax2 = key_norm_bound(h, S);
  A.B = S.budget;
  const bool pending = S.moves_pending;
  A.tail_move = pending ? S.tail_move : nullptr;
  A.move_dst = S.move_dst; A.move_j = S.move_j; A.n_moves_ptr = S.n_moves_dev;
  A.delta = pending ? S.moves_delta : nullptr;
  A.status = h->status;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(kFillSlices * kFillClusterCtas);
  cfg.blockDim = dim3(kAppendFillThreads);
  cfg.stream = st;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeClusterDimension;
  attr.val.clusterDim.x = kFillClusterCtas;
  attr.val.clusterDim.y = 1;
  attr.val.clusterDim.z = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  cudaError_t e = h->cfg.dtype == kBF16 ? cudaLaunchKernelEx(&cfg, k_append_fill<kBF16>, A, nvec)
                                        : cudaLaunchKernelEx(&cfg, k_append_fill<kF32>, A, nvec);
  if (e != cudaSuccess) return cuda_fail(e);
  LAUNCHED();
  S.moves_pending = false;
  S.moves_delta = nullptr;
  return OVGGT_OK;
}

// The attention over all n + M rows, and the bookkeeping that closes the attend half.  Attention does not care in
// which order the cached rows lie, so it reads the K/V buffer front to back in either layout.
int enqueue_attention(ovggt_cache* h, int32_t layer, const ovggt_frame_io* io, cudaStream_t st) {
  LayerState& S = h->layers[layer];
  const int kb = S.kv;
  int rc;
  {
    ProfScope ps(h, OVGGT_PROF_ATTENTION, st);
    rc = launch_attention(io->q, S.kbuf[kb], S.vbuf[kb], h->M, S.n + h->M, h->cfg.n_heads, h->cfg.dtype, io->out,
                          h->attn_scratch, h->status, st, &S.maps[kb], key_norm_bound(h, S),
                          h->cfg.score_mode == OVGGT_SCORE_ATTN ? h->attn_lse : nullptr);
  }
  if (rc) return rc;
  if (h->first_frame < 0) {
    h->first_frame = io->frame_id;
    h->last_registration = io->frame_id;   // the first frame is the initial anchor
  }
  S.pending = true;
  S.pending_frame = io->frame_id;
  return OVGGT_OK;
}

// Query-key mode (Supp. D): the criterion of the new frame's rows, from the frame's own q and k; kept in the layer's
// s_raw until the layer's compress.
int enqueue_qk_scores(ovggt_cache* h, LayerState& S, const ovggt_frame_io* io, cudaStream_t st) {
  if (h->cfg.score_mode != OVGGT_SCORE_QK) return OVGGT_OK;
  ProfScope ps(h, OVGGT_PROF_ROW_NORMS, st);
  return launch_qk_scores(io->q, io->k, h->M, h->C, h->cfg.n_heads, h->cfg.dtype, h->qk_part, h->qk_sum, S.s_raw, st);
}

// Attention-weight mode (Supp. D): the criterion of the new frame's rows, from the attention that has just been
// enqueued on st (its log2 denominators) and the frame's own q and k; kept in the layer's s_raw as well.
int enqueue_received_scores(ovggt_cache* h, LayerState& S, const ovggt_frame_io* io, cudaStream_t st) {
  if (h->cfg.score_mode != OVGGT_SCORE_ATTN) return OVGGT_OK;
  ProfScope ps(h, OVGGT_PROF_ROW_NORMS, st);
  return launch_attention_received(io->q, io->k, h->M, h->C, h->cfg.n_heads, h->cfg.dtype, h->attn_lse, h->attn_part,
                                   S.s_raw, st);
}

// Eq. 5 and the diversity score of Sec. 3.2 for the frame io describes: everything the selection needs that does not
// depend on the anchor decision.  Reads the cached keys [0, n) and the frame's residual, so it may run before the
// frame's K/V are appended.
int enqueue_scores(ovggt_cache* h, LayerState& S, const ovggt_frame_io* io, cudaStream_t st) {
  const ovggt_config& c = h->cfg;
  const int M = h->M, C = h->C, n = S.n, kb = S.kv;
  const bool hybrid = ranks_by_diversity(c.score_mode) && n > 0;
  // query-key and attention-weight modes: s_raw was written by the attend half; the residual is not read
  const void* resid = scored_at_attend(c.score_mode) ? nullptr : io->resid;
  int rc = OVGGT_OK;
  if (!hybrid) {
    if (!resid) return OVGGT_OK;
    ProfScope ps(h, OVGGT_PROF_ROW_NORMS, st);
    return launch_row_norms(resid, M, C, c.dtype, S.s_raw, st);
  }
  if (fill_layout(h)) {
    // Column sums of the cached keys: continued from the last step's sums and the corrections its move left, or
    // summed afresh (first steps, after an import, every kColsumRefreshEvery-th step); the residual norms ride in
    // the diversity launch either way.
    ProfScope ps(h, OVGGT_PROF_DIVERSITY, st);
    const bool fresh = !S.ksum_valid || S.since_refresh >= kColsumRefreshEvery;
    if (fresh) {
      rc = launch_colsum(S.kbuf[kb], n, C, c.dtype, h->colsum_part, S.ksum[S.kcur], st);
      if (rc) return rc;
      S.since_refresh = 0;
    } else {
      S.since_refresh += 1;
    }
    return launch_diversity_sliced(S.kbuf[kb], n, C, c.dtype, S.ksum[S.kcur], fresh ? 1 : 1 + kFillSlices,
                                   S.ksum[S.kcur ^ 1], S.d, resid, M, S.s_raw, st);
  }
  if (S.colsum_nparts > 0) {   // stable layout, sums left by the last compaction
    ProfScope ps(h, OVGGT_PROF_DIVERSITY, st);
    return launch_diversity_from_parts(S.kbuf[kb], n, C, c.dtype, S.colsum_part, S.colsum_nparts, h->ksum, S.d,
                                       resid, M, S.s_raw, st);
  }
  if (resid) {
    ProfScope ps(h, OVGGT_PROF_ROW_NORMS, st);
    rc = launch_row_norms(resid, M, C, c.dtype, S.s_raw, st);
  }
  if (rc) return rc;
  ProfScope ps(h, OVGGT_PROF_DIVERSITY, st);
  return launch_diversity(S.kbuf[kb], n, C, c.dtype, h->colsum_part, h->ksum, S.d, st);
}

// `mirrored`: the anchor decision of the frame as another handle took it (camera head, Supp. C) instead of the rule
// of Sec. 3.3 applied to rho.
struct MirroredDecision { bool registered; int64_t demoted_frame; };

// Argument and order checks of the compress half; nothing is changed.
int validate_compress(ovggt_cache* h, int32_t layer, const ovggt_frame_io* io, const MirroredDecision* mirrored) {
  int rc = check_layer(h, layer);
  if (rc) return rc;
  if (!io) return OVGGT_ERR_INVALID_ARG;
  if ((h->cfg.camera_head != 0) != (mirrored != nullptr)) return OVGGT_ERR_INVALID_ARG;
  if (!scored_at_attend(h->cfg.score_mode)) {   // (those modes do not read the residual)
    if (!io->resid) return OVGGT_ERR_INVALID_ARG;
    if (!aligned16(io->resid)) return OVGGT_ERR_MISALIGNED;
  }
  const LayerState& S = h->layers[layer];
  if (!S.pending || io->frame_id != S.pending_frame) return OVGGT_ERR_FRAME_ORDER;
  const int N = S.n + h->M, ncta = select_cluster_ctas(N);
  if (compress_smem_bytes((N + ncta - 1) / ncta, h->Np, h->M) > kSmemLimit)
    return OVGGT_ERR_UNSUPPORTED;   // (create already refuses such budgets)
  // The anchor state belongs to the whole handle and moves forward only: a layer that comes with a frame older
  // than the last decision would take that frame's decision a second time.
  if (io->frame_id < h->decided_frame) return OVGGT_ERR_FRAME_ORDER;
  return OVGGT_OK;
}

// Anchor decision of frame t (Sec. 3.3), taken once and shared by all layers.
void take_decision(ovggt_cache* h, const ovggt_frame_io* io, const MirroredDecision* mirrored) {
  const ovggt_config& c = h->cfg;
  const int64_t t = io->frame_id;
  if (h->decided_frame == t) return;
  h->decided_frame = t;
  h->decided_register = false;
  h->decided_demote = -1;
  if (mirrored) {
    // the frame's token is protected / the demoted frame's token released exactly when the aggregator did so
    if (t != h->first_frame && mirrored->registered && (int)h->anchors.size() < OVGGT_MAX_ANCHORS) {
      h->decided_register = true;
      h->anchors.push_back(t);
      h->last_registration = t;
    }
    if (mirrored->demoted_frame >= 0) {
      auto it = std::find(h->anchors.begin(), h->anchors.end(), mirrored->demoted_frame);
      if (it != h->anchors.end()) {
        h->decided_demote = mirrored->demoted_frame;
        h->anchors.erase(it);
      }
    }
  } else if (t != h->first_frame && c.anchor_tokens > 0 && c.k_max > 0 && io->conf != nullptr && io->rho < c.tau &&
             t - h->last_registration >= c.min_anchor_interval) {
    h->decided_register = true;
    h->anchors.push_back(t);
    h->last_registration = t;
    if ((int)h->anchors.size() > c.k_max) {
      h->decided_demote = h->anchors.front();
      h->anchors.pop_front();
    }
  }
}

// Parameter block of the fused selection kernel for the layer's pending frame.
CompressParams select_params(ovggt_cache* h, LayerState& S, const ovggt_frame_io* io) {
  const ovggt_config& c = h->cfg;
  const int b = S.cur;
  const bool first = io->frame_id == h->first_frame;
  CompressParams P;
  P.n = S.n; P.M = h->M; P.B = S.budget;
  P.n_special = c.n_special; P.grid_h = c.grid_h; P.grid_w = c.grid_w;
  P.alpha = c.alpha; P.w_center = h->w_center; P.w_edge = h->w_edge; P.w_corner = h->w_corner;
  P.beta = c.beta;
  P.mode = scored_at_attend(c.score_mode) ? OVGGT_SCORE_HYBRID : c.score_mode;   // same Eq. 6-8, other s_raw
  P.protect_new = (first && c.protect_first_frame) ? OVGGT_FLAG_INIT
                                                   : ((c.camera_head && h->decided_register) ? OVGGT_FLAG_HIST : 0);
  P.lone_new = c.camera_head ? 1.0f : -1.0f;
  P.step_key = splitmix64(c.random_seed ^ (unsigned long long)io->frame_id);
  P.register_anchor = (!c.camera_head && h->decided_register) ? 1 : 0;
  P.A = c.anchor_tokens;
  P.demote_frame = h->decided_demote;
  P.s_raw = S.s_raw; P.d = S.d; P.conf = io->conf; P.override_r = io->score_override;
  P.ids_src = S.ids[b]; P.flags_src = S.flags[b]; P.stored_src = S.stored[b];
  P.ids_dst = S.ids[b ^ 1]; P.flags_dst = S.flags[b ^ 1]; P.stored_dst = S.stored[b ^ 1];
  P.r_out = S.r; P.survivors = S.surv;
  P.status = h->status; P.n_keep_out = S.n_keep_dev;
  P.fill = fill_layout(h) ? 1 : 0;
  P.slot_src = S.slot[b]; P.slot_dst = S.slot[b ^ 1];
  P.move_src = S.move_src; P.move_dst = S.move_dst; P.move_j = S.move_j; P.tail_move = S.tail_move;
  P.n_moves_out = S.n_moves_dev;
  return P;
}

// Host bookkeeping that follows deterministically from the sizes once a layer's compress has been enqueued.
void close_compress(ovggt_cache* h, LayerState& S, const ovggt_frame_io* io) {
  const ovggt_config& c = h->cfg;
  const int N = S.n + h->M, n_keep = std::min(N, S.budget);
  const int per_anchor = c.camera_head ? 1 : c.anchor_tokens;
  if (io->frame_id == h->first_frame && c.protect_first_frame) S.n_prot_init = h->M;
  if (h->decided_register) S.n_prot_hist += per_anchor;
  if (h->decided_demote >= 0) S.n_prot_hist -= per_anchor;
  S.evicted_total += N - n_keep;
  S.last_N = N;
  S.last_keep = n_keep;
  S.n = n_keep;
  S.cur ^= 1;
  S.pending = false;
  S.frames_seen += 1;
}

// Does the hole-filling move of this step also leave corrections of the key column sums?  They continue the sums the
// step's diversity launch used and wrote to ksum[kcur ^ 1], and describe the next cache only if every slot below B
// held a cached row (n == B: steady state).
bool move_leaves_corrections(const ovggt_cache* h, const LayerState& S) {
  return ranks_by_diversity(h->cfg.score_mode) && h->C * h->elem / 16 <= kCompactSumMaxVec && S.n == S.budget;
}

// The compress half on stream st.  The stable gather writes another buffer, so the whole half may run beside an
// attention that still reads this one; the hole-filling moves are only recorded here (see enqueue_append).
int compress_impl(ovggt_cache* h, int32_t layer, const ovggt_frame_io* io, cudaStream_t st_sel,
                  const MirroredDecision* mirrored = nullptr) {
  const cudaStream_t st_move = st_sel;
  int rc = validate_compress(h, layer, io, mirrored);
  if (rc) return rc;
  LayerState& S = h->layers[layer];
  const ovggt_config& c = h->cfg;
  const int M = h->M, C = h->C, n = S.n, N = n + M, B = S.budget, b = S.cur, kb = S.kv;
  const int64_t t = io->frame_id;
  const bool fill = fill_layout(h);
  take_decision(h, io, mirrored);     // nothing below can fail on an argument any more
  h->last_stream = st_move;

  const bool prelaunched = S.scores_frame == t;    // ovggt_layer_step already enqueued them on st_sel
  S.scores_frame = -1;
  if (!prelaunched) {
    rc = enqueue_scores(h, S, io, st_sel);
    if (rc) return rc;
  }
  const CompressParams P = select_params(h, S, io);
  const int ncta = select_cluster_ctas(N);
  const size_t smem = compress_smem_bytes((N + ncta - 1) / ncta, h->Np, M);
  CK(cudaFuncSetAttribute(k_compress_select, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemLimit));
  {
    ProfScope ps(h, OVGGT_PROF_SELECT, st_sel);
    CK(launch_cluster(k_compress_select, dim3(ncta), ncta, smem, st_sel, P));
    LAUNCHED();
  }
  const int n_keep = std::min(N, B);
  if (fill) {
    // Some rows leave: the survivors above slot B have to move into the slots that open below it.  The selection
    // kernel has left the pairs; the next append of this layer carries them out (flush_moves for other readers).
    S.ksum_valid = false;
    if (N > B) {
      const bool delta = move_leaves_corrections(h, S);
      S.moves_pending = true;
      S.moves_delta = delta ? S.ksum[S.kcur ^ 1] + C : nullptr;
      if (delta) {
        S.kcur ^= 1;
        S.ksum_valid = true;
      }
    }
  } else {
    ProfScope ps(h, OVGGT_PROF_COMPACT, st_move);
    const bool fuse = ranks_by_diversity(c.score_mode) && C * h->elem / 16 <= kCompactSumMaxVec;
    S.colsum_nparts = 0;
    if (fuse)
      rc = launch_compact_colsum(S.kbuf[kb], S.vbuf[kb], S.surv, n_keep, C, c.dtype, S.kbuf[kb ^ 1], S.vbuf[kb ^ 1],
                                 S.colsum_part, &S.colsum_nparts, st_move, N, h->status);
    else
      rc = launch_compact(S.kbuf[kb], S.vbuf[kb], S.surv, n_keep, C, c.dtype, S.kbuf[kb ^ 1], S.vbuf[kb ^ 1], st_move, N,
                          h->status);
    if (rc) return rc;
    S.kv = kb ^ 1;
  }
  close_compress(h, S, io);
  return OVGGT_OK;
}

// The compress half of every layer of the handle for one frame, in two launches instead of two per layer
// (hole-filling layout; the batched kernels take one parameter block per layer as kernel arguments).
int compress_all_layers(ovggt_cache* h, const ovggt_frame_io* ios, cudaStream_t st) {
  const ovggt_config& c = h->cfg;
  const int L = (int)h->layers.size(), M = h->M, C = h->C;
  for (int l = 0; l < L; ++l) {
    int rc = validate_compress(h, l, &ios[l], nullptr);
    if (rc) return rc;
    if (ios[l].frame_id != ios[0].frame_id) return OVGGT_ERR_FRAME_ORDER;
  }
  if (!fill_layout(h)) {                     // the stable gather has no batched kernels: layer by layer
    for (int l = 0; l < L; ++l) {
      int rc = compress_impl(h, l, &ios[l], st);
      if (rc) return rc;
    }
    return OVGGT_OK;
  }
  take_decision(h, &ios[0], nullptr);
  h->last_stream = st;
  const int nvec = C * h->elem / 16;
  CK(cudaFuncSetAttribute(k_compress_select_batched, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemLimit));
  for (int l0 = 0; l0 < L; l0 += kMaxBatchLayers) {
    const int cnt = std::min(kMaxBatchLayers, L - l0);
    // ---- scores: diversity of the cached keys and the frame's residual norms
    {
      ProfScope ps(h, OVGGT_PROF_DIVERSITY, st);
      DiversityBatch db;
      int grid_x = 1;
      // Every CTA first folds its layer's column sums (up to 1 + 16 rows of C floats, from L2) and then streams key
      // rows: the more rows a CTA takes the less that set-up weighs, as long as the launch still fills the machine a
      // few times over.  (24 layers x 12288 rows, bf16: 0.57 of the copy bandwidth at 64 rows per CTA, 0.67 at 128,
      // 0.72 at 256, 0.71 at 512.)
      int rows_per_cta = 64;
      {
        long total_rows = 0;
        for (int i = 0; i < cnt; ++i)
          if (ranks_by_diversity(c.score_mode)) total_rows += h->layers[l0 + i].n;
        while (rows_per_cta < 256 && total_rows / (2 * rows_per_cta) >= 148 * 4) rows_per_cta *= 2;
      }
      for (int i = 0; i < cnt; ++i) {
        LayerState& S = h->layers[l0 + i];
        S.scores_frame = -1;
        const bool hybrid = ranks_by_diversity(c.score_mode) && S.n > 0;
        DiversityArgs& A = db.a[i];
        A = DiversityArgs{};
        A.resid = scored_at_attend(c.score_mode) ? nullptr : (const uint4*)ios[l0 + i].resid;
        A.resid_rows = M; A.s_raw = S.s_raw;
        if (hybrid) {
          const bool fresh = !S.ksum_valid || S.since_refresh >= kColsumRefreshEvery;
          if (fresh) {
            int rc = launch_colsum(S.kbuf[S.kv], S.n, C, c.dtype, h->colsum_part, S.ksum[S.kcur], st);
            if (rc) return rc;
            S.since_refresh = 0;
          } else {
            S.since_refresh += 1;
          }
          A.K = (const uint4*)S.kbuf[S.kv]; A.rows = S.n;
          A.ksum = S.ksum[S.kcur]; A.n_slices = fresh ? 1 : 1 + kFillSlices; A.ksum_out = S.ksum[S.kcur ^ 1];
          A.d = S.d;
          A.div_ctas = std::min((S.n + rows_per_cta - 1) / rows_per_cta, 148 * 8);
        }
        grid_x = std::max(grid_x, A.div_ctas + (M + 7) / 8);
      }
      if (c.dtype == kBF16) k_diversity_batched<kBF16><<<dim3(grid_x, cnt), 256, (size_t)C * 4, st>>>(db, nvec);
      else                  k_diversity_batched<kF32><<<dim3(grid_x, cnt), 256, (size_t)C * 4, st>>>(db, nvec);
      LAUNCHED();
    }
    // ---- flags, Eq. 6-8, compacted meta, move pairs: one cluster per layer
    {
      ProfScope ps(h, OVGGT_PROF_SELECT, st);
      CompressBatch cb;
      int n_max = 0;
      for (int i = 0; i < cnt; ++i) {
        LayerState& S = h->layers[l0 + i];
        cb.p[i] = select_params(h, S, &ios[l0 + i]);
        n_max = std::max(n_max, S.n + M);
      }
      const int ncta = select_cluster_ctas(n_max);
      const size_t smem = compress_smem_bytes((n_max + ncta - 1) / ncta, h->Np, M);
      CK(launch_cluster(k_compress_select_batched, dim3(ncta, cnt), ncta, smem, st, cb));
      LAUNCHED();
    }
    // ---- the moves of the layers that evict are left to each layer's next append
    for (int i = 0; i < cnt; ++i) {
      LayerState& S = h->layers[l0 + i];
      S.ksum_valid = false;
      if (S.n + M <= S.budget) continue;
      const bool delta = move_leaves_corrections(h, S);
      S.moves_pending = true;
      S.moves_delta = delta ? S.ksum[S.kcur ^ 1] + C : nullptr;
      if (delta) {
        S.kcur ^= 1;
        S.ksum_valid = true;
      }
    }
    for (int i = 0; i < cnt; ++i) close_compress(h, h->layers[l0 + i], &ios[l0 + i]);
  }
  return OVGGT_OK;
}
}  // namespace

extern "C" int ovggt_layer_attend(ovggt_cache* h, int32_t layer, const ovggt_frame_io* io, void* stream) {
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int rc = enqueue_append(h, layer, io, st);
  if (rc) return rc;
  rc = enqueue_attention(h, layer, io, st);
  if (rc) return rc;
  rc = enqueue_qk_scores(h, h->layers[layer], io, st);
  if (rc) return rc;
  return enqueue_received_scores(h, h->layers[layer], io, st);
}

extern "C" int ovggt_layer_compress(ovggt_cache* h, int32_t layer, const ovggt_frame_io* io, void* stream) {
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  return compress_impl(h, layer, io, st);
}

extern "C" int ovggt_cache_anchor_decision(ovggt_cache* h, int64_t frame_id, int32_t* registered,
                                           int64_t* demoted_frame) {
  if (!h || !registered || !demoted_frame) return OVGGT_ERR_INVALID_ARG;
  if (h->decided_frame != frame_id) return OVGGT_ERR_FRAME_ORDER;
  *registered = h->decided_register ? 1 : 0;
  *demoted_frame = h->decided_demote;
  return OVGGT_OK;
}

extern "C" int ovggt_camera_compress(ovggt_cache* h, int32_t layer, const ovggt_frame_io* io, int32_t registered,
                                     int64_t demoted_frame, void* stream) {
  if (!h || !h->cfg.camera_head) return OVGGT_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const MirroredDecision d{registered != 0, demoted_frame};
  return compress_impl(h, layer, io, st, &d);
}

extern "C" int ovggt_layers_compress(ovggt_cache* h, const ovggt_frame_io* ios, int32_t n_ios, void* stream) {
  if (!h || !ios || n_ios != (int32_t)h->layers.size() || h->cfg.camera_head) return OVGGT_ERR_INVALID_ARG;
  return compress_all_layers(h, ios, static_cast<cudaStream_t>(stream));
}

extern "C" int ovggt_layer_step(ovggt_cache* h, int32_t layer, const ovggt_frame_io* io, void* stream) {
  int rc = check_layer(h, layer);
  if (rc) return rc;
  if (h->cfg.camera_head) return OVGGT_ERR_INVALID_ARG;   // the camera head's cache needs the aggregator's decision
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const bool resid_ok = io && (scored_at_attend(h->cfg.score_mode) || (io->resid && aligned16(io->resid)));
  // (the attention-weight criterion needs the attention's own denominators: nothing to overlap it with)
  const bool can_overlap = h->side && h->overlap && resid_ok && io->q && io->k && io->v && io->out &&
                           !h->layers[layer].pending && h->cfg.score_mode != OVGGT_SCORE_ATTN;
  if (!can_overlap) {
    rc = ovggt_layer_attend(h, layer, io, stream);
    if (rc) return rc;
    return ovggt_layer_compress(h, layer, io, stream);
  }
  // Scoring and selection (Eq. 5-8) read the cache and the new rows but not the attention's output, so they run on
  // the handle's second, higher-priority stream beside the attention:
  //   stream:  append (+ the previous step's moves) . fork ... attention ........................ join
  //   side:                                            scores, selection [, stable gather] ....../
  // The stable gather writes the other K/V buffer.  The hole-filling moves would write the buffer the attention
  // reads; they wait for the next append of the layer, which has to touch the same slots anyway.
  rc = validate_attend(h, layer, io);
  if (rc) return rc;
  LayerState& S = h->layers[layer];
  rc = enqueue_append(h, layer, io, st);
  if (rc) return rc;
  CK(cudaEventRecord(h->ev_fork, st));
  CK(cudaStreamWaitEvent(h->side, h->ev_fork, 0));
  rc = enqueue_qk_scores(h, S, io, h->side);
  if (rc == OVGGT_OK) rc = enqueue_scores(h, S, io, h->side);
  if (rc == OVGGT_OK) {
    S.scores_frame = io->frame_id;
    rc = enqueue_attention(h, layer, io, st);
  }
  if (rc == OVGGT_OK) rc = compress_impl(h, layer, io, h->side);
  // join: whatever happened, the caller's stream is ordered after the side work
  S.scores_frame = -1;
  h->last_stream = st;
  cudaError_t e1 = cudaEventRecord(h->ev_join, h->side);
  cudaError_t e2 = cudaStreamWaitEvent(st, h->ev_join, 0);
  if (rc) return rc;
  if (e1 != cudaSuccess) return cuda_fail(e1);
  if (e2 != cudaSuccess) return cuda_fail(e2);
  return OVGGT_OK;
}

extern "C" int ovggt_cache_set_key_bound(ovggt_cache* h, int32_t enable) {
  if (!h) return OVGGT_ERR_INVALID_ARG;
  h->use_key_bound = enable != 0;
  return OVGGT_OK;
}

extern "C" int ovggt_cache_set_overlap(ovggt_cache* h, int32_t enable) {
  if (!h) return OVGGT_ERR_INVALID_ARG;
  h->overlap = enable != 0;
  return OVGGT_OK;
}

extern "C" int ovggt_layer_step_host(ovggt_cache* h, int32_t layer, const ovggt_frame_io* io, void* stream) {
  int rc = check_layer(h, layer);
  if (rc) return rc;
  if (!io || !io->q || !io->k || !io->v || !io->resid || !io->out || io->score_override) return OVGGT_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t bytes = (size_t)h->M * h->C * h->elem;
  // Inputs go through one of two staging sets on a copy stream of the handle's own, so that the copies of this
  // step run while the kernels of the previous step (enqueued on `stream` by the previous call) still compute.
  const int p = h->stage_next;
  h->stage_next ^= 1;
  cudaStream_t cs = h->copy ? h->copy : st;
  if (h->copy) {
    // the set was last read by the step two calls ago
    if (h->stage_used[p]) CK(cudaStreamWaitEvent(cs, h->ev_done[p], 0));
  }
  const char* hq = static_cast<const char*>(io->q);
  const bool packed = static_cast<const char*>(io->k) == hq + bytes && static_cast<const char*>(io->v) == hq + 2 * bytes &&
                      static_cast<const char*>(io->resid) == hq + 3 * bytes && h->stage_k[p] == h->stage_q[p] + bytes &&
                      h->stage_v[p] == h->stage_q[p] + 2 * bytes && h->stage_r[p] == h->stage_q[p] + 3 * bytes;
  if (packed) {   // q | k | v | resid back to back on the host: one copy instead of four
    CK(cudaMemcpyAsync(h->stage_q[p], io->q, 4 * bytes, cudaMemcpyHostToDevice, cs));
  } else {
    CK(cudaMemcpyAsync(h->stage_q[p], io->q, bytes, cudaMemcpyHostToDevice, cs));
    CK(cudaMemcpyAsync(h->stage_k[p], io->k, bytes, cudaMemcpyHostToDevice, cs));
    CK(cudaMemcpyAsync(h->stage_v[p], io->v, bytes, cudaMemcpyHostToDevice, cs));
    CK(cudaMemcpyAsync(h->stage_r[p], io->resid, bytes, cudaMemcpyHostToDevice, cs));
  }
  if (io->conf) CK(cudaMemcpyAsync(h->stage_conf[p], io->conf, (size_t)h->Np * 4, cudaMemcpyHostToDevice, cs));
  if (h->copy) {
    CK(cudaEventRecord(h->ev_h2d[p], cs));
    CK(cudaStreamWaitEvent(st, h->ev_h2d[p], 0));
  }
  ovggt_frame_io dev = *io;
  dev.q = h->stage_q[p]; dev.k = h->stage_k[p]; dev.v = h->stage_v[p]; dev.resid = h->stage_r[p];
  dev.conf = io->conf ? h->stage_conf[p] : nullptr;
  // Pinned, mapped host memory can take the output straight from the kernel (posted writes over the bus, no
  // separate copy after the step); anything else goes through the staging buffer.
  void* out_dev = nullptr;
  {
    cudaPointerAttributes attr;
    if (cudaPointerGetAttributes(&attr, io->out) == cudaSuccess && attr.type == cudaMemoryTypeHost &&
        attr.devicePointer != nullptr && aligned16(attr.devicePointer))
      out_dev = attr.devicePointer;
    else
      (void)cudaGetLastError();
  }
  dev.out = out_dev ? out_dev : h->stage_o[p];
  rc = ovggt_layer_step(h, layer, &dev, stream);
  if (rc == OVGGT_OK && !out_dev) {
    cudaError_t e = cudaMemcpyAsync(io->out, h->stage_o[p], bytes, cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) rc = cuda_fail(e);
  }
  if (h->copy) {
    cudaError_t e = cudaEventRecord(h->ev_done[p], st);
    if (e != cudaSuccess && rc == OVGGT_OK) rc = cuda_fail(e);
    h->stage_used[p] = true;
  }
  return rc;
}

extern "C" int ovggt_cache_stats(ovggt_cache* h, int32_t layer, ovggt_stats* out) {
  int rc = check_layer(h, layer);
  if (rc) return rc;
  if (!out) return OVGGT_ERR_INVALID_ARG;
  const LayerState& S = h->layers[layer];
  std::memset(out, 0, sizeof(*out));
  out->n_cached = S.n;
  out->n_protected_init = S.n_prot_init;
  out->n_protected_hist = S.n_prot_hist;
  out->n_active_anchors = (int)h->anchors.size();
  int i = 0;
  for (int64_t f : h->anchors) out->anchor_frames[i++] = f;
  out->frames_seen = S.frames_seen;
  out->evicted_total = S.evicted_total;
  out->last_n_candidates = S.last_N;
  out->last_n_survivors = S.last_keep;
  out->bytes_resident = S.kv_bytes;
  CK(cudaStreamSynchronize(h->last_stream));
  int status = 0;
  CK(cudaMemcpy(&status, h->status, sizeof(int), cudaMemcpyDeviceToHost));
  out->device_status = status;
  return status == 0 ? OVGGT_OK : status;
}

extern "C" int ovggt_cache_export(ovggt_cache* h, int32_t layer, int64_t* token_ids, uint8_t* flags, float* scores,
                                  void* k, void* v, int32_t* n_out) {
  int rc = check_layer(h, layer);
  if (rc) return rc;
  LayerState& S = h->layers[layer];
  if (S.pending) return OVGGT_ERR_FRAME_ORDER;
  rc = flush_moves(h, S, h->last_stream);
  if (rc) return rc;
  CK(cudaStreamSynchronize(h->last_stream));
  const int n = S.n, b = S.cur, kb = S.kv;
  const size_t row = (size_t)h->C * h->elem;
  if (n > 0) {
    if (token_ids) CK(cudaMemcpy(token_ids, S.ids[b], (size_t)n * 8, cudaMemcpyDeviceToHost));
    if (flags) CK(cudaMemcpy(flags, S.flags[b], (size_t)n, cudaMemcpyDeviceToHost));
    if (scores) CK(cudaMemcpy(scores, S.stored[b], (size_t)n * 4, cudaMemcpyDeviceToHost));
    if (!fill_layout(h)) {
      if (k) CK(cudaMemcpy(k, S.kbuf[kb], (size_t)n * row, cudaMemcpyDeviceToHost));
      if (v) CK(cudaMemcpy(v, S.vbuf[kb], (size_t)n * row, cudaMemcpyDeviceToHost));
    } else if (k || v) {
      // the rows lie in slot order on the device; the caller gets them in ascending token id
      std::vector<int> slot(n);
      std::vector<char> tmp((size_t)n * row);
      CK(cudaMemcpy(slot.data(), S.slot[b], (size_t)n * 4, cudaMemcpyDeviceToHost));
      for (int which = 0; which < 2; ++which) {
        char* dst = static_cast<char*>(which == 0 ? k : v);
        if (!dst) continue;
        CK(cudaMemcpy(tmp.data(), which == 0 ? S.kbuf[kb] : S.vbuf[kb], (size_t)n * row, cudaMemcpyDeviceToHost));
        for (int j = 0; j < n; ++j) {
          if (slot[j] < 0 || slot[j] >= n) return OVGGT_ERR_DEVICE_STATUS;
          std::memcpy(dst + (size_t)j * row, tmp.data() + (size_t)slot[j] * row, row);
        }
      }
    }
  }
  if (n_out) *n_out = n;
  return OVGGT_OK;
}

extern "C" int ovggt_cache_import(ovggt_cache* h, int32_t layer, const int64_t* token_ids, const uint8_t* flags,
                                  const float* scores, const void* k, const void* v, int32_t n,
                                  int64_t next_frame_id, int64_t last_registration_frame) {
  int rc = check_layer(h, layer);
  if (rc) return rc;
  LayerState& S = h->layers[layer];
  if (n < 0 || n > S.budget || (n > 0 && (!token_ids || !flags || !scores || !k || !v))) return OVGGT_ERR_INVALID_ARG;
  const int M = h->M;
  // rebuild the bookkeeping from ids and flags
  int n_init = 0, n_hist = 0;
  std::vector<int64_t> anchor_frames;
  for (int i = 0; i < n; ++i) {
    if (i > 0 && token_ids[i] <= token_ids[i - 1]) return OVGGT_ERR_INVALID_ARG;
    if (flags[i] == OVGGT_FLAG_INIT) ++n_init;
    else if (flags[i] == OVGGT_FLAG_HIST) {
      ++n_hist;
      const int64_t f = token_ids[i] / M;
      if (anchor_frames.empty() || anchor_frames.back() != f) anchor_frames.push_back(f);
    } else if (flags[i] != OVGGT_FLAG_EVICTABLE) return OVGGT_ERR_INVALID_ARG;
  }
  if ((int)anchor_frames.size() > h->cfg.k_max) return OVGGT_ERR_INVALID_ARG;
  // The anchor FIFO, the first frame and the last registration belong to the handle, not to a layer.  A handle that
  // has seen no frame adopts them from the first non-empty layer imported; every later import has to agree.
  const bool fresh = h->first_frame < 0;
  if (n > 0 && !fresh) {
    const int64_t f0 = token_ids[0] / M;
    if (h->cfg.protect_first_frame ? f0 != h->first_frame : f0 < h->first_frame) return OVGGT_ERR_INVALID_ARG;
    if (anchor_frames.size() != h->anchors.size() ||
        !std::equal(anchor_frames.begin(), anchor_frames.end(), h->anchors.begin()))
      return OVGGT_ERR_INVALID_ARG;
    if (last_registration_frame != h->last_registration) return OVGGT_ERR_INVALID_ARG;
  }
  CK(cudaStreamSynchronize(h->last_stream));
  const int b = S.cur, kb = S.kv;
  const size_t row = (size_t)h->C * h->elem;
  if (n > 0) {
    CK(cudaMemcpy(S.ids[b], token_ids, (size_t)n * 8, cudaMemcpyHostToDevice));
    CK(cudaMemcpy(S.flags[b], flags, (size_t)n, cudaMemcpyHostToDevice));
    CK(cudaMemcpy(S.stored[b], scores, (size_t)n * 4, cudaMemcpyHostToDevice));
    CK(cudaMemcpy(S.kbuf[kb], k, (size_t)n * row, cudaMemcpyHostToDevice));
    CK(cudaMemcpy(S.vbuf[kb], v, (size_t)n * row, cudaMemcpyHostToDevice));
    if (fill_layout(h)) {         // rows arrive in token order: slot = position
      std::vector<int> slot(n);
      for (int j = 0; j < n; ++j) slot[j] = j;
      CK(cudaMemcpy(S.slot[b], slot.data(), (size_t)n * 4, cudaMemcpyHostToDevice));
    }
  }
  CK(cudaMemset(S.kmax2, 0, (size_t)h->cfg.n_heads * 4));
  if (n > 0 && h->cfg.dtype == kBF16 && h->C * h->elem / 16 <= 128) {
    k_key_norm_max<<<std::min((n + 7) / 8, 148 * 8), 256>>>((const uint4*)S.kbuf[kb], n, h->C * h->elem / 16, S.kmax2);
    LAUNCHED();
    CK(cudaDeviceSynchronize());
  }
  S.n = n;
  S.colsum_nparts = 0;          // the imported keys have not been summed
  S.ksum_valid = false;
  S.moves_pending = false;      // (whatever was pending concerned rows that are gone)
  S.moves_delta = nullptr;
  S.pending = false;
  S.n_prot_init = n_init;
  S.n_prot_hist = n_hist;
  S.pending_frame = next_frame_id - 1;
  S.frames_seen = n > 0 ? 1 : 0;
  if (n > 0 && fresh) {
    h->anchors.assign(anchor_frames.begin(), anchor_frames.end());
    h->first_frame = token_ids[0] / M;
    h->last_registration = last_registration_frame;
    h->decided_frame = -1;
  }
  return OVGGT_OK;
}

extern "C" int ovggt_cache_reset(ovggt_cache* h) {
  if (!h) return OVGGT_ERR_INVALID_ARG;
  CK(cudaStreamSynchronize(h->last_stream));
  if (h->side) CK(cudaStreamSynchronize(h->side));
  for (LayerState& S : h->layers) {
    S.n = 0;
    S.cur = 0;
    S.pending = false;
    S.frames_seen = S.evicted_total = 0;
    S.pending_frame = -1;
    S.n_prot_init = S.n_prot_hist = 0;
    S.last_N = S.last_keep = 0;
    S.colsum_nparts = 0;
    S.ksum_valid = false;
    S.moves_pending = false;
    S.moves_delta = nullptr;
    S.since_refresh = 0;
    S.scores_frame = -1;
    CK(cudaMemset(S.kmax2, 0, (size_t)h->cfg.n_heads * 4));
  }
  h->anchors.clear();
  h->first_frame = h->last_registration = h->decided_frame = -1;
  h->decided_register = false;
  h->decided_demote = -1;
  CK(cudaMemset(h->status, 0, 64));
  return OVGGT_OK;
}

extern "C" int ovggt_cache_clear_status(ovggt_cache* h) {
  if (!h) return OVGGT_ERR_INVALID_ARG;
  CK(cudaStreamSynchronize(h->last_stream));
  CK(cudaMemset(h->status, 0, 64));
  return OVGGT_OK;
}

extern "C" int ovggt_cache_selftest_bounded_wait(ovggt_cache* h, uint32_t limit_us, uint64_t* waited_ns, void* stream) {
  if (!h || limit_us == 0 || limit_us > 1000000) return OVGGT_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  h->last_stream = st;
  unsigned long long* dev_ns = reinterpret_cast<unsigned long long*>(h->status + 8);   // (inside the 64-byte status block)
  k_bounded_wait_selftest<<<1, 32, 0, st>>>(h->status, (unsigned long long)limit_us * 1000ull, dev_ns);
  LAUNCHED();
  if (waited_ns) {
    CK(cudaStreamSynchronize(st));
    unsigned long long ns = 0;
    CK(cudaMemcpy(&ns, dev_ns, 8, cudaMemcpyDeviceToHost));
    *waited_ns = ns;
  }
  return OVGGT_OK;
}

extern "C" int ovggt_cache_last_selection(ovggt_cache* h, int32_t layer, float* priorities, int32_t* n_candidates,
                                          int32_t* survivors, int32_t* n_survivors) {
  int rc = check_layer(h, layer);
  if (rc) return rc;
  const LayerState& S = h->layers[layer];
  CK(cudaStreamSynchronize(h->last_stream));
  if (priorities && S.last_N > 0) CK(cudaMemcpy(priorities, S.r, (size_t)S.last_N * 4, cudaMemcpyDeviceToHost));
  if (survivors && S.last_keep > 0) CK(cudaMemcpy(survivors, S.surv, (size_t)S.last_keep * 4, cudaMemcpyDeviceToHost));
  if (n_candidates) *n_candidates = S.last_N;
  if (n_survivors) *n_survivors = S.last_keep;
  return OVGGT_OK;
}

extern "C" int ovggt_cache_profile_enable(ovggt_cache* h, int32_t enable) {
  if (!h) return OVGGT_ERR_INVALID_ARG;
  h->prof = enable != 0;
  return OVGGT_OK;
}

extern "C" int ovggt_cache_profile_read(ovggt_cache* h, double* ms, int64_t* counts, int32_t reset) {
  if (!h) return OVGGT_ERR_INVALID_ARG;
  CK(cudaStreamSynchronize(h->last_stream));
  for (auto& r : h->prof_recs) {
    float t = 0.0f;
    if (cudaEventElapsedTime(&t, r.a, r.b) == cudaSuccess) {
      h->prof_ms[r.cls] += t;
      h->prof_cnt[r.cls] += 1;
    }
    cudaEventDestroy(r.a);
    cudaEventDestroy(r.b);
  }
  h->prof_recs.clear();
  for (int i = 0; i < OVGGT_PROF_CLASSES; ++i) {
    if (ms) ms[i] = h->prof_ms[i];
    if (counts) counts[i] = h->prof_cnt[i];
    if (reset) { h->prof_ms[i] = 0.0; h->prof_cnt[i] = 0; }
  }
  return OVGGT_OK;
}

extern "C" uint64_t ovggt_kernel_launches(void) { return g_launches.load(); }
extern "C" int ovggt_last_cuda_error(void) { return g_last_cuda_error.load(); }

extern "C" const char* ovggt_strerror(int code) {
  switch (code) {
    case OVGGT_OK: return "ok";
    case OVGGT_ERR_INVALID_ARG: return "invalid argument";
    case OVGGT_ERR_BAD_LAYER: return "layer index out of range";
    case OVGGT_ERR_BUDGET_TOO_SMALL: return "budget below the protected-set bound M + K_max * A";
    case OVGGT_ERR_FRAME_ORDER: return "frame ids must increase and attend/compress must alternate";
    case OVGGT_ERR_MISALIGNED: return "pointer not sufficiently aligned";
    case OVGGT_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case OVGGT_ERR_CUDA: return "CUDA call failed";
    case OVGGT_ERR_DEVICE_STATUS: return "a kernel reported an inconsistency";
    case OVGGT_ERR_TIMEOUT: return "a bounded device-side wait ran out";
    case OVGGT_ERR_UNSUPPORTED: return "configuration not supported by this build";
    case OVGGT_ERR_TOO_LARGE: return "size exceeds the fixed capacity of the built-in scratch array";
    default: return "unknown error";
  }
}

// ------------------------------------------------------------------ single kernels

extern "C" int ovggt_k_row_norms(const void* x, int32_t rows, int32_t C, int32_t dtype, float* s, void* stream) {
  if (rows == 0) return OVGGT_OK;
  if (!x || !s || rows < 0 || C < 1 || (C * elem_bytes(dtype)) % 16 || (dtype != kF32 && dtype != kBF16))
    return OVGGT_ERR_INVALID_ARG;
  if (!aligned16(x)) return OVGGT_ERR_MISALIGNED;
  return launch_row_norms(x, rows, C, dtype, s, static_cast<cudaStream_t>(stream));
}

extern "C" size_t ovggt_k_diversity_scratch_bytes(int32_t rows, int32_t C) {
  (void)rows;
  return ((size_t)kMaxColsumParts + 1) * (size_t)C * 4;
}

extern "C" int ovggt_k_diversity(const void* K, int32_t rows, int32_t C, int32_t dtype, float* d, void* scratch,
                                 void* stream) {
  if (rows == 0) return OVGGT_OK;
  if (!K || !d || !scratch || rows < 0 || C < 1 || (C * elem_bytes(dtype)) % 16 || (dtype != kF32 && dtype != kBF16) ||
      (size_t)C * 4 > 48 * 1024)
    return OVGGT_ERR_INVALID_ARG;
  if (!aligned16(K) || !aligned16(scratch)) return OVGGT_ERR_MISALIGNED;
  float* part = static_cast<float*>(scratch);
  float* ksum = part + (size_t)kMaxColsumParts * C;
  return launch_diversity(K, rows, C, dtype, part, ksum, d, static_cast<cudaStream_t>(stream));
}

extern "C" int ovggt_k_select(const float* r, const uint8_t* flags, int32_t N, int32_t B, int32_t batch,
                              int32_t* survivors, void* scratch, void* stream) {
  if (N < 1 || B < 0 || batch < 1) return OVGGT_ERR_INVALID_ARG;
  if (B == 0) return OVGGT_OK;   // nothing can be kept: the survivor lists are empty
  if (!r || !flags || !survivors || !scratch) return OVGGT_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int* status = reinterpret_cast<int*>(scratch);
  const int ncta = select_cluster_ctas(N);
  const size_t smem = select_smem_bytes((N + ncta - 1) / ncta, 0);
  if (smem > kSmemLimit) return OVGGT_ERR_UNSUPPORTED;
  CK(cudaFuncSetAttribute(k_select, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemLimit));
  CK(cudaMemsetAsync(status, 0, 4, st));
  CK(launch_cluster(k_select, dim3(ncta, batch), ncta, smem, st, r, flags, (int)N, (int)B, (int*)survivors, status));
  LAUNCHED();
  return OVGGT_OK;
}

extern "C" int ovggt_k_compact(const void* k_src, const void* v_src, const int32_t* survivors, int32_t n_keep,
                               int32_t C, int32_t dtype, void* k_dst, void* v_dst, void* stream) {
  if (n_keep == 0) return OVGGT_OK;
  if (!k_src || !v_src || !survivors || !k_dst || !v_dst || n_keep < 0 || C < 1 || (C * elem_bytes(dtype)) % 16)
    return OVGGT_ERR_INVALID_ARG;
  if (!aligned16(k_src) || !aligned16(v_src) || !aligned16(k_dst) || !aligned16(v_dst)) return OVGGT_ERR_MISALIGNED;
  // (the caller's source row count is not part of this call: the checked build has no bound to test against here)
  return launch_compact(k_src, v_src, survivors, n_keep, C, dtype, k_dst, v_dst, static_cast<cudaStream_t>(stream),
                        0x7FFFFFFF, nullptr);
}

extern "C" size_t ovggt_k_attention_scratch_bytes(int32_t M, int32_t N, int32_t n_heads) {
  return attn_tcgen05_scratch_bytes(M, N, n_heads);
}

extern "C" int ovggt_k_attention(const void* q, const void* k, const void* v, int32_t M, int32_t N, int32_t n_heads,
                                 int32_t dtype, void* out, void* scratch, int32_t* device_status, void* stream) {
  if (!q || !k || !v || !out || M < 1 || N < 1 || n_heads < 1 || (dtype != kF32 && dtype != kBF16))
    return OVGGT_ERR_INVALID_ARG;
  if (dtype == kBF16 && (!scratch || !device_status)) return OVGGT_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out)) return OVGGT_ERR_MISALIGNED;
  return launch_attention(q, k, v, M, N, n_heads, dtype, out, scratch, device_status, static_cast<cudaStream_t>(stream));
}

extern "C" int ovggt_k_key_norm_bound(const void* K, int32_t rows, int32_t n_heads, float* kmax2, void* stream) {
  if (!kmax2 || rows < 0 || (rows > 0 && !K) || n_heads < 1 || n_heads > 16) return OVGGT_ERR_INVALID_ARG;
  if (!aligned16(K)) return OVGGT_ERR_MISALIGNED;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  CK(cudaMemsetAsync(kmax2, 0, (size_t)n_heads * 4, st));
  if (rows == 0) return OVGGT_OK;
  k_key_norm_max<<<std::min((rows + 7) / 8, 148 * 8), 256, 0, st>>>((const uint4*)K, rows, n_heads * 8, kmax2);
  LAUNCHED();
  return OVGGT_OK;
}

extern "C" int ovggt_k_attention_bounded(const void* q, const void* k, const void* v, int32_t M, int32_t N,
                                         int32_t n_heads, void* out, void* scratch, int32_t* device_status,
                                         const float* kmax2, void* stream) {
  if (!q || !k || !v || !out || M < 1 || N < 1 || n_heads < 1 || !scratch || !device_status || !kmax2)
    return OVGGT_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out)) return OVGGT_ERR_MISALIGNED;
  return launch_attention(q, k, v, M, N, n_heads, kBF16, out, scratch, device_status, static_cast<cudaStream_t>(stream),
                          nullptr, kmax2);
}

extern "C" int ovggt_k_gemm_bf16(const void* A, const void* Bm, int32_t M, int32_t N, int32_t K, void* C,
                                 int32_t* device_status, void* stream) {
  if (!A || !Bm || !C || !device_status || M < 1 || N < 1 || K < 1) return OVGGT_ERR_INVALID_ARG;
  if (K % 64 != 0 || N % 8 != 0) return OVGGT_ERR_UNSUPPORTED;
  if (!aligned16(A) || !aligned16(Bm) || !aligned16(C)) return OVGGT_ERR_MISALIGNED;
  int rc = gemm_tcgen05_launch(A, Bm, C, M, N, K, device_status, static_cast<cudaStream_t>(stream));
  if (rc == OVGGT_OK) g_launches.fetch_add(1);
  if (rc == OVGGT_ERR_CUDA) g_last_cuda_error.store(attn_tcgen05_last_error());
  return rc;
}

// ------------------------------------------------------------------ allocation-free diversity

namespace {
constexpr int kStaticDivMaxC = 1024;
// Built-in scratch of ovggt_k_diversity_static: column-sum partials [kMaxColsumParts, C] followed by the column
// sums [C], C <= kStaticDivMaxC (about 2.4 MB).  Every GPU that loads the library holds it until the process exits.
static __device__ __align__(256) float g_static_div_scratch[(kMaxColsumParts + 1) * kStaticDivMaxC];

constexpr int kMaxDevices = 64;
float* g_static_div_ptr[kMaxDevices] = {nullptr};
std::atomic<int> g_static_div_ready[kMaxDevices];

// Device address of the built-in scratch on the current device.  In host code the array's name is only a
// handle for the runtime, not an address a kernel could use; the address is asked for once per device.
int static_div_scratch(float** out) {
  int dev = 0;
  CK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return OVGGT_ERR_UNSUPPORTED;
  if (!g_static_div_ready[dev].load(std::memory_order_acquire)) {
    void* p = nullptr;
    CK(cudaGetSymbolAddress(&p, g_static_div_scratch));
    g_static_div_ptr[dev] = static_cast<float*>(p);
    g_static_div_ready[dev].store(1, std::memory_order_release);
  }
  *out = g_static_div_ptr[dev];
  return OVGGT_OK;
}
}  // namespace

extern "C" int ovggt_k_diversity_static(const void* K, int32_t rows, int32_t C, int32_t dtype, float* d,
                                        void* stream) {
  if (rows == 0) return OVGGT_OK;
  if (!K || !d || rows < 0 || C < 1 || (dtype != kF32 && dtype != kBF16) || (C * elem_bytes(dtype)) % 16)
    return OVGGT_ERR_INVALID_ARG;
  if (C > kStaticDivMaxC) return OVGGT_ERR_TOO_LARGE;
  if (!aligned16(K)) return OVGGT_ERR_MISALIGNED;
  float* scratch = nullptr;
  int rc = static_div_scratch(&scratch);
  if (rc) return rc;
  float* part = scratch;
  float* ksum = scratch + (size_t)kMaxColsumParts * C;
  return launch_diversity(K, rows, C, dtype, part, ksum, d, static_cast<cudaStream_t>(stream));
}
