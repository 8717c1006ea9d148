/*
 * ovggt.h - C ABI of the B200 streaming global-attention step of OVGGT.
 *
 * One handle (ovggt_cache) holds the bounded KV caches of all global-attention
 * layers of one frame stream.  For every incoming frame and every layer the
 * caller runs one step:
 *
 *   append  K_t, V_t to the layer's cache                           (Eq. 2)
 *   attend  the frame's queries over [cache of frame t-1 ; frame t] (Sec. 3.1)
 *   score   new tokens by FFN-residual norm, smoothed               (Eq. 5, Eq. 6)
 *           cached tokens by key diversity, hybrid-normalised       (Eq. 7)
 *   protect first-frame tokens and historical anchors (FIFO)        (Sec. 3.3)
 *   select  P u Top-k(U, B - |P|) and compact the cache             (Eq. 8)
 *
 * Conventions
 *  - Every `device` pointer is CUDA device memory of the GPU that was current at
 *    ovggt_cache_create; every `host` pointer is ordinary host memory.
 *  - Row-major, token-major tensors: [tokens, C] with C = n_heads * head_dim and head h
 *    owning columns [h*head_dim, (h+1)*head_dim).  Element type is the configured
 *    dtype (float, or bfloat16 bit patterns).  Tensors must be 16-byte aligned.
 *  - Tokens of a frame: n_special aux tokens (camera, registers) first, then the
 *    grid_h x grid_w patch tokens row-major; M = n_special + grid_h * grid_w.
 *  - The caller owns every device byte: inputs, outputs and the workspace.  The
 *    library never allocates or frees device memory and keeps no pointer of an
 *    ovggt_frame_io after the call returns.  The handle itself is host memory.
 *  - Every call enqueues its kernels on the given CUDA stream (a cudaStream_t passed
 *    as void*; NULL = the legacy default stream) and returns without synchronising,
 *    unless stated.  All layers of a handle share scratch memory, so all calls on one
 *    handle must be ordered on one stream (or otherwise serialised by the caller).
 *  - Return value: 0 on success, a negative OVGGT_ERR_* otherwise; no call aborts,
 *    throws or prints.  A handle is not thread-safe; independent handles are independent.
 */
#ifndef OVGGT_H_
#define OVGGT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define OVGGT_MAX_ANCHORS 16

enum {
  OVGGT_OK = 0,
  OVGGT_ERR_INVALID_ARG = -1,       /* NULL handle / pointer, non-positive size, unsupported head_dim or dtype */
  OVGGT_ERR_BAD_LAYER = -2,
  OVGGT_ERR_BUDGET_TOO_SMALL = -3,  /* B < M, or B below the protected-set bound M + K_max * A of Eq. 9 */
  OVGGT_ERR_FRAME_ORDER = -4,       /* frame ids must increase; attend/compress must alternate per layer */
  OVGGT_ERR_MISALIGNED = -5,        /* a device tensor or the workspace is not 16-byte (workspace: 1024-byte) aligned */
  OVGGT_ERR_WORKSPACE_TOO_SMALL = -6,
  OVGGT_ERR_CUDA = -7,              /* a CUDA runtime / driver call failed; see ovggt_last_cuda_error */
  OVGGT_ERR_DEVICE_STATUS = -8,     /* a kernel reported an inconsistency through the device status word */
  OVGGT_ERR_TIMEOUT = -9,           /* a bounded device-side wait ran out (the kernel returned cleanly) */
  OVGGT_ERR_UNSUPPORTED = -10,      /* the configuration is valid but this build has no kernel for it */
  OVGGT_ERR_TOO_LARGE = -11         /* a size exceeds the fixed capacity of a built-in scratch array */
};

enum { OVGGT_DTYPE_F32 = 0, OVGGT_DTYPE_BF16 = 1 };
/* How evictable rows are ranked.  HYBRID is the paper's method (Eq. 7).  RESIDUAL_STORED ranks every row by the
 * smoothed residual norm it had when new.  RANDOM is the random-eviction baseline of the paper's full-cache comparison
 * (Supp. A): the rows that leave are drawn uniformly at random under the same budget - every evictable row gets a
 * fresh uniform priority per step, the top 24 bits of SplitMix64(SplitMix64(random_seed ^ frame_id) + token_id)
 * scaled by 2^-24 (SplitMix64(x): z = x + 0x9E3779B97F4A7C15; z = (z ^ z >> 30) * 0xBF58476D1CE4E5B9;
 * z = (z ^ z >> 27) * 0x94D049BB133111EB; z ^ z >> 31), so that a run is reproducible from its seed.
 * QK is the query-key baseline of the scoring probe (Supp. D): the hybrid mode with the residual norm of a new token
 * (Eq. 5) replaced by a dot product of queries and keys that needs no attention matrix.  The paper prints no formula;
 * the reading built here is the mean, over the frame's M queries and the heads, of the scaled logit new token j
 * receives, s_j = 1 / (M n_heads) sum_h sum_i (q_{i,h} . k_{j,h}) / sqrt(head_dim), computed through the column sums
 * of Q.  The attend half computes it from io->q and io->k and keeps it per layer until the layer's compress half,
 * whose io->resid is then not read (it may be NULL); Eq. 6-8 and the key diversity of cached rows are unchanged.
 * ATTN is the probe's attention-weight baseline, the criterion that needs the attention matrix (reading: the
 * attention new token j receives in the frame's own attention over [cache + frame], averaged over the frame's M
 * queries and the heads, s_j = 1 / (M n_heads) sum_h sum_i P_h[i, n + j]).  The attention kernels leave each row's
 * log2 softmax denominator behind and a second pass over the frame's own M x M block recomputes those columns of P;
 * it runs in the attend half after the attention, so ovggt_layer_step does not overlap anything in this mode.  The
 * residual is not read either.
 * QK and ATTN are not available for a camera-head cache. */
enum {
  OVGGT_SCORE_HYBRID = 0, OVGGT_SCORE_RESIDUAL_STORED = 1, OVGGT_SCORE_RANDOM = 2, OVGGT_SCORE_QK = 3,
  OVGGT_SCORE_ATTN = 4
};
enum { OVGGT_FLAG_EVICTABLE = 0, OVGGT_FLAG_INIT = 1, OVGGT_FLAG_HIST = 2 };
/* Where surviving K/V rows live after Eq. 8 (the paper fixes the survivor set, not a layout):
 *  FILL_HOLES     one K/V buffer per layer; the rows admitted from the new frame are copied into the slots the
 *                 evicted rows leave (at most M rows move per step, inside the layer's next append); logical
 *                 (token id) order is kept in per-row meta and restored by ovggt_cache_export.  Attention reads the buffer front to back: the order of
 *                 cached rows does not change its result beyond fp32 summation order.
 *  STABLE_GATHER  two K/V buffers per layer; every survivor is copied, in token order, into the other buffer
 *                 (B rows move per step; rows lie in token order on the device). */
enum { OVGGT_COMPACT_FILL_HOLES = 0, OVGGT_COMPACT_STABLE_GATHER = 1 };

typedef struct ovggt_cache ovggt_cache; /* opaque host-side handle */

typedef struct {
  int32_t n_layers, n_heads, head_dim;   /* head_dim must be 64 */
  int32_t n_special, grid_h, grid_w;     /* per-frame token layout (Sec. 3.1) */
  const int32_t* budget;                 /* host [n_layers]: B^(l), tokens kept per layer between steps (Eq. 8) */
  int32_t anchor_tokens;                 /* A = ceil(eta * N_p): protected patch tokens per historical anchor */
  int32_t k_max;                         /* K_max active historical anchors, <= OVGGT_MAX_ANCHORS */
  int32_t min_anchor_interval;           /* frames between anchor registrations (paper: 100) */
  float tau, alpha, beta;                /* coverage threshold, smoothing strength (Eq. 6), hybrid balance (Eq. 7) */
  int32_t protect_first_frame;           /* 1: Global Initial Anchor (all M first-frame tokens kept for good) */
  int32_t score_mode;                    /* OVGGT_SCORE_* */
  int32_t dtype;                         /* OVGGT_DTYPE_* of q, k, v, resid, out and of the cache */
  int32_t compaction;                    /* OVGGT_COMPACT_* */
  uint64_t random_seed;                  /* OVGGT_SCORE_RANDOM only */
  int32_t camera_head;                   /* 1: the camera head's cache (Supp. C): n_special = 1, grid 0 x 0,
                                            anchor_tokens = 0; see ovggt_camera_compress.  0: an aggregator cache */
  void* workspace;                       /* device, >= ovggt_workspace_bytes(cfg), 1024-byte aligned; need not be zeroed */
  size_t workspace_bytes;
} ovggt_config;

typedef struct {
  int64_t frame_id;             /* strictly increasing over the stream; the same for all layers of a frame */
  const void* q;                /* [M, C] queries of the frame                     (attend) */
  const void* k;                /* [M, C] keys of the frame                        (attend) */
  const void* v;                /* [M, C] values of the frame                      (attend) */
  const void* resid;            /* [M, C] FFN residual rows, LayerScale included   (compress, Eq. 5; unused and
                                   optional in OVGGT_SCORE_QK and OVGGT_SCORE_ATTN) */
  const float* conf;            /* [grid_h*grid_w] per-patch confidence, or NULL = no anchor candidate (compress) */
  float rho;                    /* coverage ratio of the latest anchor in this view; NaN = no decision (compress) */
  const float* score_override;  /* [n + M] fp32 or NULL: priorities the selection ranks instead of its own (compress) */
  void* out;                    /* [M, C] attention output                         (attend) */
} ovggt_frame_io;               /* ovggt_layer_step: all pointers device.  ovggt_layer_step_host: all pointers host. */

typedef struct {
  int32_t n_cached;             /* rows held after the last completed step, <= budget */
  int32_t n_protected_init;     /* |P_init| */
  int32_t n_protected_hist;     /* |P_hist| = anchor_tokens * n_active_anchors */
  int32_t n_active_anchors;
  int64_t anchor_frames[OVGGT_MAX_ANCHORS]; /* active historical anchors, oldest first */
  int64_t frames_seen;          /* steps completed on this layer */
  int64_t evicted_total;        /* rows dropped so far */
  int32_t last_n_candidates;    /* N = n + M of the last step */
  int32_t last_n_survivors;     /* min(N, B) */
  uint64_t bytes_resident;      /* workspace bytes this layer's K/V buffers occupy: constant over the stream
                                   (2 (B + M) C elements with hole filling, twice that with the stable gather) */
  int32_t device_status;        /* 0, or the OVGGT_ERR_* a kernel raised */
} ovggt_stats;

/* Bytes of device workspace the configuration needs (0 if the configuration is invalid).
 * cfg->workspace / workspace_bytes are ignored here. */
size_t ovggt_workspace_bytes(const ovggt_config* cfg);

/* Validate cfg, lay the caches out in cfg->workspace and return a handle.  Clears a few words of the
 * workspace on the legacy default stream and synchronises.
 * OVGGT_ERR_BUDGET_TOO_SMALL if a layer's budget cannot hold the protected set (Eq. 9).
 * OVGGT_ERR_UNSUPPORTED if a layer's B + M candidates do not fit the selection kernel, which keeps them in the
 * shared memory of one 8-CTA cluster (about 18 bytes per candidate and CTA: B + M up to roughly 90,000). */
int ovggt_cache_create(const ovggt_config* cfg, ovggt_cache** out);
int ovggt_cache_destroy(ovggt_cache* cache);

/* Eq. 2 + attention: append io->k / io->v as rows [n, n+M) of the layer's cache, then write
 * softmax(Q K^T / sqrt(head_dim)) V over all n + M rows to io->out.  No mask inside the step
 * (causality is between frames).  Uses frame_id, q, k, v, out. */
int ovggt_layer_attend(ovggt_cache* cache, int32_t layer, const ovggt_frame_io* io, void* stream);

/* Eq. 5-8 and Sec. 3.3 for the frame appended by the last ovggt_layer_attend of this layer:
 * score, protect, select the survivors and compact the cache to <= B^(l) rows, order preserved.
 * The anchor decision of a frame is taken once (first layer that compresses it) from rho and the
 * interval rule and applied identically to every layer.  The anchor state belongs to the handle and only moves
 * forward: every layer has to compress frame t before any layer compresses a later frame; a layer that comes
 * with an older frame gets OVGGT_ERR_FRAME_ORDER and nothing is changed.  Uses frame_id, resid, conf, rho,
 * score_override. */
int ovggt_layer_compress(ovggt_cache* cache, int32_t layer, const ovggt_frame_io* io, void* stream);

/* ovggt_layer_compress for every layer of the handle in one call (Sec. 3.2: each layer l has its own budget B^(l),
 * given at create): ios [n_ios], n_ios = n_layers, ios[l] describing layer l's pending frame (all with the same
 * frame_id; conf and rho are taken from ios[0]).  This is the call for a model whose anchor inputs exist only after
 * its heads have run: attend layer by layer, then compress all layers together.  In the hole-filling layout the
 * scores and the selection of up to 32 layers each go out as one launch (blockIdx.y = layer; one thread-block
 * cluster per layer for the selection), so the small per-layer kernels fill the GPU together, and the moves of each
 * layer ride in that layer's next append as always; in the stable-gather layout the layers are compressed one after
 * the other.  All layers are checked before anything
 * changes; results are those of n_layers single calls. */
int ovggt_layers_compress(ovggt_cache* cache, const ovggt_frame_io* ios, int32_t n_ios, void* stream);

/* Supp. C: the camera prediction head keeps one token per frame in a cache of its own, under the same scoring and
 * protection.  Create it as a second handle with camera_head = 1 (budget[l] >= 1 + K_max tokens), run
 * ovggt_layer_attend on it with the camera token's q, k, v ([1, C]), and compress it with this call instead of
 * ovggt_layer_compress.  Differences from the aggregator's cache: no patch map, hence no smoothing (Eq. 6 does not
 * apply; the stored score is the raw residual norm); the anchor flags are not decided from rho but mirror the
 * aggregator's decision for the same frame_id - registered != 0 protects this frame's token, demoted_frame >= 0
 * releases that frame's token; the new group of Eq. 7 has one member (0/0), whose normalised score is taken as 1.
 * ovggt_cache_anchor_decision reads (registered, demoted_frame) of frame_id from the aggregator handle once one of
 * its layers has compressed that frame (OVGGT_ERR_FRAME_ORDER before that, or once a later frame was decided).
 * Uses frame_id, resid ([1, C]), score_override of io. */
int ovggt_cache_anchor_decision(ovggt_cache* aggregator, int64_t frame_id, int32_t* registered, int64_t* demoted_frame);
int ovggt_camera_compress(ovggt_cache* camera, int32_t layer, const ovggt_frame_io* io, int32_t registered,
                          int64_t demoted_frame, void* stream);

/* ovggt_layer_attend and ovggt_layer_compress of one (frame, layer): the whole hot path.  Scoring and selection
 * read the cache and the new rows but not the attention's output, so they are enqueued on a second stream that the
 * handle owns (a host object, created by ovggt_cache_create), forked from and joined back into `stream` with
 * events, and run beside the attention; so does the stable gather, which writes another buffer.  The hole-filling
 * moves would write the buffer the attention reads: the selection only records them, and the layer's next append
 * (which touches the same slots) carries them out first; ovggt_cache_export flushes them.  For the caller the call
 * is still asynchronous and ordered on `stream` alone. */
int ovggt_layer_step(ovggt_cache* cache, int32_t layer, const ovggt_frame_io* io, void* stream);

/* Turn the overlap of ovggt_layer_step off (0) or on (non-zero, the default): off, the two halves run one after the
 * other on `stream`, which is what per-kernel timing wants. */
int ovggt_cache_set_overlap(ovggt_cache* cache, int32_t enable);

/* The bf16 attention kernel may take a softmax reference that needs no tracking: per layer the library keeps a
 * running upper bound of the per-head key norms (updated by every append, recomputed by an import, cleared by a
 * reset; it never shrinks, so it stays a bound when keys are evicted), and |q| |k|_max / sqrt(64) bounds every logit
 * of a query row.  A warp whose 32 rows all find that bound within 2^48 of the true maximum of their first 96 scores
 * uses it for good and skips maximum tracking and rescaling; other warps track the maximum as before.  Results agree
 * within the attention tolerance either way.  On by default; 0 turns it off for the handle. */
int ovggt_cache_set_key_bound(ovggt_cache* cache, int32_t enable);

/* The same step with HOST tensors: q, k, v, resid, conf, out are host pointers; score_override must be NULL.
 * The host inputs must hold their values when the call is made.  They are copied into one of two sets of staging
 * buffers of the workspace on a copy stream the handle owns (not ordered after earlier work on `stream`), so with
 * pinned host memory the copies of one step overlap the kernels of the step before; the step itself runs on
 * `stream`; out is written by the kernel itself when it is pinned, mapped host memory, and copied back on `stream`
 * otherwise.  When q, k, v and resid lie back to back in that order in host memory they travel as one copy.  The
 * call returns without synchronising: once `stream` has been synchronised, out is valid and the input buffers may be
 * reused. */
int ovggt_layer_step_host(ovggt_cache* cache, int32_t layer, const ovggt_frame_io* io, void* stream);

/* Counters of one layer.  Synchronises the stream the handle last used (to read the device status word). */
int ovggt_cache_stats(ovggt_cache* cache, int32_t layer, ovggt_stats* out);

/* Copy the layer's current layout to host arrays, ascending token id = ascending row.  Any pointer may be
 * NULL.  token_ids [n] (frame_id * M + index in frame), flags [n] (OVGGT_FLAG_*), scores [n] (the smoothed
 * activation score each row had when it was new), k and v [n, C] in the configured dtype.  Synchronises. */
int ovggt_cache_export(ovggt_cache* cache, int32_t layer, int64_t* token_ids, uint8_t* flags,
                       float* scores, void* k, void* v, int32_t* n);

/* Replace the layer's content by n rows given as host arrays (ascending token ids); next_frame_id is the
 * smallest frame id the stream may continue with.  The per-layer counters are rebuilt from the flags and ids.
 * The anchor FIFO, the first frame and the last registration belong to the whole handle: a handle that has seen
 * no frame adopts them from the first non-empty layer imported (FIFO = the frames of its HIST rows, oldest first;
 * first frame = its first row's frame; last_registration_frame as given); every later non-empty import must agree
 * with them (OVGGT_ERR_INVALID_ARG otherwise, nothing changed); an empty import never touches them.  To load a
 * different stream into a used handle, call ovggt_cache_reset first.  The imported rows lie in token order on the
 * device.  With hole filling the exporting handle held the same rows in slot order, so the two handles add the
 * attention's terms in different orders from then on: their outputs agree to fp32 rounding, not bit for bit (with the
 * stable gather they are bit-identical).  Synchronises. */
int ovggt_cache_import(ovggt_cache* cache, int32_t layer, const int64_t* token_ids, const uint8_t* flags,
                       const float* scores, const void* k, const void* v, int32_t n,
                       int64_t next_frame_id, int64_t last_registration_frame);

/* Forget every frame: all layers empty, no anchors, no first frame, device status cleared.  Synchronises. */
int ovggt_cache_reset(ovggt_cache* cache);

/* Every device-side wait of the library (the attention kernel waits on shared-memory barriers for its bulk copies
 * and tensor-core instructions) is bounded: when it runs out, the kernel returns cleanly and leaves OVGGT_ERR_TIMEOUT
 * in the handle's device status word, which ovggt_cache_stats reports and which stays set until cleared.
 * ovggt_cache_selftest_bounded_wait exercises exactly that wait routine on the GPU without any copy or tensor-core
 * work: one warp waits, for at most limit_us microseconds (1 .. 1,000,000), on a barrier that nothing will ever
 * complete.  Afterwards the status word holds OVGGT_ERR_TIMEOUT; *waited_ns (host, may be NULL; non-NULL
 * synchronises) is how long the wait lasted.  ovggt_cache_clear_status zeroes the status word (synchronises), after
 * which the handle is used as before. */
int ovggt_cache_selftest_bounded_wait(ovggt_cache* cache, uint32_t limit_us, uint64_t* waited_ns, void* stream);
int ovggt_cache_clear_status(ovggt_cache* cache);

/* Results of the layer's last compress, copied to host (each pointer may be NULL): priorities [N] as the
 * library computed them (+inf on protected rows; its own values even when score_override was ranked instead),
 * survivor positions [n'] ascending, and their counts.  Synchronises. */
int ovggt_cache_last_selection(ovggt_cache* cache, int32_t layer, float* priorities, int32_t* n_candidates,
                               int32_t* survivors, int32_t* n_survivors);

/* Per-kernel-class device time.  While enabled, every step records a pair of CUDA events (host objects, no
 * device memory) around the launches of each class on the step's stream; the events add a little latency, so
 * throughput is measured with profiling off.  ovggt_cache_profile_read synchronises, adds up the elapsed
 * milliseconds and launch-group counts per class into ms / counts [OVGGT_PROF_CLASSES] (each may be NULL) and,
 * if reset is non-zero, clears the totals. */
enum {
  OVGGT_PROF_APPEND = 0,     /* Eq. 2 copy of K_t, V_t */
  OVGGT_PROF_ATTENTION = 1,  /* attention kernel and, when the KV range is split, its merge kernel */
  OVGGT_PROF_ROW_NORMS = 2,  /* Eq. 5 */
  OVGGT_PROF_DIVERSITY = 3,  /* key column sums + diversity */
  OVGGT_PROF_SELECT = 4,     /* flags, Eq. 6, Eq. 7, Eq. 8 */
  OVGGT_PROF_COMPACT = 5,    /* gather of the surviving K/V rows */
  OVGGT_PROF_CLASSES = 6
};
int ovggt_cache_profile_enable(ovggt_cache* cache, int32_t enable);
int ovggt_cache_profile_read(ovggt_cache* cache, double* ms, int64_t* counts, int32_t reset);

/* Number of kernels this library has launched since it was loaded (all handles). */
uint64_t ovggt_kernel_launches(void);

const char* ovggt_strerror(int code);
/* The cudaError_t / CUresult of the last failed CUDA call in this process (0 if none). */
int ovggt_last_cuda_error(void);

/* ------------------------------------------------------------------------------------------------
 * Single kernels, exposed for unit parity tests and scaled micro-benchmarks.  All pointers device,
 * dtype = OVGGT_DTYPE_*, asynchronous on `stream`.
 * ---------------------------------------------------------------------------------------------- */

/* Eq. 5: s[j] = ||x[j, :]||_2 for rows of x [rows, C]; fp32 accumulation in a fixed order. */
int ovggt_k_row_norms(const void* x, int32_t rows, int32_t C, int32_t dtype, float* s, void* stream);

/* Sec. 3.2 (Hybrid Scoring): d[i] = 1 - cos(K[i, :], sum of all rows of K) for K [rows, C].
 * scratch: device, >= ovggt_k_diversity_scratch_bytes(rows, C). */
size_t ovggt_k_diversity_scratch_bytes(int32_t rows, int32_t C);
int ovggt_k_diversity(const void* K, int32_t rows, int32_t C, int32_t dtype, float* d, void* scratch,
                      void* stream);

/* (No counterpart in the paper: a packaging variant of ovggt_k_diversity.)
 * The same result, d[i] = 1 - cos(K[i, :], sum of all rows of K), for callers that must not allocate device
 * memory and have no spare buffer to lend: code that runs after its host application has handed the whole GPU
 * to a pool allocator, inside a latency-bound frame loop where a driver allocation would stall the device, or
 * behind a plug-in interface that forbids allocation calls.  The intermediate column sums live in an array that
 * is compiled into the library (about 2.4 MB on every GPU that loads it, held until the process exits), so the
 * call needs K and d only and itself calls no allocating routine of CUDA or of any other library.
 *   Limit: C <= 1024 columns (any number of rows); a larger C returns OVGGT_ERR_TOO_LARGE and launches nothing.
 *   The first call on each device looks the array's device address up (cudaGetSymbolAddress, with that device
 *   current) before it launches; make that first call outside any stream capture.  Later calls on the device
 *   only launch kernels.
 *   All calls on a device share the one array, and it keeps whatever the previous call left in it.  Nothing in
 *   it has to start at zero: each call overwrites every element it later reads.  Two calls that overlap on the
 *   GPU (different streams, or different host threads without ordering) race on it; order them on one stream
 *   or with events. */
int ovggt_k_diversity_static(const void* K, int32_t rows, int32_t C, int32_t dtype, float* d, void* stream);

/* Eq. 8: survivors of N candidates with priorities r [N] and flags [N] (non-zero = protected) under budget B:
 * every protected row plus the B - |P| evictable rows of largest r, ties to the lower position, NaN ranks
 * with -inf.  survivors [min(N, B)] ascending.  scratch: device, >= 64 bytes (a status word).
 * `batch` independent problems are laid out back to back (r, flags, survivors strides N, N, min(N, B)); one
 * thread-block cluster each.  N up to about 350,000 (8 CTAs x shared memory); beyond: OVGGT_ERR_UNSUPPORTED. */
int ovggt_k_select(const float* r, const uint8_t* flags, int32_t N, int32_t B, int32_t batch,
                   int32_t* survivors, void* scratch, void* stream);

/* Order-preserving compaction: dst[j, :] = src[survivors[j], :] for K and V, j < n_keep. */
int ovggt_k_compact(const void* k_src, const void* v_src, const int32_t* survivors, int32_t n_keep, int32_t C,
                    int32_t dtype, void* k_dst, void* v_dst, void* stream);

/* out [M, C] = softmax(Q K^T / sqrt(64)) V per head over N rows; head_dim 64.  bf16: tcgen05 kernel;
 * fp32: SIMT kernel.  scratch: device, >= ovggt_k_attention_scratch_bytes(M, N, n_heads). */
size_t ovggt_k_attention_scratch_bytes(int32_t M, int32_t N, int32_t n_heads);
int ovggt_k_attention(const void* q, const void* k, const void* v, int32_t M, int32_t N, int32_t n_heads,
                      int32_t dtype, void* out, void* scratch, int32_t* device_status, void* stream);

/* The bf16 attention with a fixed softmax reference where it is safe (see ovggt_cache_set_key_bound).
 * ovggt_k_key_norm_bound: kmax2 [n_heads] (device) = max over the rows of K [rows, n_heads * 64] (bf16) of the squared
 * norm of each head's 64 columns; n_heads <= 16.  ovggt_k_attention_bounded: as ovggt_k_attention for bf16, given such
 * a bound for (at least) the N keys it attends over; a bound that is too small voids the result. */
int ovggt_k_key_norm_bound(const void* K, int32_t rows, int32_t n_heads, float* kmax2, void* stream);
int ovggt_k_attention_bounded(const void* q, const void* k, const void* v, int32_t M, int32_t N, int32_t n_heads,
                              void* out, void* scratch, int32_t* device_status, const float* kmax2, void* stream);

/* Not a step of the paper's path: the dense products a model wraps around it (QKV and output projections, MLP), so
 * that the multi-layer workloads can run their scaffold on a hand-written tcgen05 kernel as well.
 * C [M, N] = A [M, K] x B [K, N], all bf16 row-major, fp32 accumulation, device pointers, 16-byte aligned; K must be a
 * multiple of 64 and N of 8 (OVGGT_ERR_UNSUPPORTED otherwise).  device_status: device int, as for ovggt_k_attention. */
int ovggt_k_gemm_bf16(const void* A, const void* B, int32_t M, int32_t N, int32_t K, void* C, int32_t* device_status,
                      void* stream);

#ifdef __cplusplus
}
#endif
#endif
