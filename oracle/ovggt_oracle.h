/*
 * CPU oracle for the OVGGT streaming global-attention step.
 *
 * TEST INFRASTRUCTURE ONLY.  This is a plain, slow, obviously-correct CPU
 * statement of what one (frame, layer) step computes, written from the paper.
 * It shares no code with the CUDA library and must never be called from the
 * product path; only the tests, the smoke check and the benchmark's CPU
 * baseline use it.
 *
 * All arithmetic is fp64 on inputs that were already rounded to the stream's
 * storage type (the float arrays passed in hold exactly the values the GPU
 * receives).  The one place a floating-point value decides an integer - the
 * budgeted selection - compares fp32 keys, the precision the CUDA selection
 * kernel uses: the fp64 priority is rounded once to fp32 and ranked from there.
 *
 * Pins (see the CPU tests): attention against an independent dense softmax,
 * selection against a brute-force sort, smoothing / diversity / min-max
 * against closed forms and special cases, anchor FIFO against a hand-written
 * schedule, the budget and protected-size invariants (Eq. 8, Eq. 9), and the
 * full-cache footprint formula of Sec. 3.1; the camera-head cache against the aggregator's anchor schedule and
 * closed forms of its two differences.
 * Parity unpinned: the reconstruction accuracy the paper reports for the
 * method (needs its datasets and trained weights).
 */
#ifndef OVGGT_ORACLE_H_
#define OVGGT_ORACLE_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum { ORC_FLAG_EVICTABLE = 0, ORC_FLAG_INIT = 1, ORC_FLAG_HIST = 2 };
enum { ORC_SCORE_HYBRID = 0, ORC_SCORE_RESIDUAL_STORED = 1, ORC_SCORE_RANDOM = 2, ORC_SCORE_QK = 3, ORC_SCORE_ATTN = 4 };

typedef struct {
  int32_t n_heads, head_dim;             /* C = n_heads * head_dim */
  int32_t n_special, grid_h, grid_w;     /* M = n_special + grid_h * grid_w (Sec. 3.1) */
  int32_t budget;                        /* B^(l), tokens (Eq. 8) */
  int32_t anchor_tokens;                 /* ceil(eta * N_p): protected patch tokens per historical anchor */
  int32_t k_max, min_anchor_interval;    /* K_max, frames between registrations (Sec. 3.3) */
  double tau, alpha, beta;               /* coverage threshold, smoothing strength, hybrid balance */
  int32_t protect_first_frame;           /* Global Initial Anchor on/off */
  int32_t score_mode;                    /* ORC_SCORE_* */
  int32_t diversity_per_head;            /* 0: cosine on the whole C-vector; 1: mean over heads of per-head cosine */
  int32_t camera_cache;                  /* 1: the camera head's cache (Supp. C): one token per frame, grid 0 x 0 */
  uint64_t random_seed;                  /* ORC_SCORE_RANDOM: seed of the per-step uniform priorities */
} orc_config;

typedef struct orc_state orc_state;

/* ---- the pieces, each a pure function (so each can be pinned on its own) ---- */

/* Eq. 5: s_j = || r_j ||_2 for the M rows of R [M, C]. */
void orc_residual_norms(const float* R, int32_t M, int32_t C, double* s);

/* The query-key baseline of the scoring probe (Supp. D): the current-frame criterion is replaced by a dot product
 * of queries and keys that needs no attention matrix.  The paper gives no formula; the reading taken here is the
 * mean, over the frame's M queries and the heads, of the scaled attention logit that new token j receives:
 *   s_j = 1 / (M * n_heads) * sum_h sum_i  (q_{i,h} . k_{j,h}) / sqrt(head_dim),
 * Q, K [M, C] being the frame's own queries and keys.  Everything after the criterion (Eq. 6, Eq. 7 with the key
 * diversity of the cached rows, Eq. 8) is as in the hybrid mode; the residual is not used. */
void orc_qk_scores(const float* Q, const float* K, int32_t M, int32_t n_heads, int32_t head_dim, double* s);

/* The attention-weight baseline of the scoring probe (Supp. D): the criterion that needs the materialised attention
 * matrix.  Reading taken here (the paper prints no formula): the importance of a token is the attention it receives,
 * averaged over the frame's M queries and the heads,
 *   s_j = 1 / (M * n_heads) * sum_h sum_i P_h[i, first_col + j],   P_h = softmax(Q_h K_h^T / sqrt(head_dim)) over all N rows,
 * for the n_cols columns from first_col on.  Q [M, C]; K [N, C].  (Over all N columns the s_j add up to 1.) */
void orc_attention_received(const float* Q, const float* K, int32_t M, int32_t N, int32_t n_heads, int32_t head_dim,
                            int32_t first_col, int32_t n_cols, double* s);

/* Eq. 6: patch part of s (after the first n_special entries) as a grid_h x grid_w
 * map, smoothed with a 3x3 Gaussian (sigma = 1, replicate border); aux tokens copied. */
void orc_smooth(const double* s, int32_t n_special, int32_t grid_h, int32_t grid_w,
                double alpha, double* s_out);

/* Sec. 3.2, Hybrid Scoring: d_i = 1 - cos(k_i, kbar), kbar = mean of the n rows of K [n, C]. */
void orc_diversity(const float* K, int32_t n, int32_t C, int32_t n_heads, int32_t per_head,
                   double* d);

/* Eq. 7: independent min-max over the evictable historical rows (first n entries,
 * values d) and the evictable new rows (next M entries, values s); protected rows
 * (flags != 0) take no part and get +inf.  r is fp32 [n + M]. */
void orc_hybrid(const double* d, const double* s, const uint8_t* flags, int32_t n, int32_t M,
                double beta, float* r);

/* The random-eviction baseline of the paper's full-cache comparison (Supp. A): under the same budget, the rows that
 * leave are drawn uniformly at random.  Here: every evictable row gets a fresh uniform priority in [0, 1) per step
 * and Eq. 8 keeps the largest, which is a uniformly random subset.  The priority of token `token_id` in the step
 * of frame `frame_id` is a counter-based value, so that both sides of a parity test can compute it:
 *   u = top 24 bits of SplitMix64(SplitMix64(seed ^ frame_id) + token_id), scaled by 2^-24,
 * SplitMix64(x) being one output step of that generator from state x (Steele, Lea, Flood 2014):
 *   z = x + 0x9E3779B97F4A7C15; z = (z ^ z >> 30) * 0xBF58476D1CE4E5B9; z = (z ^ z >> 27) * 0x94D049BB133111EB; z ^ z >> 31. */
uint64_t orc_splitmix64(uint64_t x);
float orc_random_priority(uint64_t seed, int64_t frame_id, int64_t token_id);

/* Eq. 8: keep every protected row and the (B - |P|) evictable rows of largest r;
 * ties go to the lower position, NaN ranks with -inf.  Returns the survivor
 * positions in ascending order; n_out = min(N, B).  Returns -1 if |P| > B. */
int orc_select(const float* r, const uint8_t* flags, int32_t N, int32_t B,
               int32_t* survivors, int32_t* n_out);

/* Indices of the A largest entries of conf [n] (ties -> lower index, NaN ranks with -inf), ascending. */
void orc_top_conf(const float* conf, int32_t n, int32_t A, int32_t* idx);

/* softmax(Q_h K_h^T / sqrt(d)) V_h for the listed query rows (rows == NULL: all M).
 * Q [M, C]; K, V [N, C]; out [n_rows, C]; token-major, head h owns columns [h*d, (h+1)*d). */
void orc_attention(const float* Q, const float* K, const float* V, int32_t M, int32_t N,
                   int32_t n_heads, int32_t head_dim, const int32_t* rows, int32_t n_rows,
                   float* out);

/* ---- the streaming state of one layer ---- */

orc_state* orc_create(const orc_config* cfg);      /* NULL on an invalid config */
void orc_destroy(orc_state* st);
void orc_set_threads(int32_t n);                   /* OpenMP threads used by the loops (default 1) */
int32_t orc_get_threads(void);

int32_t orc_num_rows(const orc_state* st);
int32_t orc_num_protected(const orc_state* st, int32_t* n_init, int32_t* n_hist);
int32_t orc_active_anchors(const orc_state* st, int64_t* frames /* [k_max] */);
int64_t orc_evicted_total(const orc_state* st);

/* Eq. 2 then the layer's attention: append the frame's M rows (ids frame_id*M + j),
 * then attend the listed query rows over all n + M rows.  out may be NULL (append only). */
int orc_attend(orc_state* st, int64_t frame_id, const float* q, const float* k, const float* v,
               const int32_t* rows, int32_t n_rows, float* out);

/* Score, protect, select, compact (Eq. 5-8, Sec. 3.3) for the frame appended by the
 * last orc_attend.  conf may be NULL (no anchor candidate).  score_override, if not
 * NULL, replaces the computed priorities of evictable rows verbatim.
 * Outputs (each may be NULL): r_out [N] priorities as ranked (+inf on protected rows);
 * survivors [min(N, B)] ascending positions in the pre-compaction buffer; n_survivors;
 * registered = 1 if this frame became a historical anchor; demoted_frame = frame id of
 * the anchor released by the FIFO, or -1. */
int orc_compress(orc_state* st, const float* resid, const float* conf, double rho,
                 const float* score_override, float* r_out, int32_t* survivors,
                 int32_t* n_survivors, int32_t* registered, int64_t* demoted_frame);

/* Supp. C: the camera prediction head keeps one token per frame in a cache of its own, managed by the same scoring
 * and protection with two differences: there is no patch map, hence no smoothing (the stored score is the raw
 * residual norm), and the anchor flags are not decided here but follow the aggregator's decision for the same frame:
 * registered != 0 protects this frame's token as a historical anchor, demoted_frame >= 0 releases that frame's token.
 * Eq. 7's min-max of the new group has a single member (0/0): its normalised score is taken as 1, so the token ranks
 * at beta (with 0 it would tie with the least diverse cached token, lose by position and never enter the cache).
 * For a state created with camera_cache = 1 (n_special = 1, grid 0 x 0, anchor_tokens 0; the budget must hold
 * 1 + k_max tokens).  Other arguments as orc_compress. */
int orc_compress_camera(orc_state* st, const float* resid, int32_t registered, int64_t demoted_frame,
                        const float* score_override, float* r_out, int32_t* survivors,
                        int32_t* n_survivors);

/* Current layout, ascending token id.  Any pointer may be NULL. */
void orc_export(const orc_state* st, int64_t* ids, uint8_t* flags, float* stored, float* k, float* v);

/* Sec. 3.1: elements held by an uncompressed cache after T frames, 2*L*T*M*N_h*d. */
double orc_full_cache_elements(int32_t L, int64_t T, int32_t M, int32_t n_heads, int32_t head_dim);

#ifdef __cplusplus
}
#endif
#endif
