/*
 * CPU oracle for the OVGGT streaming global-attention step - TEST INFRASTRUCTURE ONLY.
 * See ovggt_oracle.h for what is pinned and what is not.  Plain loops, fp64, no
 * blocking, no fusion: each function is the paper's definition written out.
 */
#include "ovggt_oracle.h"

#include <algorithm>
#include <cmath>
#include <cstring>
#include <deque>
#include <limits>
#include <numeric>
#include <vector>

static int g_threads = 1;

extern "C" void orc_set_threads(int32_t n) { g_threads = n < 1 ? 1 : n; }
extern "C" int32_t orc_get_threads(void) { return g_threads; }

/* ------------------------------------------------------------------ Eq. 5 */
extern "C" void orc_residual_norms(const float* R, int32_t M, int32_t C, double* s) {
  for (int32_t j = 0; j < M; ++j) {
    double acc = 0.0;
    for (int32_t c = 0; c < C; ++c) {
      double x = (double)R[(size_t)j * C + c];
      acc += x * x;
    }
    s[j] = std::sqrt(acc);
  }
}

/* ------------------------------------------------------------------ Supp. D, query-key criterion */
extern "C" void orc_qk_scores(const float* Q, const float* K, int32_t M, int32_t n_heads, int32_t head_dim,
                              double* s) {
  const int32_t C = n_heads * head_dim;
  const double scale = 1.0 / std::sqrt((double)head_dim);
  for (int32_t j = 0; j < M; ++j) {
    double total = 0.0;
    for (int32_t h = 0; h < n_heads; ++h)
      for (int32_t i = 0; i < M; ++i) {
        double logit = 0.0;
        for (int32_t e = 0; e < head_dim; ++e)
          logit += (double)Q[(size_t)i * C + h * head_dim + e] * (double)K[(size_t)j * C + h * head_dim + e];
        total += logit * scale;
      }
    s[j] = total / ((double)M * (double)n_heads);
  }
}

/* ------------------------------------------------------------------ Eq. 6
 * G is the 3x3 Gaussian with sigma = 1, G[dy][dx] proportional to
 * exp(-(dx^2 + dy^2) / 2), normalised to sum 1.  Outside the map the nearest
 * map entry is used (replicate border), so a constant map stays constant. */
extern "C" void orc_smooth(const double* s, int32_t n_special, int32_t grid_h, int32_t grid_w,
                           double alpha, double* s_out) {
  for (int32_t j = 0; j < n_special; ++j) s_out[j] = s[j];
  double G[3][3];
  double total = 0.0;
  for (int dy = -1; dy <= 1; ++dy)
    for (int dx = -1; dx <= 1; ++dx) {
      G[dy + 1][dx + 1] = std::exp(-0.5 * (double)(dx * dx + dy * dy));
      total += G[dy + 1][dx + 1];
    }
  const double* S = s + n_special;
  for (int32_t y = 0; y < grid_h; ++y)
    for (int32_t x = 0; x < grid_w; ++x) {
      double conv = 0.0;
      for (int dy = -1; dy <= 1; ++dy)
        for (int dx = -1; dx <= 1; ++dx) {
          int32_t yy = std::min(std::max(y + dy, 0), grid_h - 1);
          int32_t xx = std::min(std::max(x + dx, 0), grid_w - 1);
          conv += (G[dy + 1][dx + 1] / total) * S[(size_t)yy * grid_w + xx];
        }
      double raw = S[(size_t)y * grid_w + x];
      s_out[n_special + (size_t)y * grid_w + x] = alpha * conv + (1.0 - alpha) * raw;
    }
}

/* ------------------------------------------------------------------ diversity
 * d_i = 1 - cos(k_i, kbar).  A zero vector has no direction: its cosine is taken as 0. */
static double cosine(const float* a, const double* b, int32_t len) {
  double dot = 0.0, na = 0.0, nb = 0.0;
  for (int32_t c = 0; c < len; ++c) {
    dot += (double)a[c] * b[c];
    na += (double)a[c] * (double)a[c];
    nb += b[c] * b[c];
  }
  if (na == 0.0 || nb == 0.0) return 0.0;
  return dot / (std::sqrt(na) * std::sqrt(nb));
}

extern "C" void orc_diversity(const float* K, int32_t n, int32_t C, int32_t n_heads,
                              int32_t per_head, double* d) {
  if (n <= 0) return;
  std::vector<double> kbar(C, 0.0);
  for (int32_t i = 0; i < n; ++i)
    for (int32_t c = 0; c < C; ++c) kbar[c] += (double)K[(size_t)i * C + c];
  for (int32_t c = 0; c < C; ++c) kbar[c] /= (double)n;
#pragma omp parallel for num_threads(g_threads) schedule(static)
  for (int32_t i = 0; i < n; ++i) {
    const float* ki = K + (size_t)i * C;
    if (!per_head) {
      d[i] = 1.0 - cosine(ki, kbar.data(), C);
    } else {
      int32_t hd = C / n_heads;
      double acc = 0.0;
      for (int32_t h = 0; h < n_heads; ++h) acc += cosine(ki + h * hd, kbar.data() + h * hd, hd);
      d[i] = 1.0 - acc / (double)n_heads;
    }
  }
}

/* ------------------------------------------------------------------ Eq. 7 */
static void minmax_group(const double* x, const uint8_t* flags, int32_t count, double weight,
                         float* r, double lone_value = 0.0) {
  double lo = std::numeric_limits<double>::infinity(), hi = -lo;
  int32_t members = 0;
  for (int32_t i = 0; i < count; ++i)
    if (flags[i] == ORC_FLAG_EVICTABLE) {
      lo = std::min(lo, x[i]);
      hi = std::max(hi, x[i]);
      ++members;
    }
  for (int32_t i = 0; i < count; ++i) {
    if (flags[i] != ORC_FLAG_EVICTABLE) {
      r[i] = std::numeric_limits<float>::infinity();
    } else {
      double hat = (members > 0 && hi > lo) ? (x[i] - lo) / (hi - lo) : 0.0;
      if (members == 1) hat = lone_value;   /* 0/0: a reading, 0 for the aggregator, 1 for the camera cache */
      r[i] = (float)(weight * hat);
    }
  }
}

extern "C" void orc_hybrid(const double* d, const double* s, const uint8_t* flags, int32_t n,
                           int32_t M, double beta, float* r) {
  minmax_group(d, flags, n, 1.0 - beta, r);
  minmax_group(s, flags + n, M, beta, r + n);
}

/* ------------------------------------------------------------------ random-eviction baseline (Supp. A) */
extern "C" uint64_t orc_splitmix64(uint64_t x) {
  uint64_t z = x + 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

extern "C" float orc_random_priority(uint64_t seed, int64_t frame_id, int64_t token_id) {
  const uint64_t step_key = orc_splitmix64(seed ^ (uint64_t)frame_id);
  const uint64_t bits = orc_splitmix64(step_key + (uint64_t)token_id);
  return (float)(bits >> 40) * (1.0f / 16777216.0f); /* 24 bits: exact in fp32, in [0, 1) */
}

/* ------------------------------------------------------------------ Eq. 8 */
/* Rank of a priority: NaN ranks with -inf (evicted first); -0 and +0 compare equal. */
static inline float rank_key(float x) {
  return std::isnan(x) ? -std::numeric_limits<float>::infinity() : x;
}

extern "C" int orc_select(const float* r, const uint8_t* flags, int32_t N, int32_t B,
                          int32_t* survivors, int32_t* n_out) {
  if (N <= B) {
    for (int32_t i = 0; i < N; ++i) survivors[i] = i;
    *n_out = N;
    return 0;
  }
  std::vector<int32_t> prot, evictable;
  for (int32_t i = 0; i < N; ++i) (flags[i] != ORC_FLAG_EVICTABLE ? prot : evictable).push_back(i);
  int64_t k = (int64_t)B - (int64_t)prot.size();
  if (k < 0) return -1;
  /* Stable sort by descending rank: equal ranks keep their order, i.e. lower position first. */
  std::stable_sort(evictable.begin(), evictable.end(),
                   [&](int32_t a, int32_t b) { return rank_key(r[a]) > rank_key(r[b]); });
  std::vector<int32_t> keep(prot);
  keep.insert(keep.end(), evictable.begin(), evictable.begin() + k);
  std::sort(keep.begin(), keep.end());
  for (size_t i = 0; i < keep.size(); ++i) survivors[i] = keep[i];
  *n_out = (int32_t)keep.size();
  return 0;
}

extern "C" void orc_top_conf(const float* conf, int32_t n, int32_t A, int32_t* idx) {
  std::vector<int32_t> order(n);
  std::iota(order.begin(), order.end(), 0);
  std::stable_sort(order.begin(), order.end(),
                   [&](int32_t a, int32_t b) { return rank_key(conf[a]) > rank_key(conf[b]); });
  std::vector<int32_t> top(order.begin(), order.begin() + std::min(A, n));
  std::sort(top.begin(), top.end());
  for (size_t i = 0; i < top.size(); ++i) idx[i] = top[i];
}

/* ------------------------------------------------------------------ attention
 * Dense softmax(Q K^T / sqrt(d)) V per head.  No mask: causality is between
 * frames, every cached row belongs to an earlier frame and the frame sees itself. */
extern "C" void orc_attention(const float* Q, const float* K, const float* V, int32_t M,
                              int32_t N, int32_t n_heads, int32_t head_dim, const int32_t* rows,
                              int32_t n_rows, float* out) {
  const int32_t C = n_heads * head_dim;
  if (rows == nullptr) n_rows = M;
  const double scale = 1.0 / std::sqrt((double)head_dim);
  const int64_t work = (int64_t)n_rows * n_heads;
#pragma omp parallel for num_threads(g_threads) schedule(dynamic, 4)
  for (int64_t w = 0; w < work; ++w) {
    const int32_t ri = (int32_t)(w / n_heads), h = (int32_t)(w % n_heads);
    const int32_t m = rows ? rows[ri] : ri;
    const float* q = Q + (size_t)m * C + (size_t)h * head_dim;
    std::vector<double> logit(N);
    double mx = -std::numeric_limits<double>::infinity();
    for (int32_t n = 0; n < N; ++n) {
      const float* kk = K + (size_t)n * C + (size_t)h * head_dim;
      double acc = 0.0;
      for (int32_t c = 0; c < head_dim; ++c) acc += (double)q[c] * (double)kk[c];
      logit[n] = acc * scale;
      mx = std::max(mx, logit[n]);
    }
    double denom = 0.0;
    for (int32_t n = 0; n < N; ++n) {
      logit[n] = std::exp(logit[n] - mx);
      denom += logit[n];
    }
    for (int32_t c = 0; c < head_dim; ++c) {
      double acc = 0.0;
      for (int32_t n = 0; n < N; ++n)
        acc += logit[n] * (double)V[(size_t)n * C + (size_t)h * head_dim + c];
      out[(size_t)ri * C + (size_t)h * head_dim + c] = (float)(acc / denom);
    }
  }
}

/* ------------------------------------------------------------------ Supp. D, attention-weight criterion */
extern "C" void orc_attention_received(const float* Q, const float* K, int32_t M, int32_t N, int32_t n_heads,
                                       int32_t head_dim, int32_t first_col, int32_t n_cols, double* s) {
  const int32_t C = n_heads * head_dim;
  const double scale = 1.0 / std::sqrt((double)head_dim);
  for (int32_t j = 0; j < n_cols; ++j) s[j] = 0.0;
  std::vector<double> p(N);
  for (int32_t h = 0; h < n_heads; ++h)
    for (int32_t i = 0; i < M; ++i) {
      /* row i of P_h, written out */
      double mx = -std::numeric_limits<double>::infinity();
      for (int32_t n = 0; n < N; ++n) {
        double acc = 0.0;
        for (int32_t c = 0; c < head_dim; ++c)
          acc += (double)Q[(size_t)i * C + h * head_dim + c] * (double)K[(size_t)n * C + h * head_dim + c];
        p[n] = acc * scale;
        mx = std::max(mx, p[n]);
      }
      double denom = 0.0;
      for (int32_t n = 0; n < N; ++n) {
        p[n] = std::exp(p[n] - mx);
        denom += p[n];
      }
      for (int32_t j = 0; j < n_cols; ++j) s[j] += p[first_col + j] / denom;
    }
  for (int32_t j = 0; j < n_cols; ++j) s[j] /= (double)M * (double)n_heads;
}

/* ------------------------------------------------------------------ state */
struct orc_state {
  orc_config cfg;
  int32_t M, C;
  std::vector<int64_t> ids;
  std::vector<uint8_t> flags;
  std::vector<float> stored;   /* smoothed activation score each row had when it was new */
  std::vector<float> k, v;     /* [rows, C] */
  std::vector<float> q_frame;  /* [M, C] queries of the pending frame (ORC_SCORE_QK only) */
  std::vector<double> received; /* [M] attention the pending frame's tokens receive (ORC_SCORE_ATTN only) */
  std::deque<int64_t> anchors; /* active historical anchor frames, oldest first */
  int64_t first_frame = -1, last_frame = -1, last_registration = -1;
  int64_t evicted_total = 0;
  bool pending = false;        /* a frame was appended and not yet compressed */
};

extern "C" orc_state* orc_create(const orc_config* cfg) {
  if (!cfg || cfg->n_heads < 1 || cfg->head_dim < 1 || cfg->n_special < 0 || cfg->anchor_tokens < 0 ||
      cfg->k_max < 0)
    return nullptr;
  if (cfg->camera_cache) {
    /* Supp. C: one camera token per frame, nothing else */
    if (cfg->n_special != 1 || cfg->grid_h != 0 || cfg->grid_w != 0 || cfg->anchor_tokens != 0) return nullptr;
  } else if (cfg->grid_h < 1 || cfg->grid_w < 1 || cfg->anchor_tokens > cfg->grid_h * cfg->grid_w) {
    return nullptr;
  }
  if (cfg->camera_cache && (cfg->score_mode == ORC_SCORE_QK || cfg->score_mode == ORC_SCORE_ATTN))
    return nullptr; /* the probe concerns the aggregator */
  const int64_t M = cfg->n_special + (int64_t)cfg->grid_h * cfg->grid_w;
  /* Eq. 9: the protected set can reach M + K_max * A; the budget must hold it.  (Camera cache: an anchor is the
   * frame's one token.) */
  const int64_t per_anchor = cfg->camera_cache ? 1 : cfg->anchor_tokens;
  const int64_t pmax = (cfg->protect_first_frame ? M : 0) + (int64_t)cfg->k_max * per_anchor;
  if (cfg->budget < M || cfg->budget < pmax) return nullptr;
  orc_state* st = new orc_state();
  st->cfg = *cfg;
  st->M = (int32_t)M;
  st->C = cfg->n_heads * cfg->head_dim;
  return st;
}

extern "C" void orc_destroy(orc_state* st) { delete st; }
extern "C" int32_t orc_num_rows(const orc_state* st) { return (int32_t)st->ids.size(); }
extern "C" int64_t orc_evicted_total(const orc_state* st) { return st->evicted_total; }

extern "C" int32_t orc_num_protected(const orc_state* st, int32_t* n_init, int32_t* n_hist) {
  int32_t a = 0, b = 0;
  for (uint8_t f : st->flags) {
    a += f == ORC_FLAG_INIT;
    b += f == ORC_FLAG_HIST;
  }
  if (n_init) *n_init = a;
  if (n_hist) *n_hist = b;
  return a + b;
}

extern "C" int32_t orc_active_anchors(const orc_state* st, int64_t* frames) {
  int32_t i = 0;
  for (int64_t f : st->anchors) {
    if (frames) frames[i] = f;
    ++i;
  }
  return i;
}

extern "C" int orc_attend(orc_state* st, int64_t frame_id, const float* q, const float* k,
                          const float* v, const int32_t* rows, int32_t n_rows, float* out) {
  if (st->pending) return -2;                 /* previous frame was never compressed */
  if (frame_id <= st->last_frame) return -3;  /* frames arrive in increasing order */
  const int32_t M = st->M, C = st->C;
  /* Eq. 2: C_t = [C_{t-1}; (K_t, V_t)] */
  for (int32_t j = 0; j < M; ++j) {
    st->ids.push_back(frame_id * (int64_t)M + j);
    st->flags.push_back(ORC_FLAG_EVICTABLE);
    st->stored.push_back(0.0f);
  }
  st->k.insert(st->k.end(), k, k + (size_t)M * C);
  st->v.insert(st->v.end(), v, v + (size_t)M * C);
  if (st->cfg.score_mode == ORC_SCORE_QK) st->q_frame.assign(q, q + (size_t)M * C);
  if (st->cfg.score_mode == ORC_SCORE_ATTN) { /* columns of the frame's own tokens in this very attention */
    const int32_t N = (int32_t)st->ids.size();
    st->received.assign(M, 0.0);
    orc_attention_received(q, st->k.data(), M, N, st->cfg.n_heads, st->cfg.head_dim, N - M, M, st->received.data());
  }
  if (st->first_frame < 0) {
    st->first_frame = frame_id;
    st->last_registration = frame_id; /* the first frame is the initial anchor */
  }
  st->last_frame = frame_id;
  st->pending = true;
  if (out)
    orc_attention(q, st->k.data(), st->v.data(), M, (int32_t)st->ids.size(), st->cfg.n_heads,
                  st->cfg.head_dim, rows, n_rows, out);
  return 0;
}

/* Budgeted retention (Eq. 8) and order-preserving compaction, given the priorities r [N]. */
static int select_and_compact(orc_state* st, const std::vector<float>& r, int32_t* survivors,
                              int32_t* n_survivors) {
  const int32_t C = st->C, N = (int32_t)st->ids.size();
  std::vector<int32_t> keep(N);
  int32_t n_keep = 0;
  if (orc_select(r.data(), st->flags.data(), N, st->cfg.budget, keep.data(), &n_keep) != 0) return -4;
  std::vector<int64_t> ids(n_keep);
  std::vector<uint8_t> flags(n_keep);
  std::vector<float> stored(n_keep), kk((size_t)n_keep * C), vv((size_t)n_keep * C);
  for (int32_t j = 0; j < n_keep; ++j) {
    const int32_t src = keep[j];
    ids[j] = st->ids[src];
    flags[j] = st->flags[src];
    stored[j] = st->stored[src];
    std::memcpy(&kk[(size_t)j * C], &st->k[(size_t)src * C], sizeof(float) * C);
    std::memcpy(&vv[(size_t)j * C], &st->v[(size_t)src * C], sizeof(float) * C);
  }
  st->evicted_total += N - n_keep;
  st->ids.swap(ids);
  st->flags.swap(flags);
  st->stored.swap(stored);
  st->k.swap(kk);
  st->v.swap(vv);
  st->pending = false;
  if (survivors) std::memcpy(survivors, keep.data(), sizeof(int32_t) * n_keep);
  if (n_survivors) *n_survivors = n_keep;
  return 0;
}

extern "C" int orc_compress(orc_state* st, const float* resid, const float* conf, double rho,
                            const float* score_override, float* r_out, int32_t* survivors,
                            int32_t* n_survivors, int32_t* registered, int64_t* demoted_frame) {
  if (!st->pending) return -2;
  const orc_config& cfg = st->cfg;
  const int32_t M = st->M, C = st->C;
  const int32_t N = (int32_t)st->ids.size(), n = N - M;
  const int64_t t = st->last_frame;

  /* Activation Value Rating (Eq. 5) and smoothing (Eq. 6) of the new frame. */
  std::vector<double> s(M), s_smooth(M);
  if (cfg.score_mode == ORC_SCORE_QK) /* Supp. D: the frame's queries against its own keys instead of Eq. 5 */
    orc_qk_scores(st->q_frame.data(), &st->k[(size_t)n * C], M, cfg.n_heads, cfg.head_dim, s.data());
  else if (cfg.score_mode == ORC_SCORE_ATTN) /* Supp. D: the attention the new tokens received */
    s = st->received;
  else
    orc_residual_norms(resid, M, C, s.data());
  orc_smooth(s.data(), cfg.n_special, cfg.grid_h, cfg.grid_w, cfg.alpha, s_smooth.data());
  for (int32_t j = 0; j < M; ++j) st->stored[n + j] = (float)s_smooth[j];

  /* Dynamic Anchor Protection (Sec. 3.3). */
  int32_t did_register = 0;
  int64_t demoted = -1;
  if (t == st->first_frame) {
    if (cfg.protect_first_frame)
      for (int32_t j = 0; j < M; ++j) st->flags[n + j] = ORC_FLAG_INIT;
  } else if (cfg.anchor_tokens > 0 && cfg.k_max > 0 && conf != nullptr && rho < cfg.tau &&
             t - st->last_registration >= cfg.min_anchor_interval) {
    std::vector<int32_t> top(cfg.anchor_tokens);
    orc_top_conf(conf, cfg.grid_h * cfg.grid_w, cfg.anchor_tokens, top.data());
    for (int32_t p : top) st->flags[n + cfg.n_special + p] = ORC_FLAG_HIST;
    st->anchors.push_back(t);
    st->last_registration = t;
    did_register = 1;
    if ((int32_t)st->anchors.size() > cfg.k_max) {
      demoted = st->anchors.front();
      st->anchors.pop_front();
      for (int32_t i = 0; i < N; ++i)
        if (st->flags[i] == ORC_FLAG_HIST && st->ids[i] / M == demoted)
          st->flags[i] = ORC_FLAG_EVICTABLE;
    }
  }

  /* Priorities (Eq. 7), or the stored-residual reading. */
  std::vector<float> r(N);
  if (cfg.score_mode == ORC_SCORE_HYBRID || cfg.score_mode == ORC_SCORE_QK || cfg.score_mode == ORC_SCORE_ATTN) {
    std::vector<double> d(std::max(n, 1));
    orc_diversity(st->k.data(), n, C, cfg.n_heads, cfg.diversity_per_head, d.data());
    orc_hybrid(d.data(), s_smooth.data(), st->flags.data(), n, M, cfg.beta, r.data());
  } else if (cfg.score_mode == ORC_SCORE_RANDOM) {
    for (int32_t i = 0; i < N; ++i)
      r[i] = st->flags[i] != ORC_FLAG_EVICTABLE ? std::numeric_limits<float>::infinity()
                                                : orc_random_priority(cfg.random_seed, t, st->ids[i]);
  } else {
    for (int32_t i = 0; i < N; ++i)
      r[i] = st->flags[i] != ORC_FLAG_EVICTABLE ? std::numeric_limits<float>::infinity()
                                                : st->stored[i];
  }
  if (score_override)
    for (int32_t i = 0; i < N; ++i)
      if (st->flags[i] == ORC_FLAG_EVICTABLE) r[i] = score_override[i];
  if (r_out) std::memcpy(r_out, r.data(), sizeof(float) * N);

  int rc = select_and_compact(st, r, survivors, n_survivors);
  if (rc != 0) return rc;
  if (registered) *registered = did_register;
  if (demoted_frame) *demoted_frame = demoted;
  return 0;
}

/* ------------------------------------------------------------------ Supp. C: the camera head's cache */
extern "C" int orc_compress_camera(orc_state* st, const float* resid, int32_t registered,
                                   int64_t demoted_frame, const float* score_override, float* r_out,
                                   int32_t* survivors, int32_t* n_survivors) {
  if (!st->pending) return -2;
  const orc_config& cfg = st->cfg;
  if (!cfg.camera_cache || st->M != 1) return -5;
  const int32_t C = st->C;
  const int32_t N = (int32_t)st->ids.size(), n = N - 1;
  const int64_t t = st->last_frame;

  /* Activation Value Rating (Eq. 5) of the frame's one token; there is no map to smooth (Eq. 6 does not apply). */
  double s = 0.0;
  orc_residual_norms(resid, 1, C, &s);
  st->stored[n] = (float)s;

  /* Protection follows the aggregator's decision for this frame (Sec. 3.3 applied there, mirrored here). */
  if (t == st->first_frame) {
    if (cfg.protect_first_frame) st->flags[n] = ORC_FLAG_INIT;
  } else if (registered) {
    st->flags[n] = ORC_FLAG_HIST;
    st->anchors.push_back(t);
    st->last_registration = t;
  }
  if (demoted_frame >= 0) {
    for (int32_t i = 0; i < N; ++i)
      if (st->flags[i] == ORC_FLAG_HIST && st->ids[i] == demoted_frame) st->flags[i] = ORC_FLAG_EVICTABLE;
    for (auto it = st->anchors.begin(); it != st->anchors.end(); ++it)
      if (*it == demoted_frame) {
        st->anchors.erase(it);
        break;
      }
  }

  std::vector<float> r(N);
  if (cfg.score_mode == ORC_SCORE_HYBRID) {
    std::vector<double> d(std::max(n, 1));
    orc_diversity(st->k.data(), n, C, cfg.n_heads, cfg.diversity_per_head, d.data());
    minmax_group(d.data(), st->flags.data(), n, 1.0 - cfg.beta, r.data());
    minmax_group(&s, st->flags.data() + n, 1, cfg.beta, r.data() + n, /*lone_value=*/1.0);
  } else {
    for (int32_t i = 0; i < N; ++i)
      r[i] = st->flags[i] != ORC_FLAG_EVICTABLE ? std::numeric_limits<float>::infinity()
                                                : st->stored[i];
  }
  if (score_override)
    for (int32_t i = 0; i < N; ++i)
      if (st->flags[i] == ORC_FLAG_EVICTABLE) r[i] = score_override[i];
  if (r_out) std::memcpy(r_out, r.data(), sizeof(float) * N);
  return select_and_compact(st, r, survivors, n_survivors);
}

extern "C" void orc_export(const orc_state* st, int64_t* ids, uint8_t* flags, float* stored,
                           float* k, float* v) {
  const size_t n = st->ids.size();
  if (ids) std::memcpy(ids, st->ids.data(), n * sizeof(int64_t));
  if (flags) std::memcpy(flags, st->flags.data(), n);
  if (stored) std::memcpy(stored, st->stored.data(), n * sizeof(float));
  if (k) std::memcpy(k, st->k.data(), n * st->C * sizeof(float));
  if (v) std::memcpy(v, st->v.data(), n * st->C * sizeof(float));
}

extern "C" double orc_full_cache_elements(int32_t L, int64_t T, int32_t M, int32_t n_heads,
                                          int32_t head_dim) {
  return 2.0 * (double)L * (double)T * (double)M * (double)n_heads * (double)head_dim;
}
