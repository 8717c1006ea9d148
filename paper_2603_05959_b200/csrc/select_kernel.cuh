// Budgeted selection (Eq. 8) as a radix select over a thread-block cluster, and the fused per-step kernel
// that prepares its input: anchor flags (Sec. 3.3), activation smoothing (Eq. 6), hybrid priorities (Eq. 7).
//
// A cluster of up to 8 CTAs x 1024 threads splits the N candidates into contiguous position ranges, one per
// CTA, held in that CTA's shared memory.  Protected rows get the largest possible key, so "every protected
// row plus the B - |P| best evictable rows" is simply "the B largest keys"; ties at the threshold are
// admitted in position order, so the result is unique.  The B-th largest key is found with four 8-bit
// most-significant-digit passes; per-CTA digit histograms and counts are combined through distributed
// shared memory with one cluster barrier per pass.
#pragma once

#include <cooperative_groups.h>

#include "common.cuh"

namespace ovggt {

namespace cg = cooperative_groups;

constexpr int kSelectThreads = 512;   // 512 x 64 registers: half an SM, so a CTA fits beside an attention CTA
constexpr int kSelectMaxCtas = 8;
constexpr uint32_t kKeyProtected = 0xFFFFFFFFu;   // above the key of +inf (0xFF800000)

struct SelectShared {
  int hist[2][256];          // this CTA's digit histogram, double-buffered across passes (read by the cluster)
  int tot[256];              // cluster-wide digit counts of the current pass
  int scan[64];
  float fscan[64];
  int digit, krem;
  int pub_gt, pub_eq;        // this CTA's counts of keys above / equal to the threshold, read by the cluster
  float pub_lo_h, pub_hi_h, pub_lo_n, pub_hi_n;
  int all_gt[kSelectMaxCtas], all_eq[kSelectMaxCtas];   // the whole cluster's counts, gathered by one warp
  int pub_up, pub_down;      // hole filling: survivors above the low range / evicted rows inside it, this CTA
  int all_up[kSelectMaxCtas], all_down[kSelectMaxCtas];
  float mm[4];               // cluster-wide lo_h, hi_h, lo_n, hi_n
};

// Range of positions owned by CTA `rank` when N positions are split over `ncta` CTAs.
__device__ __forceinline__ void cta_range(int N, int ncta, int rank, int* begin, int* end) {
  const int span = (N + ncta - 1) / ncta;
  *begin = min(N, rank * span);
  *end = min(N, *begin + span);
}

// Warp 0 finds the digit whose bin holds the krem-th largest remaining key, given bin counts tot[256].
__device__ __noinline__ void find_digit(const int* tot, int krem, SelectShared* sh) {
  const int tid = threadIdx.x;
  if (tid < 32) {
    int c[8], local = 0;
#pragma unroll
    for (int b = 0; b < 8; ++b) {
      c[b] = tot[tid * 8 + b];
      local += c[b];
    }
    int above = local;   // inclusive suffix sum over lanes: keys in this lane's bins and in all higher bins
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_down_sync(0xFFFFFFFFu, above, o);
      if (tid + o < 32) above += y;
    }
    int cum = above - local;
#pragma unroll
    for (int b = 7; b >= 0; --b) {
      if (cum < krem && cum + c[b] >= krem) {
        sh->digit = tid * 8 + b;
        sh->krem = krem - cum;
      }
      cum += c[b];
    }
  }
}

// Digit histogram of the keys that match (mask, prefix).  Keys of one step share their leading bits, so lanes
// of a warp mostly hit the same bin: lanes with equal digits are grouped and one of them adds the group's count.
__device__ __noinline__ void digit_histogram(const uint32_t* keys, int cnt, uint32_t mask, uint32_t prefix,
                                                int shift, int* hist) {
  const int tid = threadIdx.x, nthr = blockDim.x;
  for (int i0 = 0; i0 < cnt; i0 += nthr) {
    const int i = i0 + tid;
    int digit = -1;
    if (i < cnt) {
      const uint32_t key = keys[i];
      if ((key & mask) == prefix) digit = (int)((key >> shift) & 255u);
    }
    const unsigned peers = __match_any_sync(0xFFFFFFFFu, digit);
    if (digit >= 0 && (int)(__ffs(peers) - 1) == (tid & 31)) atomicAdd(&hist[digit], __popc(peers));
  }
}

// keys[0 .. cnt): this CTA's keys for positions [begin, begin + cnt).  Finds the B largest keys of the whole
// cluster (ties by position), writes the surviving global positions, ascending, to survivors[] and marks the
// kept local positions in keep[] (cnt bytes).  Returns the cluster-wide survivor count, min(N, B).
// *my_base receives the index in survivors[] of this CTA's first survivor.
__device__ inline int cluster_select(cg::cluster_group& cluster, const uint32_t* keys, uint8_t* keep, int begin,
                                     int cnt, int N, int B, int* survivors, SelectShared* sh, int* my_base,
                                     int* bad) {
  const int tid = threadIdx.x, nthr = blockDim.x;
  const int ncta = (int)cluster.num_blocks(), rank = (int)cluster.block_rank();
  const bool keep_all = N <= B;
  uint32_t T = 0;
  int need_eq = 0;
  if (!keep_all) {
    uint32_t prefix = 0, mask = 0;
    int krem = B;
    int buf = 0;
#pragma unroll 1
    for (int shift = 24; shift >= 0; shift -= 8, buf ^= 1) {
      int* hist = sh->hist[buf];
      for (int b = tid; b < 256; b += nthr) hist[b] = 0;
      __syncthreads();
      digit_histogram(keys, cnt, mask, prefix, shift, hist);
      cluster.sync();
      // every CTA folds all histograms and finds the same digit
      if (tid < 256) {
        int v[kSelectMaxCtas];
#pragma unroll
        for (int r = 0; r < kSelectMaxCtas; ++r)      // all remote loads in flight before the first add
          v[r] = r < ncta ? cluster.map_shared_rank(hist, r)[tid] : 0;
        int t = 0;
#pragma unroll
        for (int r = 0; r < kSelectMaxCtas; ++r) t += v[r];
        sh->tot[tid] = t;
      }
      __syncthreads();
      find_digit(sh->tot, krem, sh);
      __syncthreads();
      prefix |= (uint32_t)sh->digit << shift;
      mask |= 255u << shift;
      krem = sh->krem;
    }
    T = prefix;
    need_eq = krem;
  }
  // Thread t owns the contiguous local positions [t*chunk, (t+1)*chunk).
  const int chunk = (cnt + nthr - 1) / nthr;
  const int lo = min(cnt, tid * chunk), hi = min(cnt, lo + chunk);
  // One exchange settles everything: with (keys above T, keys equal to T) of every CTA, each CTA knows how
  // many of its ties are admitted (ties go to the lower position, i.e. to the lower rank first) and where its
  // survivors start in the output.
  int cnt_gt = 0, cnt_eq = 0;
  if (keep_all) {
    cnt_gt = hi - lo;
  } else {
    for (int i = lo; i < hi; ++i) {
      const uint32_t key = keys[i];
      cnt_gt += key > T;
      cnt_eq += key == T;
    }
  }
  int gt_total, eq_total;
  block_excl_scan_int(cnt_gt, sh->scan, &gt_total);
  int eq_rank = block_excl_scan_int(cnt_eq, sh->scan, &eq_total);   // ties before this thread's, within the CTA
  if (tid == 0) {
    sh->pub_gt = gt_total;
    sh->pub_eq = eq_total;
  }
  cluster.sync();
  if (tid < ncta) {                                   // one remote read per lane instead of ncta per thread
    sh->all_gt[tid] = *cluster.map_shared_rank(&sh->pub_gt, tid);
    sh->all_eq[tid] = *cluster.map_shared_rank(&sh->pub_eq, tid);
  }
  __syncthreads();
  int before = 0, all = 0, eq_before = 0, eq_all = 0;
  for (int r = 0; r < ncta; ++r) {
    const int e = sh->all_eq[r], gcount = sh->all_gt[r];
    const int adm = keep_all ? 0 : max(0, min(e, need_eq - eq_all));   // ties of rank r that are admitted
    if (r < rank) {
      before += gcount + adm;
      eq_before += e;
    }
    all += gcount + adm;
    eq_all += e;
  }
  eq_rank += eq_before;
  // more protected rows than the budget holds: only the first B of them can stay
  *bad = (!keep_all && T == kKeyProtected && eq_all > need_eq) ? 1 : 0;
  int cnt_keep = 0;
  for (int i = lo; i < hi; ++i) {
    bool k = true;
    if (!keep_all) {
      const uint32_t key = keys[i];
      k = key > T || (key == T && eq_rank++ < need_eq);
    }
    keep[i] = k ? 1 : 0;
    cnt_keep += k;
  }
  int keep_total;
  int base = block_excl_scan_int(cnt_keep, sh->scan, &keep_total);
  *my_base = before;
  base += before;
  for (int i = lo; i < hi; ++i)
    if (keep[i]) survivors[base++] = begin + i;
  __syncthreads();
  return all;
}

// Single-CTA pick used for the small top-A choice over the confidence map: marks the A largest of cnt keys
// in keep[], ties to the lower index.
__device__ inline void block_top_mark(const uint32_t* keys, uint8_t* keep, int cnt, int A, SelectShared* sh) {
  const int tid = threadIdx.x, nthr = blockDim.x;
  const bool keep_all = cnt <= A;
  uint32_t T = 0;
  int need_eq = 0;
  if (!keep_all && A > 0) {
    uint32_t prefix = 0, mask = 0;
    int krem = A;
#pragma unroll 1
    for (int shift = 24; shift >= 0; shift -= 8) {
      for (int b = tid; b < 256; b += nthr) sh->tot[b] = 0;
      __syncthreads();
      digit_histogram(keys, cnt, mask, prefix, shift, sh->tot);
      __syncthreads();
      find_digit(sh->tot, krem, sh);
      __syncthreads();
      prefix |= (uint32_t)sh->digit << shift;
      mask |= 255u << shift;
      krem = sh->krem;
      __syncthreads();
    }
    T = prefix;
    need_eq = krem;
  }
  const int chunk = (cnt + nthr - 1) / nthr;
  const int lo = min(cnt, tid * chunk), hi = min(cnt, lo + chunk);
  int cnt_eq = 0;
  if (!keep_all && A > 0)
    for (int i = lo; i < hi; ++i) cnt_eq += keys[i] == T;
  int tot;
  int eq_rank = block_excl_scan_int(cnt_eq, sh->scan, &tot);
  for (int i = lo; i < hi; ++i) {
    bool k = keep_all;
    if (!keep_all && A > 0) k = keys[i] > T || (keys[i] == T && eq_rank++ < need_eq);
    keep[i] = k ? 1 : 0;
  }
  __syncthreads();
}

// Shared memory a CTA of the selection kernels needs for `span` owned positions (+ np confidence entries).
__host__ __device__ inline size_t select_smem_bytes(int span, int np) {
  return ((sizeof(SelectShared) + 15) & ~(size_t)15) + (size_t)span * 4 + 2 * (((size_t)span + 15) & ~(size_t)15) +
         (size_t)np * 4 + (((size_t)np + 15) & ~(size_t)15) + 16;
}

// The fused per-step kernel also keeps the ids, stored scores and physical slots of its positions (16 bytes each)
// and the frame's raw residual norms (m floats) on chip.
__host__ __device__ inline size_t compress_smem_bytes(int span, int np, int m) {
  return select_smem_bytes(span, np) + (((size_t)span * 8 + 15) & ~(size_t)15) +
         2 * (((size_t)span * 4 + 15) & ~(size_t)15) + (((size_t)m * 4 + 15) & ~(size_t)15) + 16;
}

// ---- standalone selection over given priorities: one cluster per independent problem (blockIdx.y)

__global__ void __launch_bounds__(kSelectThreads) k_select(const float* __restrict__ r,
                                                           const uint8_t* __restrict__ flags_in, int N, int B,
                                                           int* __restrict__ survivors, int* status) {
  extern __shared__ __align__(16) unsigned char smem[];
  cg::cluster_group cluster = cg::this_cluster();
  SelectShared* sh = reinterpret_cast<SelectShared*>(smem);
  unsigned char* p = smem + ((sizeof(SelectShared) + 15) & ~15);
  const int ncta = (int)cluster.num_blocks();
  int begin, end;
  cta_range(N, ncta, (int)cluster.block_rank(), &begin, &end);
  const int cnt = end - begin, span = (N + ncta - 1) / ncta;
  uint32_t* keys = reinterpret_cast<uint32_t*>(p);
  uint8_t* keep = p + (size_t)span * 4;
  const size_t prob = blockIdx.y;
  const float* rr = r + prob * (size_t)N;
  const uint8_t* ff = flags_in + prob * (size_t)N;
  for (int i = threadIdx.x; i < cnt; i += blockDim.x)
    keys[i] = ff[begin + i] != 0 ? kKeyProtected : rank_key(rr[begin + i]);
  __syncthreads();
  int my_base, bad;
  const int n_keep = cluster_select(cluster, keys, keep, begin, cnt, N, B, survivors + prob * (size_t)min(N, B), sh,
                                    &my_base, &bad);
  if ((bad || n_keep != min(N, B)) && threadIdx.x == 0 && status) atomicCAS(status, 0, OVGGT_ERR_DEVICE_STATUS);
  cluster.sync();   // no CTA may exit while others still read its shared memory
}

// ---- the fused per-step kernel

struct CompressParams {
  int n, M, B;                      // cached rows, new rows, budget
  int n_special, grid_h, grid_w;
  float alpha, w_center, w_edge, w_corner;   // Eq. 6: blend and the normalised 3x3 Gaussian weights
  float beta;
  int mode;                         // OVGGT_SCORE_*
  int protect_new;                  // != 0: give every new row this flag (INIT: first frame; HIST: a camera-cache anchor)
  unsigned long long step_key;      // OVGGT_SCORE_RANDOM: SplitMix64(seed ^ frame id) of this step
  float lone_new;                   // >= 0: normalised score of a new group without a range (Eq. 7's 0/0); < 0: 0
  int register_anchor, A;           // 1: flag the A most confident patches of the new frame HIST
  long long demote_frame;           // >= 0: release the HIST rows of that frame
  const float* s_raw;               // [M] residual norms of the new rows
  const float* d;                   // key diversity (hybrid mode), indexed by the row's physical slot
  const float* conf;                // [grid_h*grid_w]
  const float* override_r;          // [N] or nullptr
  const long long* ids_src; const uint8_t* flags_src; const float* stored_src;   // [N] pre-compaction meta
  long long* ids_dst; uint8_t* flags_dst; float* stored_dst;                     // [<=B] compacted meta
  float* r_out;                     // [N] priorities as computed here
  int* survivors;                   // [min(N, B)]
  int* status;
  int* n_keep_out;
  // Hole-filling layout (fill != 0): the K/V row of logical position g lives in slot slot_src[g] (g < n) or g
  // (new rows); the K/V rows are not gathered.  Survivors whose slot is >= B have to move into the slots < B
  // that evicted rows leave: the i-th such survivor (in logical order) goes to the i-th such slot (in the logical
  // order of the rows that leave).  The kernel writes the pairs and the survivors' slots; the move kernel that
  // follows copies the rows and patches slot_dst[move_j[i]] = move_dst[i].
  int fill;
  const int* slot_src;              // [n]
  int* slot_dst;                    // [<= B]
  int* move_src; int* move_dst; int* move_j;   // [<= M] each
  int* tail_move;                   // [M]: for slot B + i, the index of the move that empties it, or -1
  int* n_moves_out;
};

// Eq. 6 for new-frame token j (aux tokens keep their raw score); s_raw: the frame's M residual norms.
__device__ __forceinline__ float smoothed_score(const CompressParams& P, const float* s_raw, int j) {
  float v = s_raw[j];
  if (j >= P.n_special) {
    const int q = j - P.n_special, y = q / P.grid_w, x = q - y * P.grid_w;
    const float* S = s_raw + P.n_special;
    float conv = 0.0f;
#pragma unroll
    for (int dy = -1; dy <= 1; ++dy)
#pragma unroll
      for (int dx = -1; dx <= 1; ++dx) {
        const int yy = min(max(y + dy, 0), P.grid_h - 1), xx = min(max(x + dx, 0), P.grid_w - 1);
        const float w = (dx == 0 && dy == 0) ? P.w_center : ((dx == 0 || dy == 0) ? P.w_edge : P.w_corner);
        conv = __fmaf_rn(w, S[yy * P.grid_w + xx], conv);
      }
    v = __fmaf_rn(P.alpha, conv, __fmul_rn(1.0f - P.alpha, v));
  }
  return v;
}

__device__ __forceinline__ void compress_select_body(const CompressParams& P, unsigned char* smem) {
  cg::cluster_group cluster = cg::this_cluster();
  const int ncta = (int)cluster.num_blocks(), rank = (int)cluster.block_rank();
  SelectShared* sh = reinterpret_cast<SelectShared*>(smem);
  unsigned char* p = smem + ((sizeof(SelectShared) + 15) & ~15);
  const int tid = threadIdx.x, nthr = blockDim.x;
  const int n = P.n, M = P.M, N = n + M, Np = P.grid_h * P.grid_w;
  int begin, end;
  cta_range(N, ncta, rank, &begin, &end);
  const int cnt = end - begin, span = (N + ncta - 1) / ncta, span16 = (span + 15) & ~15;
  uint32_t* keys = reinterpret_cast<uint32_t*>(p);        // [span] values, then the priorities' keys, in place
  float* val = reinterpret_cast<float*>(keys);
  uint8_t* fl = p + (size_t)span * 4;                      // [span] protection flags of the owned positions
  uint8_t* keep = fl + span16;                             // [span]
  uint32_t* ckeys = reinterpret_cast<uint32_t*>(keep + span16);   // [Np] confidence keys
  uint8_t* cmark = reinterpret_cast<uint8_t*>(ckeys + Np);        // [Np]
  unsigned char* q8 = smem + ((select_smem_bytes(span, Np) + 15) & ~(size_t)15);
  long long* sid = reinterpret_cast<long long*>(q8);              // [span] ids of the owned positions
  float* sst = reinterpret_cast<float*>(q8 + (((size_t)span * 8 + 15) & ~(size_t)15));   // [span] their stored scores
  int* ssl = reinterpret_cast<int*>(sst + (((size_t)span + 3) & ~(size_t)3));   // [span] their physical slots
  float* sraw = reinterpret_cast<float*>(ssl + (((size_t)span + 3) & ~(size_t)3)); // [M] the frame's residual norms

  // -- anchor registration (Sec. 3.3): the A most confident patch tokens of the new frame, ties to the lower
  //    index.  Every CTA computes the same marks and uses those of the positions it owns.
  const bool reg = P.register_anchor && P.A > 0;
  if (reg) {
    for (int i = tid; i < Np; i += nthr) ckeys[i] = rank_key(P.conf[i]);
    __syncthreads();
    block_top_mark(ckeys, cmark, Np, P.A, sh);
  }

  // -- protection flags and values of the owned positions.  A CTA that owns new rows first stages the frame's raw
  //    norms (Eq. 6 reads each nine times); all global loads of four positions are issued before any is used.
  if (end > n) {
    for (int j = tid; j < M; j += nthr) sraw[j] = P.s_raw[j];
    __syncthreads();
  }
  for (int i0 = tid; i0 < cnt; i0 += 4 * nthr) {
    uint8_t f4[4];
    long long id4[4];
    float d4[4], st4[4];
    int sl4[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int i = i0 + u * nthr, g = begin + i;
      sl4[u] = g;
      if (i < cnt) {
        f4[u] = P.flags_src[g];
        id4[u] = P.ids_src[g];
        if (g < n) {
          st4[u] = P.stored_src[g];
          if (P.fill) {
            sl4[u] = P.slot_src[g];
            if (!index_ok(sl4[u], P.B + P.M, P.status)) sl4[u] = g;
          }
        }
      }
    }
    if (P.mode == OVGGT_SCORE_HYBRID) {
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int i = i0 + u * nthr, g = begin + i;
        d4[u] = (i < cnt && g < n) ? P.d[sl4[u]] : 0.0f;
      }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int i = i0 + u * nthr, g = begin + i;
      if (i < cnt) {
        uint8_t f = f4[u] & 3;
        float x, keepscore;
        if (g >= n) {
          const int j = g - n;
          if (P.protect_new) f = (uint8_t)P.protect_new;
          if (reg && j >= P.n_special && cmark[j - P.n_special]) f = OVGGT_FLAG_HIST;
          x = smoothed_score(P, sraw, j);
          keepscore = x;           // the score the row keeps
        } else {
          if (P.demote_frame >= 0 && f == OVGGT_FLAG_HIST && id4[u] / M == P.demote_frame) f = OVGGT_FLAG_EVICTABLE;
          x = (P.mode == OVGGT_SCORE_HYBRID) ? d4[u] : st4[u];
          keepscore = st4[u];
        }
        if (P.mode == OVGGT_SCORE_RANDOM) x = random_priority(P.step_key, id4[u]);   // Supp. A: uniform, fresh per step
        fl[i] = f;
        val[i] = x;
        sid[i] = id4[u];
        sst[i] = keepscore;
        ssl[i] = sl4[u];
      }
    }
  }
  __syncthreads();

  // -- Eq. 7: min-max of each group over the whole cluster
  float lo_h = INFINITY, hi_h = -INFINITY, lo_n = INFINITY, hi_n = -INFINITY;
  if (P.mode == OVGGT_SCORE_HYBRID) {
    for (int i = tid; i < cnt; i += nthr)
      if (fl[i] == 0) {
        const float x = val[i];
        if (begin + i < n) { lo_h = fminf(lo_h, x); hi_h = fmaxf(hi_h, x); }
        else               { lo_n = fminf(lo_n, x); hi_n = fmaxf(hi_n, x); }
      }
    block_minmax(lo_h, hi_h, sh->fscan, &lo_h, &hi_h);
    block_minmax(lo_n, hi_n, sh->fscan, &lo_n, &hi_n);
    if (tid == 0) {
      sh->pub_lo_h = lo_h; sh->pub_hi_h = hi_h; sh->pub_lo_n = lo_n; sh->pub_hi_n = hi_n;
    }
    cluster.sync();
    if (tid < 32) {                                   // one warp gathers: lane r reads CTA r's four values
      float a = INFINITY, b = -INFINITY, c2 = INFINITY, d2 = -INFINITY;
      if (tid < ncta) {
        const SelectShared* o = cluster.map_shared_rank(sh, tid);
        a = o->pub_lo_h; b = o->pub_hi_h; c2 = o->pub_lo_n; d2 = o->pub_hi_n;
      }
#pragma unroll
      for (int off = 4; off > 0; off >>= 1) {         // kSelectMaxCtas = 8 lanes carry values
        a = fminf(a, __shfl_xor_sync(0xFFFFFFFFu, a, off));
        b = fmaxf(b, __shfl_xor_sync(0xFFFFFFFFu, b, off));
        c2 = fminf(c2, __shfl_xor_sync(0xFFFFFFFFu, c2, off));
        d2 = fmaxf(d2, __shfl_xor_sync(0xFFFFFFFFu, d2, off));
      }
      if (tid == 0) { sh->mm[0] = a; sh->mm[1] = b; sh->mm[2] = c2; sh->mm[3] = d2; }
    }
    __syncthreads();
    lo_h = sh->mm[0]; hi_h = sh->mm[1]; lo_n = sh->mm[2]; hi_n = sh->mm[3];
  }
  for (int i = tid; i < cnt; i += nthr) {
    const int g = begin + i;
    float r;
    uint32_t key;
    if (fl[i] != 0) {
      r = INFINITY;
      key = kKeyProtected;
    } else {
      if (P.mode == OVGGT_SCORE_HYBRID) {
        const float lo = g < n ? lo_h : lo_n, hi = g < n ? hi_h : hi_n;
        const float w = g < n ? 1.0f - P.beta : P.beta;
        r = hi > lo ? __fmul_rn(w, __fdiv_rn(val[i] - lo, hi - lo))
                    : ((g >= n && P.lone_new >= 0.0f) ? __fmul_rn(w, P.lone_new) : 0.0f);
      } else {
        r = val[i];
      }
      key = rank_key(P.override_r ? P.override_r[g] : r);
    }
    P.r_out[g] = r;          // the kernel's own priority, also when an override is ranked instead
    keys[i] = key;
  }
  __syncthreads();

  // -- Eq. 8
  int my_base, bad;
  const int n_keep = cluster_select(cluster, keys, keep, begin, cnt, N, P.B, P.survivors, sh, &my_base, &bad);

  // -- compacted meta of this CTA's survivors (order preserved)
  const int chunk = (cnt + nthr - 1) / nthr;
  const int lo = min(cnt, tid * chunk), hi = min(cnt, lo + chunk);
  int my_j;       // compacted index of this thread's first survivor
  {
    int c = 0;
    for (int i = lo; i < hi; ++i) c += keep[i];
    int tot;
    my_j = my_base + block_excl_scan_int(c, sh->scan, &tot);
    int j = my_j;
    for (int i = lo; i < hi; ++i)
      if (keep[i]) {
        if (j < P.B) {
          P.ids_dst[j] = sid[i];
          P.flags_dst[j] = fl[i];
          P.stored_dst[j] = sst[i];
          if (P.fill) P.slot_dst[j] = ssl[i];
        }
        ++j;
      }
  }
  if (rank == 0 && tid == 0) {
    *P.n_keep_out = n_keep;
    if (bad || n_keep != min(N, P.B)) atomicCAS(P.status, 0, OVGGT_ERR_DEVICE_STATUS);
  }
  if (P.fill) {
    // -- hole filling: pair the survivors that sit above slot B with the slots below B whose rows leave
    int up = 0, down = 0;
    for (int i = lo; i < hi; ++i) {
      up += keep[i] && ssl[i] >= P.B;
      down += !keep[i] && ssl[i] < P.B;
    }
    int up_tot, down_tot;
    int up_rank = block_excl_scan_int(up, sh->scan, &up_tot);
    int down_rank = block_excl_scan_int(down, sh->scan, &down_tot);
    if (tid == 0) {
      sh->pub_up = up_tot;
      sh->pub_down = down_tot;
    }
    cluster.sync();
    if (tid < ncta) {
      sh->all_up[tid] = *cluster.map_shared_rank(&sh->pub_up, tid);
      sh->all_down[tid] = *cluster.map_shared_rank(&sh->pub_down, tid);
    }
    __syncthreads();
    int up_all = 0, down_all = 0;
    for (int r = 0; r < ncta; ++r) {
      if (r < rank) {
        up_rank += sh->all_up[r];
        down_rank += sh->all_down[r];
      }
      up_all += sh->all_up[r];
      down_all += sh->all_down[r];
    }
    int j = my_j;
    for (int i = lo; i < hi; ++i) {
      if (keep[i]) {
        if (ssl[i] >= P.B && up_rank < M) {
          P.move_src[up_rank] = ssl[i];
          P.move_j[up_rank] = j;
          if (ssl[i] - P.B < M) P.tail_move[ssl[i] - P.B] = up_rank;
          ++up_rank;
        }
        ++j;
      } else if (ssl[i] < P.B) {
        if (down_rank < M) P.move_dst[down_rank++] = ssl[i];
      } else if (ssl[i] - P.B < M) {
        P.tail_move[ssl[i] - P.B] = -1;           // a row above slot B that leaves: its slot is simply free
      }
    }
    // slots above B that no row occupies yet (the cache has just filled up) hold nothing to move
    if (rank == 0)
      for (int i = max(0, N - P.B) + tid; i < M; i += nthr) P.tail_move[i] = -1;
    if (rank == 0 && tid == 0) {
      // the two counts agree whenever the slots below min(N, B) were all occupied, which the layout guarantees
      const bool consistent = up_all == down_all && up_all <= M;
      *P.n_moves_out = consistent ? up_all : 0;
      if (!consistent) atomicCAS(P.status, 0, OVGGT_ERR_DEVICE_STATUS);
    }
  }
  cluster.sync();   // no CTA may exit while others still read its shared memory
}

__global__ void __launch_bounds__(kSelectThreads) k_compress_select(const CompressParams P) {
  extern __shared__ __align__(16) unsigned char smem[];
  compress_select_body(P, smem);
}

// The same step for several layers in one launch (Sec. 3.2: every layer has its own budget B^(l) and cache): one
// cluster per layer, blockIdx.y = position in the batch.  The parameter blocks travel as kernel arguments.
constexpr int kMaxBatchLayers = 32;
struct CompressBatch {
  CompressParams p[kMaxBatchLayers];
};
__global__ void __launch_bounds__(kSelectThreads) k_compress_select_batched(const __grid_constant__ CompressBatch batch) {
  extern __shared__ __align__(16) unsigned char smem[];
  compress_select_body(batch.p[blockIdx.y], smem);
}

}  // namespace ovggt
