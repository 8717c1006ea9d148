// Budgeted selection (Eq. 8) as a single-CTA radix select, and the fused per-step kernel that
// prepares its input: anchor flags (Sec. 3.3), activation smoothing (Eq. 6), hybrid priorities (Eq. 7).
//
// One CTA of 1024 threads holds all N keys and flags in shared memory (N <= ~44K; larger N keeps the
// keys in a global scratch array).  The k-th largest key is found with four 8-bit most-significant-digit
// passes; rows tied with it are admitted in position order, so the result is unique.
#pragma once

#include "common.cuh"

namespace ovggt {

constexpr int kSelectThreads = 1024;
constexpr uint8_t kKeepBit = 0x80;

struct SelectShared {
  int hist[256];
  int scan[64];
  float fscan[64];
  int digit, krem;
};

// Selection core.  keys[N]: rank keys; flags[N]: low bits non-zero = protected (flags == nullptr: none);
// bit 7 of flags is used as the keep mark when flags != nullptr, otherwise `mark` (N bytes) is used.
// Writes survivors[0 .. n_keep) ascending and returns n_keep (= min(N, B) unless |P| > B, which sets *bad).
__device__ inline int select_core(const uint32_t* keys, uint8_t* flags, uint8_t* mark, int N, int B,
                                  int* survivors, SelectShared* sh, int* bad) {
  const int tid = threadIdx.x, nthr = blockDim.x;
  uint8_t* fl = flags ? flags : mark;
  if (!flags)
    for (int i = tid; i < N; i += nthr) mark[i] = 0;
  __syncthreads();
  int prot = 0;
  for (int i = tid; i < N; i += nthr) prot += (fl[i] & 3) != 0;
  prot = block_sum_int(prot, sh->scan);
  const bool keep_all = N <= B;
  int k = B - prot;
  if (!keep_all && k < 0) {
    if (tid == 0) *bad = 1;
    k = 0;
  }
  uint32_t T = 0;
  int need_eq = 0;
  if (!keep_all && k > 0) {
    uint32_t prefix = 0, mask = 0;
    int krem = k;
    for (int shift = 24; shift >= 0; shift -= 8) {
      for (int b = tid; b < 256; b += nthr) sh->hist[b] = 0;
      __syncthreads();
      for (int i = tid; i < N; i += nthr)
        if ((fl[i] & 3) == 0 && (keys[i] & mask) == prefix) atomicAdd(&sh->hist[(keys[i] >> shift) & 255], 1);
      __syncthreads();
      if (tid < 32) {
        int c[8], local = 0;
#pragma unroll
        for (int b = 0; b < 8; ++b) {
          c[b] = sh->hist[tid * 8 + b];
          local += c[b];
        }
        // number of matching rows in bins above this lane's bins
        int above = local;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          int y = __shfl_down_sync(0xFFFFFFFFu, above, o);
          if (tid + o < 32) above += y;
        }
        above -= local;
        int cum = above;
#pragma unroll
        for (int b = 7; b >= 0; --b) {
          if (cum < krem && cum + c[b] >= krem) {
            sh->digit = tid * 8 + b;
            sh->krem = krem - cum;
          }
          cum += c[b];
        }
      }
      __syncthreads();
      prefix |= (uint32_t)sh->digit << shift;
      mask |= 255u << shift;
      krem = sh->krem;
      __syncthreads();
    }
    T = prefix;
    need_eq = krem;
  }
  // Mark keepers: thread t owns the contiguous positions [t*chunk, (t+1)*chunk).
  const int chunk = (N + nthr - 1) / nthr;
  const int lo = min(N, tid * chunk), hi = min(N, lo + chunk);
  int cnt_eq = 0;
  if (!keep_all && k > 0)
    for (int i = lo; i < hi; ++i) cnt_eq += ((fl[i] & 3) == 0 && keys[i] == T);
  int tot;
  int eq_rank = block_excl_scan_int(cnt_eq, sh->scan, &tot);
  int cnt_keep = 0;
  for (int i = lo; i < hi; ++i) {
    bool keep;
    if (keep_all) {
      keep = true;
    } else if ((fl[i] & 3) != 0) {
      keep = true;
    } else if (k <= 0) {
      keep = false;
    } else {
      const uint32_t key = keys[i];
      keep = key > T || (key == T && eq_rank++ < need_eq);
    }
    fl[i] = (uint8_t)((fl[i] & 3) | (keep ? kKeepBit : 0));
    cnt_keep += keep;
  }
  int n_keep;
  int base = block_excl_scan_int(cnt_keep, sh->scan, &n_keep);
  for (int i = lo; i < hi; ++i)
    if (fl[i] & kKeepBit) {
      if (base < B || keep_all) survivors[base] = i;
      ++base;
    }
  __syncthreads();
  if (!keep_all && n_keep > B) {   // only when |P| > B: keep the first B marked rows
    if (tid == 0) *bad = 1;
    n_keep = B;
  }
  return n_keep;
}

// ---- standalone selection over given priorities (one CTA per independent problem)

__global__ void __launch_bounds__(kSelectThreads) k_select(const float* __restrict__ r,
                                                           const uint8_t* __restrict__ flags_in, int N, int B,
                                                           int* __restrict__ survivors, uint32_t* gkeys,
                                                           int keys_in_smem, int* status) {
  extern __shared__ __align__(16) unsigned char smem[];
  SelectShared* sh = reinterpret_cast<SelectShared*>(smem);
  unsigned char* p = smem + ((sizeof(SelectShared) + 15) & ~15);
  const size_t prob = blockIdx.x;
  uint32_t* keys = keys_in_smem ? reinterpret_cast<uint32_t*>(p) : gkeys + prob * (size_t)N;
  if (keys_in_smem) p += (size_t)N * 4;
  uint8_t* fl = p;
  const float* rr = r + prob * (size_t)N;
  const uint8_t* ff = flags_in + prob * (size_t)N;
  for (int i = threadIdx.x; i < N; i += blockDim.x) {
    keys[i] = rank_key(rr[i]);
    fl[i] = ff[i] ? 1 : 0;
  }
  __syncthreads();
  int bad = 0;
  select_core(keys, fl, nullptr, N, B, survivors + prob * (size_t)min(N, B), sh, &bad);
  if (bad && threadIdx.x == 0 && status) atomicCAS(status, 0, OVGGT_ERR_DEVICE_STATUS);
}

// ---- the fused per-step kernel

struct CompressParams {
  int n, M, B;                      // cached rows, new rows, budget
  int n_special, grid_h, grid_w;
  float alpha, w_center, w_edge, w_corner;   // Eq. 6: blend and the normalised 3x3 Gaussian weights
  float beta;
  int mode;                         // OVGGT_SCORE_*
  int protect_new;                  // 1: flag the new rows INIT (first frame)
  int register_anchor, A;           // 1: flag the A most confident patches of the new frame HIST
  long long demote_frame;           // >= 0: release the HIST rows of that frame
  const float* s_raw;               // [M] residual norms of the new rows
  const float* d;                   // [n] key diversity (hybrid mode)
  const float* conf;                // [grid_h*grid_w]
  const float* override_r;          // [N] or nullptr
  const long long* ids_src; const uint8_t* flags_src; const float* stored_src;   // [N] pre-compaction meta
  long long* ids_dst; uint8_t* flags_dst; float* stored_dst;                     // [<=B] compacted meta
  float* r_out;                     // [N] priorities as ranked
  int* survivors;                   // [min(N, B)]
  uint32_t* gkeys;                  // [N] key scratch when shared memory is too small
  int keys_in_smem;
  int* status;
  int* n_keep_out;
};

__global__ void __launch_bounds__(kSelectThreads) k_compress_select(const CompressParams P) {
  extern __shared__ __align__(16) unsigned char smem[];
  SelectShared* sh = reinterpret_cast<SelectShared*>(smem);
  unsigned char* p = smem + ((sizeof(SelectShared) + 15) & ~15);
  const int tid = threadIdx.x, nthr = blockDim.x;
  const int n = P.n, M = P.M, N = n + M, Np = P.grid_h * P.grid_w;
  float* s_new = reinterpret_cast<float*>(p);            // [M] smoothed activation scores
  p += ((size_t)M * 4 + 15) & ~(size_t)15;
  uint32_t* keys = P.keys_in_smem ? reinterpret_cast<uint32_t*>(p) : P.gkeys;
  if (P.keys_in_smem) p += (size_t)N * 4;
  uint8_t* fl = p;                                       // [N]
  float* val = reinterpret_cast<float*>(keys);           // values, then priorities, then keys, in place
  int bad = 0;

  // -- protection flags (Sec. 3.3)
  for (int i = tid; i < N; i += nthr) {
    uint8_t f = P.flags_src[i] & 3;
    if (i >= n && P.protect_new) f = OVGGT_FLAG_INIT;
    if (i < n && P.demote_frame >= 0 && f == OVGGT_FLAG_HIST && P.ids_src[i] / M == P.demote_frame)
      f = OVGGT_FLAG_EVICTABLE;
    fl[i] = f;
  }
  __syncthreads();
  if (P.register_anchor && P.A > 0) {
    // the A most confident patch tokens of the new frame, ties to the lower index
    uint8_t* mark = reinterpret_cast<uint8_t*>(s_new);   // Np <= 4*M bytes, free until smoothing
    for (int i = tid; i < Np; i += nthr) keys[i] = rank_key(P.conf[i]);
    __syncthreads();
    const int na = select_core(keys, nullptr, mark, Np, P.A, P.survivors, sh, &bad);
    __syncthreads();
    for (int j = tid; j < na; j += nthr) fl[n + P.n_special + P.survivors[j]] = OVGGT_FLAG_HIST;
    __syncthreads();
  }

  // -- Eq. 6 on the patch grid; aux tokens keep their raw score
  for (int j = tid; j < M; j += nthr) {
    float v = P.s_raw[j];
    if (j >= P.n_special) {
      const int q = j - P.n_special, y = q / P.grid_w, x = q - y * P.grid_w;
      const float* S = P.s_raw + P.n_special;
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
    s_new[j] = v;
  }
  __syncthreads();

  // -- values, then priorities (Eq. 7 or the stored-residual reading)
  for (int i = tid; i < N; i += nthr)
    val[i] = i >= n ? s_new[i - n] : (P.mode == OVGGT_SCORE_HYBRID ? P.d[i] : P.stored_src[i]);
  __syncthreads();
  float lo_h = INFINITY, hi_h = -INFINITY, lo_n = INFINITY, hi_n = -INFINITY;
  if (P.mode == OVGGT_SCORE_HYBRID) {
    for (int i = tid; i < N; i += nthr)
      if (fl[i] == 0) {
        const float x = val[i];
        if (i < n) { lo_h = fminf(lo_h, x); hi_h = fmaxf(hi_h, x); }
        else       { lo_n = fminf(lo_n, x); hi_n = fmaxf(hi_n, x); }
      }
    block_minmax(lo_h, hi_h, sh->fscan, &lo_h, &hi_h);
    block_minmax(lo_n, hi_n, sh->fscan, &lo_n, &hi_n);
  }
  __syncthreads();
  for (int i = tid; i < N; i += nthr) {
    float r;
    if (fl[i] != 0) {
      r = INFINITY;
    } else if (P.mode == OVGGT_SCORE_HYBRID) {
      const float lo = i < n ? lo_h : lo_n, hi = i < n ? hi_h : hi_n;
      const float w = i < n ? 1.0f - P.beta : P.beta;
      r = hi > lo ? __fmul_rn(w, __fdiv_rn(val[i] - lo, hi - lo)) : 0.0f;
    } else {
      r = val[i];
    }
    P.r_out[i] = r;                                      // the kernel's own priority, also under teacher forcing
    if (fl[i] == 0 && P.override_r) r = P.override_r[i];
    keys[i] = rank_key(r);
  }
  __syncthreads();

  // -- Eq. 8
  const int n_keep = select_core(keys, fl, nullptr, N, P.B, P.survivors, sh, &bad);
  __syncthreads();
  for (int j = tid; j < n_keep; j += nthr) {
    const int src = P.survivors[j];
    P.ids_dst[j] = P.ids_src[src];
    P.flags_dst[j] = fl[src] & 3;
    P.stored_dst[j] = src >= n ? s_new[src - n] : P.stored_src[src];
  }
  if (tid == 0) {
    *P.n_keep_out = n_keep;
    if (bad || n_keep != min(N, P.B)) atomicCAS(P.status, 0, OVGGT_ERR_DEVICE_STATUS);
  }
}

}  // namespace ovggt
