// Scoring kernels: residual norms (Eq. 5), key column sums and key diversity (Sec. 3.2).
// All of them stream rows of [rows, C] once with 16-byte loads and accumulate in fp32 in an
// order that depends only on the shapes, so results are reproducible run to run.
#pragma once

#include "common.cuh"

namespace ovggt {

// s[row] = sqrt(sum_c x[row, c]^2); one warp per row.  Lane l owns vectors l, l+32, ... and
// folds them in that order; lanes are combined by the fixed butterfly of warp_sum.
template <int DT>
__device__ __forceinline__ void warp_row_norm(const uint4* __restrict__ x, int row, int nvec, float* __restrict__ s) {
  constexpr int VEC = VecOf<DT>::n;
  const int lane = threadIdx.x & 31;
  const uint4* p = x + (size_t)row * nvec;
  float acc = 0.0f;
  for (int v0 = lane; v0 < nvec; v0 += 128) {
    uint4 u[4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
      if (v0 + 32 * i < nvec) u[i] = ld_nc(p + v0 + 32 * i);
#pragma unroll
    for (int i = 0; i < 4; ++i)
      if (v0 + 32 * i < nvec) {
        float f[VEC];
        unpack<DT>(u[i], f);
#pragma unroll
        for (int e = 0; e < VEC; ++e) acc = __fmaf_rn(f[e], f[e], acc);
      }
  }
  acc = warp_sum(acc);
  if (lane == 0) s[row] = __fsqrt_rn(acc);
}

template <int DT>
__global__ void __launch_bounds__(256) k_row_norms(const uint4* __restrict__ x, int rows, int nvec,
                                                   float* __restrict__ s) {
  const int row = (int)((blockIdx.x * (unsigned)blockDim.x + threadIdx.x) >> 5);
  if (row < rows) warp_row_norm<DT>(x, row, nvec, s);
}

// out[row] = scale * sum_c x[row, c] * vec[c]; one warp per row, the same order of accumulation as warp_row_norm.
// With vec = the column sums of the frame's queries and scale = 1 / (M H sqrt(d)) this is the query-key criterion of
// the scoring probe (Supp. D): the mean scaled logit the key of row `row` receives from the M queries over all heads.
template <int DT>
__global__ void __launch_bounds__(256) k_row_dots(const uint4* __restrict__ x, int rows, int nvec,
                                                  const float* __restrict__ vec, float scale, float* __restrict__ out) {
  constexpr int VEC = VecOf<DT>::n;
  const int row = (int)((blockIdx.x * (unsigned)blockDim.x + threadIdx.x) >> 5);
  if (row >= rows) return;                       // whole warps leave together: a row belongs to one warp
  const int lane = threadIdx.x & 31;
  const uint4* p = x + (size_t)row * nvec;
  float acc = 0.0f;
  for (int v = lane; v < nvec; v += 32) {
    float f[VEC];
    unpack<DT>(ld_nc(p + v), f);
    const float* w = vec + (size_t)v * VEC;
#pragma unroll
    for (int e = 0; e < VEC; ++e) acc = __fmaf_rn(f[e], __ldg(w + e), acc);
  }
  acc = warp_sum(acc);
  if (lane == 0) out[row] = acc * scale;
}

// Column sums of K [rows, C], stage 1: CTA p sums its contiguous chunk of rows, in row order,
// into part[p, C].  Thread t owns vector columns t, t + blockDim, ...
template <int DT>
__global__ void __launch_bounds__(256) k_colsum_partial(const uint4* __restrict__ K, int rows, int nvec,
                                                        int rows_per_cta, float* __restrict__ part) {
  constexpr int VEC = VecOf<DT>::n;
  const int r0 = blockIdx.x * rows_per_cta;
  const int r1 = min(rows, r0 + rows_per_cta);
  for (int v = threadIdx.x; v < nvec; v += blockDim.x) {
    float acc[VEC];
#pragma unroll
    for (int e = 0; e < VEC; ++e) acc[e] = 0.0f;
    int r = r0;
    for (; r + 4 <= r1; r += 4) {
      uint4 u[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) u[i] = ld_nc(K + (size_t)(r + i) * nvec + v);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        float f[VEC];
        unpack<DT>(u[i], f);
#pragma unroll
        for (int e = 0; e < VEC; ++e) acc[e] += f[e];
      }
    }
    for (; r < r1; ++r) {
      float f[VEC];
      unpack<DT>(ld_nc(K + (size_t)r * nvec + v), f);
#pragma unroll
      for (int e = 0; e < VEC; ++e) acc[e] += f[e];
    }
    float* o = part + (size_t)blockIdx.x * nvec * VEC + (size_t)v * VEC;
#pragma unroll
    for (int e = 0; e < VEC; ++e) o[e] = acc[e];
  }
}

// Stage 2: ksum[c] = sum_p part[p, c].  A CTA of 32 x 32 threads owns 32 columns; thread (py, cx)
// folds partials py, py + 32, ... in order, then the 32 py-values are folded in order.
__global__ void __launch_bounds__(1024) k_colsum_final(const float* __restrict__ part, int nparts, int C,
                                                       float* __restrict__ ksum) {
  __shared__ float sh[32][33];
  const int cx = threadIdx.x & 31, py = threadIdx.x >> 5;
  const int c = blockIdx.x * 32 + cx;
  float acc = 0.0f;
  if (c < C)
    for (int p = py; p < nparts; p += 32) acc += part[(size_t)p * C + c];
  sh[py][cx] = acc;
  __syncthreads();
  if (py == 0 && c < C) {
    float t = 0.0f;
#pragma unroll
    for (int i = 0; i < 32; ++i) t += sh[i][cx];
    ksum[c] = t;
  }
}

// Stage 2 for many partials (the compaction kernel leaves one per CTA): CTA (x, y) folds the partials
// p = y, y + gridDim.y, ... of its 32 columns into slice y; the CTA of a column block that finishes last folds the
// gridDim.y slices, in slice order, into ksum.  arrived: one counter per column block, zero before and after.
__global__ void __launch_bounds__(1024) k_colsum_final_sliced(const float* __restrict__ part, int nparts, int C,
                                                              float* __restrict__ ksum_slices,
                                                              float* __restrict__ ksum, int* __restrict__ arrived) {
  __shared__ float sh[32][33];
  __shared__ int is_last;
  const int cx = threadIdx.x & 31, py = threadIdx.x >> 5;
  const int c = blockIdx.x * 32 + cx;
  float acc = 0.0f;
  if (c < C) {
#pragma unroll 8
    for (int p = blockIdx.y + py * gridDim.y; p < nparts; p += 32 * gridDim.y) acc += part[(size_t)p * C + c];
  }
  sh[py][cx] = acc;
  __syncthreads();
  if (py == 0 && c < C) {
    float t = 0.0f;
#pragma unroll
    for (int i = 0; i < 32; ++i) t += sh[i][cx];
    ksum_slices[(size_t)blockIdx.y * C + c] = t;
    __threadfence();
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const int old = atomicAdd(&arrived[blockIdx.x], 1);
    is_last = old == (int)gridDim.y - 1;
    if (is_last) arrived[blockIdx.x] = 0;
  }
  __syncthreads();
  if (is_last && py == 0 && c < C) {
    __threadfence();
    float t = 0.0f;
    for (int y = 0; y < (int)gridDim.y; ++y) t += __ldcg(&ksum_slices[(size_t)y * C + c]);
    ksum[c] = t;
  }
}

// d[row] = 1 - (k_row . ksum) / (|k_row| |ksum|); the cosine with the centroid equals the cosine
// with the column sum.  ksum is given as n_slices rows of C floats that every CTA adds up in row order (one row: the
// sums themselves; more: a base row plus corrections, as the hole-filling compaction leaves them).  A zero vector has cosine 0.  One warp per pair of rows; ksum is staged in shared memory
// once per CTA and, for rows of up to 128 vectors, kept in registers by the lanes that meet its columns;
// |ksum|^2 is folded by every warp in the same order, so all CTAs agree on it.
struct DiversityArgs {
  const uint4* K; int rows;                 // cached keys [rows, C]
  const float* ksum; int n_slices;          // [n_slices, C]
  float* ksum_out;                          // [C] or nullptr
  float* d;                                 // [rows]
  int div_ctas;                             // CTAs [0, div_ctas) of the launch work on d; later ones on the norms
  const uint4* resid; int resid_rows;       // [resid_rows, C] or nullptr
  float* s_raw;                             // [resid_rows]
};

template <int DT>
__device__ __forceinline__ void diversity_body(const DiversityArgs& A, int nvec, float* sh_ksum) {
  constexpr int VEC = VecOf<DT>::n;
  const uint4* __restrict__ K = A.K;
  const float* __restrict__ ksum = A.ksum;
  float* __restrict__ ksum_out = A.ksum_out;
  float* __restrict__ d = A.d;
  const int rows = A.rows, n_slices = A.n_slices, div_ctas = A.div_ctas;
  // CTAs past the first div_ctas carry a second, independent job in the same launch: the residual norms of
  // Eq. 5 (one warp per row), so that a step pays one launch for both scores.
  if ((int)blockIdx.x >= div_ctas) {
    const int row = (int)((((int)blockIdx.x - div_ctas) * (unsigned)blockDim.x + threadIdx.x) >> 5);
    if (A.resid != nullptr && row < A.resid_rows) warp_row_norm<DT>(A.resid, row, nvec, A.s_raw);
    return;
  }
  const int C = nvec * VEC;
  const int lane = threadIdx.x & 31;
  const int warps_total = (int)((div_ctas * (unsigned)blockDim.x) >> 5);
  // Two rows per iteration, eight 16-byte loads per lane in flight (rows of up to 128 vectors; longer rows loop).
  // The first pair is requested before the centroid is staged, so that its DRAM latency runs under the set-up.
  int row = (int)((blockIdx.x * (unsigned)blockDim.x + threadIdx.x) >> 5) * 2;
  uint4 u[2][4];
  auto load_pair = [&](int r0, int v0) {
    const uint4* p0 = K + (size_t)r0 * nvec;
    const uint4* p1 = p0 + (r0 + 1 < rows ? nvec : 0);
#pragma unroll
    for (int i = 0; i < 4; ++i)
      if (v0 + 32 * i < nvec) {
        u[0][i] = ld_nc(p0 + v0 + 32 * i);
        u[1][i] = ld_nc(p1 + v0 + 32 * i);
      }
  };
  if (row < rows) load_pair(row, lane);
  for (int c = threadIdx.x; c < C; c += blockDim.x) {   // ksum: [n_slices, C], folded in slice order
    float t = ksum[c];
    for (int sl = 1; sl < n_slices; ++sl) t += ksum[(size_t)sl * C + c];
    sh_ksum[c] = t;
    if (ksum_out != nullptr && blockIdx.x == 0) ksum_out[c] = t;   // the folded sums, for whoever continues from them
  }
  __syncthreads();
  float kn = 0.0f;
  for (int v = lane; v < nvec; v += 32)
#pragma unroll
    for (int e = 0; e < VEC; e += 4) {
      const float4 k4 = *reinterpret_cast<const float4*>(sh_ksum + v * VEC + e);
      kn = __fmaf_rn(k4.x, k4.x, kn);
      kn = __fmaf_rn(k4.y, k4.y, kn);
      kn = __fmaf_rn(k4.z, k4.z, kn);
      kn = __fmaf_rn(k4.w, k4.w, kn);
    }
  kn = warp_sum(kn);
  // A lane meets the same columns in every row; when a row fits one round of loads (nvec <= 128) the lane keeps
  // its 4 x VEC centroid values in registers, and the row loop does not touch shared memory at all.
  const bool in_regs = nvec <= 128;
  float kreg[4][VEC];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int e = 0; e < VEC; e += 4) {
      float4 k4 = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
      if (in_regs && lane + 32 * i < nvec) k4 = *reinterpret_cast<const float4*>(sh_ksum + (lane + 32 * i) * VEC + e);
      kreg[i][e] = k4.x; kreg[i][e + 1] = k4.y; kreg[i][e + 2] = k4.z; kreg[i][e + 3] = k4.w;
    }
  for (; row < rows; row += 2 * warps_total) {
    const bool two = row + 1 < rows;
    float dot[2] = {0.0f, 0.0f}, nrm[2] = {0.0f, 0.0f};
    for (int v0 = lane; v0 < nvec; v0 += 128) {
      if (v0 != lane) load_pair(row, v0);
#pragma unroll
      for (int i = 0; i < 4; ++i)
        if (v0 + 32 * i < nvec) {
          float ks[VEC];
          if (in_regs) {
#pragma unroll
            for (int e = 0; e < VEC; ++e) ks[e] = kreg[i][e];
          } else {
            // 16-byte reads: consecutive lanes are VEC floats apart, which scalar reads would serialise eight ways
#pragma unroll
            for (int e = 0; e < VEC; e += 4)
              *reinterpret_cast<float4*>(ks + e) =
                  *reinterpret_cast<const float4*>(sh_ksum + (v0 + 32 * i) * VEC + e);
          }
#pragma unroll
          for (int r = 0; r < 2; ++r) {
            float f[VEC];
            unpack<DT>(u[r][i], f);
#pragma unroll
            for (int e = 0; e < VEC; ++e) {
              dot[r] = __fmaf_rn(f[e], ks[e], dot[r]);
              nrm[r] = __fmaf_rn(f[e], f[e], nrm[r]);
            }
          }
        }
    }
    const int next = row + 2 * warps_total;
    if (next < rows) load_pair(next, lane);           // the next pair travels during the reductions
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      const float dt = warp_sum(dot[r]), nr = warp_sum(nrm[r]);
      if (lane == 0 && (r == 0 || two)) {
        float cosv = 0.0f;
        if (nr > 0.0f && kn > 0.0f) cosv = __fdiv_rn(dt, __fmul_rn(__fsqrt_rn(nr), __fsqrt_rn(kn)));
        d[row + r] = 1.0f - cosv;
      }
    }
  }
}

template <int DT>
__global__ void __launch_bounds__(256) k_diversity(const uint4* __restrict__ K, int rows, int nvec,
                                                   const float* __restrict__ ksum, int n_slices,
                                                   float* __restrict__ ksum_out,
                                                   float* __restrict__ d, int div_ctas,
                                                   const uint4* __restrict__ resid, int resid_rows,
                                                   float* __restrict__ s_raw) {
  extern __shared__ __align__(16) float sh_ksum[];
  const DiversityArgs A{K, rows, ksum, n_slices, ksum_out, d, div_ctas, resid, resid_rows, s_raw};
  diversity_body<DT>(A, nvec, sh_ksum);
}

// Both scores of several layers in one launch: blockIdx.y = position in the batch, every layer with its own cache,
// sums and residual; the grid's x extent is the largest layer's, smaller layers leave their surplus CTAs idle.
constexpr int kMaxScoreBatch = 32;
struct DiversityBatch {
  DiversityArgs a[kMaxScoreBatch];
};
template <int DT>
__global__ void __launch_bounds__(256) k_diversity_batched(const __grid_constant__ DiversityBatch batch, int nvec) {
  extern __shared__ __align__(16) float sh_ksum[];
  diversity_body<DT>(batch.a[blockIdx.y], nvec, sh_ksum);
}

// Supp. D, attention-weight criterion: part[h, j] = sum_i 2^(c q_i,h . k_j,h - lse[i, h]), the attention key j of the
// frame receives from the frame's M queries in head h, given each row's log2 softmax denominator over ALL keys (lse,
// written by the attention kernels).  One CTA per (64 keys, head): the key tile and one 64-query tile at a time sit
// in shared memory as fp32, thread (ty, tx) of 16 x 16 owns a 4 x 4 block of the 64 x 64 logits.  The sums over i
// run in a fixed order (query tiles in order, then the 16 thread rows in order), so results are reproducible.
constexpr int kRecvTile = 64;
template <int DT>
__global__ void __launch_bounds__(256) k_attn_received(const uint4* __restrict__ q, const uint4* __restrict__ k, int M,
                                                       int H, const float* __restrict__ lse, float* __restrict__ part) {
  constexpr int D = 64, VEC = VecOf<DT>::n, VPR = D / VEC;
  __shared__ float Ks[kRecvTile][D + 1];
  __shared__ float Qs[kRecvTile][D + 1];
  __shared__ float Ls[kRecvTile];
  __shared__ float red[16][kRecvTile];
  const int h = blockIdx.y, j0 = blockIdx.x * kRecvTile;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const size_t row_vecs = (size_t)H * VPR;
  const float c = 1.4426950408889634f * 0.125f;              // log2(e) / sqrt(64)
  for (int idx = threadIdx.x; idx < kRecvTile * VPR; idx += 256) {
    const int r = idx / VPR, i = idx - r * VPR;
    float f[VEC];
#pragma unroll
    for (int e = 0; e < VEC; ++e) f[e] = 0.0f;
    if (j0 + r < M) unpack<DT>(k[(size_t)(j0 + r) * row_vecs + (size_t)h * VPR + i], f);
#pragma unroll
    for (int e = 0; e < VEC; ++e) Ks[r][i * VEC + e] = f[e];
  }
  float col[4] = {0.0f, 0.0f, 0.0f, 0.0f};
  for (int i0 = 0; i0 < M; i0 += kRecvTile) {
    __syncthreads();
    for (int idx = threadIdx.x; idx < kRecvTile * VPR; idx += 256) {
      const int r = idx / VPR, i = idx - r * VPR;
      float f[VEC];
#pragma unroll
      for (int e = 0; e < VEC; ++e) f[e] = 0.0f;
      if (i0 + r < M) unpack<DT>(q[(size_t)(i0 + r) * row_vecs + (size_t)h * VPR + i], f);
#pragma unroll
      for (int e = 0; e < VEC; ++e) Qs[r][i * VEC + e] = f[e];
    }
    if (threadIdx.x < kRecvTile) Ls[threadIdx.x] = i0 + threadIdx.x < M ? lse[(size_t)(i0 + threadIdx.x) * H + h] : INFINITY;
    __syncthreads();
    float acc[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
      for (int b = 0; b < 4; ++b) acc[a][b] = 0.0f;
    for (int d = 0; d < D; ++d) {
      float qa[4], kb[4];
#pragma unroll
      for (int a = 0; a < 4; ++a) qa[a] = Qs[ty * 4 + a][d];
#pragma unroll
      for (int b = 0; b < 4; ++b) kb[b] = Ks[tx * 4 + b][d];
#pragma unroll
      for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] = fmaf(qa[a], kb[b], acc[a][b]);
    }
#pragma unroll
    for (int a = 0; a < 4; ++a) {
      const float l2 = Ls[ty * 4 + a];                         // +inf for rows past M: their weight is 2^-inf = 0
#pragma unroll
      for (int b = 0; b < 4; ++b) col[b] += exp2f(fmaf(acc[a][b], c, -l2));
    }
  }
#pragma unroll
  for (int b = 0; b < 4; ++b) red[ty][tx * 4 + b] = col[b];
  __syncthreads();
  if (threadIdx.x < kRecvTile && j0 + threadIdx.x < M) {
    float t = 0.0f;
#pragma unroll
    for (int r = 0; r < 16; ++r) t += red[r][threadIdx.x];
    part[(size_t)h * M + j0 + threadIdx.x] = t;
  }
}

// s[j] = scale * sum_h part[h, j], heads in order.
__global__ void __launch_bounds__(256) k_fold_heads(const float* __restrict__ part, int M, int H, float scale,
                                                    float* __restrict__ s) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= M) return;
  float t = 0.0f;
  for (int h = 0; h < H; ++h) t += part[(size_t)h * M + j];
  s[j] = t * scale;
}

}  // namespace ovggt
