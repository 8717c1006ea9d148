// Cache append (Eq. 2) and order-preserving compaction of the surviving rows (Eq. 8).
// Rows are 16-byte-vector arrays; one warp moves one K or V row at a time with all of its
// loads issued before its stores, so many independent 16-byte transactions are in flight per SM.
#pragma once

#include <cooperative_groups.h>

#include "common.cuh"

namespace ovggt {

__device__ __forceinline__ void warp_copy_row(const uint4* __restrict__ src, uint4* __restrict__ dst, int nvec,
                                              int lane) {
  for (int v0 = lane; v0 < nvec; v0 += 128) {
    uint4 u[4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
      if (v0 + 32 * i < nvec) u[i] = ld_nc(src + v0 + 32 * i);
#pragma unroll
    for (int i = 0; i < 4; ++i)
      if (v0 + 32 * i < nvec) dst[v0 + 32 * i] = u[i];
  }
}

// dst[j, :] = src[survivors[j], :] for K and V.  Work item 2j is K row j, 2j+1 is V row j.
__global__ void __launch_bounds__(256) k_compact(const uint4* __restrict__ k_src, const uint4* __restrict__ v_src,
                                                 const int* __restrict__ survivors, int n_keep, int nvec,
                                                 uint4* __restrict__ k_dst, uint4* __restrict__ v_dst, int n_src,
                                                 int* status) {
  const int lane = threadIdx.x & 31;
  const int warps_total = (int)((gridDim.x * (unsigned)blockDim.x) >> 5);
  for (int item = (int)((blockIdx.x * (unsigned)blockDim.x + threadIdx.x) >> 5); item < 2 * n_keep;
       item += warps_total) {
    const int j = item >> 1;
    const int src = survivors[j];
    if (!index_ok(src, n_src, status)) continue;
    if (item & 1) warp_copy_row(v_src + (size_t)src * nvec, v_dst + (size_t)j * nvec, nvec, lane);
    else          warp_copy_row(k_src + (size_t)src * nvec, k_dst + (size_t)j * nvec, nvec, lane);
  }
}

constexpr int kCompactSumMaxVec = 128;   // rows of up to 128 16-byte vectors (C <= 1024 bf16) in the fused variant

// The same gather that also sums, per CTA, the columns of the K rows it writes: part[blockIdx.x, c] = sum of
// k_dst[j, c] over this CTA's rows.  A warp takes two survivors per iteration, j and j + (warps in the grid), and
// moves the K and the V row of both with all 16 loads of a lane issued before the first store: when the kernel
// shares the SMs with the attention it is the bytes in flight per occupied register that decide how long it holds
// them.  A warp folds its K rows in the order it meets them; the CTA folds its warps 4..7 onto 0..3 and then 0..3 in
// order, so the sums do not depend on timing.  The sums over all CTAs are the column sums of the compacted keys: the
// centroid the next step's diversity score needs, without another pass over K.  Requires nvec <= kCompactSumMaxVec.
template <int DT>
__global__ void __launch_bounds__(256) k_compact_colsum(const uint4* __restrict__ k_src, const uint4* __restrict__ v_src,
                                                        const int* __restrict__ survivors, int n_keep, int nvec,
                                                        uint4* __restrict__ k_dst, uint4* __restrict__ v_dst,
                                                        float* __restrict__ part, int n_src, int* status) {
  constexpr int VEC = VecOf<DT>::n;
  __shared__ __align__(16) float red[4][kCompactSumMaxVec * VEC];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int warps_total = (int)((gridDim.x * (unsigned)blockDim.x) >> 5);
  float acc[4][VEC];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int e = 0; e < VEC; ++e) acc[i][e] = 0.0f;
  for (int j0 = (int)((blockIdx.x * (unsigned)blockDim.x + threadIdx.x) >> 5); j0 < n_keep; j0 += 2 * warps_total) {
    const int j1 = j0 + warps_total;
    const bool two = j1 < n_keep;
    int s0 = survivors[j0], s1 = two ? survivors[j1] : s0;
    if (!index_ok(s0, n_src, status)) s0 = 0;     // (checked build: a bad index is reported and row 0 copied instead)
    if (!index_ok(s1, n_src, status)) s1 = 0;
    const uint4 *ka = k_src + (size_t)s0 * nvec, *va = v_src + (size_t)s0 * nvec;
    const uint4 *kb = k_src + (size_t)s1 * nvec, *vb = v_src + (size_t)s1 * nvec;
    uint4 uk[2][4], uv[2][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
      if (lane + 32 * i < nvec) {
        uk[0][i] = ld_nc(ka + lane + 32 * i);
        uv[0][i] = ld_nc(va + lane + 32 * i);
        uk[1][i] = ld_nc(kb + lane + 32 * i);
        uv[1][i] = ld_nc(vb + lane + 32 * i);
      }
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      if (r == 1 && !two) break;
      const size_t j = (size_t)(r == 0 ? j0 : j1);
#pragma unroll
      for (int i = 0; i < 4; ++i)
        if (lane + 32 * i < nvec) {
          k_dst[j * nvec + lane + 32 * i] = uk[r][i];
          v_dst[j * nvec + lane + 32 * i] = uv[r][i];
          float f[VEC];
          unpack<DT>(uk[r][i], f);
#pragma unroll
          for (int e = 0; e < VEC; ++e) acc[i][e] += f[e];
        }
    }
  }
  // fold the eight warps: 4..7 park their sums, 0..3 add them to their own and park the result, then four columns-wise
  auto park = [&](int slot, bool add) {
#pragma unroll
    for (int i = 0; i < 4; ++i)
      if (lane + 32 * i < nvec)
#pragma unroll
        for (int e = 0; e < VEC; e += 4) {
          float4* p = reinterpret_cast<float4*>(&red[slot][(lane + 32 * i) * VEC + e]);
          float4 t = make_float4(acc[i][e], acc[i][e + 1], acc[i][e + 2], acc[i][e + 3]);
          if (add) {
            const float4 o = *p;
            t.x += o.x; t.y += o.y; t.z += o.z; t.w += o.w;
          }
          *p = t;
        }
  };
  if (warp >= 4) park(warp - 4, false);
  __syncthreads();
  if (warp < 4) park(warp, true);
  __syncthreads();
  const int C = nvec * VEC;
  for (int c = threadIdx.x; c < C; c += blockDim.x)
    part[(size_t)blockIdx.x * C + c] = ((red[0][c] + red[1][c]) + red[2][c]) + red[3][c];
}

// Running upper bound of the squared per-head key norms of a bf16 cache, head_dim 64: kmax2[h] = max(kmax2[h],
// |K[row, 64h .. 64h+63]|^2).  A warp holds the row as 16-byte vectors (lane + 32 i); a head is eight consecutive
// vectors, i.e. eight neighbouring lanes of one i.  Non-negative floats order like their bit patterns, so the maximum
// is an integer atomicMax, which does not depend on the order of arrival.
__device__ __forceinline__ void warp_key_norm_max(const uint4* u, int nvec, int lane, float* kmax2) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float ss = 0.0f;
    if (lane + 32 * i < nvec) {
      const uint32_t w[4] = {u[i].x, u[i].y, u[i].z, u[i].w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float lo = __uint_as_float(w[e] << 16), hi = __uint_as_float(w[e] & 0xFFFF0000u);
        ss = fmaf(lo, lo, ss);
        ss = fmaf(hi, hi, ss);
      }
    }
    ss += __shfl_xor_sync(0xFFFFFFFFu, ss, 1);
    ss += __shfl_xor_sync(0xFFFFFFFFu, ss, 2);
    ss += __shfl_xor_sync(0xFFFFFFFFu, ss, 4);
    if ((lane & 7) == 0 && lane + 32 * i < nvec) {
      const int head = (lane + 32 * i) >> 3;
      if (ss > kmax2[head]) atomicMax(reinterpret_cast<int*>(kmax2) + head, __float_as_int(ss));
    }
  }
}

// kmax2 over rows [0, rows) of K (after an import).  bf16, nvec <= 128.
__global__ void __launch_bounds__(256) k_key_norm_max(const uint4* __restrict__ K, int rows, int nvec,
                                                      float* __restrict__ kmax2) {
  const int lane = threadIdx.x & 31;
  const int warps_total = (int)((gridDim.x * (unsigned)blockDim.x) >> 5);
  for (int r = (int)((blockIdx.x * (unsigned)blockDim.x + threadIdx.x) >> 5); r < rows; r += warps_total) {
    uint4 u[4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
      if (lane + 32 * i < nvec) u[i] = ld_nc(K + (size_t)r * nvec + lane + 32 * i);
    warp_key_norm_max(u, nvec, lane, kmax2);
  }
}

// Rows [n, n+M) of the cache := the frame's K and V; their meta: ids frame*M + j, evictable, score 0 and, in the
// hole-filling layout (slot != nullptr), the physical slot n + j.  With kmax2 (bf16 rows of up to 128 vectors) the
// running bound of the key norms takes the new keys in.
__global__ void __launch_bounds__(256) k_append(const uint4* __restrict__ k_new, const uint4* __restrict__ v_new,
                                                int M, int nvec, int n, long long frame_id,
                                                uint4* __restrict__ k_cache, uint4* __restrict__ v_cache,
                                                long long* __restrict__ ids, uint8_t* __restrict__ flags,
                                                float* __restrict__ stored, int* __restrict__ slot,
                                                float* __restrict__ kmax2) {
  const int lane = threadIdx.x & 31;
  const int gtid = blockIdx.x * blockDim.x + threadIdx.x;
  const int warps_total = (int)((gridDim.x * (unsigned)blockDim.x) >> 5);
  for (int item = gtid >> 5; item < 2 * M; item += warps_total) {
    const int j = item >> 1;
    if (item & 1) {
      warp_copy_row(v_new + (size_t)j * nvec, v_cache + (size_t)(n + j) * nvec, nvec, lane);
    } else if (kmax2 == nullptr) {
      warp_copy_row(k_new + (size_t)j * nvec, k_cache + (size_t)(n + j) * nvec, nvec, lane);
    } else {
      uint4 u[4];
#pragma unroll
      for (int i = 0; i < 4; ++i)
        if (lane + 32 * i < nvec) u[i] = ld_nc(k_new + (size_t)j * nvec + lane + 32 * i);
#pragma unroll
      for (int i = 0; i < 4; ++i)
        if (lane + 32 * i < nvec) k_cache[(size_t)(n + j) * nvec + lane + 32 * i] = u[i];
      warp_key_norm_max(u, nvec, lane, kmax2);
    }
  }
  for (int j = gtid; j < M; j += gridDim.x * blockDim.x) {
    ids[n + j] = frame_id * (long long)M + j;
    flags[n + j] = OVGGT_FLAG_EVICTABLE;
    stored[n + j] = 0.0f;
    if (slot) slot[n + j] = n + j;
  }
}

// ---- hole-filling compaction (Eq. 8 fixes the survivor set, not where the rows live)
//
// The selection kernel leaves n_moves pairs: the K/V row in slot move_src[i] (a survivor above slot B) goes to
// slot move_dst[i] (a slot below B whose row was evicted), and the survivor's meta entry move_j[i] learns its new
// slot.  Nothing else moves, so a step at steady state copies at most M rows instead of B.
// With `delta` the kernel also leaves what the move does to the column sums of the keys in slots [0, B):
//   delta[c] = sum_i (K[move_src[i], c] - K[move_dst[i], c])     (keys admitted minus keys evicted)
// as kFillSlices partial rows, one per 8-CTA cluster: a warp folds its moves in order, the CTA folds its warps in
// order, the cluster folds its CTAs in rank order through distributed shared memory.  The next step's diversity
// kernel adds the slices, in slice order, to the sums it used this step, so no pass over all keys is needed and the
// result does not depend on timing.  Requires nvec <= kCompactSumMaxVec when delta is asked for.
constexpr int kFillSlices = 16;
constexpr int kFillClusterCtas = 8;
static_assert(kFillClusterCtas <= 8, "the cluster folds below read eight ranks at most");
constexpr int kFillThreads = 256;

struct FillArgs {
  uint4* k_cache; uint4* v_cache;
  const int* move_src; const int* move_dst; const int* move_j; const int* n_moves_ptr;
  int max_moves;
  int* slot_meta;
  float* delta;                 // [kFillSlices, C] or nullptr
  int rows_cap, n_meta;         // slots of the K/V buffer, entries of slot_meta (range checks of the checked build)
  int* status;
};

template <int DT>
__device__ __forceinline__ void fill_holes_body(const FillArgs& A, int nvec) {
  constexpr int VEC = VecOf<DT>::n;
  __shared__ __align__(16) float red[4][kCompactSumMaxVec * VEC];
  __shared__ __align__(16) float cta_part[kCompactSumMaxVec * VEC];
  uint4* __restrict__ k_cache = A.k_cache;
  uint4* __restrict__ v_cache = A.v_cache;
  const int* __restrict__ move_src = A.move_src;
  const int* __restrict__ move_dst = A.move_dst;
  const int* __restrict__ move_j = A.move_j;
  const int* __restrict__ n_moves_ptr = A.n_moves_ptr;
  int* __restrict__ slot_meta = A.slot_meta;
  float* __restrict__ delta = A.delta;
  const int max_moves = A.max_moves;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int warps_total = (int)((gridDim.x * (unsigned)blockDim.x) >> 5);
  const int n_moves = min(*n_moves_ptr, max_moves);
  const bool sum = delta != nullptr;
  float acc[4][VEC];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int e = 0; e < VEC; ++e) acc[i][e] = 0.0f;
  for (int m = (int)((blockIdx.x * (unsigned)blockDim.x + threadIdx.x) >> 5); m < n_moves; m += warps_total) {
    const int src = move_src[m], dst = move_dst[m];
    if (!index_ok(src, A.rows_cap, A.status) || !index_ok(dst, A.rows_cap, A.status) ||
        !index_ok(move_j[m], A.n_meta, A.status))
      continue;
    for (int v0 = lane; v0 < nvec; v0 += 128) {
      uint4 uk[4], uv[4], uo[4];
#pragma unroll
      for (int i = 0; i < 4; ++i)
        if (v0 + 32 * i < nvec) {
          uk[i] = ld_nc(k_cache + (size_t)src * nvec + v0 + 32 * i);
          uv[i] = ld_nc(v_cache + (size_t)src * nvec + v0 + 32 * i);
          if (sum) uo[i] = ld_nc(k_cache + (size_t)dst * nvec + v0 + 32 * i);
        }
#pragma unroll
      for (int i = 0; i < 4; ++i)
        if (v0 + 32 * i < nvec) {
          k_cache[(size_t)dst * nvec + v0 + 32 * i] = uk[i];
          v_cache[(size_t)dst * nvec + v0 + 32 * i] = uv[i];
          if (sum) {
            float a[VEC], b[VEC];
            unpack<DT>(uk[i], a);
            unpack<DT>(uo[i], b);
#pragma unroll
            for (int e = 0; e < VEC; ++e) acc[i][e] += a[e] - b[e];
          }
        }
    }
    if (lane == 0) slot_meta[move_j[m]] = dst;
  }
  if (!sum) return;
  // CTA fold: warps 4..7 park, 0..3 add their own, then the four are added in order (as in k_compact_colsum)
  auto park = [&](int slot, bool add) {
#pragma unroll
    for (int i = 0; i < 4; ++i)
      if (lane + 32 * i < nvec)
#pragma unroll
        for (int e = 0; e < VEC; e += 4) {
          float4* p = reinterpret_cast<float4*>(&red[slot][(lane + 32 * i) * VEC + e]);
          float4 t = make_float4(acc[i][e], acc[i][e + 1], acc[i][e + 2], acc[i][e + 3]);
          if (add) {
            const float4 o = *p;
            t.x += o.x; t.y += o.y; t.z += o.z; t.w += o.w;
          }
          *p = t;
        }
  };
  if (warp >= 4) park(warp - 4, false);
  __syncthreads();
  if (warp < 4) park(warp, true);
  __syncthreads();
  const int C = nvec * VEC;
  for (int c = threadIdx.x; c < C; c += blockDim.x) cta_part[c] = ((red[0][c] + red[1][c]) + red[2][c]) + red[3][c];
  // cluster fold through distributed shared memory: CTA r of the cluster owns every 8th group of 32 columns
  cooperative_groups::cluster_group cluster = cooperative_groups::this_cluster();
  cluster.sync();
  const int ncta = (int)cluster.num_blocks(), rank = (int)cluster.block_rank();
  const int cid = (int)blockIdx.x / ncta;
  for (int c = rank * 32 + (threadIdx.x & 31) + (threadIdx.x >> 5) * 32 * ncta; c < C;
       c += 32 * ncta * (blockDim.x >> 5)) {
    float v[8];                                   // all remote reads in flight before the first add (clusters of <= 8)
#pragma unroll
    for (int q = 0; q < 8; ++q) v[q] = q < ncta ? cluster.map_shared_rank(cta_part, q)[c] : 0.0f;
    float t = 0.0f;
#pragma unroll
    for (int q = 0; q < 8; ++q) t += v[q];        // rank order
    delta[(size_t)cid * C + c] = t;
  }
  cluster.sync();   // no CTA may exit while others still read its shared memory
}

template <int DT>
__global__ void __launch_bounds__(kFillThreads) k_fill_holes(uint4* __restrict__ k_cache, uint4* __restrict__ v_cache,
                                                             const int* __restrict__ move_src,
                                                             const int* __restrict__ move_dst,
                                                             const int* __restrict__ move_j,
                                                             const int* __restrict__ n_moves_ptr, int max_moves,
                                                             int nvec, int* __restrict__ slot_meta,
                                                             float* __restrict__ delta /* [kFillSlices, C] or null */,
                                                             int rows_cap, int n_meta, int* status) {
  const FillArgs A{k_cache, v_cache, move_src, move_dst, move_j, n_moves_ptr, max_moves, slot_meta, delta,
                   rows_cap, n_meta, status};
  fill_holes_body<DT>(A, nvec);
}

// Eq. 2 together with the move the previous step left behind.  The hole-filling move of step t and the append of
// step t + 1 touch the same slots - the rows admitted at step t sit in slots >= B, exactly where frame t + 1 goes -
// and nothing reads the cache in between, so one kernel does both and a step has one small launch less on its critical
// path.  A warp owns new row j (slot n + j): if that slot still holds an admitted row (tail_move says which move), the
// warp first carries it down to its destination, then writes the new K/V row over it; program order inside the warp
// is all the ordering this needs.  Meta of the new rows and the corrections of the key column sums as in k_append and
// k_fill_holes.  Launched as kFillSlices clusters of kFillClusterCtas CTAs.
struct AppendFillArgs {
  const uint4* k_new; const uint4* v_new;     // the frame's rows [M, C]
  int M, n; long long frame_id;
  uint4* k_cache; uint4* v_cache;
  long long* ids; uint8_t* flags; float* stored; int* slot;   // meta of the layer, logical order
  float* kmax2;                               // running bound of the key norms, or nullptr
  int B;                                      // slots >= B may hold rows that still have to move
  const int* tail_move; const int* move_dst; const int* move_j; const int* n_moves_ptr;   // nullptr: nothing pending
  float* delta;                               // [kFillSlices, C] or nullptr
  int* status;                                // where the checked build reports a bad move index
};

constexpr int kAppendFillThreads = 384;      // 16 clusters x 8 CTAs x 12 warps: a warp per row up to 1536 new rows

template <int DT>
__global__ void __launch_bounds__(kAppendFillThreads) k_append_fill(const __grid_constant__ AppendFillArgs A, int nvec) {
  constexpr int VEC = VecOf<DT>::n;
  __shared__ __align__(16) float red[4][kCompactSumMaxVec * VEC];
  __shared__ __align__(16) float cta_part[kCompactSumMaxVec * VEC];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int gtid = blockIdx.x * blockDim.x + threadIdx.x;
  const int warps_total = (int)((gridDim.x * (unsigned)blockDim.x) >> 5);
  const bool pending = A.tail_move != nullptr;
  const bool sum = A.delta != nullptr;
  float acc[4][VEC];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int e = 0; e < VEC; ++e) acc[i][e] = 0.0f;
  for (int j = gtid >> 5; j < A.M; j += warps_total) {
    const int s = A.n + j;                                   // the new row's slot
    const bool tail = pending && s >= A.B && s - A.B < A.M;
    // everything that does not depend on another load goes out first: the move's index, the number of moves, the
    // new rows, and (speculatively, when a move may be pending for this slot) the rows that sit in the slot
    int m = tail ? A.tail_move[s - A.B] : -1;
    const int n_moves = tail ? min(*A.n_moves_ptr, A.M) : 0;
    uint4 nk[4], nv[4], uk[4], uv[4], uo[4];
    const int first = lane;                                  // rows longer than 128 vectors take further rounds below
#pragma unroll
    for (int i = 0; i < 4; ++i)
      if (first + 32 * i < nvec) {
        nk[i] = ld_nc(A.k_new + (size_t)j * nvec + first + 32 * i);
        nv[i] = ld_nc(A.v_new + (size_t)j * nvec + first + 32 * i);
        if (tail) {   // (plain loads: these cache lines are rewritten by this very kernel)
          uk[i] = A.k_cache[(size_t)s * nvec + first + 32 * i];
          uv[i] = A.v_cache[(size_t)s * nvec + first + 32 * i];
        }
      }
    // (a warp collective: every lane of the warp is here, whatever part of the row it holds; rows of up to 128
    //  vectors only, which is all the bound is kept for)
    if (A.kmax2 != nullptr) warp_key_norm_max(nk, nvec, lane, A.kmax2);
    if (m >= n_moves) m = -1;
    int dst = m >= 0 ? A.move_dst[m] : 0;
    if (m >= 0 && (!index_ok(dst, A.B, A.status) || !index_ok(A.move_j[m], A.B, A.status))) m = -1;
    for (int v0 = lane; v0 < nvec; v0 += 128) {
      if (v0 != lane) {
#pragma unroll
        for (int i = 0; i < 4; ++i)
          if (v0 + 32 * i < nvec) {
            nk[i] = ld_nc(A.k_new + (size_t)j * nvec + v0 + 32 * i);
            nv[i] = ld_nc(A.v_new + (size_t)j * nvec + v0 + 32 * i);
            if (m >= 0) {
              uk[i] = A.k_cache[(size_t)s * nvec + v0 + 32 * i];
              uv[i] = A.v_cache[(size_t)s * nvec + v0 + 32 * i];
            }
          }
      }
      if (m >= 0 && sum) {
#pragma unroll
        for (int i = 0; i < 4; ++i)
          if (v0 + 32 * i < nvec) uo[i] = A.k_cache[(size_t)dst * nvec + v0 + 32 * i];
      }
#pragma unroll
      for (int i = 0; i < 4; ++i)
        if (v0 + 32 * i < nvec) {
          if (m >= 0) {
            A.k_cache[(size_t)dst * nvec + v0 + 32 * i] = uk[i];
            A.v_cache[(size_t)dst * nvec + v0 + 32 * i] = uv[i];
            if (sum) {
              float a[VEC], b[VEC];
              unpack<DT>(uk[i], a);
              unpack<DT>(uo[i], b);
#pragma unroll
              for (int e = 0; e < VEC; ++e) acc[i][e] += a[e] - b[e];
            }
          }
          A.k_cache[(size_t)s * nvec + v0 + 32 * i] = nk[i];
          A.v_cache[(size_t)s * nvec + v0 + 32 * i] = nv[i];
        }
    }
    if (lane == 0) {
      if (m >= 0) A.slot[A.move_j[m]] = dst;
      A.ids[s] = A.frame_id * (long long)A.M + j;
      A.flags[s] = OVGGT_FLAG_EVICTABLE;
      A.stored[s] = 0.0f;
      A.slot[s] = s;
    }
  }
  if (!sum) return;
  // CTA fold in a fixed order: warps 8..11 park their sums in the four slots, 4..7 add theirs, 0..3 add theirs, then
  // the four slots are added in order
  auto park = [&](int slot_, bool add) {
#pragma unroll
    for (int i = 0; i < 4; ++i)
      if (lane + 32 * i < nvec)
#pragma unroll
        for (int e = 0; e < VEC; e += 4) {
          float4* p = reinterpret_cast<float4*>(&red[slot_][(lane + 32 * i) * VEC + e]);
          float4 t = make_float4(acc[i][e], acc[i][e + 1], acc[i][e + 2], acc[i][e + 3]);
          if (add) {
            const float4 o = *p;
            t.x += o.x; t.y += o.y; t.z += o.z; t.w += o.w;
          }
          *p = t;
        }
  };
  static_assert(kAppendFillThreads == 384, "the fold below is written for twelve warps");
  if (warp >= 8) park(warp - 8, false);
  __syncthreads();
  if (warp >= 4 && warp < 8) park(warp - 4, true);
  __syncthreads();
  if (warp < 4) park(warp, true);
  __syncthreads();
  const int C = nvec * VEC;
  for (int c = threadIdx.x; c < C; c += blockDim.x) cta_part[c] = ((red[0][c] + red[1][c]) + red[2][c]) + red[3][c];
  cooperative_groups::cluster_group cluster = cooperative_groups::this_cluster();
  cluster.sync();
  const int ncta = (int)cluster.num_blocks(), rank = (int)cluster.block_rank();
  const int cid = (int)blockIdx.x / ncta;
  for (int c = rank * 32 + (threadIdx.x & 31) + (threadIdx.x >> 5) * 32 * ncta; c < C;
       c += 32 * ncta * (blockDim.x >> 5)) {
    float v[8];                                   // all remote reads in flight before the first add (clusters of <= 8)
#pragma unroll
    for (int q = 0; q < 8; ++q) v[q] = q < ncta ? cluster.map_shared_rank(cta_part, q)[c] : 0.0f;
    float t = 0.0f;
#pragma unroll
    for (int q = 0; q < 8; ++q) t += v[q];        // rank order, as a loop over the ranks would add them
    A.delta[(size_t)cid * C + c] = t;
  }
  cluster.sync();   // no CTA may exit while others still read its shared memory
}

}  // namespace ovggt
