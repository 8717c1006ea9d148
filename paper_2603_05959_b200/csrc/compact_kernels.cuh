// Cache append (Eq. 2) and order-preserving compaction of the surviving rows (Eq. 8).
// Rows are 16-byte-vector arrays; one warp moves one K or V row at a time with all of its
// loads issued before its stores, so many independent 16-byte transactions are in flight per SM.
#pragma once

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
                                                 uint4* __restrict__ k_dst, uint4* __restrict__ v_dst) {
  const int lane = threadIdx.x & 31;
  const int warps_total = (int)((gridDim.x * (unsigned)blockDim.x) >> 5);
  for (int item = (int)((blockIdx.x * (unsigned)blockDim.x + threadIdx.x) >> 5); item < 2 * n_keep;
       item += warps_total) {
    const int j = item >> 1;
    const int src = survivors[j];
    if (item & 1) warp_copy_row(v_src + (size_t)src * nvec, v_dst + (size_t)j * nvec, nvec, lane);
    else          warp_copy_row(k_src + (size_t)src * nvec, k_dst + (size_t)j * nvec, nvec, lane);
  }
}

// Rows [n, n+M) of the cache := the frame's K and V; their meta: ids frame*M + j, evictable, score 0.
__global__ void __launch_bounds__(256) k_append(const uint4* __restrict__ k_new, const uint4* __restrict__ v_new,
                                                int M, int nvec, int n, long long frame_id,
                                                uint4* __restrict__ k_cache, uint4* __restrict__ v_cache,
                                                long long* __restrict__ ids, uint8_t* __restrict__ flags,
                                                float* __restrict__ stored) {
  const int lane = threadIdx.x & 31;
  const int gtid = blockIdx.x * blockDim.x + threadIdx.x;
  const int warps_total = (int)((gridDim.x * (unsigned)blockDim.x) >> 5);
  for (int item = gtid >> 5; item < 2 * M; item += warps_total) {
    const int j = item >> 1;
    if (item & 1) warp_copy_row(v_new + (size_t)j * nvec, v_cache + (size_t)(n + j) * nvec, nvec, lane);
    else          warp_copy_row(k_new + (size_t)j * nvec, k_cache + (size_t)(n + j) * nvec, nvec, lane);
  }
  for (int j = gtid; j < M; j += gridDim.x * blockDim.x) {
    ids[n + j] = frame_id * (long long)M + j;
    flags[n + j] = OVGGT_FLAG_EVICTABLE;
    stored[n + j] = 0.0f;
  }
}

}  // namespace ovggt
