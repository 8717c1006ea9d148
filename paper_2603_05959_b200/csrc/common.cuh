// Shared device helpers of the OVGGT step kernels: element access, block primitives.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/ovggt.h"

namespace ovggt {

constexpr int kF32 = OVGGT_DTYPE_F32;
constexpr int kBF16 = OVGGT_DTYPE_BF16;

// Elements per 16-byte vector of a stored row.
template <int DT> struct VecOf { static constexpr int n = (DT == kBF16) ? 8 : 4; };

__host__ __device__ inline int elem_bytes(int dtype) { return dtype == kBF16 ? 2 : 4; }

// Expand one 16-byte vector of stored elements to floats (exact).
template <int DT>
__device__ __forceinline__ void unpack(const uint4& u, float* f) {
  if constexpr (DT == kBF16) {
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      f[2 * i] = __uint_as_float(w[i] << 16);
      f[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
  } else {
    f[0] = __uint_as_float(u.x);
    f[1] = __uint_as_float(u.y);
    f[2] = __uint_as_float(u.z);
    f[3] = __uint_as_float(u.w);
  }
}

__device__ __forceinline__ uint4 ld_nc(const uint4* p) {
  uint4 r;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
               : "l"(p));
  return r;
}

// Sum over the warp in a fixed butterfly order; every lane gets the result.
__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xFFFFFFFFu, x, o);
  return x;
}

// Priority -> unsigned key whose integer order is the ranking order:
// NaN ranks with -inf, -0 equals +0, larger float = larger key.
__device__ __forceinline__ uint32_t rank_key(float x) {
  if (x != x) x = -INFINITY;
  if (x == 0.0f) x = 0.0f;
  uint32_t u = __float_as_uint(x);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// One output step of the SplitMix64 generator from state x (Steele, Lea, Flood 2014), and the uniform priority in
// [0, 1) that the random-eviction mode gives token `token_id` in the step of frame `frame_id`: the top 24 bits of
// SplitMix64(SplitMix64(seed ^ frame_id) + token_id), exact in fp32.
__host__ __device__ __forceinline__ unsigned long long splitmix64(unsigned long long x) {
  unsigned long long z = x + 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}
__host__ __device__ __forceinline__ float random_priority(unsigned long long step_key, long long token_id) {
  return (float)(splitmix64(step_key + (unsigned long long)token_id) >> 40) * (1.0f / 16777216.0f);
}

// Range check of an index that a kernel has read from device memory (survivor lists, slots, move lists).  In the
// ordinary build it costs nothing.  Built with -DOVGGT_BOUNDS_CHECK, an index outside [0, n) is not used: the access
// is skipped and OVGGT_ERR_DEVICE_STATUS goes to the status word, which the next ovggt_cache_stats reports - no trap,
// the kernel runs to its end.
#ifdef OVGGT_BOUNDS_CHECK
__device__ __forceinline__ bool index_ok(long long i, long long n, int* status) {
  if (i >= 0 && i < n) return true;
  if (status != nullptr) atomicCAS(status, 0, OVGGT_ERR_DEVICE_STATUS);
  return false;
}
#else
__device__ __forceinline__ bool index_ok(long long, long long, int*) { return true; }
#endif

// ---- block-wide primitives for a block of up to 1024 threads; `sh` holds >= 33 words.

__device__ inline int block_sum_int(int x, int* sh) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = (blockDim.x + 31) >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xFFFFFFFFu, x, o);
  __syncthreads();
  if (lane == 0) sh[warp] = x;
  __syncthreads();
  int t = 0;
  for (int w = 0; w < nwarp; ++w) t += sh[w];
  return t;
}

// Exclusive prefix sum of x over the threads of the block in thread order; *total = block sum.
__device__ __noinline__ int block_excl_scan_int(int x, int* sh, int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = (blockDim.x + 31) >> 5;
  int incl = x;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int y = __shfl_up_sync(0xFFFFFFFFu, incl, o);
    if (lane >= o) incl += y;
  }
  __syncthreads();
  if (lane == 31) sh[warp] = incl;
  __syncthreads();
  int base = 0, tot = 0;
  for (int w = 0; w < nwarp; ++w) {
    if (w < warp) base += sh[w];
    tot += sh[w];
  }
  *total = tot;
  return base + incl - x;
}

__device__ __noinline__ void block_minmax(float lo, float hi, float* sh, float* out_lo, float* out_hi) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = (blockDim.x + 31) >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    lo = fminf(lo, __shfl_xor_sync(0xFFFFFFFFu, lo, o));
    hi = fmaxf(hi, __shfl_xor_sync(0xFFFFFFFFu, hi, o));
  }
  __syncthreads();
  if (lane == 0) {
    sh[warp] = lo;
    sh[32 + warp] = hi;
  }
  __syncthreads();
  float a = sh[0], b = sh[32];
  for (int w = 1; w < nwarp; ++w) {
    a = fminf(a, sh[w]);
    b = fmaxf(b, sh[32 + w]);
  }
  *out_lo = a;
  *out_hi = b;
}

}  // namespace ovggt
