// bf16 GEMM for sm_100a: C [M, N] = A [M, K] x B [K, N], row-major, fp32 accumulation in tensor memory.
//
// Not part of the streaming step itself: it is what a model wraps around it (QKV / output projections, MLP), provided
// so that the 24-layer workloads can run their scaffold on hand-written kernels too.  Built from the same pieces as
// the attention kernel (TMA with 128-byte swizzle, mbarriers, tcgen05.mma issued by one elected lane, tcgen05.ld
// epilogue), in the simplest arrangement that keeps the tensor pipe fed:
//   CTA tile 128 x 128, K in steps of 64: A tile [128 rows, 64 k] K-major (16 KB), B tile [64 k, 128 n] as two
//   [64 k, 64 n] boxes, N-major as the tensor lies in memory (2 x 8 KB); four stages (128 KB of shared memory);
//   warp 0 produces (TMA), warp 1 issues the MMAs (two N = 64 MMAs per 16 k, accumulators in TMEM columns [0, 128)),
//   warps 2-5 read the accumulators back (one thread per output row), round to bf16 and store.
// Requirements: K a multiple of 64, N a multiple of 8 (TMA row pitch of 16 bytes), 16-byte aligned bases.  Every
// barrier wait is bounded (about one second); on expiry the CTA records OVGGT_ERR_TIMEOUT and leaves through the
// common teardown, after the MMAs it issued have drained.
#pragma once

#include "attn_tcgen05.cuh"

namespace ovggt {

constexpr int kGemmBM = 128, kGemmBN = 128, kGemmBK = 64, kGemmStages = 4;
constexpr int kGemmThreads = 192;
constexpr int kGemmATile = kGemmBM * kGemmBK * 2;          // 16 KB
constexpr int kGemmBBox = kGemmBK * 64 * 2;                // 8 KB: [64 k, 64 n]
constexpr int kGemmBTile = 2 * kGemmBBox;                  // 16 KB
constexpr int kGemmTmemCols = 128;

struct GemmBarriers {
  unsigned long long full[kGemmStages], empty[kGemmStages], acc_full, drain;
  uint32_t tmem_base;
  int abort_flag;
};
constexpr size_t kGemmSmemBytes = (size_t)kGemmStages * (kGemmATile + kGemmBTile) + sizeof(GemmBarriers) + 64;

// The bounded wait of the attention kernel, for a barrier block of another shape.
__device__ __forceinline__ bool gemm_wait(void* bar, uint32_t parity, GemmBarriers* B, int* status) {
  if (mbar_try_wait(bar, parity)) return true;
  unsigned long long t0 = 0;
  for (uint32_t spins = 1;; ++spins) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((spins & 1023u) == 0) {
      if (*(volatile int*)&B->abort_flag) return false;
      const unsigned long long now = global_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > kWaitLimitNs) {
        *(volatile int*)&B->abort_flag = 1;
        atomicCAS(status, 0, OVGGT_ERR_TIMEOUT);
        return false;
      }
    }
  }
}

__global__ void __launch_bounds__(kGemmThreads, 1)
k_gemm_bf16_tcgen05(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                    __nv_bfloat16* __restrict__ C, int M, int N, int K, int* status) {
  extern __shared__ __align__(1024) unsigned char smem[];
  if (smem_u32(smem) & 1023u) {
    if (threadIdx.x == 0) atomicCAS(status, 0, OVGGT_ERR_DEVICE_STATUS);
    return;
  }
  unsigned char* sA = smem;
  unsigned char* sB = sA + kGemmStages * kGemmATile;
  GemmBarriers* B = reinterpret_cast<GemmBarriers*>(sB + kGemmStages * kGemmBTile);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m0 = blockIdx.y * kGemmBM, n0 = blockIdx.x * kGemmBN;
  const int k_tiles = K / kGemmBK;

  if (warp == 0 && lane == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_a) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_b) : "memory");
    for (int s = 0; s < kGemmStages; ++s) {
      mbar_init(&B->full[s], 1);
      mbar_init(&B->empty[s], 1);
    }
    mbar_init(&B->acc_full, 1);
    mbar_init(&B->drain, 1);
    B->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&B->tmem_base)),
                 "r"((uint32_t)kGemmTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *(volatile uint32_t*)&B->tmem_base;

  if (warp == 0) {
    // ------------------------------------------------ TMA producer
    if (lane == 0) {
      int issued = 0;
      bool ok = true;
      for (int kt = 0; kt < k_tiles && ok; ++kt) {
        const int s = kt % kGemmStages;
        const uint32_t ph = (uint32_t)(kt / kGemmStages) & 1u;
        if (kt >= kGemmStages) ok = gemm_wait(&B->empty[s], ph ^ 1u, B, status);
        if (!ok) break;
        mbar_expect_tx(&B->full[s], kGemmATile + kGemmBTile);
        tma_load_2d(sA + s * kGemmATile, &tm_a, kt * kGemmBK, m0, &B->full[s]);
        tma_load_2d(sB + s * kGemmBTile, &tm_b, n0, kt * kGemmBK, &B->full[s]);
        tma_load_2d(sB + s * kGemmBTile + kGemmBBox, &tm_b, n0 + 64, kt * kGemmBK, &B->full[s]);
        ++issued;
      }
      if (!ok)   // leave no bulk copy in flight into this CTA's shared memory
        for (int i = max(0, issued - kGemmStages); i < issued; ++i)
          gemm_wait(&B->full[i % kGemmStages], (uint32_t)(i / kGemmStages) & 1u, B, status);
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------ MMA issuer (whole warp in step, one elected lane issues)
    const bool leader = elect_one();
    const uint32_t tm = __reduce_or_sync(0xFFFFFFFFu, tmem);
    constexpr uint32_t idesc = idesc_bf16(64, true);            // A K-major, B N-major, N = 64
    bool ok = true;
    for (int kt = 0; kt < k_tiles && ok; ++kt) {
      const int s = kt % kGemmStages;
      const uint32_t ph = (uint32_t)(kt / kGemmStages) & 1u;
      ok = __all_sync(0xFFFFFFFFu, gemm_wait(&B->full[s], ph, B, status)) != 0;
      if (!ok) break;
      tc_fence_after();
      const uint64_t da = smem_desc_sw128(smem_u32(sA + s * kGemmATile));
      if (leader) {
#pragma unroll
        for (int nb = 0; nb < 2; ++nb) {
          const uint64_t db = smem_desc_sw128(smem_u32(sB + s * kGemmBTile + nb * kGemmBBox));
#pragma unroll
          for (int kk = 0; kk < kGemmBK / 16; ++kk)   // A: 16 k = 32 bytes inside the swizzled row; B: 16 k-rows = 2048 bytes
            mma_ss(tm + nb * 64, da + (uint64_t)(kk * 2), db + (uint64_t)(kk * 128), idesc, (kt > 0 || kk > 0));
        }
        tc_commit(&B->empty[s]);
      }
    }
    if (ok) {
      if (leader) tc_commit(&B->acc_full);
    } else {
      if (leader) tc_commit(&B->drain);             // let every issued MMA finish before TMEM is freed
      __all_sync(0xFFFFFFFFu, gemm_wait(&B->drain, 0, B, status));
    }
    __syncwarp();
  } else {
    // ------------------------------------------------ epilogue: warps 2..5 own the TMEM lane quarters 2, 3, 0, 1
    const int quad = warp & 3;
    const int row = quad * 32 + lane;
    const uint32_t t_row = tmem + ((uint32_t)(quad * 32) << 16);
    const bool ok = __all_sync(0xFFFFFFFFu, gemm_wait(&B->acc_full, 0, B, status)) != 0;
    if (ok) {
      tc_fence_after();
      const int m = m0 + row;
#pragma unroll
      for (int j = 0; j < kGemmBN / 32; ++j) {
        uint32_t o[32];
        tmem_ld32(t_row + j * 32, o);
        tmem_wait_ld();
        if (m < M) {
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int n = n0 + j * 32 + e * 8;
            if (n < N) {                              // N is a multiple of 8: a group of 8 columns is in or out
              uint4 w;
              w.x = pack_bf16(__uint_as_float(o[8 * e + 0]), __uint_as_float(o[8 * e + 1]));
              w.y = pack_bf16(__uint_as_float(o[8 * e + 2]), __uint_as_float(o[8 * e + 3]));
              w.z = pack_bf16(__uint_as_float(o[8 * e + 4]), __uint_as_float(o[8 * e + 5]));
              w.w = pack_bf16(__uint_as_float(o[8 * e + 6]), __uint_as_float(o[8 * e + 7]));
              *reinterpret_cast<uint4*>(C + (size_t)m * N + n) = w;
            }
          }
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)kGemmTmemCols) : "memory");
  }
}

// [rows, cols] bf16 row-major; box = 64 columns x box_rows rows, 128-byte swizzle, zero fill outside.
inline int gemm_tcgen05_launch(const void* A, const void* Bm, void* C, int M, int N, int K, int* status, cudaStream_t st) {
  CUtensorMap ta, tb;
  int rc = make_rows_map(&ta, A, M, K, kGemmBM);       // 64 k-columns x 128 rows per box
  if (rc) return rc;
  rc = make_rows_map(&tb, Bm, K, N, kGemmBK);          // 64 n-columns x 64 k-rows per box
  if (rc) return rc;
  static cudaError_t attr = cudaFuncSetAttribute(k_gemm_bf16_tcgen05, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                 (int)kGemmSmemBytes);
  if (attr != cudaSuccess) { g_attn_last_error = (int)attr; return OVGGT_ERR_CUDA; }
  dim3 grid((N + kGemmBN - 1) / kGemmBN, (M + kGemmBM - 1) / kGemmBM);
  k_gemm_bf16_tcgen05<<<grid, kGemmThreads, kGemmSmemBytes, st>>>(ta, tb, static_cast<__nv_bfloat16*>(C), M, N, K, status);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) { g_attn_last_error = (int)e; return OVGGT_ERR_CUDA; }
  return OVGGT_OK;
}

}  // namespace ovggt
