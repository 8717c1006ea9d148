// bf16 flash attention for sm_100a: out = softmax(Q K^T / sqrt(64)) V per head, head_dim 64, no mask.
//
// One CTA owns one 128-row query tile of one head and a contiguous range of 192-row KV tiles.  Each KV
// tile is processed as two 96-row halves with their own S buffer in tensor memory, so the MMAs of one half
// run while the softmax warps work on the other and the softmax never waits for a whole QK^T -> PV chain.
//   warps 0-3   softmax: one thread per query row reads its 96 S values of a half with tcgen05.ld and turns them into
//               p = 2^(s c - reference).  Where the cache supplies a bound of the key norms, the reference is fixed
//               once (the bound of this row's logits, moved a whole number of powers of two above the first half's
//               maximum): nothing is tracked and O is never rescaled.  Without a bound the reference is a running
//               maximum, gathered inside the exponential pass, and O is rescaled only when it grows by more than 2^8
//               (the pass is then repeated).  One pair of exponentials in three is a cubic on the FMA pipes, the rest
//               go to the special-function unit; P is written as bf16 over the first 48 columns of that half; at
//               the end the warps normalise and store O (or the split's partial O, maximum and sum)
//   warp 4      TMA producer: Q once, then K and V tiles into 128-byte-swizzled shared-memory stages
//   warp 5      allocates tensor memory and issues tcgen05.mma:  S_h = Q K_h^T  (SS, fp32 in TMEM),
//               O += P_h V_h (P read from TMEM as the A operand, V MN-major from shared memory); the whole warp
//               walks the loop so that descriptors stay warp-uniform, one elected lane issues
//   warps 6-7   only complete the second warpgroup, which hands its registers to the softmax warpgroup
// With head_dim 64 a 128 x 128 tile needs 512 tensor-pipe cycles but 1024 cycles of the 16-per-clock
// exponential unit, so the softmax rounds bound the kernel (a 96-column round is about 1,700 cycles, 1,200 of them
// the exponential pass, whose instruction mix tops out near 0.15 columns per cycle per scheduler); two CTAs are
// resident per SM (256 TMEM columns and ~115 KB shared memory each) to keep that unit fed from two independent query
// tiles.  The KV range may be split across CTAs; partial (O, max, sum) triples are merged by a second kernel.  Every
// mbarrier wait is bounded: on expiry the CTA records OVGGT_ERR_TIMEOUT in the status word and leaves through the
// common teardown.
#pragma once

#include <cuda.h>

#include <algorithm>
#include <type_traits>

#include "common.cuh"

namespace ovggt {

constexpr int kBM = 128;            // query rows per CTA
constexpr int kBN = 192;            // KV rows per tile
constexpr int kCtasPerSm = 2;       // resident CTAs per SM
constexpr int kHD = 64;             // head dim
constexpr int kKVStages = 2;
constexpr int kAttnThreads = 256;
// setmaxnreg only moves registers inside the pool the CTA was launched with (threads x launch registers), and an
// increase that the pool cannot serve waits for ever: the two warpgroups must fit 256 x 128.
constexpr int kRegsLaunch = 128;    // what __launch_bounds__(256, 2) gives: 65536 / 512
constexpr int kRegsSoftmax = 216, kRegsOther = 40;
static_assert(128 * kRegsSoftmax + 128 * kRegsOther <= kAttnThreads * kRegsLaunch, "register pool of the CTA exceeded");
constexpr int kQBytes = kBM * kHD * 2;           // 16 KB
constexpr int kTileBytes = kBN * kHD * 2;          // 24 KB
constexpr int kHalf = kBN / 2;      // KV rows per S buffer
constexpr int kTmemCols = 256;
constexpr int kColS = 0, kColO = 2 * kHalf;   // S_0 at columns [0, 96), S_1 at [96, 192), O at [192, 256): all 256 columns
constexpr float kRescaleThreshold = 8.0f;          // log2 units
// A row whose logits have a known upper bound (|q| x the largest |k| of the cache, Cauchy-Schwarz) may take that bound
// as its softmax reference for good: nothing can outgrow it, so the maximum need not be tracked and O never rescaled.
// The price is that every exponential comes out 2^-(bound - true maximum) smaller than it could; fp32 sums and bf16
// probabilities keep their relative precision as long as that stays far from the underflow threshold (2^-126).
constexpr float kFixedRefMaxGap = 48.0f;           // log2 units between the bound and the first half's true maximum
#ifndef OVGGT_ATTN_POLY_NUM
#define OVGGT_ATTN_POLY_NUM 1
#define OVGGT_ATTN_POLY_DEN 3
#endif
// kPolyNum pairs of exponentials in every kPolyDen go to the FMA pipes instead of the special-function unit
constexpr int kPolyNum = OVGGT_ATTN_POLY_NUM, kPolyDen = OVGGT_ATTN_POLY_DEN;
__host__ __device__ constexpr bool pair_on_fma_pipes(int pair) { return (pair * kPolyNum) % kPolyDen < kPolyNum; }
constexpr int kMaxSplits = 16;

struct AttnBarriers {
  unsigned long long q_full, s_full[2], p_full[2], pv_done, o_full, drain;
  unsigned long long k_full[kKVStages], k_empty[kKVStages], v_full[kKVStages], v_empty[kKVStages];
  uint32_t tmem_base;
  int abort_flag;
};

// (no slack for aligning the base by hand: two CTAs of 114.9 KB must fit one SM; the base is checked instead)
constexpr size_t kAttnSmemBytes = (size_t)kQBytes + (size_t)kTileBytes * 2 * kKVStages + sizeof(AttnBarriers) + 64;

// ---------------------------------------------------------------- PTX wrappers

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(void* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(void* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(void* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(void* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
// Wait for the phase with the given parity, for at most limit_ns (about one second unless stated).  On expiry the
// CTA's abort flag is raised, OVGGT_ERR_TIMEOUT goes to the status word and the caller gets false; so does every
// other waiter of the CTA the next time it looks at the flag.
constexpr unsigned long long kWaitLimitNs = 1000000000ull;
__device__ __forceinline__ bool mbar_wait(void* bar, uint32_t parity, AttnBarriers* B, int* status,
                                          unsigned long long limit_ns = kWaitLimitNs) {
  if (mbar_try_wait(bar, parity)) return true;
  unsigned long long t0 = 0;
  for (uint32_t spins = 1;; ++spins) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((spins & 1023u) == 0) {
      if (*(volatile int*)&B->abort_flag) return false;
      const unsigned long long now = global_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > limit_ns) {
        *(volatile int*)&B->abort_flag = 1;
        atomicCAS(status, 0, OVGGT_ERR_TIMEOUT);
        return false;
      }
    }
  }
}

__device__ __forceinline__ void tma_load_2d(void* smem_dst, const CUtensorMap* map, int x, int y, void* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(smem_u32(smem_dst)), "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar))
      : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(void* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}

// Shared-memory matrix descriptor for a 128-byte-swizzled tile whose 8-row groups are 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
  d |= (uint64_t)1 << 16;                  // leading byte offset (unused for one swizzle atom): 16 B
  d |= (uint64_t)(1024 >> 4) << 32;        // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;                  // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                  // 128-byte swizzle
  return d;
}

// Instruction descriptor: bf16 x bf16 -> fp32, M = 128.
__host__ __device__ constexpr uint32_t idesc_bf16(int n, bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((uint32_t)(n >> 3) << 17) |
         ((uint32_t)(128 >> 4) << 24);
}

__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
      " tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n" ::"r"(d_tmem), "l"(a_desc), "l"(b_desc),
      "r"(idesc), "r"(acc)
      : "memory");
}
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
      " tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}\n" ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc),
      "r"(idesc), "r"(acc)
      : "memory");
}

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
      "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
      "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]),
      "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]),
      "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
      "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
// (a.x * b.x + c.x, a.y * b.y + c.y) and (a.x + b.x, a.y + b.y) as single packed instructions
__device__ __forceinline__ float2 fma2(float2 a, float2 b, float2 c) {
  float2 d;
  asm("{\n .reg .b64 ra, rb, rc, rd;\n mov.b64 ra, {%2, %3};\n mov.b64 rb, {%4, %5};\n mov.b64 rc, {%6, %7};\n"
      " fma.rn.f32x2 rd, ra, rb, rc;\n mov.b64 {%0, %1}, rd;\n}\n"
      : "=f"(d.x), "=f"(d.y)
      : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y), "f"(c.x), "f"(c.y));
  return d;
}
__device__ __forceinline__ float2 add2(float2 a, float2 b) {
  float2 d;
  asm("{\n .reg .b64 ra, rb, rd;\n mov.b64 ra, {%2, %3};\n mov.b64 rb, {%4, %5};\n"
      " add.rn.f32x2 rd, ra, rb;\n mov.b64 {%0, %1}, rd;\n}\n"
      : "=f"(d.x), "=f"(d.y)
      : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
  return d;
}
// True in exactly one lane of a converged warp.
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile(
      "{\n\t.reg .pred p;\n\telect.sync _|p, 0xFFFFFFFF;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(pred));
  return pred != 0;
}
// 2^x for a pair on the FMA pipes, for the share of the exponentials taken off the 16-per-clock special-function
// unit: x = n + f with n = round(x) (magic-number rounding) and f in [-0.5, 0.5], a cubic for 2^f (Chebyshev nodes,
// relative error 1e-4, below bf16 rounding), and n added into the exponent field.  x is clamped at -125 so that the
// exponent field cannot wrap; larger x than the rescale threshold only occurs in a pass whose result is discarded.
__device__ __forceinline__ float2 ex2_poly2(float2 x) {
  const float kMagic = 12582912.0f;                  // 1.5 * 2^23
  x.x = fmaxf(x.x, -125.0f);
  x.y = fmaxf(x.y, -125.0f);
  const float2 t = add2(x, make_float2(kMagic, kMagic));
  const float2 n = add2(t, make_float2(-kMagic, -kMagic));
  const float2 f = fma2(n, make_float2(-1.0f, -1.0f), x);
  float2 p = fma2(f, make_float2(0.05583828315138817f, 0.05583828315138817f),
                  make_float2(0.2426394820213318f, 0.2426394820213318f));
  p = fma2(p, f, make_float2(0.6931367516517639f, 0.6931367516517639f));
  p = fma2(p, f, make_float2(0.9999245405197144f, 0.9999245405197144f));
  return make_float2(__int_as_float(__float_as_int(p.x) + (__float_as_int(t.x) << 23)),
                     __int_as_float(__float_as_int(p.y) + (__float_as_int(t.y) << 23)));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  uint32_t d;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}

// ---------------------------------------------------------------- the kernel

struct AttnParams {
  int M, N, H;
  int splits, tiles_per_split, tiles_total;
  const float* kmax2;     // [H] upper bound of |k_j,h|^2 over all N keys, or nullptr (the maximum is tracked)
  __nv_bfloat16* out;     // [M, C]            (splits == 1)
  float* o_part;          // [splits, M, C]    un-normalised partial outputs
  float2* ml_part;        // [splits, M, H]    (reference maximum in log2 units, row sum)
  float* lse;             // [M, H] or nullptr: log2 of each row's softmax denominator (reference + log2 of the sum)
  int* status;
};

__global__ void __launch_bounds__(kAttnThreads, kCtasPerSm)
k_attn_tcgen05(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
               const __grid_constant__ CUtensorMap tm_v, const AttnParams P) {
  extern __shared__ __align__(1024) unsigned char smem[];
  if (smem_u32(smem) & 1023u) {                      // the 128-byte swizzle needs 1024-byte aligned tiles
    if (threadIdx.x == 0) atomicCAS(P.status, 0, OVGGT_ERR_DEVICE_STATUS);
    return;
  }
  unsigned char* sQ = smem;
  unsigned char* sK = sQ + kQBytes;
  unsigned char* sV = sK + kKVStages * kTileBytes;
  AttnBarriers* B = reinterpret_cast<AttnBarriers*>(sV + kKVStages * kTileBytes);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int qt = blockIdx.x, h = blockIdx.y, split = blockIdx.z;
  const int t_begin = split * P.tiles_per_split;
  const int n_tiles = min(P.tiles_total, t_begin + P.tiles_per_split) - t_begin;   // >= 1 by construction
  const int C = P.H * kHD;

  // The producer's elected thread sets the barriers up and sends the first loads (Q and the first K/V tile) on their
  // way at once, so that they travel while tensor memory is allocated and the CTA meets at its first barrier.
  if (warp == 4 && lane == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_q) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_k) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_v) : "memory");
    mbar_init(&B->q_full, 1);
    for (int hf = 0; hf < 2; ++hf) {
      mbar_init(&B->s_full[hf], 1);
      mbar_init(&B->p_full[hf], 128);
    }
    mbar_init(&B->pv_done, 1);
    mbar_init(&B->o_full, 1);
    mbar_init(&B->drain, 1);
    for (int s = 0; s < kKVStages; ++s) {
      mbar_init(&B->k_full[s], 1);
      mbar_init(&B->k_empty[s], 1);
      mbar_init(&B->v_empty[s], 1);
      mbar_init(&B->v_full[s], 1);
    }
    B->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    mbar_expect_tx(&B->q_full, kQBytes);
    tma_load_2d(sQ, &tm_q, h * kHD, qt * kBM, &B->q_full);
    mbar_expect_tx(&B->k_full[0], kTileBytes);
    tma_load_2d(sK, &tm_k, h * kHD, t_begin * kBN, &B->k_full[0]);
    mbar_expect_tx(&B->v_full[0], kTileBytes);
    tma_load_2d(sV, &tm_v, h * kHD, t_begin * kBN, &B->v_full[0]);
  }
  if (warp == 5) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&B->tmem_base)),
                 "r"((uint32_t)kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *(volatile uint32_t*)&B->tmem_base;

  if (warp >= 4) {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsOther));
  if (warp == 4) {
    // ------------------------------------------------ TMA producer
    if (lane == 0) {
      int issued_k = 1, issued_v = 1;                // Q and tile 0 were sent during set-up
      bool ok = true;
      for (int it = 1; it < n_tiles && ok; ++it) {
        const int s = it % kKVStages;
        const uint32_t ph = (uint32_t)(it / kKVStages) & 1u;
        const int row = (t_begin + it) * kBN;
        ok = mbar_wait(&B->k_empty[s], ph ^ 1u, B, P.status);
        if (!ok) break;
        mbar_expect_tx(&B->k_full[s], kTileBytes);
        tma_load_2d(sK + s * kTileBytes, &tm_k, h * kHD, row, &B->k_full[s]);
        ++issued_k;
        ok = mbar_wait(&B->v_empty[s], ph ^ 1u, B, P.status);
        if (!ok) break;
        mbar_expect_tx(&B->v_full[s], kTileBytes);
        tma_load_2d(sV + s * kTileBytes, &tm_v, h * kHD, row, &B->v_full[s]);
        ++issued_v;
      }
      if (!ok) {
        // leave no bulk copy in flight into this CTA's shared memory
        mbar_wait(&B->q_full, 0, B, P.status);
        for (int i = max(0, issued_k - kKVStages); i < issued_k; ++i)
          mbar_wait(&B->k_full[i % kKVStages], (uint32_t)(i / kKVStages) & 1u, B, P.status);
        for (int i = max(0, issued_v - kKVStages); i < issued_v; ++i)
          mbar_wait(&B->v_full[i % kKVStages], (uint32_t)(i / kKVStages) & 1u, B, P.status);
      }
    }
    __syncwarp();
  } else if (warp == 5) {
    // ------------------------------------------------ MMA issuer
    // Issue order (the tensor pipe executes one thread's MMAs in order):
    //   QK(0,0) QK(0,1) | PV(0,0) QK(1,0) PV(0,1) QK(1,1) | PV(1,0) QK(2,0) PV(1,1) QK(2,1) | ...
    // QK(t+1,h) overwrites S_h only after PV(t,h) has read P_h from it.
    // The whole warp walks the loop in step (every wait result goes through a vote, the tensor-memory base through
    // a warp reduction), so addresses and descriptors are warp-uniform values; one elected lane issues.
    {
      const bool leader = elect_one();
      const uint32_t tm = __reduce_or_sync(0xFFFFFFFFu, tmem);
      constexpr uint32_t idesc_qk = idesc_bf16(kHalf, false);
      constexpr uint32_t idesc_pv = idesc_bf16(kHD, true);
      const uint64_t dq = smem_desc_sw128(smem_u32(sQ));
      // S_hf = Q K_hf^T for the KV tile held in stage `st` (8 rows = one 1024-byte swizzle group)
      auto issue_qk = [&](int st, int hf) {
        const uint64_t dk = smem_desc_sw128(smem_u32(sK + st * kTileBytes + hf * (kTileBytes / 2)));
        if (leader) {
#pragma unroll
          for (int kk = 0; kk < kHD / 16; ++kk)     // 16 elements of head dim = 32 bytes inside the swizzled row
            mma_ss(tm + kColS + hf * kHalf, dq + (uint64_t)(kk * 2), dk + (uint64_t)(kk * 2), idesc_qk, kk > 0);
        }
      };
      auto wait_all = [&](void* bar, uint32_t parity) {
        return __all_sync(0xFFFFFFFFu, mbar_wait(bar, parity, B, P.status)) != 0;
      };
      bool ok = wait_all(&B->q_full, 0);
      if (ok) ok = wait_all(&B->k_full[0], 0);
      if (ok) {
        tc_fence_after();
        issue_qk(0, 0);
        if (leader) tc_commit(&B->s_full[0]);
        issue_qk(0, 1);
        if (leader) {
          tc_commit(&B->s_full[1]);
          tc_commit(&B->k_empty[0]);
        }
      }
      for (int it = 0; it < n_tiles && ok; ++it) {
        const int s = it % kKVStages, s1 = (it + 1) % kKVStages;
        const uint32_t ph = (uint32_t)(it / kKVStages) & 1u, ph1 = (uint32_t)((it + 1) / kKVStages) & 1u;
        const bool more = it + 1 < n_tiles;
        ok = wait_all(&B->v_full[s], ph);
        if (!ok) break;
        const uint64_t dv = smem_desc_sw128(smem_u32(sV + s * kTileBytes));
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          ok = wait_all(&B->p_full[hf], (uint32_t)it & 1u);
          if (!ok) break;
          tc_fence_after();
          if (leader) {
#pragma unroll
            for (int kk = 0; kk < kHalf / 16; ++kk)   // 16 KV rows = 2048 bytes; P: 8 TMEM columns per 16 bf16
              mma_ts(tm + kColO, tm + kColS + hf * kHalf + kk * 8, dv + (uint64_t)((hf * (kHalf / 16) + kk) * 128),
                     idesc_pv, (it > 0 || hf > 0 || kk > 0));
            if (hf == 1) tc_commit(&B->v_empty[s]);
            if (!more && hf == 0) tc_commit(&B->pv_done);   // (the last half has no later score MMA to tell it by)
          }
          if (more) {
            if (hf == 0) {
              ok = wait_all(&B->k_full[s1], ph1);
              if (!ok) break;
              tc_fence_after();
            }
            issue_qk(s1, hf);
            if (leader) {
              tc_commit(&B->s_full[hf]);
              if (hf == 1) tc_commit(&B->k_empty[s1]);
            }
          }
        }
      }
      if (ok) {
        if (leader) tc_commit(&B->o_full);
        wait_all(&B->o_full, 0);
      } else {
        if (leader) tc_commit(&B->drain);           // let every issued MMA finish before TMEM is freed
        wait_all(&B->drain, 0);
      }
    }
    __syncwarp();
  }
  } else {
    // ------------------------------------------------ softmax, correction and epilogue (128 threads)
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsSoftmax));
    const int quad = warp;
    const int row = quad * 32 + lane;
    const uint32_t t_row = tmem + ((uint32_t)(quad * 32) << 16);
    const float c = 1.4426950408889634f * 0.125f;     // log2(e) / sqrt(64)
    float mref = 0.0f, l = 0.0f;
    bool ok = true;
    // Upper bound of this row's logits in log2 units: |q_row,h| |k|_max log2(e) / 8.  The row's 64 query values are
    // the eight 16-byte chunks of its 128-byte line in the (swizzled) Q tile, in whatever order.
    float bound = 0.0f;
    bool fixed_ref = false;
    if (P.kmax2 != nullptr) {
      ok = __all_sync(0xFFFFFFFFu, mbar_wait(&B->q_full, 0, B, P.status)) != 0;
      if (ok) {
        float qn2 = 0.0f;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const uint4 u = *reinterpret_cast<const uint4*>(sQ + row * 128 + ((j ^ (row & 7)) << 4));
          const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float lo = __uint_as_float(w[e] << 16), hi = __uint_as_float(w[e] & 0xFFFF0000u);
            qn2 = fmaf(lo, lo, qn2);
            qn2 = fmaf(hi, hi, qn2);
          }
        }
        bound = sqrtf(qn2 * __ldg(P.kmax2 + h)) * c;
      }
    }
    for (int idx = 0; idx < 2 * n_tiles && ok; ++idx) {       // idx = 2 * tile + half
      const int it = idx >> 1, hf = idx & 1;
      // (every wait result is made warp-uniform before the warp meets an .aligned tensor-memory instruction)
      ok = __all_sync(0xFFFFFFFFu, mbar_wait(&B->s_full[hf], (uint32_t)it & 1u, B, P.status)) != 0;
      if (!ok) break;
      tc_fence_after();
      uint32_t s[kHalf];
      auto load_scores = [&]() {
#pragma unroll
        for (int j = 0; j < kHalf / 32; ++j) tmem_ld32(t_row + kColS + hf * kHalf + j * 32, s + j * 32);
        tmem_wait_ld();
        const int col0 = (t_begin + it) * kBN + hf * kHalf;
        if (col0 + kHalf > P.N) {
#pragma unroll
          for (int j = 0; j < kHalf; ++j)
            if (col0 + j >= P.N) s[j] = 0xFF800000u;     // -inf on columns past the last row
        }
      };
      // p = 2^(s * c - mref) on pairs, packed to bf16 over the front of s[]; returns the row's sum of p (four
      // independent packed partial sums, folded in a fixed order).  With `track` the raw row maximum is gathered in
      // the same pass (four chains of 3-input maxima), where it hides behind the exponentials.
      auto exp_pass = [&](auto track, float& raw_max) -> float {
        const float2 c2 = make_float2(c, c), nm2 = make_float2(-mref, -mref);
        float2 acc[4];
        float m4[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          acc[q] = make_float2(0.0f, 0.0f);
          m4[q] = -INFINITY;
        }
#pragma unroll
        for (int j = 0; j < kHalf; j += 2) {
          const float s0 = __uint_as_float(s[j]), s1 = __uint_as_float(s[j + 1]);
          if constexpr (decltype(track)::value) m4[(j >> 1) & 3] = max3(m4[(j >> 1) & 3], s0, s1);
          const float2 x = fma2(make_float2(s0, s1), c2, nm2);
          const float2 p = pair_on_fma_pipes(j >> 1) ? ex2_poly2(x) : make_float2(ex2(x.x), ex2(x.y));
          acc[(j >> 1) & 3] = add2(acc[(j >> 1) & 3], p);
          s[j >> 1] = pack_bf16(p.x, p.y);
        }
        raw_max = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
        const float2 t = add2(add2(acc[0], acc[1]), add2(acc[2], acc[3]));
        return t.x + t.y;
      };
      load_scores();
      float add, raw;
      if (idx == 0) {
        // the first half fixes the reference: its maximum has to be known before any exponential
        float m4[4];
        constexpr int kChain = kHalf / 4;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          m4[q] = fmaxf(__uint_as_float(s[kChain * q]), __uint_as_float(s[kChain * q + 1]));
#pragma unroll
          for (int j = 2; j < kChain; j += 2)
            m4[q] = max3(m4[q], __uint_as_float(s[kChain * q + j]), __uint_as_float(s[kChain * q + j + 1]));
        }
        mref = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3])) * c;
        if (P.kmax2 != nullptr) {
          // take the bound as the reference if it is a bound for what was seen and not absurdly far above it; the
          // decision is per warp, so that the warp stays in step
          const bool safe = bound >= mref && bound - mref <= kFixedRefMaxGap;
          fixed_ref = __all_sync(0xFFFFFFFFu, safe) != 0;
          // a whole number of powers of two above the true maximum of this half: its largest probability is then an
          // exact power of two, as it is (2^0) when the maximum itself is the reference, so a row that one early key
          // dominates loses nothing to the bf16 rounding of P
          if (fixed_ref) mref += ceilf(bound - mref);
        }
        add = exp_pass(std::false_type{}, raw);
      } else if (fixed_ref) {
        add = exp_pass(std::false_type{}, raw);          // no score can exceed the reference: nothing to track
      } else {
        // Later halves compute p under the reference they inherit while the maximum is gathered, and keep the
        // result unless the maximum outgrew the reference by more than the threshold (rare); then O is rescaled,
        // the scores are read again (P has not been written over them yet) and p is recomputed.
        add = exp_pass(std::true_type{}, raw);
        const float mx = raw * c;
        const bool grow = mx - mref > kRescaleThreshold;
        if (__any_sync(0xFFFFFFFFu, grow)) {
          // O may still be accumulating the previous half.  PV(idx - 1) is issued just before the scores of half
          // idx + 1, so the completion of those scores covers it; the last half has a barrier of its own.
          ok = idx + 1 < 2 * n_tiles ? mbar_wait(&B->s_full[hf ^ 1], (uint32_t)((idx + 1) >> 1) & 1u, B, P.status)
                                     : mbar_wait(&B->pv_done, 0, B, P.status);
          ok = __all_sync(0xFFFFFFFFu, ok) != 0;
          if (!ok) break;
          tc_fence_after();
          const float a = grow ? ex2(mref - mx) : 1.0f;
          if (grow) {
            mref = mx;
            l *= a;
          }
          uint32_t o[16];
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            tmem_ld16(t_row + kColO + j * 16, o);
            tmem_wait_ld();
#pragma unroll
            for (int e = 0; e < 16; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * a);
            tmem_st16(t_row + kColO + j * 16, o);
          }
          load_scores();
          add = exp_pass(std::false_type{}, raw);
        }
      }
      l += add;
      // P: bf16 pairs over the first kHalf / 2 columns of S_hf
      if constexpr (kHalf / 2 >= 32) tmem_st32(t_row + kColS + hf * kHalf, s);
      if constexpr ((kHalf / 2) % 32 == 16) tmem_st16(t_row + kColS + hf * kHalf + (kHalf / 64) * 32, s + (kHalf / 64) * 32);
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(&B->p_full[hf]);
    }
    if (ok) ok = mbar_wait(&B->o_full, 0, B, P.status);
    ok = __all_sync(0xFFFFFFFFu, ok) != 0;
    if (ok) {
      tc_fence_after();
      const int m = qt * kBM + row;
      const float inv = 1.0f / l;
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        uint32_t o[32];
        tmem_ld32(t_row + kColO + j * 32, o);
        tmem_wait_ld();
        if (m < P.M) {
          if (P.splits == 1) {
            uint4* dst = reinterpret_cast<uint4*>(P.out + (size_t)m * C + (size_t)h * kHD + j * 32);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              uint4 w;
              w.x = pack_bf16(__uint_as_float(o[8 * e + 0]) * inv, __uint_as_float(o[8 * e + 1]) * inv);
              w.y = pack_bf16(__uint_as_float(o[8 * e + 2]) * inv, __uint_as_float(o[8 * e + 3]) * inv);
              w.z = pack_bf16(__uint_as_float(o[8 * e + 4]) * inv, __uint_as_float(o[8 * e + 5]) * inv);
              w.w = pack_bf16(__uint_as_float(o[8 * e + 6]) * inv, __uint_as_float(o[8 * e + 7]) * inv);
              dst[e] = w;
            }
          } else {
            uint4* dst = reinterpret_cast<uint4*>(P.o_part + ((size_t)split * P.M + m) * C + (size_t)h * kHD + j * 32);
#pragma unroll
            for (int e = 0; e < 8; ++e) dst[e] = make_uint4(o[4 * e], o[4 * e + 1], o[4 * e + 2], o[4 * e + 3]);
          }
        }
      }
      if (P.splits > 1 && m < P.M) P.ml_part[((size_t)split * P.M + m) * P.H + h] = make_float2(mref, l);
      if (P.splits == 1 && P.lse != nullptr && m < P.M) P.lse[(size_t)m * P.H + h] = mref + log2f(l);
    }
  }

  // ------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (warp == 5) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)kTmemCols) : "memory");
  }
}

// out[m, h*64 + c] = sum_s O_s 2^(m_s - m*) / sum_s l_s 2^(m_s - m*), m* = max_s m_s, splits folded in order.
// One thread per 4 columns; all loads of a thread are issued before the arithmetic that needs them.
__global__ void __launch_bounds__(256) k_attn_merge(const float* __restrict__ o_part, const float2* __restrict__ ml_part,
                                                    int M, int H, int splits, __nv_bfloat16* __restrict__ out,
                                                    float* __restrict__ lse) {
  const int C = H * kHD;
  const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const size_t total = (size_t)M * (C / 4);
  // launched with programmatic stream serialisation: its CTAs may become resident while the last attention CTAs
  // drain; the partials are complete and visible once this wait returns
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (idx >= total) return;
  const int m = (int)(idx / (C / 4)), c4 = (int)(idx % (C / 4)), h = (c4 * 4) / kHD;
  float2 ml[kMaxSplits];
  float4 o[kMaxSplits];
#pragma unroll
  for (int s = 0; s < kMaxSplits; ++s)
    if (s < splits) {
      ml[s] = ml_part[((size_t)s * M + m) * H + h];
      o[s] = *reinterpret_cast<const float4*>(o_part + ((size_t)s * M + m) * C + c4 * 4);
    }
  float mstar = -INFINITY;
#pragma unroll
  for (int s = 0; s < kMaxSplits; ++s)
    if (s < splits) mstar = fmaxf(mstar, ml[s].x);
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  float den = 0.0f;
#pragma unroll
  for (int s = 0; s < kMaxSplits; ++s)
    if (s < splits) {
      const float w = exp2f(ml[s].x - mstar);
      acc.x = fmaf(w, o[s].x, acc.x);
      acc.y = fmaf(w, o[s].y, acc.y);
      acc.z = fmaf(w, o[s].z, acc.z);
      acc.w = fmaf(w, o[s].w, acc.w);
      den = fmaf(w, ml[s].y, den);
    }
  const float inv = 1.0f / den;
  if (lse != nullptr && (c4 * 4) % kHD == 0) lse[(size_t)m * H + h] = mstar + log2f(den);
  uint2 w;
  w.x = pack_bf16(acc.x * inv, acc.y * inv);
  w.y = pack_bf16(acc.z * inv, acc.w * inv);
  *reinterpret_cast<uint2*>(out + (size_t)m * C + c4 * 4) = w;
}

// Self-test of the bounded wait: one CTA sets up a barrier that expects one arrival, nobody arrives, and the wait is
// given limit_ns.  The kernel must come back with OVGGT_ERR_TIMEOUT in the status word (no tensor memory, no bulk
// copy, nothing in flight when it returns).  waited_ns receives how long the wait lasted.
__global__ void __launch_bounds__(32) k_bounded_wait_selftest(int* status, unsigned long long limit_ns,
                                                              unsigned long long* waited_ns) {
  __shared__ AttnBarriers B;
  if (threadIdx.x == 0) {
    mbar_init(&B.q_full, 1);
    B.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  const unsigned long long t0 = global_ns();
  const bool ok = __all_sync(0xFFFFFFFFu, mbar_wait(&B.q_full, 0, &B, status, limit_ns)) != 0;
  if (threadIdx.x == 0 && waited_ns) *waited_ns = global_ns() - t0;
  if (ok && threadIdx.x == 0) atomicCAS(status, 0, OVGGT_ERR_DEVICE_STATUS);   // a wait nobody ends must not succeed
}

// ---------------------------------------------------------------- host side

inline int g_attn_last_error = 0;
inline int attn_tcgen05_last_error() { return g_attn_last_error; }

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// [rows, C] bf16 row-major; box = 64 columns x box_rows rows, 128-byte swizzle, zero fill outside.
inline int make_rows_map(CUtensorMap* map, const void* base, int rows, int C, int box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return OVGGT_ERR_CUDA;
  cuuint64_t dims[2] = {(cuuint64_t)C, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)C * 2};
  cuuint32_t box[2] = {(cuuint32_t)kHD, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    g_attn_last_error = (int)r;
    return OVGGT_ERR_CUDA;
  }
  return OVGGT_OK;
}

// Number of KV splits: minimise (waves of CTAs over 2 x 148 slots) x (tiles per CTA + fixed overhead).
inline int attn_choose_splits(int M, int N, int H) {
  const int q_tiles = (M + kBM - 1) / kBM, tiles = (N + kBN - 1) / kBN;
  const long slots = (long)kCtasPerSm * 148;
  int best = 1;
  long best_cost = -1;
  for (int s = 1; s <= kMaxSplits && s <= tiles; ++s) {
    const int per = (tiles + s - 1) / s;
    const int eff = (tiles + per - 1) / per;
    if (eff != s) continue;
    const long ctas = (long)q_tiles * H * s;
    const long waves = (ctas + slots - 1) / slots;
    const long cost = waves * (per + 384 / kBN) + (s > 1 ? 256 / kBN : 0);
    if (best_cost < 0 || cost < best_cost) {
      best_cost = cost;
      best = s;
    }
  }
  return best;
}

inline size_t attn_tcgen05_scratch_bytes(int M, int N, int H) {
  (void)N;
  const size_t C = (size_t)H * kHD;
  return (size_t)kMaxSplits * M * C * 4 + (size_t)kMaxSplits * M * H * 8 + 1024;
}

inline int attn_tcgen05_num_launches(int M, int N, int H) { return attn_choose_splits(M, N, H) > 1 ? 2 : 1; }

// Tensor maps of a K/V buffer pair, kept by the caller between launches: a cache that lives in one buffer with a
// row count that stops changing needs them encoded once, not once per step.
struct AttnKvMaps {
  CUtensorMap k, v;
  const void *k_base = nullptr, *v_base = nullptr;
  int rows = -1, C = 0;
};

inline int attn_kv_maps(AttnKvMaps* m, const void* k, const void* v, int N, int C) {
  if (m->k_base == k && m->v_base == v && m->rows == N && m->C == C) return OVGGT_OK;
  m->rows = -1;
  int rc = make_rows_map(&m->k, k, N, C, kBN);
  if (rc) return rc;
  rc = make_rows_map(&m->v, v, N, C, kBN);
  if (rc) return rc;
  m->k_base = k; m->v_base = v; m->rows = N; m->C = C;
  return OVGGT_OK;
}

inline int attn_tcgen05_launch(const void* q, const void* k, const void* v, int M, int N, int H, void* out,
                               void* scratch, int* status, cudaStream_t st, AttnKvMaps* kv_maps = nullptr,
                               int force_splits = 0, const float* kmax2 = nullptr, float* lse = nullptr) {
  const int C = H * kHD;
  CUtensorMap tq;
  AttnKvMaps local;
  AttnKvMaps* maps = kv_maps ? kv_maps : &local;
  int rc = make_rows_map(&tq, q, M, C, kBM);
  if (rc) return rc;
  rc = attn_kv_maps(maps, k, v, N, C);
  if (rc) return rc;
  const CUtensorMap& tk = maps->k;
  const CUtensorMap& tv = maps->v;
  AttnParams P;
  P.M = M; P.N = N; P.H = H;
  P.tiles_total = (N + kBN - 1) / kBN;
  P.splits = force_splits > 0 ? std::min(force_splits, std::min(kMaxSplits, P.tiles_total)) : attn_choose_splits(M, N, H);
  P.tiles_per_split = (P.tiles_total + P.splits - 1) / P.splits;
  P.splits = (P.tiles_total + P.tiles_per_split - 1) / P.tiles_per_split;     // no empty split
  P.out = static_cast<__nv_bfloat16*>(out);
  P.o_part = static_cast<float*>(scratch);
  P.ml_part = reinterpret_cast<float2*>(static_cast<char*>(scratch) + (size_t)kMaxSplits * M * C * 4);
  P.status = status;
  P.kmax2 = kmax2;
  P.lse = lse;
  cudaError_t e = cudaFuncSetAttribute(k_attn_tcgen05, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kAttnSmemBytes);
  if (e != cudaSuccess) { g_attn_last_error = (int)e; return OVGGT_ERR_CUDA; }
  dim3 grid((M + kBM - 1) / kBM, H, P.splits);
  k_attn_tcgen05<<<grid, kAttnThreads, kAttnSmemBytes, st>>>(tq, tk, tv, P);
  e = cudaGetLastError();
  if (e != cudaSuccess) { g_attn_last_error = (int)e; return OVGGT_ERR_CUDA; }
  if (P.splits > 1) {
    const size_t total = (size_t)M * (C / 4);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)((total + 255) / 256));
    cfg.blockDim = dim3(256);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg, k_attn_merge, (const float*)P.o_part, (const float2*)P.ml_part, M, H, P.splits, P.out,
                           lse);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) { g_attn_last_error = (int)e; return OVGGT_ERR_CUDA; }
  }
  return OVGGT_OK;
}

}  // namespace ovggt
