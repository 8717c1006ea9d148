// fp32-accumulating SIMT attention: out = softmax(Q K^T / sqrt(64)) V per head, head_dim 64.
// This is the kernel of the fp32 configuration (tensor cores have no fp32 input path) and works for
// bf16 storage too.  One thread owns one query row of one head and streams the keys through
// shared-memory tiles with an online (running-max) softmax in base 2.
#pragma once

#include "common.cuh"

namespace ovggt {

constexpr int kSimtRows = 128;   // query rows per CTA
constexpr int kSimtTile = 32;    // keys per shared-memory tile

template <int DT>
__global__ void __launch_bounds__(kSimtRows) k_attn_simt(const void* __restrict__ q, const void* __restrict__ k,
                                                         const void* __restrict__ v, int M, int N, int H,
                                                         void* __restrict__ out, float* __restrict__ lse = nullptr) {
  constexpr int D = 64, VEC = VecOf<DT>::n, VPR = D / VEC;   // vectors per head-row
  __shared__ __align__(16) float Ks[kSimtTile][D];
  __shared__ __align__(16) float Vs[kSimtTile][D];
  const int h = blockIdx.y, m = blockIdx.x * kSimtRows + threadIdx.x;
  const int C = H * D;
  const size_t row_vecs = (size_t)C / VEC;
  const float scale = 1.4426950408889634f * 0.125f;          // log2(e) / sqrt(64)
  float qr[D], acc[D];
#pragma unroll
  for (int c = 0; c < D; ++c) { qr[c] = 0.0f; acc[c] = 0.0f; }
  if (m < M) {
    const uint4* qp = reinterpret_cast<const uint4*>(q) + (size_t)m * row_vecs + (size_t)h * VPR;
#pragma unroll
    for (int i = 0; i < VPR; ++i) {
      float f[VEC];
      unpack<DT>(qp[i], f);
#pragma unroll
      for (int e = 0; e < VEC; ++e) qr[i * VEC + e] = f[e] * scale;
    }
  }
  float mref = -INFINITY, l = 0.0f;
  for (int t0 = 0; t0 < N; t0 += kSimtTile) {
    __syncthreads();
    for (int idx = threadIdx.x; idx < kSimtTile * VPR; idx += kSimtRows) {
      const int r = idx / VPR, i = idx - r * VPR;
      float fk[VEC], fv[VEC];
      if (t0 + r < N) {
        const size_t off = (size_t)(t0 + r) * row_vecs + (size_t)h * VPR + i;
        unpack<DT>(reinterpret_cast<const uint4*>(k)[off], fk);
        unpack<DT>(reinterpret_cast<const uint4*>(v)[off], fv);
      } else {
#pragma unroll
        for (int e = 0; e < VEC; ++e) { fk[e] = 0.0f; fv[e] = 0.0f; }
      }
#pragma unroll
      for (int e = 0; e < VEC; ++e) { Ks[r][i * VEC + e] = fk[e]; Vs[r][i * VEC + e] = fv[e]; }
    }
    __syncthreads();
    float s[kSimtTile];
    float tmax = -INFINITY;
#pragma unroll
    for (int j = 0; j < kSimtTile; ++j) {
      float a = 0.0f;
#pragma unroll
      for (int c = 0; c < D; ++c) a = fmaf(qr[c], Ks[j][c], a);
      s[j] = (t0 + j < N) ? a : -INFINITY;
      tmax = fmaxf(tmax, s[j]);
    }
    const float mnew = fmaxf(mref, tmax);
    const float corr = (mref == -INFINITY) ? 0.0f : exp2f(mref - mnew);
    l *= corr;
#pragma unroll
    for (int c = 0; c < D; ++c) acc[c] *= corr;
#pragma unroll
    for (int j = 0; j < kSimtTile; ++j) {
      const float p = exp2f(s[j] - mnew);
      l += p;
#pragma unroll
      for (int c = 0; c < D; ++c) acc[c] = fmaf(p, Vs[j][c], acc[c]);
    }
    mref = mnew;
  }
  if (m < M) {
    const float inv = 1.0f / l;
    if (lse != nullptr) lse[(size_t)m * H + h] = mref + log2f(l);   // log2 of the row's softmax denominator
    if constexpr (DT == kBF16) {
      __nv_bfloat16* o = reinterpret_cast<__nv_bfloat16*>(out) + (size_t)m * C + (size_t)h * D;
#pragma unroll
      for (int c = 0; c < D; c += 2)
        *reinterpret_cast<__nv_bfloat162*>(o + c) = __floats2bfloat162_rn(acc[c] * inv, acc[c + 1] * inv);
    } else {
      float* o = reinterpret_cast<float*>(out) + (size_t)m * C + (size_t)h * D;
#pragma unroll
      for (int c = 0; c < D; c += 4)
        *reinterpret_cast<float4*>(o + c) = make_float4(acc[c] * inv, acc[c + 1] * inv, acc[c + 2] * inv, acc[c + 3] * inv);
    }
  }
}

}  // namespace ovggt
