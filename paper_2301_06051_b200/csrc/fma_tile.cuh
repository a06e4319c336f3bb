// fp32 FMA building blocks shared by the fused layer kernel and the pooling kernel: a tile GEMM that
// streams a row-major [out][in] weight matrix (float or bfloat16) through shared memory, and warp
// reductions.
#pragma once
#include "dsvt_common.cuh"

namespace dsvt_fma {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kNC = 64;  // output columns per GEMM column block
constexpr int kKC = 32;  // K elements staged per step

__device__ __forceinline__ float gelu_erf(float t) { return 0.5f * t * (1.0f + erff(t * 0.70710678118654752440f)); }

__device__ __forceinline__ void load8(const float* p, float (&w)[8]) {
  const float4 a = *reinterpret_cast<const float4*>(p);
  const float4 b = *reinterpret_cast<const float4*>(p + 4);
  w[0] = a.x; w[1] = a.y; w[2] = a.z; w[3] = a.w; w[4] = b.x; w[5] = b.y; w[6] = b.z; w[7] = b.w;
}
__device__ __forceinline__ void load8(const __nv_bfloat16* p, float (&w)[8]) {
  const uint4 a = *reinterpret_cast<const uint4*>(p);
  const uint32_t u[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    w[2 * i] = __uint_as_float(u[i] << 16);
    w[2 * i + 1] = __uint_as_float(u[i] & 0xFFFF0000u);
  }
}

// Os[r][o] = act(sum_k As[r][k] * W[o][k] + bias[o]) for rows r < 16 * rm_used, o < N.
// 256 threads: tx = tid % 16 owns 4 adjacent columns of a 64-column block, ty = tid / 16 owns rows
// ty, ty + 16, ...  W is streamed through shared memory 32 K-elements at a time, transposed so that
// the inner loop reads it with 128-bit conflict-free loads.
template <typename WT, int RM>
__device__ void gemm_tile(const float* __restrict__ As, int lda, int rm_used, const WT* __restrict__ W, int K, int N,
                          const float* __restrict__ bias, float* __restrict__ Os, int ldo, bool gelu,
                          float* __restrict__ Wst) {
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int o_l = tid & 63, kq = tid >> 6;  // staging role: column o_l, K-octet kq
  for (int n0 = 0; n0 < N; n0 += kNC) {
    float acc[RM][4];
#pragma unroll
    for (int i = 0; i < RM; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
    float wreg[8];
    auto fetch = [&](int k0) {
      const int o = n0 + o_l, k = k0 + kq * 8;
      if (o < N && k < K) {
        load8(W + (size_t)o * K + k, wreg);
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) wreg[i] = 0.f;
      }
    };
    fetch(0);
    for (int k0 = 0; k0 < K; k0 += kKC) {
      __syncthreads();  // previous step's readers are done with Wst
#pragma unroll
      for (int i = 0; i < 8; ++i) Wst[(kq * 8 + i) * kNC + o_l] = wreg[i];
      __syncthreads();
      if (k0 + kKC < K) fetch(k0 + kKC);
      const int kmax = min(kKC, K - k0);
      for (int kk = 0; kk < kmax; kk += 4) {
        float4 a4[RM];
#pragma unroll
        for (int i = 0; i < RM; ++i)
          if (i < rm_used) a4[i] = *reinterpret_cast<const float4*>(As + (size_t)(ty + 16 * i) * lda + k0 + kk);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const float4 w4 = *reinterpret_cast<const float4*>(Wst + (kk + u) * kNC + tx * 4);
#pragma unroll
          for (int i = 0; i < RM; ++i)
            if (i < rm_used) {
              const float a = u == 0 ? a4[i].x : u == 1 ? a4[i].y : u == 2 ? a4[i].z : a4[i].w;
              acc[i][0] = fmaf(a, w4.x, acc[i][0]);
              acc[i][1] = fmaf(a, w4.y, acc[i][1]);
              acc[i][2] = fmaf(a, w4.z, acc[i][2]);
              acc[i][3] = fmaf(a, w4.w, acc[i][3]);
            }
        }
      }
    }
    const int col = n0 + tx * 4;
    if (col < N) {
      float4 b4 = make_float4(0.f, 0.f, 0.f, 0.f);
      if (bias) b4 = *reinterpret_cast<const float4*>(bias + col);
#pragma unroll
      for (int i = 0; i < RM; ++i)
        if (i < rm_used) {
          float4 v = make_float4(acc[i][0] + b4.x, acc[i][1] + b4.y, acc[i][2] + b4.z, acc[i][3] + b4.w);
          if (gelu) { v.x = gelu_erf(v.x); v.y = gelu_erf(v.y); v.z = gelu_erf(v.z); v.w = gelu_erf(v.w); }
          *reinterpret_cast<float4*>(Os + (size_t)(ty + 16 * i) * ldo + col) = v;
        }
    }
  }
  __syncthreads();
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ int warp_max_int(int v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = max(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

}  // namespace dsvt_fma
