// A measurement aid, not a step of the method: a kernel that does nothing but dependent-free fp32 fused
// multiply-adds, so that a benchmark can time the FP32 FMA rate of the device it runs on (the bound of the fp32
// layer path, whose arithmetic runs on the FMA pipes and not on the tensor cores).
#include "dsvt_common.cuh"

namespace {

constexpr int kChains = 8;  // independent accumulators per thread

__global__ void __launch_bounds__(1024) fma_probe_kernel(int32_t iters, float seed, float* __restrict__ sink) {
  float acc[kChains];
#pragma unroll
  for (int c = 0; c < kChains; ++c) acc[c] = seed + (float)(threadIdx.x + c);
  const float m = 1.0f + seed * 1e-7f, a = seed * 1e-3f;
  for (int i = 0; i < iters; ++i) {
#pragma unroll
    for (int c = 0; c < kChains; ++c) acc[c] = fmaf(acc[c], m, a);
  }
  float s = 0.f;
#pragma unroll
  for (int c = 0; c < kChains; ++c) s += acc[c];
  if (s == 123.456f) sink[0] = s;  // (never true in practice: keeps the chains alive)
}

}  // namespace

extern "C" int dsvt_fma_probe(dsvt_ctx* ctx, int32_t blocks, int32_t threads, int32_t iters, float* sink,
                              int64_t* flops) {
  if (!ctx || !sink || blocks < 1 || threads < 32 || threads > 1024 || threads % 32 != 0 || iters < 1)
    return DSVT_ERR_INVALID_ARG;
  fma_probe_kernel<<<(unsigned)blocks, (unsigned)threads, 0, ctx->stream>>>(iters, 1.0f, sink);
  DSVT_LAUNCHED(ctx);
  if (flops) *flops = (int64_t)blocks * threads * (int64_t)iters * kChains * 2;
  return DSVT_OK;
}
