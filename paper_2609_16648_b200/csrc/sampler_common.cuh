// Arithmetic shared by the two sampler kernels (cluster-per-sequence and CTA-per-sequence): one definition of the
// probability p(x), of the running (max, sum) merge and of the integer weight, so that both kernels make their
// decisions on identical formulas.
#pragma once

#include "common.cuh"
#include "kernels.h"

namespace gm {

constexpr int SAMP_WARPS = SAMP_THREADS / 32;
constexpr int SAMP_MAX_ROWS = 2 * GM_MAX_K_ + 1;

struct MZ { float m, z; };                        // running maximum (raw logit units) and sum of 2^((x - m) s)

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ MZ mz_merge(MZ a, MZ b, float s) {
  const float m = fmaxf(a.m, b.m);
  if (m == -INFINITY) return MZ{m, 0.f};
  return MZ{m, a.z * ex2((a.m - m) * s) + b.z * ex2((b.m - m) * s)};
}
// softmax probability of a raw logit x given s, c = -fl(max * s) and 1 / Z
__device__ __forceinline__ float prob_of(float x, float s, float c, float inv_z) {
  return __fmul_rn(ex2(__fmaf_rn(x, s, c)), inv_z);
}
__device__ __forceinline__ void unpack8(const uint4 &v, float (&x)[8]) {
  x[0] = bf16_lo(v.x); x[1] = bf16_hi(v.x); x[2] = bf16_lo(v.y); x[3] = bf16_hi(v.y);
  x[4] = bf16_lo(v.z); x[5] = bf16_hi(v.z); x[6] = bf16_lo(v.w); x[7] = bf16_hi(v.w);
}
__device__ __forceinline__ uint32_t bmax2(uint32_t a, uint32_t b) {          // packed bf16x2 maximum
  __nv_bfloat162 r = __hmax2(*reinterpret_cast<__nv_bfloat162 *>(&a), *reinterpret_cast<__nv_bfloat162 *>(&b));
  return *reinterpret_cast<uint32_t *>(&r);
}
__device__ __forceinline__ uint64_t step_of(const SamplerArgs &A) { return A.step_ptr ? *A.step_ptr : A.step; }
// integer weight of one residual entry: trunc(r * 2^44) for r > 0, else 0 (the product is an exact scaling)
__device__ __forceinline__ unsigned long long weight_of(float p, float q, bool use_q) {
  const float r = use_q ? __fsub_rn(p, q) : p;
  return r > 0.f ? __float2ull_rz(__fmul_rn(r, 17592186044416.0f /* 2^44 */)) : 0ull;
}


}  // namespace gm
