// LayerNorm over the d channels of one row held by d / 8 consecutive lanes, eight consecutive channels
// per lane (LN_q / LN_k of the front end: Appendix, time mixer of the backbone).  One definition of the
// arithmetic - fp32 statistics, biased variance, eps inside the root, affine map, result rounded to
// bf16 - shared by the stand-alone kernel (kvm_head_layernorm) and by the ingest kernels that apply it
// on the fly, so that the two routes give the same bits.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>

namespace kvm {

// v: this lane's eight channels (in: raw values, out: normalised values rounded to bf16, as floats);
// w8 / b8: this lane's eight weights and biases.  Every lane of the warp must call (shuffles).
template <int D>
__device__ __forceinline__ void ln_chunk8(float (&v)[8], const float (&w8)[8], const float (&b8)[8], float eps) {
  constexpr int LPR = D / 8;
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < 8; ++i) s += v[i];
#pragma unroll
  for (int o = LPR / 2; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  const float mean = s * (1.f / D);
  float q = 0.f;
#pragma unroll
  for (int i = 0; i < 8; ++i) q = fmaf(v[i] - mean, v[i] - mean, q);
#pragma unroll
  for (int o = LPR / 2; o > 0; o >>= 1) q += __shfl_xor_sync(0xffffffffu, q, o);
  const float rstd = rsqrtf(q * (1.f / D) + eps);
#pragma unroll
  for (int i = 0; i < 8; ++i) v[i] = __bfloat162float(__float2bfloat16_rn(fmaf((v[i] - mean) * rstd, w8[i], b8[i])));
}

// this lane's eight weights / biases of head h ([H, D] fp32 arrays; NULL = 1 / 0)
template <int D>
__device__ __forceinline__ void ln_load_affine(const float* __restrict__ weight, const float* __restrict__ bias, int h, int sub,
                                               float (&w8)[8], float (&b8)[8]) {
#pragma unroll
  for (int i = 0; i < 8; ++i) { w8[i] = 1.f; b8[i] = 0.f; }
  if (weight) {
    const float4 a = *reinterpret_cast<const float4*>(weight + (int64_t)h * D + sub * 8), b = *reinterpret_cast<const float4*>(weight + (int64_t)h * D + sub * 8 + 4);
    w8[0] = a.x; w8[1] = a.y; w8[2] = a.z; w8[3] = a.w; w8[4] = b.x; w8[5] = b.y; w8[6] = b.z; w8[7] = b.w;
  }
  if (bias) {
    const float4 a = *reinterpret_cast<const float4*>(bias + (int64_t)h * D + sub * 8), b = *reinterpret_cast<const float4*>(bias + (int64_t)h * D + sub * 8 + 4);
    b8[0] = a.x; b8[1] = a.y; b8[2] = a.z; b8[3] = a.w; b8[4] = b.x; b8[5] = b.y; b8[6] = b.z; b8[7] = b.w;
  }
}

}  // namespace kvm
