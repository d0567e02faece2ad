// Merge gate of the layer's front end (Section 3.2 "KVM weight preparation", Eq. 2):
//     g_t = 1 + ELU(x_t W_g),   one scalar per token and kv head,
// i.e. g = 1 + z for z > 0 and exp(z) otherwise, z = x_t . W_g[h].  The result is the `gate`
// argument of kvm_prefill / kvm_decode_step.
//
// A skinny product [tokens x d_model] x [d_model x heads] with at most 64 heads: every x element is
// needed once per head, so the kernel is bound by reading x (2 d_model bytes per token) as long as
// the FMA pipe keeps up.  A CTA takes 64 tokens; thread (token, part) owns one token, all heads and
// one quarter of every 128-channel slice: its share of the x row streams through registers, eight
// channels (16 bytes) per load, and is never shared; the W_g rows go through shared memory slice by
// slice and are read as broadcasts (every lane of a warp wants the same weights), so a step of eight
// channels costs 2 HT shared-memory loads for 8 HT FMAs.  The four partial sums of a token meet in
// shared memory at the end (fixed order: reproducible), and the stores run along the token axis of
// gate[B, heads, T].
#include "kvm_internal.h"

namespace kvm {

constexpr int kGateTokens = 64;   // tokens per CTA
constexpr int kGateParts = 4;     // threads per token, each a quarter of the channels of a slice
constexpr int kGateThreads = kGateTokens * kGateParts;
constexpr int kGateK = 128;       // channels per shared-memory slice of W_g

template <int HT>                 // heads, padded to 8, 16, 32 or 64
__global__ void __launch_bounds__(kGateThreads) merge_gate_kernel(const __nv_bfloat16* __restrict__ x, const float* __restrict__ w,
                                                                  float* __restrict__ gate, int64_t T, int dm, int H) {
  __shared__ __align__(16) float ws[HT * kGateK];   // W_g slice [HT][128]; afterwards the partial sums
  const int tid = threadIdx.x, tok = tid % kGateTokens, part = tid / kGateTokens;   // a warp shares `part`
  const int b = blockIdx.y;
  const int64_t t = (int64_t)blockIdx.x * kGateTokens + tok;
  const bool valid = t < T;
  const __nv_bfloat16* row = x + ((int64_t)b * T + (valid ? t : 0)) * dm;
  float acc[HT];
#pragma unroll
  for (int h = 0; h < HT; ++h) acc[h] = 0.f;
  for (int k0 = 0; k0 < dm; k0 += kGateK) {
    __syncthreads();   // the previous slice is no longer read
    for (int e = tid; e < HT * kGateK; e += kGateThreads) {
      const int h = e / kGateK, c = e % kGateK;
      ws[e] = (h < H && k0 + c < dm) ? w[(int64_t)h * dm + k0 + c] : 0.f;
    }
    __syncthreads();
#pragma unroll 2
    for (int j = 0; j < kGateK / 8 / kGateParts; ++j) {
      const int c = 8 * (part * (kGateK / 8 / kGateParts) + j);   // first of eight channels inside the slice
      if (k0 + c >= dm) break;                                    // d_model is a multiple of 8
      const uint4 raw = *reinterpret_cast<const uint4*>(row + k0 + c);
      const __nv_bfloat162* p2 = reinterpret_cast<const __nv_bfloat162*>(&raw);
      const float2 f0 = __bfloat1622float2(p2[0]), f1 = __bfloat1622float2(p2[1]);
      const float2 f2 = __bfloat1622float2(p2[2]), f3 = __bfloat1622float2(p2[3]);
#pragma unroll
      for (int h = 0; h < HT; ++h) {
        const float4 wa = *reinterpret_cast<const float4*>(&ws[h * kGateK + c]);       // one address per warp: broadcast
        const float4 wb = *reinterpret_cast<const float4*>(&ws[h * kGateK + c + 4]);
        float a = acc[h];
        a = fmaf(f0.x, wa.x, a); a = fmaf(f0.y, wa.y, a); a = fmaf(f1.x, wa.z, a); a = fmaf(f1.y, wa.w, a);
        a = fmaf(f2.x, wb.x, a); a = fmaf(f2.y, wb.y, a); a = fmaf(f3.x, wb.z, a); a = fmaf(f3.y, wb.w, a);
        acc[h] = a;
      }
    }
  }
  // parts 2, 3 -> parts 0, 1, then part 1 -> part 0, through the slice buffer (2 x 64 x HT floats fit it)
  __syncthreads();
  if (part >= 2) {
#pragma unroll
    for (int h = 0; h < HT; ++h) ws[((part - 2) * HT + h) * kGateTokens + tok] = acc[h];
  }
  __syncthreads();
  if (part < 2) {
#pragma unroll
    for (int h = 0; h < HT; ++h) acc[h] += ws[(part * HT + h) * kGateTokens + tok];
  }
  __syncthreads();
  if (part == 1) {
#pragma unroll
    for (int h = 0; h < HT; ++h) ws[h * kGateTokens + tok] = acc[h];
  }
  __syncthreads();
  if (part == 0 && valid) {
#pragma unroll
    for (int h = 0; h < HT; ++h) {
      const float z = acc[h] + ws[h * kGateTokens + tok];
      if (h < H) gate[((int64_t)b * H + h) * T + t] = z > 0.f ? 1.f + z : expf(z);   // 1 + ELU(z), alpha = 1
    }
  }
}

}  // namespace kvm

using namespace kvm;

extern "C" __attribute__((visibility("default")))
kvm_status_t kvm_merge_gate(const void* x, const float* w_gate, int32_t batch, int64_t n_tokens, int32_t d_model,
                                    int32_t n_kv_heads, float* gate, void* cuda_stream) {
  if (!x || !w_gate || !gate || batch < 1 || n_tokens < 1 || d_model < 8 || n_kv_heads < 1) return KVM_ERR_INVALID_ARG;
  if (d_model % 8 || ((uintptr_t)x & 15) || ((uintptr_t)w_gate & 3) || ((uintptr_t)gate & 3)) return KVM_ERR_INVALID_ARG;
  if (n_kv_heads > 64) return KVM_ERR_UNSUPPORTED;
  if (batch > 65535) return KVM_ERR_UNSUPPORTED;
  cudaStream_t s = (cudaStream_t)cuda_stream;
  const dim3 grid((unsigned)((n_tokens + kGateTokens - 1) / kGateTokens), (unsigned)batch);
  const __nv_bfloat16* xp = (const __nv_bfloat16*)x;
  if (n_kv_heads <= 8) merge_gate_kernel<8><<<grid, kGateThreads, 0, s>>>(xp, w_gate, gate, n_tokens, d_model, n_kv_heads);
  else if (n_kv_heads <= 16) merge_gate_kernel<16><<<grid, kGateThreads, 0, s>>>(xp, w_gate, gate, n_tokens, d_model, n_kv_heads);
  else if (n_kv_heads <= 32) merge_gate_kernel<32><<<grid, kGateThreads, 0, s>>>(xp, w_gate, gate, n_tokens, d_model, n_kv_heads);
  else merge_gate_kernel<64><<<grid, kGateThreads, 0, s>>>(xp, w_gate, gate, n_tokens, d_model, n_kv_heads);
  return cudaGetLastError() == cudaSuccess ? KVM_OK : KVM_ERR_CUDA;
}
