// Merge gate of the layer's front end (Section 3.2 "KVM weight preparation", Eq. 2):
//     g_t = 1 + ELU(x_t W_g),   one scalar per token and kv head,
// i.e. g = 1 + z for z > 0 and exp(z) otherwise, z = x_t . W_g[h].  The result is the `gate`
// argument of kvm_prefill / kvm_decode_step.
//
// A skinny product [tokens x d_model] x [d_model x heads] with at most 64 heads: every x element is
// needed once per head, so the kernel is bound by reading x (2 d_model bytes per token) as long as
// the FMA pipe keeps up.  One CTA takes 64 tokens: 64-channel slices of their x rows and of all
// W_g rows go through shared memory, thread (tx, ty) accumulates tokens tx, tx + 32 against heads
// ty*HPT .. ty*HPT + HPT - 1 in fp32, and the results leave through shared memory so that the stores
// run along the token axis of gate[B, heads, T].
#include "kvm_internal.h"

namespace kvm {

constexpr int kGateTokens = 64;   // tokens per CTA
constexpr int kGateK = 64;        // channels per shared-memory slice

template <int HPT>
__global__ void __launch_bounds__(256) merge_gate_kernel(const __nv_bfloat16* __restrict__ x, const float* __restrict__ w,
                                                         float* __restrict__ gate, int64_t T, int dm, int H) {
  constexpr int HP = 8 * HPT;   // heads, padded
  __shared__ float xs[kGateTokens][kGateK + 1];
  __shared__ float ws[HP][kGateK];
  float (*outs)[kGateK + 1] = xs;   // the results reuse the x slice (HP <= 64 rows of 64 tokens) once the products are done
  static_assert(HP <= kGateTokens && kGateK == kGateTokens, "result tile must fit the x slice");
  const int tid = threadIdx.x, tx = tid & 31, ty = tid >> 5;
  const int b = blockIdx.y;
  const int64_t t0 = (int64_t)blockIdx.x * kGateTokens;
  float acc[2][HPT];
#pragma unroll
  for (int h = 0; h < HPT; ++h) acc[0][h] = acc[1][h] = 0.f;
  for (int k0 = 0; k0 < dm; k0 += kGateK) {
    // x slice: 64 tokens x 64 channels, eight bf16 (16 bytes) per load
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const int e = (tid + i * 256) * 8;
      const int tk = e / kGateK, ch = e % kGateK;
      float v[8];
      if (t0 + tk < T && k0 + ch < dm) {   // d_model is a multiple of 8: a run of eight is inside or outside
        const uint4 raw = *reinterpret_cast<const uint4*>(x + ((int64_t)b * T + t0 + tk) * dm + k0 + ch);
        const __nv_bfloat162* p2 = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float2 f = __bfloat1622float2(p2[j]);
          v[2 * j] = f.x; v[2 * j + 1] = f.y;
        }
      } else {
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] = 0.f;
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) xs[tk][ch + j] = v[j];
    }
    // W_g slice: all heads x 64 channels
    for (int e = tid; e < HP * kGateK; e += 256) {
      const int h = e / kGateK, c = e % kGateK;
      ws[h][c] = (h < H && k0 + c < dm) ? w[(int64_t)h * dm + k0 + c] : 0.f;
    }
    __syncthreads();
#pragma unroll 8
    for (int kk = 0; kk < kGateK; ++kk) {
      const float x0 = xs[tx][kk], x1 = xs[tx + 32][kk];
#pragma unroll
      for (int h = 0; h < HPT; ++h) {
        const float wv = ws[ty * HPT + h][kk];   // one address per warp: broadcast
        acc[0][h] = fmaf(x0, wv, acc[0][h]);
        acc[1][h] = fmaf(x1, wv, acc[1][h]);
      }
    }
    __syncthreads();
  }
#pragma unroll
  for (int h = 0; h < HPT; ++h) {
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const float z = acc[i][h];
      outs[ty * HPT + h][tx + 32 * i] = z > 0.f ? 1.f + z : expf(z);   // 1 + ELU(z), alpha = 1
    }
  }
  __syncthreads();
  for (int e = tid; e < H * kGateTokens; e += 256) {
    const int h = e / kGateTokens, tk = e % kGateTokens;
    if (t0 + tk < T) gate[((int64_t)b * H + h) * T + t0 + tk] = outs[h][tk];
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
  const int hpt = (n_kv_heads + 7) / 8;
  if (hpt <= 1) merge_gate_kernel<1><<<grid, 256, 0, s>>>(xp, w_gate, gate, n_tokens, d_model, n_kv_heads);
  else if (hpt <= 2) merge_gate_kernel<2><<<grid, 256, 0, s>>>(xp, w_gate, gate, n_tokens, d_model, n_kv_heads);
  else if (hpt <= 4) merge_gate_kernel<4><<<grid, 256, 0, s>>>(xp, w_gate, gate, n_tokens, d_model, n_kv_heads);
  else merge_gate_kernel<8><<<grid, 256, 0, s>>>(xp, w_gate, gate, n_tokens, d_model, n_kv_heads);
  return cudaGetLastError() == cudaSuccess ? KVM_OK : KVM_ERR_CUDA;
}
