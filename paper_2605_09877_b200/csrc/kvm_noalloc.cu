// kvm_attend_rows_noalloc: the split single-query attention of the decode step, for callers that
// must not allocate device memory.
//
// Who needs this: code that runs where cudaMalloc is off limits -- a serving loop that handed all
// device memory to its own pool at start-up, a plugin living inside another framework's memory
// plan, a region that must not synchronise the device (cudaMalloc / cudaFree may) -- but that
// already holds key / value rows in buffers of its own (for instance a readout cache obtained with
// kvm_state_export plus the window tokens) and wants them attended with the decode kernel.  The
// regular decode path keeps the partial results of its row splits in a buffer that
// kvm_state_create allocated; here the same partials live in a fixed array that is part of the
// loaded library image, so the call itself allocates nothing.
//
// The scratch is one file-scope __device__ array: every GPU that loads the library carries it
// (about 4.3 MB) until the process exits, all calls share it, and it keeps whatever the last call
// left in it.  Nothing in it has to start at zero: each call overwrites every (head, split) slot it
// later reads.  Two calls that overlap on the same GPU (different streams, or different host
// threads) would race on it; callers serialise them.
#include <mutex>

#include "kvm_internal.h"

namespace kvm {

constexpr int kNoAllocMaxSlots = 8192;                    // n_heads * n_splits must not exceed this
constexpr int kNoAllocSlotFloats = 128 + 2;               // accumulator (up to head_dim 128) + max + sum
constexpr int kNoAllocMaxDevices = 64;

static __device__ __align__(256) float g_noalloc_partials[kNoAllocMaxSlots * kNoAllocSlotFloats];

// Host-side copies of the array's device address, one per GPU.  The symbol's name is only a
// stand-in in host code; the address a kernel can use comes from cudaGetSymbolAddress, asked once
// per device while that device is current.
static float* g_noalloc_ptr[kNoAllocMaxDevices] = {nullptr};
static std::mutex g_noalloc_mutex;

__device__ __forceinline__ void na_unpack8(const uint4& w, float (&f)[8]) {
  const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&w.x));
  const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&w.y));
  const float2 c = __half22float2(*reinterpret_cast<const __half2*>(&w.z));
  const float2 e = __half22float2(*reinterpret_cast<const __half2*>(&w.w));
  f[0] = a.x; f[1] = a.y; f[2] = b.x; f[3] = b.y; f[4] = c.x; f[5] = c.y; f[6] = e.x; f[7] = e.y;
}

// grid (nsplit, n_heads), 256 threads.  Same streaming scheme as the decode kernel: D/8 lanes per
// row with 16-byte loads, online softmax per warp, warps merged through shared memory; the
// (max, sum, accumulator) of the split goes to `part`.
template <int D>
__global__ void __launch_bounds__(256) noalloc_attend_kernel(const __half* __restrict__ q, const __half* __restrict__ keys,
                                                             const __half* __restrict__ values, float* __restrict__ part,
                                                             int64_t n_rows, int nsplit, float scale_log2) {
  constexpr int LPR = D / 8;
  constexpr int RPW = 32 / LPR;
  constexpr int UNR = 4;
  constexpr int STEP = RPW * UNR;
  __shared__ float s_m[8], s_l[8];
  __shared__ float s_acc[8][D];
  const int split = blockIdx.x, h = blockIdx.y;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int grp = lane / LPR, gl = lane % LPR;
  int64_t per = (n_rows + nsplit - 1) / nsplit;
  per = (per + 8 * STEP - 1) / (8 * STEP) * (8 * STEP);
  const int64_t r0 = (int64_t)split * per;
  const int64_t r1 = min(n_rows, r0 + per);
  float qf[8];
  na_unpack8(*reinterpret_cast<const uint4*>(q + (int64_t)h * D + gl * 8), qf);
  const __half* kh = keys + (int64_t)h * n_rows * D;
  const __half* vh = values + (int64_t)h * n_rows * D;
  float m_run = -INFINITY, l_run = 0.f;
  float acc[8];
#pragma unroll
  for (int c = 0; c < 8; ++c) acc[c] = 0.f;
  for (int64_t base = r0 + (int64_t)warp * STEP; base < r1; base += 8 * STEP) {
    uint4 kw[UNR], vw[UNR];
    bool ok[UNR];
#pragma unroll
    for (int i = 0; i < UNR; ++i) {
      const int64_t row = base + i * RPW + grp;
      ok[i] = row < r1;
      kw[i] = ok[i] ? *reinterpret_cast<const uint4*>(kh + row * D + gl * 8) : make_uint4(0, 0, 0, 0);
      vw[i] = ok[i] ? *reinterpret_cast<const uint4*>(vh + row * D + gl * 8) : make_uint4(0, 0, 0, 0);
    }
    float lg[UNR];
    float tmax = -INFINITY;
#pragma unroll
    for (int i = 0; i < UNR; ++i) {
      float kf[8];
      na_unpack8(kw[i], kf);
      float dot = 0.f;
#pragma unroll
      for (int c = 0; c < 8; ++c) dot = fmaf(qf[c], kf[c], dot);
#pragma unroll
      for (int o = LPR / 2; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
      lg[i] = ok[i] ? dot * scale_log2 : -INFINITY;
      tmax = fmaxf(tmax, lg[i]);
    }
#pragma unroll
    for (int o = 16; o >= LPR; o >>= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, o));
    if (tmax == -INFINITY) continue;
    const float mnew = fmaxf(m_run, tmax);
    const float corr = exp2f(m_run - mnew);
    m_run = mnew;
    l_run *= corr;
#pragma unroll
    for (int c = 0; c < 8; ++c) acc[c] *= corr;
#pragma unroll
    for (int i = 0; i < UNR; ++i) {
      const float pr = exp2f(lg[i] - mnew);
      l_run += pr;
      float vf[8];
      na_unpack8(vw[i], vf);
#pragma unroll
      for (int c = 0; c < 8; ++c) acc[c] = fmaf(pr, vf[c], acc[c]);
    }
  }
#pragma unroll
  for (int o = 16; o >= LPR; o >>= 1) {
    l_run += __shfl_xor_sync(0xffffffffu, l_run, o);
#pragma unroll
    for (int c = 0; c < 8; ++c) acc[c] += __shfl_xor_sync(0xffffffffu, acc[c], o);
  }
  if (grp == 0) {
#pragma unroll
    for (int c = 0; c < 8; ++c) s_acc[warp][gl * 8 + c] = acc[c];
    if (gl == 0) { s_m[warp] = m_run; s_l[warp] = l_run; }
  }
  __syncthreads();
  if (tid < D) {
    float mx = -INFINITY;
#pragma unroll
    for (int w = 0; w < 8; ++w) mx = fmaxf(mx, s_m[w]);
    float l = 0.f, a = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) {
      const float f = (s_m[w] == -INFINITY) ? 0.f : exp2f(s_m[w] - mx);
      l += s_l[w] * f;
      a += s_acc[w][tid] * f;
    }
    // every slot that the combine kernel reads is written here, also by an empty split
    float* dst = part + ((int64_t)h * nsplit + split) * kNoAllocSlotFloats;
    dst[tid] = a;
    if (tid == 0) { dst[128] = mx; dst[129] = l; }
  }
}

template <int D>
__global__ void noalloc_combine_kernel(const float* __restrict__ part, __nv_bfloat16* __restrict__ out, int nsplit) {
  const int h = blockIdx.x, x = threadIdx.x;
  if (x >= D) return;
  const float* src = part + (int64_t)h * nsplit * kNoAllocSlotFloats;
  float mx = -INFINITY;
  for (int s = 0; s < nsplit; ++s) mx = fmaxf(mx, src[s * kNoAllocSlotFloats + 128]);
  float l = 0.f, a = 0.f;
  for (int s = 0; s < nsplit; ++s) {
    const float ms = src[s * kNoAllocSlotFloats + 128];
    const float f = (ms == -INFINITY) ? 0.f : exp2f(ms - mx);
    l += src[s * kNoAllocSlotFloats + 129] * f;
    a += src[s * kNoAllocSlotFloats + x] * f;
  }
  out[(int64_t)h * D + x] = __float2bfloat16_rn(a / l);
}

}  // namespace kvm

using namespace kvm;

extern "C" __attribute__((visibility("default")))
kvm_status_t kvm_attend_rows_noalloc(const void* q, const void* keys, const void* values, int32_t n_heads,
                                     int64_t n_rows, int32_t head_dim, float scale, void* out, void* cuda_stream) {
  if (!q || !keys || !values || !out) return KVM_ERR_INVALID_ARG;
  if (n_heads < 1 || n_rows < 1) return KVM_ERR_INVALID_ARG;
  if (head_dim != 64 && head_dim != 128) return KVM_ERR_UNSUPPORTED;
  if (((uintptr_t)q & 15) || ((uintptr_t)keys & 15) || ((uintptr_t)values & 15) || ((uintptr_t)out & 1)) return KVM_ERR_INVALID_ARG;
  // splits: fill the GPU (about four CTAs per SM) but keep at least 256 rows per split
  int64_t want = (4 * 148 + n_heads - 1) / n_heads;
  const int64_t maxs = (n_rows + 255) / 256;
  if (want > maxs) want = maxs;
  if (want > kMaxSplits) want = kMaxSplits;
  if (want < 1) want = 1;
  const int nsplit = (int)want;
  if ((int64_t)n_heads * nsplit > kNoAllocMaxSlots) return KVM_ERR_CAPACITY;   // the fixed scratch holds 8192 partials

  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kNoAllocMaxDevices) { cudaGetLastError(); return KVM_ERR_CUDA; }
  float* part = nullptr;
  {
    // set-up, once per device, with that device current: ask the runtime where the array lives
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!g_noalloc_ptr[dev]) {
      float* p = nullptr;
      if (cudaGetSymbolAddress((void**)&p, g_noalloc_partials) != cudaSuccess || !p) { cudaGetLastError(); return KVM_ERR_CUDA; }
      g_noalloc_ptr[dev] = p;
    }
    part = g_noalloc_ptr[dev];
  }
  cudaStream_t s = (cudaStream_t)cuda_stream;
  const float scale_log2 = scale * 1.4426950408889634f;
  dim3 grid(nsplit, n_heads);
  if (head_dim == 128) {
    noalloc_attend_kernel<128><<<grid, 256, 0, s>>>((const __half*)q, (const __half*)keys, (const __half*)values, part, n_rows, nsplit, scale_log2);
    noalloc_combine_kernel<128><<<n_heads, 128, 0, s>>>(part, (__nv_bfloat16*)out, nsplit);
  } else {
    noalloc_attend_kernel<64><<<grid, 256, 0, s>>>((const __half*)q, (const __half*)keys, (const __half*)values, part, n_rows, nsplit, scale_log2);
    noalloc_combine_kernel<64><<<n_heads, 64, 0, s>>>(part, (__nv_bfloat16*)out, nsplit);
  }
  return cudaGetLastError() == cudaSuccess ? KVM_OK : KVM_ERR_CUDA;
}
