// Scalar-core (SIMT) attention over [state rows ; window] for one chunk (Section 3.2 "Readout").
// One warp per query, keys streamed through shared memory in tiles of 32, online softmax per
// warp.  This is the cross-check path (KVM_FLAG_SIMT_ATTENTION) and the path for shapes the
// tensor-core kernel does not tile; the default prefill path is the tcgen05 kernel.
#include "kvm_internal.h"

namespace kvm {

struct AttnSimtParams {
  const __half *stQ, *stK, *stV, *Khat, *Vhat;
  const float *tau_s, *tau_b;
  __nv_bfloat16* out;
  int64_t Tcall, stRows, Mcap;
  int64_t q_row0, t0, m, win_row0, b, out_t0;
  int64_t so0, so1, so2;
  int nq, Hq, Hkv, G;
  int no_state_temp;
};

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

template <int D>
__global__ void __launch_bounds__(256) attn_simt_kernel(AttnSimtParams p) {
  constexpr int CH = D / 32;      // output channels per lane
  constexpr int RW = D / 2 + 1;   // padded row stride in 32-bit words (conflict-free per-lane rows)
  __shared__ uint32_t sK[32 * RW];
  __shared__ uint32_t sV[32 * RW];
  __shared__ float sQ[8][D];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int bh = blockIdx.y;
  const int bb = bh / p.Hq, hq = bh % p.Hq, hk = hq / p.G;
  const int64_t u = (int64_t)bb * p.Hkv + hk;
  const int qi = blockIdx.x * 8 + warp;
  const bool valid = qi < p.nq;
  const int64_t t = p.t0 + qi;
  const int64_t m = p.m;

  if (valid) {
    const __half* qrow = p.stQ + ((int64_t)bh * p.Tcall + p.q_row0 + qi) * D;
    for (int x = lane; x < D; x += 32) sQ[warp][x] = __half2float(qrow[x]);
  }
  const int qlast = min(blockIdx.x * 8 + 7, p.nq - 1);
  const int64_t limit = valid ? m + (t - p.b + 1) : 0;
  const int64_t limit_max = m + (p.t0 + qlast - p.b + 1);
  const float kLog2e = 1.4426950408889634f;
  const float scale_s = p.tau_s[hq] * rsqrtf((float)D) * kLog2e;
  const float scale_b = p.tau_b[hq] * rsqrtf((float)D) * kLog2e;

  float m_run = -INFINITY, l_run = 0.f;
  float acc[CH];
#pragma unroll
  for (int c = 0; c < CH; ++c) acc[c] = 0.f;

  for (int64_t tile0 = 0; tile0 < limit_max; tile0 += 32) {
    __syncthreads();
    for (int wd = tid; wd < 32 * (D / 2); wd += 256) {
      const int row = wd / (D / 2), cw = wd % (D / 2);
      const int64_t kk = tile0 + row;
      uint32_t wk = 0u, wv = 0u;
      if (kk < limit_max) {
        const __half *srcK, *srcV;
        if (kk < m) {
          srcK = p.Khat + (u * p.Mcap + kk) * D;
          srcV = p.Vhat + (u * p.Mcap + kk) * D;
        } else {
          srcK = p.stK + (u * p.stRows + p.win_row0 + (kk - m)) * D;
          srcV = p.stV + (u * p.stRows + p.win_row0 + (kk - m)) * D;
        }
        wk = reinterpret_cast<const uint32_t*>(srcK)[cw];
        wv = reinterpret_cast<const uint32_t*>(srcV)[cw];
      }
      sK[row * RW + cw] = wk;
      sV[row * RW + cw] = wv;
    }
    __syncthreads();
    if (valid && tile0 < limit) {
      const int64_t kk = tile0 + lane;
      float logit = -INFINITY;
      if (kk < limit) {
        float dot = 0.f;
        const uint32_t* kr = sK + lane * RW;
#pragma unroll 8
        for (int cw = 0; cw < D / 2; ++cw) {
          const float2 kf = __half22float2(*reinterpret_cast<const __half2*>(&kr[cw]));
          dot = fmaf(sQ[warp][2 * cw], kf.x, dot);
          dot = fmaf(sQ[warp][2 * cw + 1], kf.y, dot);
        }
        logit = dot * (kk < m ? scale_s : scale_b);
      }
      const float tmax = warp_max(logit);
      const float mnew = fmaxf(m_run, tmax);
      const float corr = exp2f(m_run - mnew);
      const float pj = (kk < limit) ? exp2f(logit - mnew) : 0.f;
      l_run = l_run * corr + warp_sum(pj);
      m_run = mnew;
#pragma unroll
      for (int c = 0; c < CH; ++c) acc[c] *= corr;
      for (int j = 0; j < 32; ++j) {
        const float pb = __shfl_sync(0xffffffffu, pj, j);
        if (pb != 0.f) {
          const uint32_t* vr = sV + j * RW + lane * (CH / 2);
#pragma unroll
          for (int c2 = 0; c2 < CH / 2; ++c2) {
            const float2 vf = __half22float2(*reinterpret_cast<const __half2*>(&vr[c2]));
            acc[2 * c2] = fmaf(pb, vf.x, acc[2 * c2]);
            acc[2 * c2 + 1] = fmaf(pb, vf.y, acc[2 * c2 + 1]);
          }
        }
      }
    }
  }
  if (valid) {
    const float inv = 1.f / l_run;
    __nv_bfloat16* orow = p.out + bb * p.so0 + hq * p.so1 + (p.out_t0 + qi) * p.so2;
#pragma unroll
    for (int c2 = 0; c2 < CH / 2; ++c2) {
      reinterpret_cast<__nv_bfloat162*>(orow + lane * CH)[c2] =
          __floats2bfloat162_rn(acc[2 * c2] * inv, acc[2 * c2 + 1] * inv);
    }
  }
}

int launch_attn_simt(State* st, const AttnArgs& a, cudaStream_t s) {
  AttnSimtParams p;
  p.stQ = st->stQ; p.stK = st->stK; p.stV = st->stV; p.Khat = st->KhatBuf[st->nfolds & 1]; p.Vhat = st->VhatBuf[st->nfolds & 1];
  p.tau_s = st->tau_s; p.tau_b = st->tau_b;
  p.out = a.out;
  p.Tcall = st->Tcall; p.stRows = st->stRows; p.Mcap = st->Mcap;
  p.q_row0 = a.q_row0; p.t0 = a.t0; p.m = a.m; p.win_row0 = a.win_row0; p.b = a.b; p.out_t0 = a.out_t0;
  p.so0 = a.so[0]; p.so1 = a.so[1]; p.so2 = a.so[2];
  p.nq = a.nq; p.Hq = st->Hq; p.Hkv = st->Hkv; p.G = st->G;
  p.no_state_temp = 0;
  dim3 grid((a.nq + 7) / 8, st->B * st->Hq);
  if (st->d == 128) attn_simt_kernel<128><<<grid, 256, 0, s>>>(p);
  else attn_simt_kernel<64><<<grid, 256, 0, s>>>(p);
  return 1;
}

}  // namespace kvm
