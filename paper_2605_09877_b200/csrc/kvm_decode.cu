// Single-token decode (Table 1 "Decode time per token"): one query per head attends over the
// m readout rows of the state plus the window tokens [b, t].  The step is bound by HBM
// bandwidth (it streams K_hat, V_hat and the window once), so the kernel is a streaming
// reduction: every warp walks its share of the rows with 16-byte loads, keeps an online
// softmax in registers, warps are merged with shuffles and shared memory, and row splits
// (when there are too few heads to fill the GPU) are merged by a small second kernel.
#include "kvm_internal.h"

namespace kvm {

// Rotates q and k of the new token, stores k, v, gate in the window ring and the rotated query
// (rounded to bf16 exactly like the prefill staging) in decQ.
__global__ void decode_ingest_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                                     const __nv_bfloat16* __restrict__ v, const float* __restrict__ gate,
                                     const double* __restrict__ inv_freq, __half* __restrict__ decQ,
                                     __half* __restrict__ ringK, __half* __restrict__ ringV,
                                     float* __restrict__ ringG, int nQ, int nKV, int d, int r, int64_t t,
                                     int64_t ringCap, int64_t ringLen, int32_t* __restrict__ sat_counter) {
  // blocks [0, nQ): query heads; blocks [nQ, nQ + nKV): kv units
  const int x = threadIdx.x;
  if (x >= d) return;
  const int half = r >> 1;
  float cs = 1.f, sn = 0.f;
  int partner = x;
  if (x < r) {
    const int pidx = x < half ? x : x - half;
    double s, c;
    sincos((double)t * inv_freq[pidx], &s, &c);
    cs = (float)c; sn = (float)s;
    partner = x < half ? x + half : x - half;
  }
  if ((int)blockIdx.x < nQ) {
    const __nv_bfloat16* row = q + (int64_t)blockIdx.x * d;
    const float val = __bfloat162float(row[x]);
    const float oth = __bfloat162float(row[partner]);
    const float o = (x < r) ? (x < half ? val * cs - oth * sn : oth * sn + val * cs) : val;
    if (!(fabsf(o) <= 65504.f)) atomicAdd(sat_counter, 1);   // (clamped: counted for the debug counter)
    decQ[(int64_t)blockIdx.x * d + x] = __float2half_rn(fminf(fmaxf(o, -65504.f), 65504.f));
  } else {
    const int u = blockIdx.x - nQ;
    const __nv_bfloat16* row = k + (int64_t)u * d;
    const float val = __bfloat162float(row[x]);
    const float oth = __bfloat162float(row[partner]);
    const float o = (x < r) ? (x < half ? val * cs - oth * sn : oth * sn + val * cs) : val;
    const int64_t rrow = (int64_t)u * ringCap + (t % ringLen);
    const float vv = __bfloat162float(v[(int64_t)u * d + x]);
    const int nsat = (!(fabsf(o) <= 65504.f) ? 1 : 0) + (!(fabsf(vv) <= 65504.f) ? 1 : 0);
    if (nsat) atomicAdd(sat_counter, nsat);
    ringK[rrow * d + x] = __float2half_rn(fminf(fmaxf(o, -65504.f), 65504.f));
    ringV[rrow * d + x] = __float2half_rn(fminf(fmaxf(vv, -65504.f), 65504.f));
    if (x == 0) ringG[rrow] = gate ? gate[u] : 1.0f;
  }
}

struct DecodeParams {
  const __half *decQ, *Khat, *Vhat, *ringK, *ringV;
  const float *tau_s, *tau_b;
  __nv_bfloat16* out;
  float* part;     // [B*Hq, nsplit, D + 2]
  int64_t Mcap, ringCap, ringLen, m, b, t;
  int Hq, Hkv, G, nsplit;
};

__device__ __forceinline__ void unpack8(const uint4& w, float (&f)[8]) {
  const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&w.x));
  const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&w.y));
  const float2 c = __half22float2(*reinterpret_cast<const __half2*>(&w.z));
  const float2 e = __half22float2(*reinterpret_cast<const __half2*>(&w.w));
  f[0] = a.x; f[1] = a.y; f[2] = b.x; f[3] = b.y; f[4] = c.x; f[5] = c.y; f[6] = e.x; f[7] = e.y;
}

__device__ __forceinline__ uint4 ldg_stream(const void* p) {
  uint4 r;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
  return r;
}

// grid (nsplit, B*Hq); block 256 = 8 warps.  LPR = D/8 lanes cover one row with 16-byte loads,
// a warp covers RPW = 32/LPR rows per load instruction and UNR such instructions per step.
template <int D>
__global__ void __launch_bounds__(256) decode_attn_kernel(DecodeParams p) {
  constexpr int LPR = D / 8;
  constexpr int RPW = 32 / LPR;
  constexpr int UNR = 4;
  constexpr int STEP = RPW * UNR;       // rows per warp per iteration
  __shared__ float s_m[8], s_l[8];
  __shared__ float s_acc[8][D];

  const int split = blockIdx.x, bh = blockIdx.y;
  const int bb = bh / p.Hq, hq = bh % p.Hq, hk = hq / p.G;
  const int64_t u = (int64_t)bb * p.Hkv + hk;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int grp = lane / LPR, gl = lane % LPR;   // row group inside the warp, lane inside the row

  const int64_t m = p.m;
  const int64_t n = m + (p.t - p.b + 1);
  int64_t per = (n + p.nsplit - 1) / p.nsplit;
  per = (per + 8 * STEP - 1) / (8 * STEP) * (8 * STEP);
  const int64_t r0 = (int64_t)split * per;
  const int64_t r1 = min(n, r0 + per);

  const float kLog2e = 1.4426950408889634f;
  const float scale_s = p.tau_s[hq] * rsqrtf((float)D) * kLog2e;
  const float scale_b = p.tau_b[hq] * rsqrtf((float)D) * kLog2e;

  float qf[8];
  {
    const uint4 qw = *reinterpret_cast<const uint4*>(p.decQ + (int64_t)bh * D + gl * 8);
    unpack8(qw, qf);
  }
  float m_run = -INFINITY, l_run = 0.f;
  float acc[8];
#pragma unroll
  for (int c = 0; c < 8; ++c) acc[c] = 0.f;

  const __half* KhatU = p.Khat + u * p.Mcap * D;
  const __half* VhatU = p.Vhat + u * p.Mcap * D;
  const __half* ringKU = p.ringK + u * p.ringCap * D;
  const __half* ringVU = p.ringV + u * p.ringCap * D;

  for (int64_t base = r0 + (int64_t)warp * STEP; base < r1; base += 8 * STEP) {
    uint4 kw[UNR], vw[UNR];
    bool ok[UNR];
    bool st_[UNR];
#pragma unroll
    for (int i = 0; i < UNR; ++i) {
      const int64_t row = base + i * RPW + grp;
      ok[i] = row < r1;
      st_[i] = row < m;
      if (ok[i]) {
        const __half *kp, *vp;
        if (st_[i]) {
          kp = KhatU + row * D;
          vp = VhatU + row * D;
        } else {
          const int64_t slot = (p.b + (row - m)) % p.ringLen;
          kp = ringKU + slot * D;
          vp = ringVU + slot * D;
        }
        kw[i] = ldg_stream(kp + gl * 8);
        vw[i] = ldg_stream(vp + gl * 8);
      } else {
        kw[i] = make_uint4(0, 0, 0, 0);
        vw[i] = make_uint4(0, 0, 0, 0);
      }
    }
    float lg[UNR];
    float tmax = -INFINITY;
#pragma unroll
    for (int i = 0; i < UNR; ++i) {
      float kf[8];
      unpack8(kw[i], kf);
      float dot = 0.f;
#pragma unroll
      for (int c = 0; c < 8; ++c) dot = fmaf(qf[c], kf[c], dot);
#pragma unroll
      for (int o = LPR / 2; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
      lg[i] = ok[i] ? dot * (st_[i] ? scale_s : scale_b) : -INFINITY;
      tmax = fmaxf(tmax, lg[i]);
    }
    // maximum over the row groups of the warp
#pragma unroll
    for (int o = 16; o >= LPR; o >>= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, o));
    if (tmax == -INFINITY) continue;   // warp-uniform: no valid row in this step
    const float mnew = fmaxf(m_run, tmax);
    const float corr = exp2f(m_run - mnew);
    m_run = mnew;
    l_run *= corr;
#pragma unroll
    for (int c = 0; c < 8; ++c) acc[c] *= corr;
#pragma unroll
    for (int i = 0; i < UNR; ++i) {
      const float pr = exp2f(lg[i] - mnew);   // 0 for invalid rows
      l_run += pr;
      float vf[8];
      unpack8(vw[i], vf);
#pragma unroll
      for (int c = 0; c < 8; ++c) acc[c] = fmaf(pr, vf[c], acc[c]);
    }
  }
  // merge the row groups of the warp (all share m_run; l_run is per group)
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
    if (p.nsplit == 1) {
      p.out[(int64_t)bh * D + tid] = __float2bfloat16_rn(a / l);
    } else {
      float* dst = p.part + ((int64_t)bh * p.nsplit + split) * (D + 2);
      dst[tid] = a;
      if (tid == 0) { dst[D] = mx; dst[D + 1] = l; }
    }
  }
}

template <int D>
__global__ void decode_combine_kernel(const float* __restrict__ part, __nv_bfloat16* __restrict__ out, int nsplit) {
  const int bh = blockIdx.x, x = threadIdx.x;
  if (x >= D) return;
  const float* src = part + (int64_t)bh * nsplit * (D + 2);
  float mx = -INFINITY;
  for (int s = 0; s < nsplit; ++s) mx = fmaxf(mx, src[s * (D + 2) + D]);
  float l = 0.f, a = 0.f;
  for (int s = 0; s < nsplit; ++s) {
    const float ms = src[s * (D + 2) + D];
    const float f = (ms == -INFINITY) ? 0.f : exp2f(ms - mx);
    l += src[s * (D + 2) + D + 1] * f;
    a += src[s * (D + 2) + x] * f;
  }
  out[(int64_t)bh * D + x] = __float2bfloat16_rn(a / l);
}

int launch_decode(State* st, const DecodeArgs& a, cudaStream_t s) {
  int launches = 0;
  const int D = st->d;
  const int nQ = st->B * st->Hq, nKV = st->U;
  decode_ingest_kernel<<<nQ + nKV, D, 0, s>>>(a.q, a.k, a.v, a.gate, st->inv_freq, st->decQ, st->ringK, st->ringV,
                                              st->ringG, nQ, nKV, D, st->r, a.t, (int64_t)st->w * st->Cmax,
                                              st->ringLen, st->status + 4);
  ++launches;
  DecodeParams p;
  p.decQ = st->decQ; p.Khat = st->KhatBuf[st->nfolds & 1]; p.Vhat = st->VhatBuf[st->nfolds & 1]; p.ringK = st->ringK; p.ringV = st->ringV;
  p.tau_s = st->tau_s; p.tau_b = st->tau_b; p.out = a.out; p.part = st->decPart;
  p.Mcap = st->Mcap; p.ringCap = (int64_t)st->w * st->Cmax; p.ringLen = st->ringLen;
  p.m = a.m; p.b = a.b; p.t = a.t;
  p.Hq = st->Hq; p.Hkv = st->Hkv; p.G = st->G;
  // splits: fill ~4 CTAs per SM, keep at least 256 rows per split
  const int64_t n = a.m + (a.t - a.b + 1);
  int64_t want = (4 * 148 + nQ - 1) / nQ;
  int64_t maxs = (n + 255) / 256;
  int nsplit = (int)(want < maxs ? want : maxs);
  if (nsplit < 1) nsplit = 1;
  if (nsplit > st->nsplitDec) nsplit = st->nsplitDec;
  p.nsplit = nsplit;
  dim3 grid(nsplit, nQ);
  if (D == 128) decode_attn_kernel<128><<<grid, 256, 0, s>>>(p);
  else decode_attn_kernel<64><<<grid, 256, 0, s>>>(p);
  ++launches;
  if (nsplit > 1) {
    if (D == 128) decode_combine_kernel<128><<<nQ, 128, 0, s>>>(st->decPart, a.out, nsplit);
    else decode_combine_kernel<64><<<nQ, 64, 0, s>>>(st->decPart, a.out, nsplit);
    ++launches;
  }
  return launches;
}

}  // namespace kvm
