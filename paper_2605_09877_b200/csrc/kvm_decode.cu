// Single-token decode (Table 1 "Decode time per token"): one query per head attends over the
// m readout rows of the state plus the window tokens [b, t].  The step is bound by HBM
// bandwidth (it streams K_hat, V_hat and the window once), so the kernel is a streaming
// reduction: every warp walks its share of the rows with 16-byte loads, keeps an online
// softmax in registers, warps are merged with shuffles and shared memory, and row splits
// (when there are too few heads to fill the GPU) are merged by a small second kernel.
#include "kvm_internal.h"
#include "ln_rows.cuh"

namespace kvm {

// One rotary channel: `val` with its partner `oth` of the other rotary half.
__device__ __forceinline__ float rope_pair(float val, float oth, float cs, float sn, bool lower) {
  return lower ? val * cs - oth * sn : oth * sn + val * cs;
}

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
    const float o = (x < r) ? rope_pair(val, oth, cs, sn, x < half) : val;
    if (!(fabsf(o) <= 65504.f)) atomicAdd(sat_counter, 1);   // (clamped: counted for the debug counter)
    decQ[(int64_t)blockIdx.x * d + x] = __float2half_rn(fminf(fmaxf(o, -65504.f), 65504.f));
  } else {
    const int u = blockIdx.x - nQ;
    const __nv_bfloat16* row = k + (int64_t)u * d;
    const float val = __bfloat162float(row[x]);
    const float oth = __bfloat162float(row[partner]);
    const float o = (x < r) ? rope_pair(val, oth, cs, sn, x < half) : val;
    const int64_t rrow = (int64_t)u * ringCap + (t % ringLen);
    const float vv = __bfloat162float(v[(int64_t)u * d + x]);
    const int nsat = (!(fabsf(o) <= 65504.f) ? 1 : 0) + (!(fabsf(vv) <= 65504.f) ? 1 : 0);
    if (nsat) atomicAdd(sat_counter, nsat);
    ringK[rrow * d + x] = __float2half_rn(fminf(fmaxf(o, -65504.f), 65504.f));
    ringV[rrow * d + x] = __float2half_rn(fminf(fmaxf(vv, -65504.f), 65504.f));
    if (x == 0) ringG[rrow] = gate ? gate[u] : 1.0f;
  }
}

// The same with LN_q / LN_k applied first (fused front end): one warp per head, d / 8 lanes hold the row as
// eight channels each (ln_chunk8: the arithmetic of kvm_head_layernorm), the other lane groups compute
// copies and store nothing.  Rotation as in decode_ingest_kernel, the partner channel comes from the lane
// that holds it.
template <int D>
__global__ void __launch_bounds__(32) decode_ingest_ln_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                                        const __nv_bfloat16* __restrict__ v, const float* __restrict__ gate,
                                        const double* __restrict__ inv_freq, __half* __restrict__ decQ,
                                        __half* __restrict__ ringK, __half* __restrict__ ringV, float* __restrict__ ringG,
                                        int nQ, int nKV, int Hq, int Hkv, int r, int64_t t, int64_t ringCap, int64_t ringLen,
                                        int32_t* __restrict__ sat_counter, const float* __restrict__ lnq_w,
                                        const float* __restrict__ lnq_b, const float* __restrict__ lnk_w,
                                        const float* __restrict__ lnk_b, float eps) {
  constexpr int LPR = D / 8;
  const int lane = threadIdx.x, sub = lane % LPR;
  const bool store = lane < LPR;
  const bool isq = (int)blockIdx.x < nQ;
  const int idx = isq ? blockIdx.x : blockIdx.x - nQ;
  const int h = isq ? idx % Hq : idx % Hkv;
  const __nv_bfloat16* row = (isq ? q : k) + (int64_t)idx * D;
  float x[8];
  {
    const uint4 raw = *reinterpret_cast<const uint4*>(row + sub * 8);
    const __nv_bfloat162* pv = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 f = __bfloat1622float2(pv[i]);
      x[2 * i] = f.x; x[2 * i + 1] = f.y;
    }
  }
  float w8[8], b8[8];
  ln_load_affine<D>(isq ? lnq_w : lnk_w, isq ? lnq_b : lnk_b, h, sub, w8, b8);
  ln_chunk8<D>(x, w8, b8, eps);
  const int half = r >> 1;
  float o[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) o[i] = x[i];
  if (r > 0) {   // (uniform; r / 2 is a multiple of 8, so a partner chunk is a whole lane's)
    const int ch0 = sub * 8;
    const bool inr = ch0 < r, lower = ch0 < half;
    const int src = (lane & ~(LPR - 1)) + (inr ? (lower ? sub + half / 8 : sub - half / 8) : sub);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float oth = __shfl_sync(0xffffffffu, x[i], src);
      if (inr) {
        const int pidx = (lower ? ch0 : ch0 - half) + i;
        double sn, cs;
        sincos((double)t * inv_freq[pidx], &sn, &cs);
        o[i] = rope_pair(x[i], oth, (float)cs, (float)sn, lower);
      }
    }
  }
  if (!store) return;
  int nsat = 0;
  __half hv[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    nsat += !(fabsf(o[i]) <= 65504.f) ? 1 : 0;
    hv[i] = __float2half_rn(fminf(fmaxf(o[i], -65504.f), 65504.f));
  }
  if (isq) {
    *reinterpret_cast<uint4*>(decQ + (int64_t)idx * D + sub * 8) = *reinterpret_cast<const uint4*>(hv);
  } else {
    const int64_t rrow = (int64_t)idx * ringCap + (t % ringLen);
    *reinterpret_cast<uint4*>(ringK + rrow * D + sub * 8) = *reinterpret_cast<const uint4*>(hv);
    __half vh[8];
    const uint4 raw = *reinterpret_cast<const uint4*>(v + (int64_t)idx * D + sub * 8);
    const __nv_bfloat162* pv = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 f = __bfloat1622float2(pv[i]);
      nsat += (!(fabsf(f.x) <= 65504.f) ? 1 : 0) + (!(fabsf(f.y) <= 65504.f) ? 1 : 0);
      vh[2 * i] = __float2half_rn(fminf(fmaxf(f.x, -65504.f), 65504.f));
      vh[2 * i + 1] = __float2half_rn(fminf(fmaxf(f.y, -65504.f), 65504.f));
    }
    *reinterpret_cast<uint4*>(ringV + rrow * D + sub * 8) = *reinterpret_cast<const uint4*>(vh);
    if (sub == 0) ringG[rrow] = gate ? gate[idx] : 1.0f;
  }
  if (nsat) atomicAdd(sat_counter, nsat);
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

// grid (nsplit, B*Hq / GQ); block 256 = 8 warps.  LPR = D/8 lanes cover one row with 16-byte loads,
// a warp covers RPW = 32/LPR rows per load instruction and UNR such instructions per step.  A CTA
// serves GQ query heads that share one kv head (grouped queries): every key / value row is loaded
// once and meets all GQ queries, so the bytes streamed per step do not grow with the group size.
template <int D, int GQ>
__global__ void __launch_bounds__(256) decode_attn_kernel(DecodeParams p) {
  constexpr int LPR = D / 8;
  constexpr int RPW = 32 / LPR;
  constexpr int UNR = 4;
  constexpr int STEP = RPW * UNR;       // rows per warp per iteration
  __shared__ float s_m[8][GQ], s_l[8][GQ];
  __shared__ float s_acc[8][GQ][D];

  const int split = blockIdx.x;
  const int bh0 = blockIdx.y * GQ;                 // first query head of this CTA (GQ divides the group size G)
  const int bb = bh0 / p.Hq, hq0 = bh0 % p.Hq, hk = hq0 / p.G;
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
  float scale_s[GQ], scale_b[GQ];
  float qf[GQ][8];
#pragma unroll
  for (int g = 0; g < GQ; ++g) {
    scale_s[g] = p.tau_s[hq0 + g] * rsqrtf((float)D) * kLog2e;
    scale_b[g] = p.tau_b[hq0 + g] * rsqrtf((float)D) * kLog2e;
    const uint4 qw = *reinterpret_cast<const uint4*>(p.decQ + (int64_t)(bh0 + g) * D + gl * 8);
    unpack8(qw, qf[g]);
  }
  float m_run[GQ], l_run[GQ];
  float acc[GQ][8];
#pragma unroll
  for (int g = 0; g < GQ; ++g) {
    m_run[g] = -INFINITY; l_run[g] = 0.f;
#pragma unroll
    for (int c = 0; c < 8; ++c) acc[g][c] = 0.f;
  }

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
    float lg[GQ][UNR];
#pragma unroll
    for (int i = 0; i < UNR; ++i) {
      float kf[8];
      unpack8(kw[i], kf);
#pragma unroll
      for (int g = 0; g < GQ; ++g) {
        float dot = 0.f;
#pragma unroll
        for (int c = 0; c < 8; ++c) dot = fmaf(qf[g][c], kf[c], dot);
#pragma unroll
        for (int o = LPR / 2; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
        lg[g][i] = ok[i] ? dot * (st_[i] ? scale_s[g] : scale_b[g]) : -INFINITY;
      }
    }
#pragma unroll
    for (int g = 0; g < GQ; ++g) {
      float tmax = lg[g][0];
#pragma unroll
      for (int i = 1; i < UNR; ++i) tmax = fmaxf(tmax, lg[g][i]);
      // maximum over the row groups of the warp
#pragma unroll
      for (int o = 16; o >= LPR; o >>= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, o));
      if (tmax == -INFINITY) continue;   // warp-uniform: no valid row in this step
      const float mnew = fmaxf(m_run[g], tmax);
      const float corr = exp2f(m_run[g] - mnew);
      m_run[g] = mnew;
      l_run[g] *= corr;
#pragma unroll
      for (int c = 0; c < 8; ++c) acc[g][c] *= corr;
#pragma unroll
      for (int i = 0; i < UNR; ++i) {
        const float pr = exp2f(lg[g][i] - mnew);   // 0 for invalid rows
        l_run[g] += pr;
        float vf[8];
        unpack8(vw[i], vf);
#pragma unroll
        for (int c = 0; c < 8; ++c) acc[g][c] = fmaf(pr, vf[c], acc[g][c]);
      }
    }
  }
  // merge the row groups of the warp (all share m_run; l_run is per group)
#pragma unroll
  for (int g = 0; g < GQ; ++g) {
#pragma unroll
    for (int o = 16; o >= LPR; o >>= 1) {
      l_run[g] += __shfl_xor_sync(0xffffffffu, l_run[g], o);
#pragma unroll
      for (int c = 0; c < 8; ++c) acc[g][c] += __shfl_xor_sync(0xffffffffu, acc[g][c], o);
    }
    if (grp == 0) {
#pragma unroll
      for (int c = 0; c < 8; ++c) s_acc[warp][g][gl * 8 + c] = acc[g][c];
      if (gl == 0) { s_m[warp][g] = m_run[g]; s_l[warp][g] = l_run[g]; }
    }
  }
  __syncthreads();
  if (tid < D) {
#pragma unroll
    for (int g = 0; g < GQ; ++g) {
      float mx = -INFINITY;
#pragma unroll
      for (int w = 0; w < 8; ++w) mx = fmaxf(mx, s_m[w][g]);
      float l = 0.f, a = 0.f;
#pragma unroll
      for (int w = 0; w < 8; ++w) {
        const float f = (s_m[w][g] == -INFINITY) ? 0.f : exp2f(s_m[w][g] - mx);
        l += s_l[w][g] * f;
        a += s_acc[w][g][tid] * f;
      }
      const int64_t bh = bh0 + g;
      if (p.nsplit == 1) {
        p.out[bh * D + tid] = __float2bfloat16_rn(a / l);
      } else {
        float* dst = p.part + (bh * p.nsplit + split) * (D + 2);
        dst[tid] = a;
        if (tid == 0) { dst[D] = mx; dst[D + 1] = l; }
      }
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
  if (st->fusedLn) {
#define KVM_DEC_LN(DD)                                                                                                        \
    decode_ingest_ln_kernel<DD><<<nQ + nKV, 32, 0, s>>>(a.q, a.k, a.v, a.gate, st->inv_freq, st->decQ, st->ringK, st->ringV,   \
                                                        st->ringG, nQ, nKV, st->Hq, st->Hkv, st->r, a.t,                      \
                                                        (int64_t)st->w * st->Cmax, st->ringLen, st->status + 4, st->lnq_w,    \
                                                        st->lnq_b, st->lnk_w, st->lnk_b, st->qk_ln_eps)
    if (D == 128) { KVM_DEC_LN(128); } else { KVM_DEC_LN(64); }
#undef KVM_DEC_LN
  } else {
    decode_ingest_kernel<<<nQ + nKV, D, 0, s>>>(a.q, a.k, a.v, a.gate, st->inv_freq, st->decQ, st->ringK, st->ringV,
                                                st->ringG, nQ, nKV, D, st->r, a.t, (int64_t)st->w * st->Cmax,
                                                st->ringLen, st->status + 4);
  }
  ++launches;
  DecodeParams p;
  p.decQ = st->decQ; p.Khat = st->KhatBuf[st->nfolds & 1]; p.Vhat = st->VhatBuf[st->nfolds & 1]; p.ringK = st->ringK; p.ringV = st->ringV;
  p.tau_s = st->tau_s; p.tau_b = st->tau_b; p.out = a.out; p.part = st->decPart;
  p.Mcap = st->Mcap; p.ringCap = (int64_t)st->w * st->Cmax; p.ringLen = st->ringLen;
  p.m = a.m; p.b = a.b; p.t = a.t;
  p.Hq = st->Hq; p.Hkv = st->Hkv; p.G = st->G;
  // query heads of one kv group share a CTA (the largest of 8, 4, 2, 1 that divides the group size)
  const int GQ = (st->G % 8 == 0) ? 8 : (st->G % 4 == 0) ? 4 : (st->G % 2 == 0) ? 2 : 1;
  const int nCta = nQ / GQ;
  // splits: fill ~4 CTAs per SM, keep at least 256 rows per split
  const int64_t n = a.m + (a.t - a.b + 1);
  int64_t want = (4 * 148 + nCta - 1) / nCta;
  int64_t maxs = (n + 255) / 256;
  int nsplit = (int)(want < maxs ? want : maxs);
  if (nsplit < 1) nsplit = 1;
  if (nsplit > st->nsplitDec) nsplit = st->nsplitDec;
  p.nsplit = nsplit;
  dim3 grid(nsplit, nCta);
#define KVM_DEC(DD, GG) decode_attn_kernel<DD, GG><<<grid, 256, 0, s>>>(p)
  if (D == 128) { if (GQ == 8) KVM_DEC(128, 8); else if (GQ == 4) KVM_DEC(128, 4); else if (GQ == 2) KVM_DEC(128, 2); else KVM_DEC(128, 1); }
  else { if (GQ == 8) KVM_DEC(64, 8); else if (GQ == 4) KVM_DEC(64, 4); else if (GQ == 2) KVM_DEC(64, 2); else KVM_DEC(64, 1); }
#undef KVM_DEC
  ++launches;
  if (nsplit > 1) {
    if (D == 128) decode_combine_kernel<128><<<nQ, 128, 0, s>>>(st->decPart, a.out, nsplit);
    else decode_combine_kernel<64><<<nQ, 64, 0, s>>>(st->decPart, a.out, nsplit);
    ++launches;
  }
  return launches;
}

}  // namespace kvm
