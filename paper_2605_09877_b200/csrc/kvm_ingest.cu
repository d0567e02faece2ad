// Ingest: partial RoPE of q and k (Section 3.1 "Positional Encoding"; Appendix C "RoPE query/key")
// and staging of the call's tokens behind the not-yet-folded history taken from the window ring.
//
// Staging layout per unit u (rows of d bf16):  [ history tokens hist_start .. pos0-1 | new tokens ]
// so that the attention kernels address every window key of the call by (t - hist_start).
#include "kvm_internal.h"
#include "ln_rows.cuh"

namespace kvm {

// cos/sin of t * base^(-2p/r) for the call's tokens; the angle is formed in fp64 because at
// t ~ 1e5 an fp32 product already loses ~1e-2 rad.
__global__ void rope_table_kernel(float2* __restrict__ cs, const double* __restrict__ inv_freq,
                                  int64_t pos0, int64_t n, int half) {
  int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= n * half) return;
  int64_t i = idx / half;
  int p = (int)(idx % half);
  double ang = (double)(pos0 + i) * inv_freq[p];
  double s, c;
  sincos(ang, &s, &c);
  cs[idx] = make_float2((float)c, (float)s);
}

// Copies history tokens [hist_start, pos0) from the ring into staging rows [0, nhist).
__global__ void ingest_hist_kernel(__half* __restrict__ stK, __half* __restrict__ stV,
                                   float* __restrict__ stG, const __half* __restrict__ ringK,
                                   const __half* __restrict__ ringV, const float* __restrict__ ringG,
                                   int64_t stRows, int64_t ringCap, int64_t ringLen, int64_t hist_start,
                                   int64_t nhist, int d) {
  const int u = blockIdx.y;
  const int hw = d / 2;
  int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= nhist * hw) return;
  int64_t i = idx / hw;
  int c2 = (int)(idx % hw);
  int64_t slot = (hist_start + i) % ringLen;
  const uint32_t* sk = reinterpret_cast<const uint32_t*>(ringK + ((int64_t)u * ringCap + slot) * d);
  const uint32_t* sv = reinterpret_cast<const uint32_t*>(ringV + ((int64_t)u * ringCap + slot) * d);
  uint32_t* dk = reinterpret_cast<uint32_t*>(stK + ((int64_t)u * stRows + i) * d);
  uint32_t* dv = reinterpret_cast<uint32_t*>(stV + ((int64_t)u * stRows + i) * d);
  dk[c2] = sk[c2];
  dv[c2] = sv[c2];
  if (c2 == 0) stG[(int64_t)u * stRows + i] = ringG[(int64_t)u * ringCap + slot];
}

// bf16 inputs are carried as fp16 inside the library (same tensor-core rate, 3 more mantissa
// bits for the rotated values, the readout cache and the softmax weights).  Every bf16 value
// with 2^-14 <= |x| <= 65504 converts exactly; larger magnitudes saturate, smaller ones round
// with an absolute error below 2^-25.
// (nsat counts the values that did not fit - magnitudes above 65504, infinities, NaNs - for the debug counter)
__device__ __forceinline__ __half2 to_half2_sat(float a, float b, int& nsat) {
  nsat += (!(fabsf(a) <= 65504.f) ? 1 : 0) + (!(fabsf(b) <= 65504.f) ? 1 : 0);
  a = fminf(fmaxf(a, -65504.f), 65504.f);
  b = fminf(fmaxf(b, -65504.f), 65504.f);
  return __floats2half2_rn(a, b);
}

__device__ __forceinline__ float rope_channel(const __nv_bfloat16* row, int ch, int r, const float2* cs) {
  float val = __bfloat162float(row[ch]);
  if (ch >= r) return val;
  const int half = r >> 1;
  if (ch < half) {
    float other = __bfloat162float(row[ch + half]);
    float2 c = cs[ch];
    return val * c.x - other * c.y;
  }
  float other = __bfloat162float(row[ch - half]);
  float2 c = cs[ch - half];
  return other * c.y + val * c.x;
}

// New keys / values / gates of the call: rotate k, copy v, stage both, and write the tokens that
// stay in the window after this call (t >= tail_start) into the ring.
__global__ void ingest_kv_kernel(__half* __restrict__ stK, __half* __restrict__ stV,
                                 float* __restrict__ stG, __half* __restrict__ ringK,
                                 __half* __restrict__ ringV, float* __restrict__ ringG,
                                 const __nv_bfloat16* __restrict__ k, const __nv_bfloat16* __restrict__ v,
                                 const float* __restrict__ gate, const float2* __restrict__ ropeCS,
                                 int64_t sk0, int64_t sk1, int64_t sk2, int64_t sv0, int64_t sv1, int64_t sv2,
                                 int64_t sg0, int64_t sg1, int64_t sg2, int Hkv, int d, int r,
                                 int64_t stRows, int64_t ringCap, int64_t ringLen, int64_t pos0, int64_t n,
                                 int64_t nhist, int64_t tail_start, int32_t* __restrict__ sat_counter) {
  const int u = blockIdx.y;
  const int b = u / Hkv, hk = u % Hkv;
  const int hw = d / 2;
  int nsat = 0;
  int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= n * hw) return;
  int64_t j = idx / hw;
  int c2 = (int)(idx % hw);
  const __nv_bfloat16* krow = k + b * sk0 + hk * sk1 + j * sk2;
  const __nv_bfloat16* vrow = v + b * sv0 + hk * sv1 + j * sv2;
  const float2* cs = ropeCS + j * (r >> 1);
  const __half2 kk = to_half2_sat(rope_channel(krow, 2 * c2, r, cs), rope_channel(krow, 2 * c2 + 1, r, cs), nsat);
  const __half2 vv = to_half2_sat(__bfloat162float(vrow[2 * c2]), __bfloat162float(vrow[2 * c2 + 1]), nsat);
  if (nsat) atomicAdd(sat_counter, nsat);
  float g = gate ? gate[b * sg0 + hk * sg1 + j * sg2] : 1.0f;
  const int64_t row = (int64_t)u * stRows + nhist + j;
  reinterpret_cast<__half2*>(stK + row * d)[c2] = kk;
  reinterpret_cast<__half2*>(stV + row * d)[c2] = vv;
  if (c2 == 0) stG[row] = g;
  const int64_t t = pos0 + j;
  if (t >= tail_start) {
    const int64_t slot = t % ringLen;
    const int64_t rrow = (int64_t)u * ringCap + slot;
    reinterpret_cast<__half2*>(ringK + rrow * d)[c2] = kk;
    reinterpret_cast<__half2*>(ringV + rrow * d)[c2] = vv;
    if (c2 == 0) ringG[rrow] = g;
  }
}

__global__ void ingest_q_kernel(__half* __restrict__ stQ, const __nv_bfloat16* __restrict__ q,
                                const float2* __restrict__ ropeCS, int64_t sq0, int64_t sq1, int64_t sq2,
                                int Hq, int d, int r, int64_t Tcall, int64_t n, int32_t* __restrict__ sat_counter) {
  const int bh = blockIdx.y;
  const int b = bh / Hq, h = bh % Hq;
  const int hw = d / 2;
  int nsat = 0;
  int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= n * hw) return;
  int64_t j = idx / hw;
  int c2 = (int)(idx % hw);
  const __nv_bfloat16* qrow = q + b * sq0 + h * sq1 + j * sq2;
  const float2* cs = ropeCS + j * (r >> 1);
  reinterpret_cast<__half2*>(stQ + ((int64_t)bh * Tcall + j) * d)[c2] =
      to_half2_sat(rope_channel(qrow, 2 * c2, r, cs), rope_channel(qrow, 2 * c2 + 1, r, cs), nsat);
  if (nsat) atomicAdd(sat_counter, nsat);
}

// ---- 16-byte versions (rows 16-byte aligned, rotary half a multiple of 8 channels): a thread
//      converts eight consecutive channels of one token; same arithmetic as the scalar kernels ----

// Rotation of eight consecutive rotary channels `out` with their partners `oth` (the same channels of the
// other rotary half); c4 = the (cos, sin) pairs of these channels, two per float4.
__device__ __forceinline__ void rope_rotate8(float (&out)[8], const float (&oth)[8], const float4* __restrict__ c4, bool lower) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float4 cc = c4[i];   // cos0 sin0 cos1 sin1
    if (lower) {
      out[2 * i] = out[2 * i] * cc.x - oth[2 * i] * cc.y;
      out[2 * i + 1] = out[2 * i + 1] * cc.z - oth[2 * i + 1] * cc.w;
    } else {
      out[2 * i] = oth[2 * i] * cc.y + out[2 * i] * cc.x;
      out[2 * i + 1] = oth[2 * i + 1] * cc.w + out[2 * i + 1] * cc.z;
    }
  }
}

// Eight bf16 channels starting at channel c8*8 of a row: `raw` holds them, `rawo` their partners of the other
// rotary half (only read when the channels lie in the rotary range); rotated when they do.
__device__ __forceinline__ void rope8_from(const uint4& raw, const uint4& rawo, int c8, int r,
                                           const float2* __restrict__ cs, float (&out)[8]) {
  const __nv_bfloat162* pv = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 f = __bfloat1622float2(pv[i]);
    out[2 * i] = f.x; out[2 * i + 1] = f.y;
  }
  const int ch0 = c8 * 8;
  if (ch0 >= r) return;
  const int half = r >> 1;
  const bool lower = ch0 < half;
  const __nv_bfloat162* po = reinterpret_cast<const __nv_bfloat162*>(&rawo);
  float oth[8];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 o = __bfloat1622float2(po[i]);
    oth[2 * i] = o.x; oth[2 * i + 1] = o.y;
  }
  rope_rotate8(out, oth, reinterpret_cast<const float4*>(cs + (lower ? ch0 : ch0 - half)), lower);
}
// where the partners of chunk c8 start (any chunk outside the rotary range: itself, never used)
__device__ __forceinline__ int rope_partner8(int c8, int r) {
  const int ch0 = c8 * 8, half = r >> 1;
  return ch0 >= r ? ch0 : (ch0 < half ? ch0 + half : ch0 - half);
}

// Eight values -> eight fp16, clamped; nsat counts the values that did not fit.  The conversion itself saturates
// (cvt.rn.satfinite: a value beyond the fp16 range becomes +-65504, which no bf16 input converts to exactly -
// its neighbours are 65280 and 65536), so the packed result is tested first - one SIMD compare per pair, which
// also catches a NaN - and the values are only looked at one by one, and a NaN replaced by -65504 as a plain
// fmin/fmax clamp would, when it shows a hit.
__device__ __forceinline__ uint4 pack8_sat(const float (&x)[8], int& nsat) {
  uint4 o;
  uint32_t w[4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
    asm("cvt.rn.satfinite.f16x2.f32 %0, %1, %2;" : "=r"(w[i]) : "f"(x[2 * i + 1]), "f"(x[2 * i]));   // (first source: upper half)
  const uint32_t any = (__vcmpgeu2(w[0] & 0x7fff7fffu, 0x7bff7bffu) | __vcmpgeu2(w[1] & 0x7fff7fffu, 0x7bff7bffu)) |
                       (__vcmpgeu2(w[2] & 0x7fff7fffu, 0x7bff7bffu) | __vcmpgeu2(w[3] & 0x7fff7fffu, 0x7bff7bffu));
  if (any) {
#pragma unroll
    for (int i = 0; i < 8; ++i) nsat += !(fabsf(x[i]) <= 65504.f) ? 1 : 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const __half2 h = __floats2half2_rn(fminf(fmaxf(x[2 * i], -65504.f), 65504.f), fminf(fmaxf(x[2 * i + 1], -65504.f), 65504.f));
      w[i] = *reinterpret_cast<const uint32_t*>(&h);
    }
  }
  o.x = w[0]; o.y = w[1]; o.z = w[2]; o.w = w[3];
  return o;
}

// Tokens per thread of the 16-byte kernels: all loads of a thread's tokens are issued before the first value
// is looked at (a thread with one token had 32 bytes in flight, and a CTA lived for 16 tokens).
constexpr int kIngestTok = 2;

__global__ void __launch_bounds__(256) ingest_kv_vec_kernel(
    __half* __restrict__ stK, __half* __restrict__ stV, float* __restrict__ stG, __half* __restrict__ ringK,
    __half* __restrict__ ringV, float* __restrict__ ringG, const __nv_bfloat16* __restrict__ k,
    const __nv_bfloat16* __restrict__ v, const float* __restrict__ gate, const float2* __restrict__ ropeCS,
    int64_t sk0, int64_t sk1, int64_t sk2, int64_t sv0, int64_t sv1, int64_t sv2, int64_t sg0, int64_t sg1,
    int64_t sg2, int Hkv, int d, int r, int64_t stRows, int64_t ringCap, int64_t ringLen, int64_t pos0, int64_t n,
    int64_t nhist, int64_t tail_start, int32_t* __restrict__ sat_counter) {
  const int u = blockIdx.y;
  const int b = u / Hkv, hk = u % Hkv;
  const int w8 = d / 8;                       // 16-byte chunks per row
  const int tpb = 256 / w8;                   // tokens per pass of the block
  const int64_t j0 = (int64_t)blockIdx.x * tpb * kIngestTok + threadIdx.x / w8;
  const int c8 = threadIdx.x % w8;
  const int po = rope_partner8(c8, r);
  const bool rot = c8 * 8 < r;
  uint4 kr[kIngestTok], ko[kIngestTok], vr[kIngestTok];
  float g[kIngestTok];
#pragma unroll
  for (int it = 0; it < kIngestTok; ++it) {
    const int64_t j = j0 + (int64_t)it * tpb;
    kr[it] = ko[it] = vr[it] = make_uint4(0u, 0u, 0u, 0u);
    g[it] = 1.0f;
    if (j < n) {
      const __nv_bfloat16* krow = k + b * sk0 + hk * sk1 + j * sk2;
      kr[it] = *reinterpret_cast<const uint4*>(krow + c8 * 8);
      if (rot) ko[it] = *reinterpret_cast<const uint4*>(krow + po);
      vr[it] = *reinterpret_cast<const uint4*>(v + b * sv0 + hk * sv1 + j * sv2 + c8 * 8);
      if (gate) g[it] = gate[b * sg0 + hk * sg1 + j * sg2];
    }
  }
  int nsat = 0;
#pragma unroll
  for (int it = 0; it < kIngestTok; ++it) {
    const int64_t j = j0 + (int64_t)it * tpb;
    if (j >= n) continue;
    float kx[8], vx[8];
    rope8_from(kr[it], ko[it], c8, r, ropeCS + j * (r >> 1), kx);
    const __nv_bfloat162* pv = reinterpret_cast<const __nv_bfloat162*>(&vr[it]);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 f = __bfloat1622float2(pv[i]);
      vx[2 * i] = f.x; vx[2 * i + 1] = f.y;
    }
    const uint4 kk = pack8_sat(kx, nsat), vv = pack8_sat(vx, nsat);
    const int64_t row = (int64_t)u * stRows + nhist + j;
    reinterpret_cast<uint4*>(stK + row * d)[c8] = kk;
    reinterpret_cast<uint4*>(stV + row * d)[c8] = vv;
    if (c8 == 0) stG[row] = g[it];
    const int64_t t = pos0 + j;
    if (t >= tail_start) {
      const int64_t rrow = (int64_t)u * ringCap + t % ringLen;
      reinterpret_cast<uint4*>(ringK + rrow * d)[c8] = kk;
      reinterpret_cast<uint4*>(ringV + rrow * d)[c8] = vv;
      if (c8 == 0) ringG[rrow] = g[it];
    }
  }
  if (nsat) atomicAdd(sat_counter, nsat);
}

__global__ void __launch_bounds__(256) ingest_q_vec_kernel(__half* __restrict__ stQ, const __nv_bfloat16* __restrict__ q,
                                                           const float2* __restrict__ ropeCS, int64_t sq0, int64_t sq1,
                                                           int64_t sq2, int Hq, int d, int r, int64_t Tcall, int64_t n,
                                                           int32_t* __restrict__ sat_counter) {
  const int bh = blockIdx.y;
  const int b = bh / Hq, h = bh % Hq;
  const int w8 = d / 8, tpb = 256 / w8;
  const int64_t j0 = (int64_t)blockIdx.x * tpb * kIngestTok + threadIdx.x / w8;
  const int c8 = threadIdx.x % w8;
  const int po = rope_partner8(c8, r);
  const bool rot = c8 * 8 < r;
  uint4 qr[kIngestTok], qo[kIngestTok];
#pragma unroll
  for (int it = 0; it < kIngestTok; ++it) {
    const int64_t j = j0 + (int64_t)it * tpb;
    qr[it] = qo[it] = make_uint4(0u, 0u, 0u, 0u);
    if (j < n) {
      const __nv_bfloat16* qrow = q + b * sq0 + h * sq1 + j * sq2;
      qr[it] = *reinterpret_cast<const uint4*>(qrow + c8 * 8);
      if (rot) qo[it] = *reinterpret_cast<const uint4*>(qrow + po);
    }
  }
  int nsat = 0;
#pragma unroll
  for (int it = 0; it < kIngestTok; ++it) {
    const int64_t j = j0 + (int64_t)it * tpb;
    if (j >= n) continue;
    float qx[8];
    rope8_from(qr[it], qo[it], c8, r, ropeCS + j * (r >> 1), qx);
    reinterpret_cast<uint4*>(stQ + ((int64_t)bh * Tcall + j) * d)[c8] = pack8_sat(qx, nsat);
  }
  if (nsat) atomicAdd(sat_counter, nsat);
}

// ---- LN_q / LN_k applied on the way in (fused front end): the d / 8 threads that convert a token's row
//      first take its LayerNorm (ln_chunk8: the arithmetic of kvm_head_layernorm, result rounded to bf16
//      as that kernel stores it), fetch the rotary partner chunk from the lane that holds it, rotate and
//      stage.  Saves the read-modify-write pass of the stand-alone kernel over q and k. ----

// this lane's eight channels of `row` after LN and partial RoPE (every lane of the warp must call)
template <int D>
__device__ __forceinline__ void ln_rope8(const __nv_bfloat16* __restrict__ row, int c8, int r, const float2* __restrict__ cs,
                                         const float* __restrict__ lnw, const float* __restrict__ lnb, int h, float eps,
                                         float (&out)[8]) {
  constexpr int W8 = D / 8;
  const uint4 raw = *reinterpret_cast<const uint4*>(row + c8 * 8);
  const __nv_bfloat162* pv = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 f = __bfloat1622float2(pv[i]);
    out[2 * i] = f.x; out[2 * i + 1] = f.y;
  }
  float w8[8], b8[8];
  ln_load_affine<D>(lnw, lnb, h, c8, w8, b8);
  ln_chunk8<D>(out, w8, b8, eps);
  if (r == 0) return;   // (uniform)
  const int half = r >> 1, ch0 = c8 * 8;
  const bool inr = ch0 < r, lower = ch0 < half;
  const int lane = threadIdx.x & 31;
  const int src = (lane & ~(W8 - 1)) + (inr ? (lower ? c8 + half / 8 : c8 - half / 8) : c8);
  float oth[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) oth[i] = __shfl_sync(0xffffffffu, out[i], src);
  if (inr) rope_rotate8(out, oth, reinterpret_cast<const float4*>(cs + (lower ? ch0 : ch0 - half)), lower);
}

template <int D>
__global__ void __launch_bounds__(256) ingest_kv_ln_kernel(
    __half* __restrict__ stK, __half* __restrict__ stV, float* __restrict__ stG, __half* __restrict__ ringK,
    __half* __restrict__ ringV, float* __restrict__ ringG, const __nv_bfloat16* __restrict__ k,
    const __nv_bfloat16* __restrict__ v, const float* __restrict__ gate, const float2* __restrict__ ropeCS,
    int64_t sk0, int64_t sk1, int64_t sk2, int64_t sv0, int64_t sv1, int64_t sv2, int64_t sg0, int64_t sg1,
    int64_t sg2, int Hkv, int r, int64_t stRows, int64_t ringCap, int64_t ringLen, int64_t pos0, int64_t n,
    int64_t nhist, int64_t tail_start, int32_t* __restrict__ sat_counter, const float* __restrict__ lnw,
    const float* __restrict__ lnb, float eps) {
  constexpr int d = D, w8 = D / 8, tpb = 256 / w8;
  const int u = blockIdx.y;
  const int b = u / Hkv, hk = u % Hkv;
  const int64_t j0 = (int64_t)blockIdx.x * tpb + threadIdx.x / w8;
  const int c8 = threadIdx.x % w8;
  const bool live = j0 < n;                 // (rows past the end compute a copy of the last row: the shuffles need every lane)
  const int64_t j = live ? j0 : n - 1;
  float kx[8], vx[8];
  ln_rope8<D>(k + b * sk0 + hk * sk1 + j * sk2, c8, r, ropeCS + j * (r >> 1), lnw, lnb, hk, eps, kx);
  if (!live) return;
  {
    const uint4 raw = *reinterpret_cast<const uint4*>(v + b * sv0 + hk * sv1 + j * sv2 + c8 * 8);
    const __nv_bfloat162* pv = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 f = __bfloat1622float2(pv[i]);
      vx[2 * i] = f.x; vx[2 * i + 1] = f.y;
    }
  }
  int nsat = 0;
  const uint4 kk = pack8_sat(kx, nsat), vv = pack8_sat(vx, nsat);
  if (nsat) atomicAdd(sat_counter, nsat);
  const float g = gate ? gate[b * sg0 + hk * sg1 + j * sg2] : 1.0f;
  const int64_t row = (int64_t)u * stRows + nhist + j;
  reinterpret_cast<uint4*>(stK + row * d)[c8] = kk;
  reinterpret_cast<uint4*>(stV + row * d)[c8] = vv;
  if (c8 == 0) stG[row] = g;
  const int64_t t = pos0 + j;
  if (t >= tail_start) {
    const int64_t rrow = (int64_t)u * ringCap + t % ringLen;
    reinterpret_cast<uint4*>(ringK + rrow * d)[c8] = kk;
    reinterpret_cast<uint4*>(ringV + rrow * d)[c8] = vv;
    if (c8 == 0) ringG[rrow] = g;
  }
}

template <int D>
__global__ void __launch_bounds__(256) ingest_q_ln_kernel(__half* __restrict__ stQ, const __nv_bfloat16* __restrict__ q,
                                                          const float2* __restrict__ ropeCS, int64_t sq0, int64_t sq1,
                                                          int64_t sq2, int Hq, int r, int64_t Tcall, int64_t n,
                                                          int32_t* __restrict__ sat_counter, const float* __restrict__ lnw,
                                                          const float* __restrict__ lnb, float eps) {
  constexpr int w8 = D / 8, tpb = 256 / w8;
  const int bh = blockIdx.y;
  const int b = bh / Hq, h = bh % Hq;
  const int64_t j0 = (int64_t)blockIdx.x * tpb + threadIdx.x / w8;
  const int c8 = threadIdx.x % w8;
  const bool live = j0 < n;
  const int64_t j = live ? j0 : n - 1;
  float qx[8];
  ln_rope8<D>(q + b * sq0 + h * sq1 + j * sq2, c8, r, ropeCS + j * (r >> 1), lnw, lnb, h, eps, qx);
  if (!live) return;
  int nsat = 0;
  reinterpret_cast<uint4*>(stQ + ((int64_t)bh * Tcall + j) * D)[c8] = pack8_sat(qx, nsat);
  if (nsat) atomicAdd(sat_counter, nsat);
}

// Can this call take the 16-byte ingest kernels (which the fused front end requires)?
bool ingest_rows_aligned(int r, const IngestArgs& a) {
  auto al16 = [](const void* ptr, const int64_t* st3) {
    return ((uintptr_t)ptr & 15) == 0 && (st3[0] & 7) == 0 && (st3[1] & 7) == 0 && (st3[2] & 7) == 0;
  };
  const bool rope_ok = r == 0 || ((r / 2) % 8) == 0;
  return rope_ok && al16(a.k, a.sk) && al16(a.v, a.sv) && al16(a.q, a.sq);
}

int launch_ingest(State* st, const IngestArgs& a, cudaStream_t s) {
  int launches = 0;
  const int d = st->d, hw = d / 2;
  const int threads = 256;
  if (st->r > 0) {
    int64_t tot = a.n * (st->r / 2);
    rope_table_kernel<<<(unsigned)((tot + threads - 1) / threads), threads, 0, s>>>(st->ropeCS, st->inv_freq,
                                                                                  a.pos0, a.n, st->r / 2);
    ++launches;
  }
  if (a.nhist > 0) {
    dim3 grid((unsigned)((a.nhist * hw + threads - 1) / threads), st->U);
    ingest_hist_kernel<<<grid, threads, 0, s>>>(st->stK, st->stV, st->stG, st->ringK, st->ringV, st->ringG,
                                                st->stRows, (int64_t)st->w * st->Cmax, st->ringLen,
                                                a.hist_start, a.nhist, d);
    ++launches;
  }
  // 16-byte path: every row of q, k, v starts on a 16-byte boundary and a rotary half is whole chunks
  auto al16 = [](const void* ptr, const int64_t* st3) {
    return ((uintptr_t)ptr & 15) == 0 && (st3[0] & 7) == 0 && (st3[1] & 7) == 0 && (st3[2] & 7) == 0;
  };
  const bool rope_ok = st->r == 0 || ((st->r / 2) % 8) == 0;
  const int tpb = 256 / (d / 8);
  if (st->fusedLn) {   // (the caller has checked ingest_rows_aligned)
    dim3 gk((unsigned)((a.n + tpb - 1) / tpb), st->U), gq((unsigned)((a.n + tpb - 1) / tpb), st->B * st->Hq);
#define KVM_LN_INGEST(DD)                                                                                                   \
    ingest_kv_ln_kernel<DD><<<gk, 256, 0, s>>>(st->stK, st->stV, st->stG, st->ringK, st->ringV, st->ringG, a.k, a.v, a.gate, \
                                               st->ropeCS, a.sk[0], a.sk[1], a.sk[2], a.sv[0], a.sv[1], a.sv[2], a.sg[0],   \
                                               a.sg[1], a.sg[2], st->Hkv, st->r, st->stRows, (int64_t)st->w * st->Cmax,     \
                                               st->ringLen, a.pos0, a.n, a.nhist, a.tail_start, st->status + 4, st->lnk_w,  \
                                               st->lnk_b, st->qk_ln_eps);                                                   \
    ingest_q_ln_kernel<DD><<<gq, 256, 0, s>>>(st->stQ, a.q, st->ropeCS, a.sq[0], a.sq[1], a.sq[2], st->Hq, st->r, st->Tcall, \
                                              a.n, st->status + 4, st->lnq_w, st->lnq_b, st->qk_ln_eps)
    if (d == 128) { KVM_LN_INGEST(128); } else { KVM_LN_INGEST(64); }
#undef KVM_LN_INGEST
    return launches + 2;
  }
  if (rope_ok && al16(a.k, a.sk) && al16(a.v, a.sv)) {
    dim3 grid((unsigned)((a.n + tpb * kIngestTok - 1) / (tpb * kIngestTok)), st->U);
    ingest_kv_vec_kernel<<<grid, 256, 0, s>>>(st->stK, st->stV, st->stG, st->ringK, st->ringV, st->ringG, a.k,
                                              a.v, a.gate, st->ropeCS, a.sk[0], a.sk[1], a.sk[2], a.sv[0],
                                              a.sv[1], a.sv[2], a.sg[0], a.sg[1], a.sg[2], st->Hkv, d, st->r,
                                              st->stRows, (int64_t)st->w * st->Cmax, st->ringLen, a.pos0, a.n,
                                              a.nhist, a.tail_start, st->status + 4);
    ++launches;
  } else {
    dim3 grid((unsigned)((a.n * hw + threads - 1) / threads), st->U);
    ingest_kv_kernel<<<grid, threads, 0, s>>>(st->stK, st->stV, st->stG, st->ringK, st->ringV, st->ringG, a.k,
                                              a.v, a.gate, st->ropeCS, a.sk[0], a.sk[1], a.sk[2], a.sv[0],
                                              a.sv[1], a.sv[2], a.sg[0], a.sg[1], a.sg[2], st->Hkv, d, st->r,
                                              st->stRows, (int64_t)st->w * st->Cmax, st->ringLen, a.pos0, a.n,
                                              a.nhist, a.tail_start, st->status + 4);
    ++launches;
  }
  if (rope_ok && al16(a.q, a.sq)) {
    dim3 grid((unsigned)((a.n + tpb * kIngestTok - 1) / (tpb * kIngestTok)), st->B * st->Hq);
    ingest_q_vec_kernel<<<grid, 256, 0, s>>>(st->stQ, a.q, st->ropeCS, a.sq[0], a.sq[1], a.sq[2], st->Hq, d,
                                             st->r, st->Tcall, a.n, st->status + 4);
    ++launches;
  } else {
    dim3 grid((unsigned)((a.n * hw + threads - 1) / threads), st->B * st->Hq);
    ingest_q_kernel<<<grid, threads, 0, s>>>(st->stQ, a.q, st->ropeCS, a.sq[0], a.sq[1], a.sq[2], st->Hq, d,
                                             st->r, st->Tcall, a.n, st->status + 4);
    ++launches;
  }
  return launches;
}

}  // namespace kvm
