// The fold of one overflow block into the state (Section 3.2 "Append", "Merge", budget rule,
// value-radius preservation) for every unit:
//   1. kbar_kernel          memory keys kbar_j = LN_s(zero_r(k_j))            (Eq. 1) in fp64 and
//                           fp16, the keys LN_s(kbar_j) of the rows the tokens would create (fp16, and
//                           their LayerNorm statistics); computed for a batch of blocks ahead of the folds,
//                           together with the tensor-core products LN_s(kbar_a) . kbar_j (new-row filter)
//   2. routing filter       approximate similarities kbar_j . LN_s(s^K_i) in fp16 x fp16 -> fp32
//                           (tcgen05 kernel in kvm_route_tc.cu, scalar-core cross-check here),
//                           the rows within the rounding window of the best one, per token and row split
//   3. fold_decide_kernel   exact fp64 similarities of the candidates, append selection, merge
//                           routing against s_+ (new rows: filtered by the products of step 1, the few
//                           contenders exactly), grouping of the merged tokens by target row; several CTAs
//                           per unit share the refinement, the last one to finish takes the block-wide steps
//   4. fold_apply_kernel    one warp per touched row: creates appended rows, accumulates the
//                           members in ascending token order (deterministic), refreshes the
//                           readout cache (LN_s of the key sum, value-radius readout) in the readout
//                           copy of the new state version
//   (prev_copy_kernel brings the rows the previous fold touched over to that copy first.)
//
// Integer decisions (which tokens are appended, which row each token merges into) are taken on
// fp64 similarities computed from fp64 key sums, so they agree with an fp64 reference unless two
// similarities agree to ~1e-12.  The fp16 pass only prunes: a row is a candidate when its
// approximate similarity is within 2*eps of the best one, eps being a rigorous bound on the fp16
// rounding error of the dot product, so the true arg max is always among the candidates.
#include "kvm_internal.h"

namespace kvm {

__device__ __forceinline__ double warp_sum_d(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// LN_s statistics of one row held as D/32 strided channels per lane.
template <int CH>
__device__ __forceinline__ void row_stats(const double (&x)[CH], int D, double eps, double& mean, double& rstd) {
  double s = 0.0;
#pragma unroll
  for (int i = 0; i < CH; ++i) s += x[i];
  mean = warp_sum_d(s) / D;
  double q = 0.0;
#pragma unroll
  for (int i = 0; i < CH; ++i) q += (x[i] - mean) * (x[i] - mean);
  rstd = 1.0 / sqrt(warp_sum_d(q) / D + eps);
}

// The memory key kbar_j = LN_s(zero_r(k_j)) (Eq. 1) in fp64 is two thirds of everything the memory-key kernel
// writes, and the decision and application kernels read it back row by row.  States with enough units to
// fill the GPU - where the folds are bound by memory traffic, not by their chain of dependent launches - do
// not keep it (RK = true): every kernel that needs kbar_j recomputes it from the fp16 key and the token's
// (mean, rstd), with the roundings pinned so that all of them get the same bits.
__device__ __forceinline__ double ln_affine(double v, double mean, double rstd, double w, double b) {
  return __dadd_rn(__dmul_rn(w, __dmul_rn(__dsub_rn(v, mean), rstd)), b);
}
template <int D, bool RK>
struct KbarRows {            // the memory keys of one unit's folded block
  const double* k64;         // !RK: [C][D] fp64
  const __half* k16;         // RK: the block's keys [C][D] fp16 ...
  const double2* stat;       //     ... and (mean, rstd) of zero_r(k_j) per token
  int r;                     //     leading channels that zero_r clears
  // channel x of kbar_j; g, b = LN_s weight and bias of that channel
  __device__ __forceinline__ double at(int j, int x, double g, double b) const {
    if (!RK) return k64[(int64_t)j * D + x];
    const double2 st = stat[j];
    const double v = x < r ? 0.0 : (double)__half2float(k16[(int64_t)j * D + x]);
    return ln_affine(v, st.x, st.y, g, b);
  }
};

// channels x .. x + 3 of kbar_j (x a multiple of 4) for the kernels that hold rows as runs of four channels
template <int D, bool RK>
__device__ __forceinline__ void kbar_run4(const KbarRows<D, RK>& kr, int j, int x, const float* __restrict__ ln_w_h,
                                          const float* __restrict__ ln_b_h, double (&out)[4]) {
  if (!RK) {
    const double* kb = kr.k64 + (int64_t)j * D + x;
    const double2 k01 = *reinterpret_cast<const double2*>(kb), k23 = *reinterpret_cast<const double2*>(kb + 2);
    out[0] = k01.x; out[1] = k01.y; out[2] = k23.x; out[3] = k23.y;
  } else {
    alignas(8) __half hv[4];
    *reinterpret_cast<uint2*>(hv) = *reinterpret_cast<const uint2*>(kr.k16 + (int64_t)j * D + x);
    const float4 w4 = *reinterpret_cast<const float4*>(ln_w_h + x), b4 = *reinterpret_cast<const float4*>(ln_b_h + x);
    const float wv[4] = {w4.x, w4.y, w4.z, w4.w}, bv[4] = {b4.x, b4.y, b4.z, b4.w};
    const double2 st = kr.stat[j];
#pragma unroll
    for (int e = 0; e < 4; ++e)
      out[e] = ln_affine(x + e < kr.r ? 0.0 : (double)__half2float(hv[e]), st.x, st.y, (double)wv[e], (double)bv[e]);
  }
}

// ------------------------------------------------------------------------------------------
// 1. memory keys (one warp per overflow token)

// Four token rows per warp, eight lanes per row: every fp64 reduction step, divide and square root
// is an instruction of the whole warp whatever the number of rows it serves, and with one row per
// warp those made up most of the ~375 instructions per row (the kernel was bound by the fp64 pipe,
// not by memory).  Lane `sub` of a row's group holds channels 32 i + 4 sub .. + 3, so that the eight
// lanes of a group read and write contiguous runs.
constexpr int kKbarRowsPerWarp = 4;
constexpr int kKbarRowsPerCta = 8 * kKbarRowsPerWarp;

__device__ __forceinline__ double group8_sum_d(double v) {
#pragma unroll
  for (int o = 4; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

template <int D, bool RK>
__global__ void __launch_bounds__(256, RK ? 4 : 2) kbar_kernel(const __half* __restrict__ ok, int64_t unit_stride,
                                                      const float* __restrict__ ln_w, const float* __restrict__ ln_b,
                                                      double* __restrict__ kbar64, __half* __restrict__ kbarH,
                                                      float* __restrict__ kbarNorm, double2* __restrict__ kbarHatStat,
                                                      __half* __restrict__ kbarHatH, int C, int Cmax, int CbarRows, int U, int Hkv, int r,
                                                      double ln_eps, int write_hat, double2* __restrict__ kbarStat) {
  constexpr int NI = D / 32;          // runs of four channels per lane
  constexpr int NC = 4 * NI;          // channels per lane
  constexpr double inv_d = 1.0 / D;   // D is a power of two: the multiplication is the division, exactly
  const int u = blockIdx.y, hk = u % Hkv;
  const int g = blockIdx.z;   // block of the batch = slot
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int sub = lane & 7;
  const int j = (blockIdx.x * 8 + warp) * kKbarRowsPerWarp + (lane >> 3);
  const bool live = j < C;            // (dead groups compute a copy of the last row and store nothing:
  const int jj = live ? j : C - 1;    //  the shuffles below need every lane)
  const __half* row = ok + (int64_t)u * unit_stride + ((int64_t)g * C + jj) * D;
  double val[NC];
  float valf[NC];   // (the same values in fp32, for the launches that need nothing else in fp64)
#pragma unroll
  for (int i = 0; i < NI; ++i) {
    alignas(8) __half hv[4];
    *reinterpret_cast<uint2*>(hv) = *reinterpret_cast<const uint2*>(row + 32 * i + 4 * sub);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      valf[4 * i + e] = (32 * i + 4 * sub + e < r) ? 0.f : __half2float(hv[e]);
      val[4 * i + e] = (double)valf[4 * i + e];
    }
  }
  double sum = 0.0;
#pragma unroll
  for (int c = 0; c < NC; ++c) sum += val[c];
  const double mean = group8_sum_d(sum) * inv_d;
  double dev = 0.0;
#pragma unroll
  for (int c = 0; c < NC; ++c) dev += (val[c] - mean) * (val[c] - mean);
  const double rstd = 1.0 / sqrt(group8_sum_d(dev) * inv_d + ln_eps);
  const int64_t o = (((int64_t)g * U + u) * Cmax + jj) * D;
  const int64_t oh = (((int64_t)g * U + u) * CbarRows + jj) * D;
  if (RK && write_hat < 0) {
    // Nothing below is kept in fp64 for such a launch: the fp64 memory key is recomputed where it is needed from
    // (mean, rstd), which stay exact as above; what is written here - the fp16 key for the routing filter and its
    // norm for the filter's window - only has to be as good as an fp16 operand, so the affine map runs in fp32.
    // (|fp16(fp32 result) - kbar| exceeds half an fp16 ulp by < 2^-22 of the operands' magnitudes, inside the
    // 2^-13 |a| |b| that the window keeps in reserve; the norm is rounded up by more than its fp32 summation error.)
    const float mean_f = (float)mean, rstd_f = (float)rstd;
    float n2f = 0.f;
#pragma unroll
    for (int i = 0; i < NI; ++i) {
      const int x = 32 * i + 4 * sub;
      const float4 w4 = *reinterpret_cast<const float4*>(ln_w + hk * D + x), b4 = *reinterpret_cast<const float4*>(ln_b + hk * D + x);
      const float wv[4] = {w4.x, w4.y, w4.z, w4.w}, bv[4] = {b4.x, b4.y, b4.z, b4.w};
      alignas(8) __half kh[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float tf = fmaf(wv[e], (valf[4 * i + e] - mean_f) * rstd_f, bv[e]);
        kh[e] = __float2half_rn(tf);
        n2f = fmaf(tf, tf, n2f);
      }
      if (live) *reinterpret_cast<uint2*>(kbarH + oh + x) = *reinterpret_cast<const uint2*>(kh);
    }
#pragma unroll
    for (int o2 = 4; o2 > 0; o2 >>= 1) n2f += __shfl_xor_sync(0xffffffffu, n2f, o2);
    if (live && sub == 0) {
      kbarNorm[((int64_t)g * U + u) * Cmax + j] = sqrtf(n2f) * 1.00002f;
      kbarStat[((int64_t)g * U + u) * Cmax + j] = make_double2(mean, rstd);
    }
    return;
  }
  double kb[NC];
  double n2 = 0.0;
#pragma unroll
  for (int i = 0; i < NI; ++i) {
    const int x = 32 * i + 4 * sub;
    const float4 w4 = *reinterpret_cast<const float4*>(ln_w + hk * D + x), b4 = *reinterpret_cast<const float4*>(ln_b + hk * D + x);
    const float wv[4] = {w4.x, w4.y, w4.z, w4.w}, bv[4] = {b4.x, b4.y, b4.z, b4.w};
    alignas(8) __half kh[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const double t = RK ? ln_affine(val[4 * i + e], mean, rstd, (double)wv[e], (double)bv[e])
                          : (double)wv[e] * ((val[4 * i + e] - mean) * rstd) + (double)bv[e];
      kb[4 * i + e] = t;
      kh[e] = __float2half_rn((float)t);
      n2 += t * t;
    }
    if (live) {
      if (!RK) {
        reinterpret_cast<double2*>(kbar64 + o + x)[0] = make_double2(kb[4 * i], kb[4 * i + 1]);
        reinterpret_cast<double2*>(kbar64 + o + x)[1] = make_double2(kb[4 * i + 2], kb[4 * i + 3]);
      }
      *reinterpret_cast<uint2*>(kbarH + oh + x) = *reinterpret_cast<const uint2*>(kh);
    }
  }
  n2 = group8_sum_d(n2);
  if (live && sub == 0) {
    kbarNorm[((int64_t)g * U + u) * Cmax + j] = (float)sqrt(n2) * 1.000001f;
    if (RK) kbarStat[((int64_t)g * U + u) * Cmax + j] = make_double2(mean, rstd);
  }
  // (write_hat < 0: the decision kernel takes these statistics itself, for the few tokens that create rows)
  if (write_hat < 0) return;
  // LN_s applied to kbar itself: the readout key of the row that this token would create
  sum = 0.0;
#pragma unroll
  for (int c = 0; c < NC; ++c) sum += kb[c];
  const double mu2 = group8_sum_d(sum) * inv_d;
  dev = 0.0;
#pragma unroll
  for (int c = 0; c < NC; ++c) dev += (kb[c] - mu2) * (kb[c] - mu2);
  const double rs2 = 1.0 / sqrt(group8_sum_d(dev) * inv_d + ln_eps);
#pragma unroll
  for (int i = 0; i < NI; ++i) {
    const int x = 32 * i + 4 * sub;
    const float4 w4 = *reinterpret_cast<const float4*>(ln_w + hk * D + x), b4 = *reinterpret_cast<const float4*>(ln_b + hk * D + x);
    const float wv[4] = {w4.x, w4.y, w4.z, w4.w}, bv[4] = {b4.x, b4.y, b4.z, b4.w};
    alignas(8) __half kh[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const double hat = (double)wv[e] * ((kb[4 * i + e] - mu2) * rs2) + (double)bv[e];
      kh[e] = __float2half_rn((float)hat);
    }
    if (live && write_hat) *reinterpret_cast<uint2*>(kbarHatH + oh + x) = *reinterpret_cast<const uint2*>(kh);
  }
  if (live && sub == 0) kbarHatStat[((int64_t)g * U + u) * Cmax + j] = make_double2(mu2, rs2);
}

// Rows that the last fold touched are current in one readout copy only: bring them over to the
// other one (warp j takes the j-th appended row and the j-th merge target, as the apply kernel did).
struct PrevFoldCopy {
  int all_append, n_append, C, Cmax;
  int64_t m, Mcap;                       // rows before that fold; row capacity per unit
  const int32_t *pi, *sorted, *nmerge;   // that fold's decisions
  const __half *Ksrc, *Vsrc;
  __half *Kdst, *Vdst;
};

template <int D>
__global__ void __launch_bounds__(256) prev_copy_kernel(PrevFoldCopy pc) {
  const int u = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int j = blockIdx.x * 8 + warp;
  if (j >= pc.C) return;
  const int64_t tb = (int64_t)u * pc.Cmax;
  int64_t cpo[2] = {-1, -1};
  if (j < pc.n_append) cpo[0] = ((int64_t)u * pc.Mcap + pc.m + j) * D;
  if (!pc.all_append) {
    const int nm = pc.nmerge[u];
    int s0 = pc.sorted[tb + j], s1 = pc.sorted[tb + (j > 0 ? j - 1 : 0)];
    s0 = (unsigned)s0 < (unsigned)pc.Cmax ? s0 : 0;   // entries past nmerge are not defined
    s1 = (unsigned)s1 < (unsigned)pc.Cmax ? s1 : 0;
    const int r1 = pc.pi[tb + s0], r0 = pc.pi[tb + s1];
    if (j < nm && r1 >= 0 && r1 < pc.m && (j == 0 || r0 != r1)) cpo[1] = ((int64_t)u * pc.Mcap + r1) * D;
  }
  uint2 cpK[2], cpV[2];
#pragma unroll
  for (int t = 0; t < 2; ++t)
    if (cpo[t] >= 0 && lane < D / 4) {   // 8 bytes per lane
      cpK[t] = reinterpret_cast<const uint2*>(pc.Ksrc + cpo[t])[lane];
      cpV[t] = reinterpret_cast<const uint2*>(pc.Vsrc + cpo[t])[lane];
    }
#pragma unroll
  for (int t = 0; t < 2; ++t)
    if (cpo[t] >= 0 && lane < D / 4) {
      reinterpret_cast<uint2*>(pc.Kdst + cpo[t])[lane] = cpK[t];
      reinterpret_cast<uint2*>(pc.Vdst + cpo[t])[lane] = cpV[t];
    }
}

// ------------------------------------------------------------------------------------------
// 2. routing filter on the scalar cores (cross-check path; the default filter runs on tcgen05)

template <int D>
__global__ void __launch_bounds__(256) route_filter_simt_kernel(const __half* __restrict__ kbarH,
                                                                const __half* __restrict__ Khat,
                                                                float* __restrict__ candV,
                                                                int32_t* __restrict__ candI, int C, int Cmax,
                                                                int CbarRows, int64_t Mcap, int64_t m, int nsplit,
                                                                const float* __restrict__ kbarNorm, float thr_coeff,
                                                                int S) {
  __shared__ __half2 sH[32 * (D / 2)];
  const int split = blockIdx.x, u = blockIdx.y;
  const int j = threadIdx.x;
  const bool active = j < C;
  int64_t per = (m + nsplit - 1) / nsplit;
  per = (per + 127) / 128 * 128;
  const int64_t i0 = (int64_t)split * per;
  const int64_t i1 = min(m, i0 + per);

  __half2 kb[D / 2];
  if (active) {
    const __half2* src = reinterpret_cast<const __half2*>(kbarH + ((int64_t)u * CbarRows + j) * D);
#pragma unroll
    for (int c = 0; c < D / 2; ++c) kb[c] = src[c];
  }
  float tv[kTopK];
  int ti[kTopK];
#pragma unroll
  for (int k = 0; k < kTopK; ++k) { tv[k] = -INFINITY; ti[k] = -1; }

  for (int64_t tile = i0; tile < i1; tile += 32) {
    __syncthreads();
    for (int wd = threadIdx.x; wd < 32 * (D / 2); wd += 256) {
      const int row = wd / (D / 2), cw = wd % (D / 2);
      const int64_t i = tile + row;
      sH[wd] = (i < i1) ? reinterpret_cast<const __half2*>(Khat + ((int64_t)u * Mcap + i) * D)[cw]
                        : __floats2half2_rn(0.f, 0.f);
    }
    __syncthreads();
    if (active) {
      const int nrow = (int)min((int64_t)32, i1 - tile);
      for (int rr = 0; rr < nrow; ++rr) {
        float acc = 0.f;
#pragma unroll
        for (int c = 0; c < D / 2; ++c) {
          const float2 a = __half22float2(kb[c]);
          const float2 b = __half22float2(sH[rr * (D / 2) + c]);
          acc = fmaf(a.x, b.x, acc);
          acc = fmaf(a.y, b.y, acc);
        }
        if (acc > tv[kTopK - 1]) {
          tv[kTopK - 1] = acc;
          ti[kTopK - 1] = (int)(tile + rr);
#pragma unroll
          for (int k = kTopK - 1; k > 0; --k) {
            if (tv[k] > tv[k - 1]) {
              const float fv = tv[k]; tv[k] = tv[k - 1]; tv[k - 1] = fv;
              const int iv = ti[k]; ti[k] = ti[k - 1]; ti[k - 1] = iv;
            }
          }
        }
      }
    }
  }
  if (active) {
    // same output format as the tensor-core filter: candidate rows within the window of the split's
    // maximum over rows >= S, that maximum, and the candidate count (kTopK + 1 = overflow)
    const int64_t o = (((int64_t)u * nsplit + split) * Cmax + j) * kTopK;
    float mx = -INFINITY;
#pragma unroll
    for (int k = 0; k < kTopK; ++k) if (ti[k] >= S) mx = fmaxf(mx, tv[k]);
    const float cut = mx - (thr_coeff * kbarNorm[(int64_t)u * Cmax + j] + 1e-5f);
    int n = 0;
#pragma unroll
    for (int k = 0; k < kTopK; ++k) {
      const bool in = ti[k] >= 0 && tv[k] >= cut;
      candI[o + k] = in ? ti[k] : -1;
      n += in ? 1 : 0;
    }
    candV[o] = mx;
    candV[o + 1] = (float)(n == kTopK ? kTopK + 1 : n);
  }
}

// ------------------------------------------------------------------------------------------
// 3. decisions

struct FoldDecideParams {
  const double* kbar64;
  const __half* ok;          // (RK) keys of the folded block: unit u at ok + u * unit_stride, [C][D]
  int64_t unit_stride;
  const double2* kbarStat;   // (RK) [U, Cmax] (mean, rstd) of zero_r(k_j)
  int r;
  const float* kbarNorm;
  const double2* kbarHatStat;   // (mean, rstd) of kbar_j: LN_s(kbar_j), the key of the row token j would create,
                                // is gam * ((kbar_j - mean) * rstd) + bet, the expression of the memory-key kernel
  const float* gramT;        // [U, Cmax, Cmax] approximate kbarHat_a . kbar_j at [a][j] (fp16 operands); folds that append more than kGramOnTheFly rows
  const __half* kbarH;       // [U, CbarRows, D] memory keys in fp16 (operand of the products that small folds compute themselves)
  int CbarRows;
  int otf_max;               // folds that append at most this many rows compute those products themselves (0: never)
  const float* candV;
  const int32_t* candI;
  const float *ln_w, *ln_b;
  const double* sumK;
  const double *kmu, *krstd;
  int32_t *pi, *sorted, *creator, *segnew, *nmerge;   // outputs, [U, Cmax] (nmerge [U])
  double *xScore, *xBest;   // [U, Cmax] per-token results handed from the slice CTAs to the last one
  int32_t *xArg, *xCount;   // [U, Cmax]; [U] ticket counter (zero between launches)
  int32_t* counters;   // debug: [0] tokens on the exhaustive path, [1] candidate pairs, [2] tokens decided
  int64_t Mcap, m;
  int C, Cmax, Hkv, S, n_append, nsplit;
  float thr_coeff;
  double ln_eps;
};

constexpr int kPairCap = 1536;
constexpr int kPairPerTok = 24;

constexpr int kDecideThreads = 512;
constexpr int kDecideWarps = kDecideThreads / 32;
static_assert(kDecideThreads == 2 * kMaxBlock, "the ranking loops give every token two threads");

// The candidate rows (kTopK entries, -1 = none) of one token in one split: two 16-byte loads.
__device__ __forceinline__ void load_cand_rows(const int32_t* candI, int64_t o, int (&i)[kTopK]) {
  static_assert(kTopK == 8, "list loads are written for 8 entries");
  const int4 i0 = *reinterpret_cast<const int4*>(candI + o), i1 = *reinterpret_cast<const int4*>(candI + o + 4);
  i[0] = i0.x; i[1] = i0.y; i[2] = i0.z; i[3] = i0.w; i[4] = i1.x; i[5] = i1.y; i[6] = i1.z; i[7] = i1.w;
}

// Sums four per-lane partials over the warp with six exchanges instead of twenty: after the call a
// lane holds the full sum of partial number t = 2*bit4(lane) + bit3(lane) (all 8 lanes of that
// group agree).  Fixed exchange order, so results are reproducible.
__device__ __forceinline__ double warp_reduce4(double v0, double v1, double v2, double v3, int lane) {
  const bool hi16 = lane & 16, hi8 = lane & 8;
  const double r0 = __shfl_xor_sync(0xffffffffu, hi16 ? v0 : v2, 16);
  const double r1 = __shfl_xor_sync(0xffffffffu, hi16 ? v1 : v3, 16);
  const double w0 = (hi16 ? v2 : v0) + r0;
  const double w1 = (hi16 ? v3 : v1) + r1;
  double z = (hi8 ? w1 : w0) + __shfl_xor_sync(0xffffffffu, hi8 ? w0 : w1, 8);
  z += __shfl_xor_sync(0xffffffffu, z, 4);
  z += __shfl_xor_sync(0xffffffffu, z, 2);
  z += __shfl_xor_sync(0xffffffffu, z, 1);
  return z;
}

// kb . LN_s(row) with the row's statistics given; channels are strided over the lanes of a warp.
template <int CH>
__device__ __forceinline__ double warp_sim(const double (&kb)[CH], const double* __restrict__ row, double mu, double rs,
                                           const double (&g)[CH], const double (&b)[CH], int lane) {
  double acc = 0.0;
#pragma unroll
  for (int i = 0; i < CH; ++i) acc += kb[i] * (g[i] * ((row[lane + 32 * i] - mu) * rs) + b[i]);
  return warp_sum_d(acc);
}

// Bitonic sort of N = 128 or 256 (key, val) pairs, ascending by key and then val, held one per thread
// by the first N threads of the CTA (the only callers; the others must not call): stages that stay
// inside a warp exchange through shuffles, those that cross warps (three for 128, six for 256) through
// shared memory (sk / sv, N entries each) and a named barrier of those N threads.  Afterwards thread t
// holds the pair of rank t.
template <typename K, int N>
__device__ __forceinline__ void sort_n(K& key, int& val, K* sk, int* sv, int t) {
  for (int k = 2; k <= N; k <<= 1) {
    for (int j = k >> 1; j > 0; j >>= 1) {
      K ok;
      int ov;
      if (j < 32) {
        ok = __shfl_xor_sync(0xffffffffu, key, j);
        ov = __shfl_xor_sync(0xffffffffu, val, j);
      } else {
        sk[t] = key; sv[t] = val;
        asm volatile("bar.sync 2, %0;" ::"n"(N) : "memory");
        ok = sk[t ^ j]; ov = sv[t ^ j];
        asm volatile("bar.sync 2, %0;" ::"n"(N) : "memory");
      }
      const bool take_min = ((t & j) == 0) == ((t & k) == 0);   // lower index of the pair in an ascending run
      const bool other_less = ok < key || (ok == key && ov < val);
      if (other_less == take_min) { key = ok; val = ov; }
    }
  }
}

// PER_SM = 2 for grids that fill the GPU twice over (64 registers, a few spills), 1 for the small grids
// of chain-bound shapes, where a CTA has an SM to itself anyway and keeps everything in registers.
template <int D, int PER_SM, bool RK>
__global__ void __launch_bounds__(kDecideThreads, PER_SM) fold_decide_kernel(FoldDecideParams p) {
  constexpr int CH = D / 32;
  __shared__ double s_score[kMaxBlock], s_best[kMaxBlock];
  __shared__ int s_barg[kMaxBlock], s_pi[kMaxBlock], s_creator[kMaxBlock];
  __shared__ int s_pstart[kMaxBlock], s_pcnt[kMaxBlock];
  __shared__ unsigned char s_app[kMaxBlock], s_exh[kMaxBlock];
  __shared__ int s_prow[kPairCap];
  __shared__ unsigned short s_ptok[kPairCap];
  __shared__ double s_pval[kPairCap];
  __shared__ int s_np, s_nmerge, s_nexh, s_last;
  __shared__ int s_wsum[kDecideWarps];
  __shared__ int s_gmaxi[kMaxBlock], s_fill[kMaxBlock];
  __shared__ float s_thr[kMaxBlock];
  __shared__ __align__(16) __half s_hat[kGramOnTheFly][D];   // LN_s(kbar_a) of the rows a small fold appends

  // grid (R, U): CTA r of a unit refines the candidates of tokens [jlo, jhi); the CTA of the unit
  // that finishes last (a ticket, nobody waits) takes the decisions that need every token
  const int u = blockIdx.y, hk = u % p.Hkv;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int C = p.C;
  const int R = gridDim.x;
  const int jlo = (int)blockIdx.x * ((C + R - 1) / R), jhi = min(C, jlo + (C + R - 1) / R);
  const int64_t m = p.m;
  const int n_a = p.n_append;
  const int64_t rowBase = (int64_t)u * p.Mcap;
  const int64_t tokBase = (int64_t)u * p.Cmax;
  KbarRows<D, RK> kbarU;
  kbarU.k64 = p.kbar64 + (int64_t)u * p.Cmax * D; kbarU.k16 = p.ok + (int64_t)u * p.unit_stride;
  kbarU.stat = p.kbarStat + tokBase; kbarU.r = p.r;

  double gam[CH], bet[CH];
#pragma unroll
  for (int i = 0; i < CH; ++i) {
    gam[i] = (double)p.ln_w[hk * D + lane + 32 * i];
    bet[i] = (double)p.ln_b[hk * D + lane + 32 * i];
  }
  if (tid == 0) { s_np = 0; s_nmerge = 0; s_nexh = 0; }
  if (tid < kMaxBlock) {
    s_app[tid] = 0; s_exh[tid] = 0; s_pcnt[tid] = 0; s_pstart[tid] = 0; s_pi[tid] = -1;
    s_best[tid] = -INFINITY; s_barg[tid] = -1; s_score[tid] = -INFINITY; s_creator[tid] = -1;
    s_gmaxi[tid] = (int)0x80000000; s_fill[tid] = 0; s_thr[tid] = 0.f;
  }
  // everything above reads parameters and writes shared memory only; the routing filter's lists are
  // read, and global memory is written, from here on
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (tid < p.Cmax && tid < kMaxBlock) p.segnew[tokBase + tid] = -1;
  __syncthreads();

  // ---- A1/A2: candidate pairs from the filter lists.  The work items are (token of the slice, split),
  //      consecutive threads taking consecutive tokens of one split, in three rounds: the maximum over
  //      the splits per token; the number of pairs per token; the pairs themselves, into the token's
  //      segment of the pair list (order inside a segment does not matter to what follows).
  //      A split keeps its candidates when its own maximum is within the window of the global one;
  //      sink rows (< S) only matter for the append score and are kept whenever rows are appended. ----
  const int nslice = jhi - jlo;
  const int nitems = nslice > 0 ? nslice * p.nsplit : 0;
  const int64_t ostep = (int64_t)p.Cmax * kTopK;
  const int64_t obase = (int64_t)u * p.nsplit * p.Cmax * kTopK;
  for (int it = tid; it < nitems; it += kDecideThreads) {
    const int sp = it / nslice, j = jlo + it % nslice;
    const int vi = __float_as_int(p.candV[obase + sp * ostep + (int64_t)j * kTopK]);
    atomicMax(&s_gmaxi[j], vi >= 0 ? vi : vi ^ 0x7fffffff);   // order-preserving integer image of the float
    if (sp == 0) s_thr[j] = p.thr_coeff * p.kbarNorm[tokBase + j] + 1e-5f;
  }
  __syncthreads();
  for (int it = tid; it < nitems; it += kDecideThreads) {
    const int sp = it / nslice, j = jlo + it % nslice;
    const int gi = s_gmaxi[j];
    const float gmax = __int_as_float(gi >= 0 ? gi : gi ^ 0x7fffffff);
    if (!(gmax > -INFINITY)) { s_exh[j] = 1; continue; }
    const int64_t o = obase + sp * ostep + (int64_t)j * kTopK;
    const float2 hd = *reinterpret_cast<const float2*>(p.candV + o);
    int i[kTopK];
    load_cand_rows(p.candI, o, i);
    const bool keep = hd.x >= gmax - s_thr[j];
    if (hd.y > (float)kTopK && (keep || (n_a > 0 && sp == 0))) s_exh[j] = 1;   // list overflowed
    int c = 0;
#pragma unroll
    for (int k = 0; k < kTopK; ++k)
      if (i[k] >= 0 && (i[k] < p.S ? n_a > 0 : keep)) ++c;
    if (c > 0) atomicAdd(&s_pcnt[j], c);
  }
  __syncthreads();
  {   // segment starts: exclusive prefix sum over the slice's tokens, one token per thread
    const int j = jlo + tid;
    const bool mine = tid < nslice;
    int c = 0;
    bool exh = false, single = false;
    if (mine) {
      c = s_pcnt[j];
      exh = s_exh[j] != 0 || c > kPairPerTok;
      if (exh) c = 0;
      // A fold that appends nothing needs no scores, and the true arg max is always among the
      // candidates: a token with a single candidate is decided without the exact similarity
      // (it takes no room in the pair list).
      if (n_a == 0 && c == 1) { single = true; c = 0; }
    }
    int incl = c;
#pragma unroll
    for (int o2 = 1; o2 < 32; o2 <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, incl, o2);
      if (lane >= o2) incl += v;
    }
    if (lane == 31) s_wsum[warp] = incl;
    __syncthreads();
    int start = incl - c;
    for (int w = 0; w < warp; ++w) start += s_wsum[w];
    if (mine) {
      // a list that would pass the end of the pair buffer is dropped (so are the lists behind it):
      // those tokens are scanned exactly instead
      if (start + c > kPairCap) { exh = true; c = 0; }
      s_pstart[j] = start;
      s_pcnt[j] = c;
      s_fill[j] = (single && !exh) ? -1 : 0;
      s_exh[j] = exh ? 1 : 0;
    }
    // pairs of the lists that were kept form a prefix of the buffer: its end, one atomic per warp
    // (256 atomics on one shared-memory word serialise)
    const unsigned wend = __reduce_max_sync(0xffffffffu, (unsigned)((mine && c > 0) ? start + c : 0));
    if (lane == 0 && wend > 0) atomicMax(&s_np, (int)wend);
    const int ne = __syncthreads_count(mine && exh);   // tokens of the slice that take the exhaustive path
    if (tid == 0) s_nexh += ne;
  }
  __syncthreads();
  for (int it = tid; it < nitems; it += kDecideThreads) {
    const int sp = it / nslice, j = jlo + it % nslice;
    if (s_exh[j]) continue;
    const int gi = s_gmaxi[j];
    const float gmax = __int_as_float(gi >= 0 ? gi : gi ^ 0x7fffffff);
    const int64_t o = obase + sp * ostep + (int64_t)j * kTopK;
    const bool keep = p.candV[o] >= gmax - s_thr[j];
    int i[kTopK];
    load_cand_rows(p.candI, o, i);
    int c = 0;
#pragma unroll
    for (int k = 0; k < kTopK; ++k)
      if (i[k] >= 0 && (i[k] < p.S ? n_a > 0 : keep)) ++c;
    if (c == 0) continue;
    if (s_fill[j] < 0) {   // the token's only candidate: its row is the merge target
#pragma unroll
      for (int k = 0; k < kTopK; ++k)
        if (i[k] >= 0 && (i[k] < p.S ? n_a > 0 : keep)) s_barg[j] = i[k];
      continue;
    }
    int w = s_pstart[j] + atomicAdd(&s_fill[j], c);
#pragma unroll
    for (int k = 0; k < kTopK; ++k) {
      if (i[k] >= 0 && (i[k] < p.S ? n_a > 0 : keep)) {
        s_prow[w] = i[k];
        s_ptok[w] = (unsigned short)j;
        ++w;
      }
    }
  }
  __syncthreads();
  // ---- A3: exact fp64 similarity of every candidate pair, one warp per pair, eight in flight
  //      (the loads of a pair hang on one another: pair list -> rows -> statistics) ----
  const int np = min(s_np, kPairCap);
  for (int q0 = warp; q0 < np; q0 += 8 * kDecideWarps) {
    double part[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const int q = min(q0 + k * kDecideWarps, np - 1);   // clamped duplicates are computed and dropped
      const int j = s_ptok[q], i = s_prow[q];
      const double* sk = p.sumK + (rowBase + i) * D;
      const double mu = p.kmu[rowBase + i], rs = p.krstd[rowBase + i];
      double acc = 0.0;
#pragma unroll
      for (int c = 0; c < CH; ++c)
        acc += kbarU.at(j, lane + 32 * c, gam[c], bet[c]) * (gam[c] * ((sk[lane + 32 * c] - mu) * rs) + bet[c]);
      part[k] = acc;
    }
    const double z0 = warp_reduce4(part[0], part[1], part[2], part[3], lane);
    const double z1 = warp_reduce4(part[4], part[5], part[6], part[7], lane);
    if ((lane & 7) == 0) {   // lanes 0, 8, 16, 24 hold pairs 0..3 of z0 and 4..7 of z1
      const int qa = q0 + (lane >> 3) * kDecideWarps, qb = qa + 4 * kDecideWarps;
      if (qa < np) s_pval[qa] = z0;
      if (qb < np) s_pval[qb] = z1;
    }
  }
  __syncthreads();
  // ---- A4: per-token reduction (ties: lowest row) ----
  if (jlo + tid < jhi && !s_exh[jlo + tid] && s_fill[jlo + tid] >= 0) {
    const int j = jlo + tid;
    double score = -INFINITY, best = -INFINITY;
    int barg = -1;
    const int st0 = s_pstart[j];
    for (int q = st0; q < st0 + s_pcnt[j]; ++q) {
      const double v = s_pval[q];
      const int i = s_prow[q];
      if (v > score) score = v;
      if (i >= p.S && (v > best || (v == best && i < barg))) { best = v; barg = i; }
    }
    s_score[j] = score;
    s_best[j] = best;
    s_barg[j] = barg;
  }
  // ---- A5: exhaustive path for flagged tokens: one warp per token, rows in sequence ----
  for (int j = jlo + warp; j < jhi; j += kDecideWarps) {
    if (!s_exh[j]) continue;
    double kb[CH];
#pragma unroll
    for (int i = 0; i < CH; ++i) kb[i] = kbarU.at(j, lane + 32 * i, gam[i], bet[i]);
    double score = -INFINITY, best = -INFINITY;
    int barg = -1;
    for (int64_t i = 0; i < m; ++i) {
      const double acc = warp_sim<CH>(kb, p.sumK + (rowBase + i) * D, p.kmu[rowBase + i], p.krstd[rowBase + i], gam, bet, lane);
      if (acc > score) score = acc;
      if (i >= p.S && acc > best) { best = acc; barg = (int)i; }
    }
    if (lane == 0) { s_score[j] = score; s_best[j] = best; s_barg[j] = barg; }
  }
  __syncthreads();
  if (R > 1) {
    // hand the slice's results over; the last CTA of the unit to get here carries on with all of them
    if (jlo + tid < jhi) {
      const int j = jlo + tid;
      p.xScore[tokBase + j] = s_score[j];
      p.xBest[tokBase + j] = s_best[j];
      p.xArg[tokBase + j] = s_barg[j];
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) {
      atomicAdd(&p.counters[0], s_nexh);
      atomicAdd(&p.counters[1], min(s_np, kPairCap));
      s_last = atomicAdd(&p.xCount[u], 1) == R - 1 ? 1 : 0;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    if (tid == 0) { p.xCount[u] = 0; s_nexh = 0; s_np = 0; }
    if (tid < C) {   // read past the L1, which may hold stale lines of these arrays
      s_score[tid] = __ldcg(p.xScore + tokBase + tid);
      s_best[tid] = __ldcg(p.xBest + tokBase + tid);
      s_barg[tid] = __ldcg(p.xArg + tokBase + tid);
    }
    __syncthreads();
  }
  // ---- B: append selection: the n_a smallest scores, ties to the smaller token index ----
  if (n_a > 0) {
    // rank of every token in the order (score, token): the n_a lowest are appended.  Counted, not sorted: two
    // threads per token, each over half of the other tokens (a 256-entry bitonic sort is 36 dependent stages,
    // six of them through shared memory and barriers; this is 128 independent compare-and-adds per thread).
    {
      unsigned long long* skey = reinterpret_cast<unsigned long long*>(s_pval);   // (the pair list is idle here)
      if (tid < kMaxBlock) {
        unsigned long long kbits = ~0ull;
        if (tid < C) {   // order-preserving integer image of the double
          const long long bits = __double_as_longlong(s_score[tid]);
          kbits = (unsigned long long)bits ^ (bits < 0 ? ~0ull : 0x8000000000000000ull);
        }
        skey[tid] = kbits;
        s_fill[tid] = 0;   // (idle here: the rank)
      }
      __syncthreads();
      const int j = tid & (kMaxBlock - 1), h = tid / kMaxBlock;   // kDecideThreads == 2 kMaxBlock
      if (j < C) {
        const unsigned long long kj = skey[j];
        const int half_n = (C + 1) / 2, i0 = h * half_n, i1 = min(C, i0 + half_n);
        int cnt = 0;
#pragma unroll 4
        for (int i = i0; i < i1; ++i) {
          const unsigned long long ki = skey[i];
          cnt += (ki < kj || (ki == kj && i < j)) ? 1 : 0;
        }
        atomicAdd(&s_fill[j], cnt);
      }
      __syncthreads();
      if (tid < C) s_app[tid] = s_fill[tid] < n_a ? 1 : 0;
    }
    __syncthreads();
    // rows are laid down in ascending token order: position of an appended token = appended tokens before it
    if (tid < kMaxBlock) {
      const bool ap = tid < C && s_app[tid];
      const unsigned bal = __ballot_sync(0xffffffffu, ap);
      if (lane == 0) s_fill[warp] = __popc(bal);   // (s_fill is idle here)
      __syncwarp();
      s_pcnt[tid] = __popc(bal & ((1u << lane) - 1u));   // appended tokens before this one inside its warp
    }
    __syncthreads();
    if (tid < C && s_app[tid]) {
      int before = s_pcnt[tid];
      for (int wq = 0; wq < warp; ++wq) before += s_fill[wq];
      s_creator[before] = tid;
    }
    __syncthreads();
  }
  // ---- D: merge target against s_+ = old rows (best exact similarity known from A) and the rows
  //      appended by this fold.  The tensor-core products gramT[a][j] ~ kbarHat_a . kbar_j are within
  //      eps_j = thr_j / 2 of the exact values, so a new row can only win when its approximate value
  //      plus eps_j reaches both the exact best old value and (best approximate new value - eps_j).
  //      Those few pairs are recomputed in fp64; everything else is decided by the bound. ----
  if (tid == 0) { atomicAdd(&p.counters[1], min(s_np, kPairCap)); s_np = 0; }
  __syncthreads();
  // A fold that appends only a few rows (n_a <= kGramOnTheFly, i.e. nearly every fold of a growing state)
  // computes the approximate products itself, fp16 x fp16 -> fp32 on the scalar cores, against the new rows'
  // keys LN_s(kbar_a) rounded to fp16 in shared memory: n_a x C products instead of the C x C that the
  // batched tensor-core product of the block's token pairs holds.  The error bound is the same (fp16
  // rounding of both operands; fp32 accumulation errs less than the tensor core's).
  const bool otf = n_a <= p.otf_max;
  if (n_a > 0 && otf) {
    for (int a = warp; a < n_a; a += kDecideWarps) {
      const int jc = s_creator[a];
      const double2 hs = p.kbarHatStat[tokBase + jc];
#pragma unroll
      for (int c = 0; c < CH; ++c)
        s_hat[a][lane + 32 * c] =
            __float2half_rn((float)(gam[c] * ((kbarU.at(jc, lane + 32 * c, gam[c], bet[c]) - hs.x) * hs.y) + bet[c]));
    }
    __syncthreads();
  }
  if (n_a > 0 && tid < C) {
    const int j = tid;
    s_pcnt[j] = 0;
    s_exh[j] = 0;
    if (!s_app[j]) {
      const double eps = 0.5 * (double)(p.thr_coeff * p.kbarNorm[tokBase + j] + 1e-5f);
      const double best_old = s_best[j];
      // one pass over the products with the new rows, ascending a: contenders are kept while they reach the
      // running bar (which only rises: a superset) and pruned against the final bar afterwards
      float gm = -INFINITY;
      int cntc = 0, ca[4] = {0, 0, 0, 0};
      float cp[4] = {0.f, 0.f, 0.f, 0.f};
      auto consider = [&](int a, float pv) {
        gm = fmaxf(gm, pv);
        if ((double)pv >= fmax(best_old, (double)gm - eps) - eps) {
#pragma unroll
          for (int k = 0; k < 4; ++k)
            if (k == cntc) { ca[k] = a; cp[k] = pv; }
          ++cntc;
        }
      };
      if (otf) {
        const __half* kj = p.kbarH + ((int64_t)u * p.CbarRows + j) * D;
        for (int a0 = 0; a0 < n_a; a0 += 4) {
          float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 2
          for (int ch = 0; ch < D / 8; ++ch) {
            const uint4 kw = *reinterpret_cast<const uint4*>(kj + 8 * ch);
            const __half2* kh = reinterpret_cast<const __half2*>(&kw);
            float2 kf[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) kf[q] = __half22float2(kh[q]);
#pragma unroll
            for (int t = 0; t < 4; ++t) {
              const int a = min(a0 + t, n_a - 1);   // (a clamped duplicate is computed and dropped)
              const uint4 hw = *reinterpret_cast<const uint4*>(&s_hat[a][8 * ch]);
              const __half2* hh = reinterpret_cast<const __half2*>(&hw);
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                const float2 hf = __half22float2(hh[q]);
                acc[t] = fmaf(kf[q].x, hf.x, acc[t]);
                acc[t] = fmaf(kf[q].y, hf.y, acc[t]);
              }
            }
          }
#pragma unroll
          for (int t = 0; t < 4; ++t)
            if (a0 + t < n_a) consider(a0 + t, acc[t]);
        }
      } else {
        // (all loads of a batch in flight before the first product is looked at)
        const float* gcol = p.gramT + (int64_t)u * p.Cmax * p.Cmax + j;
        for (int a0 = 0; a0 < n_a; a0 += 16) {
          float pv[16];
#pragma unroll
          for (int t = 0; t < 16; ++t) pv[t] = a0 + t < n_a ? gcol[(int64_t)s_creator[a0 + t] * p.Cmax] : 0.f;
#pragma unroll
          for (int t = 0; t < 16; ++t)
            if (a0 + t < n_a) consider(a0 + t, pv[t]);
        }
      }
      bool exh = cntc > 4;   // more than four contenders: every new row exactly
      if (!exh) {            // prune against the final bar (order kept: ascending new-row index)
        const double bar = fmax(best_old, (double)gm - eps) - eps;
        int kept = 0;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          if (k < cntc && (double)cp[k] >= bar) {
#pragma unroll
            for (int k2 = 0; k2 < 4; ++k2)
              if (k2 == kept) ca[k2] = ca[k];
            ++kept;
          }
        }
        cntc = kept;
      }
      int start = 0;
      if (!exh && cntc > 0) {
        start = atomicAdd(&s_np, cntc);
        if (start + cntc > kPairCap) exh = true;
      }
      if (!exh && cntc > 0) {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          if (k < cntc) {
            s_prow[start + k] = ca[k];          // index of the new row, ascending within a token
            s_ptok[start + k] = (unsigned short)j;
          }
        }
        s_pstart[j] = start;
        s_pcnt[j] = cntc;
      }
      s_exh[j] = exh ? 1 : 0;
      if (exh) atomicAdd(&s_nexh, 1);
    }
  }
  __syncthreads();
  if (n_a > 0) {
    const int np2 = min(s_np, kPairCap);
    for (int q0 = warp; q0 < np2; q0 += 8 * kDecideWarps) {
      double part[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int q = min(q0 + k * kDecideWarps, np2 - 1);
        const int jt = s_ptok[q];
        const int jc = s_creator[s_prow[q]];
        const double2 hs = p.kbarHatStat[tokBase + jc];
        double acc = 0.0;
#pragma unroll
        for (int c = 0; c < CH; ++c) {
          const double hat = gam[c] * ((kbarU.at(jc, lane + 32 * c, gam[c], bet[c]) - hs.x) * hs.y) + bet[c];
          acc += kbarU.at(jt, lane + 32 * c, gam[c], bet[c]) * hat;
        }
        part[k] = acc;
      }
      const double z0 = warp_reduce4(part[0], part[1], part[2], part[3], lane);
      const double z1 = warp_reduce4(part[4], part[5], part[6], part[7], lane);
      if ((lane & 7) == 0) {
        const int qa = q0 + (lane >> 3) * kDecideWarps, qb = qa + 4 * kDecideWarps;
        if (qa < np2) s_pval[qa] = z0;
        if (qb < np2) s_pval[qb] = z1;
      }
    }
    // tokens whose candidate list did not fit: every new row exactly, one warp per token
    for (int j = warp; j < C; j += kDecideWarps) {
      if (!s_exh[j]) continue;
      double kb[CH];
#pragma unroll
      for (int c = 0; c < CH; ++c) kb[c] = kbarU.at(j, lane + 32 * c, gam[c], bet[c]);
      double best = s_best[j];
      int arg = s_barg[j];
      for (int a = 0; a < n_a; ++a) {
        const int jc = s_creator[a];
        const double2 hs = p.kbarHatStat[tokBase + jc];
        double acc = 0.0;
#pragma unroll
        for (int c = 0; c < CH; ++c) {
          const double hat = gam[c] * ((kbarU.at(jc, lane + 32 * c, gam[c], bet[c]) - hs.x) * hs.y) + bet[c];
          acc += kb[c] * hat;
        }
        acc = warp_sum_d(acc);
        if (acc > best) { best = acc; arg = (int)m + a; }
      }
      if (lane == 0) { s_best[j] = best; s_barg[j] = arg; }
    }
  }
  __syncthreads();
  const bool merged = tid < C && !s_app[tid];
  if (merged) {
    double best = s_best[tid];
    int arg = s_barg[tid];
    if (n_a > 0 && !s_exh[tid]) {
      const int st0 = s_pstart[tid];
      for (int q = st0; q < st0 + s_pcnt[tid]; ++q) {   // ascending new-row index: the first maximum wins
        const double v = s_pval[q];
        if (v > best) { best = v; arg = (int)m + s_prow[q]; }
      }
    }
    s_pi[tid] = arg;
  }
  {   // number of merged tokens: a block-wide count (an atomic per token on one word would serialise)
    const int nm = __syncthreads_count(merged);
    if (tid == 0) s_nmerge = nm;
  }
  // ---- E: order merged tokens by (row, token); publish ----
  {   // (ranks counted as in the append selection; keys of merged tokens are distinct, the others go last)
    unsigned* ekey = reinterpret_cast<unsigned*>(s_prow);   // (the pair list is idle here)
    unsigned* ukey = ekey + 256;                             // unsorted keys
    if (tid < kMaxBlock) {
      const int pj = tid < C ? s_pi[tid] : -1;
      ukey[tid] = pj >= 0 ? (((unsigned)pj << 9) | (unsigned)tid) : 0xffffffffu;   // rows < 2^23, tokens < 2^9
      ekey[tid] = 0xffffffffu;
      s_fill[tid] = 0;
      if (tid < C) {
        p.pi[tokBase + tid] = pj;
        p.creator[tokBase + tid] = s_creator[tid];
      }
    }
    __syncthreads();
    const int j = tid & (kMaxBlock - 1), h = tid / kMaxBlock;
    const unsigned kj = ukey[j];
    if (j < C && kj != 0xffffffffu) {
      const int half_n = (C + 1) / 2, i0 = h * half_n, i1 = min(C, i0 + half_n);
      int cnt = 0;
#pragma unroll 4
      for (int i = i0; i < i1; ++i) cnt += ukey[i] < kj ? 1 : 0;
      atomicAdd(&s_fill[j], cnt);
    }
    __syncthreads();
    if (tid < C && ukey[tid] != 0xffffffffu) ekey[s_fill[tid]] = ukey[tid];   // ranks 0 .. nmerge-1
    __syncthreads();
    const unsigned kq = tid < kMaxBlock ? ekey[tid] : 0xffffffffu;
    if (kq != 0xffffffffu) {
      const int rowq = (int)(kq >> 9);
      p.sorted[tokBase + tid] = (int)(kq & 511u);
      const bool head = tid == 0 || (int)(ekey[tid - 1] >> 9) != rowq;
      if (head && rowq >= m) p.segnew[tokBase + (rowq - (int)m)] = tid;
    }
  }
  if (tid == 0) {
    p.nmerge[u] = s_nmerge;
    atomicAdd(&p.counters[0], s_nexh);
    atomicAdd(&p.counters[1], min(s_np, kPairCap));
    atomicAdd(&p.counters[2], C);
  }
}

// ------------------------------------------------------------------------------------------
// 3b. decisions for states with more units than SMs (one CTA per unit, four CTAs per SM), folds that append rows
//
// With thousands of units the exact similarities are what the decision costs: every pair reads a 1 KB row of
// fp64 key sums from HBM, and a fold that appends rows asked for the exact score (best similarity over all
// rows) of every token just to rank them.  Here the routing filter's maxima rank them first: the exact score
// of token j lies in [gmax_j - eps_j, gmax_j + eps_j] (eps_j = the bound on the fp16 rounding of its
// products, half the filter's window), so a token is appended for certain when fewer than n_a others can
// rank before it, merged for certain when n_a others rank before it for certain, and only the tokens in
// between are scored exactly (first exact pass).  A token that is merged for certain with a single candidate row and
// no new row in reach needs no exact similarity at all; the others get their old candidates and the new rows
// in reach compared exactly in a second exact pass.  The decisions are those of the kernel above bit for bit: the bounds
// only remove work whose outcome they fix.
// The products with the rows a small fold appends (n_a <= kGramOnTheFly) run on the tensor cores
// (mma.sync m16n8k16, fp16 x fp16 -> fp32): tokens x new rows, the new rows' keys in shared memory.

constexpr int kPrunedThreads = 256;
constexpr int kPrunedWarps = kPrunedThreads / 32;
constexpr int kPairCap2 = 1024;
static_assert(kPrunedThreads == kMaxBlock, "one thread per token of the block");

__device__ __forceinline__ void mma_m16n8k16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

template <int D, bool RK>
__global__ void __launch_bounds__(kPrunedThreads, 4) fold_decide_pruned_kernel(FoldDecideParams p) {
  constexpr int CH = D / 32;
  constexpr int HS = D + 32;   // row stride of the new rows' keys in halves: consecutive rows start 16 banks apart
  __shared__ double s_lo[kMaxBlock], s_hi[kMaxBlock];   // bounds of the score; then exact score / exact best of scored tokens
  __shared__ int s_barg[kMaxBlock], s_pi[kMaxBlock], s_creator[kMaxBlock];
  __shared__ int s_pstart[kMaxBlock], s_pcnt[kMaxBlock], s_nold[kMaxBlock];
  __shared__ int s_gmaxi[kMaxBlock], s_fill[kMaxBlock], s_ulist[kMaxBlock];
  __shared__ float s_thr[kMaxBlock];
  __shared__ unsigned char s_app[kMaxBlock], s_exh[kMaxBlock], s_cls[kMaxBlock], s_sink[kMaxBlock], s_ccnt[kMaxBlock];
  __shared__ unsigned char s_cont[4 * kMaxBlock];
  __shared__ int s_prow[kPairCap2];
  __shared__ unsigned short s_ptok[kPairCap2];
  __shared__ double s_pval[kPairCap2];
  __shared__ int s_np, s_nexh, s_nunc, s_npairs;
  __shared__ int s_wsum[kPrunedWarps];
  __shared__ __align__(16) __half s_hat[kGramOnTheFly * HS];
  __shared__ double2 s_hs[kGramOnTheFly];   // (mean, rstd) of LN_s(kbar_c) for the creators of a small fold

  const int u = blockIdx.y, hk = u % p.Hkv;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int C = p.C;
  const int nsort = C <= 128 ? 128 : 256;
  const int64_t m = p.m;
  const int n_a = p.n_append;
  const int64_t rowBase = (int64_t)u * p.Mcap;
  const int64_t tokBase = (int64_t)u * p.Cmax;
  KbarRows<D, RK> kbarU;
  kbarU.k64 = p.kbar64 + (int64_t)u * p.Cmax * D; kbarU.k16 = p.ok + (int64_t)u * p.unit_stride;
  kbarU.stat = p.kbarStat + tokBase; kbarU.r = p.r;
  const float* lnwH = p.ln_w + hk * D;
  const float* lnbH = p.ln_b + hk * D;
  enum { UNSURE = 0, SURE_APPEND = 1, SURE_MERGE = 2 };

  if (tid == 0) { s_np = 0; s_nexh = 0; s_nunc = 0; s_npairs = 0; }
  s_app[tid] = 0; s_exh[tid] = 0; s_cls[tid] = UNSURE; s_sink[tid] = 0; s_ccnt[tid] = 0;
  s_pcnt[tid] = 0; s_nold[tid] = 0; s_pstart[tid] = 0; s_pi[tid] = -1; s_barg[tid] = -1; s_creator[tid] = -1;
  s_gmaxi[tid] = (int)0x80000000; s_fill[tid] = 0; s_thr[tid] = 0.f;
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (tid < p.Cmax) p.segnew[tokBase + tid] = -1;
  __syncthreads();

  // a fold that appends few rows computes the products with them itself, and the statistics of their keys
  const bool otf = n_a <= p.otf_max;
  // (mean, rstd) of LN_s(kbar_c) of new row a, created by token jc
  auto hat_stat = [&](int a, int jc) { return otf ? s_hs[a] : p.kbarHatStat[tokBase + jc]; };
  // exact fp64 value of the pairs [0, np) of the list: rows < m are rows of the state, kbar_j . LN_s(s^K_i);
  // rows >= m are rows this fold appends, kbar_j . LN_s(kbar_c) with c the creator of row (i - m).  One warp
  // per pair, eight pairs in flight per warp.
  auto exact_pairs = [&](int np) {
    double gam[CH], bet[CH];
#pragma unroll
    for (int c = 0; c < CH; ++c) { gam[c] = (double)lnwH[lane + 32 * c]; bet[c] = (double)lnbH[lane + 32 * c]; }
    for (int q0 = warp; q0 < np; q0 += 8 * kPrunedWarps) {
      double part[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int q = min(q0 + k * kPrunedWarps, np - 1);   // clamped duplicates are computed and dropped
        const int j = s_ptok[q], i = s_prow[q];
        double acc = 0.0;
        if (i < m) {
          const double* sk = p.sumK + (rowBase + i) * D;
          const double mu = p.kmu[rowBase + i], rs = p.krstd[rowBase + i];
#pragma unroll
          for (int c = 0; c < CH; ++c)
            acc += kbarU.at(j, lane + 32 * c, gam[c], bet[c]) * (gam[c] * ((sk[lane + 32 * c] - mu) * rs) + bet[c]);
        } else {
          const int jc = s_creator[i - (int)m];
          const double2 hs = hat_stat(i - (int)m, jc);
#pragma unroll
          for (int c = 0; c < CH; ++c) {
            const double hat = gam[c] * ((kbarU.at(jc, lane + 32 * c, gam[c], bet[c]) - hs.x) * hs.y) + bet[c];
            acc += kbarU.at(j, lane + 32 * c, gam[c], bet[c]) * hat;
          }
        }
        part[k] = acc;
      }
      const double z0 = warp_reduce4(part[0], part[1], part[2], part[3], lane);
      const double z1 = warp_reduce4(part[4], part[5], part[6], part[7], lane);
      if ((lane & 7) == 0) {
        const int qa = q0 + (lane >> 3) * kPrunedWarps, qb = qa + 4 * kPrunedWarps;
        if (qa < np) s_pval[qa] = z0;
        if (qb < np) s_pval[qb] = z1;
      }
    }
  };
  // exclusive prefix sum of c over the threads of the CTA (all threads call)
  auto block_scan = [&](int c) {
    int incl = c;
#pragma unroll
    for (int o2 = 1; o2 < 32; o2 <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, incl, o2);
      if (lane >= o2) incl += v;
    }
    __syncthreads();   // (s_wsum may still be read from an earlier call)
    if (lane == 31) s_wsum[warp] = incl;
    __syncthreads();
    int start = incl - c;
    for (int w = 0; w < warp; ++w) start += s_wsum[w];
    return start;
  };

  // ---- 1: per token, the filter's maximum over the splits (rows >= S), the window, the number of candidates ----
  const int nitems = C * p.nsplit;
  const int64_t ostep = (int64_t)p.Cmax * kTopK;
  const int64_t obase = (int64_t)u * p.nsplit * p.Cmax * kTopK;
  for (int it = tid; it < nitems; it += kPrunedThreads) {
    const int sp = it / C, j = it % C;
    const int vi = __float_as_int(p.candV[obase + sp * ostep + (int64_t)j * kTopK]);
    atomicMax(&s_gmaxi[j], vi >= 0 ? vi : vi ^ 0x7fffffff);
    if (sp == 0) s_thr[j] = p.thr_coeff * p.kbarNorm[tokBase + j] + 1e-5f;
  }
  __syncthreads();
  for (int it = tid; it < nitems; it += kPrunedThreads) {
    const int sp = it / C, j = it % C;
    const int gi = s_gmaxi[j];
    const float gmax = __int_as_float(gi >= 0 ? gi : gi ^ 0x7fffffff);
    if (!(gmax > -INFINITY)) { s_exh[j] = 1; continue; }
    const int64_t o = obase + sp * ostep + (int64_t)j * kTopK;
    const float2 hd = *reinterpret_cast<const float2*>(p.candV + o);
    int i[kTopK];
    load_cand_rows(p.candI, o, i);
    const bool keep = hd.x >= gmax - s_thr[j];
    if (hd.y > (float)kTopK && (keep || sp == 0)) s_exh[j] = 1;   // list overflowed
    int call = 0, cold = 0;
#pragma unroll
    for (int k = 0; k < kTopK; ++k) {
      if (i[k] >= 0 && (i[k] < p.S || keep)) ++call;
      if (i[k] >= p.S && keep) ++cold;
      if (i[k] >= 0 && i[k] < p.S) s_sink[j] = 1;   // a sink row in reach: its product is not among the maxima
    }
    if (call > 0) atomicAdd(&s_pcnt[j], call);
    if (cold > 0) atomicAdd(&s_nold[j], cold);
  }
  __syncthreads();
  // ---- 2: which tokens are appended or merged whatever their exact scores turn out to be ----
  {
    const bool have = tid < C;
    const bool open = have && (s_exh[tid] || s_sink[tid]);   // no usable bounds: scored exactly
    double lo = INFINITY, hi = INFINITY;                      // (threads past the block rank after everything)
    if (have) {
      const int gi = s_gmaxi[tid];
      const double g = (double)__int_as_float(gi >= 0 ? gi : gi ^ 0x7fffffff);
      const double eps = 0.5 * (double)s_thr[tid];
      lo = open ? -INFINITY : g - eps;
      hi = open ? INFINITY : g + eps;
    }
    s_lo[tid] = lo; s_hi[tid] = hi;
    __syncthreads();
    int may = 0, must = 0;   // tokens that may / must rank before this one (ties may)
    for (int i = 0; i < C; ++i) {
      may += s_lo[i] <= hi ? 1 : 0;
      must += s_hi[i] < lo ? 1 : 0;
    }
    may -= 1;   // (itself)
    if (have && !open) s_cls[tid] = may <= n_a - 1 ? SURE_APPEND : (must >= n_a ? SURE_MERGE : UNSURE);
    __syncthreads();
  }
  // ---- 3: first exact pass: score and best old row of the unsure tokens ----
  {
    const bool unsure = tid < C && s_cls[tid] == UNSURE;
    bool exh = unsure && s_exh[tid];
    int c = (unsure && !exh) ? s_pcnt[tid] : 0;
    if (c > kPairPerTok) { exh = true; c = 0; }
    const int start = block_scan(c);
    if (start + c > kPairCap2) { exh = unsure; c = 0; }
    s_pstart[tid] = start; s_pcnt[tid] = c; s_fill[tid] = 0; s_exh[tid] = exh ? 1 : 0;
    const unsigned wend = __reduce_max_sync(0xffffffffu, (unsigned)(c > 0 ? start + c : 0));
    if (lane == 0 && wend > 0) atomicMax(&s_np, (int)wend);
    const int ne = __syncthreads_count(exh);
    if (tid == 0) s_nexh += ne;
  }
  __syncthreads();
  for (int it = tid; it < nitems; it += kPrunedThreads) {
    const int sp = it / C, j = it % C;
    if (s_cls[j] != UNSURE || s_exh[j] || s_pcnt[j] == 0) continue;
    const int gi = s_gmaxi[j];
    const float gmax = __int_as_float(gi >= 0 ? gi : gi ^ 0x7fffffff);
    const int64_t o = obase + sp * ostep + (int64_t)j * kTopK;
    const bool keep = p.candV[o] >= gmax - s_thr[j];
    int i[kTopK];
    load_cand_rows(p.candI, o, i);
    int c = 0;
#pragma unroll
    for (int k = 0; k < kTopK; ++k)
      if (i[k] >= 0 && (i[k] < p.S || keep)) ++c;
    if (c == 0) continue;
    int w = s_pstart[j] + atomicAdd(&s_fill[j], c);
#pragma unroll
    for (int k = 0; k < kTopK; ++k) {
      if (i[k] >= 0 && (i[k] < p.S || keep)) {
        s_prow[w] = i[k];
        s_ptok[w] = (unsigned short)j;
        ++w;
      }
    }
  }
  __syncthreads();
  {
    const int np = min(s_np, kPairCap2);
    exact_pairs(np);
    if (tid == 0) s_npairs += np;
  }
  __syncthreads();
  if (tid < C && s_cls[tid] == UNSURE && !s_exh[tid]) {
    double score = -INFINITY, best = -INFINITY;
    int barg = -1;
    const int st0 = s_pstart[tid];
    for (int q = st0; q < st0 + s_pcnt[tid]; ++q) {
      const double v = s_pval[q];
      const int i = s_prow[q];
      if (v > score) score = v;
      if (i >= p.S && (v > best || (v == best && i < barg))) { best = v; barg = i; }
    }
    s_lo[tid] = score; s_hi[tid] = best; s_barg[tid] = barg;
  }
  for (int j = warp; j < C; j += kPrunedWarps) {   // no usable list: every row exactly, one warp per token
    if (!s_exh[j]) continue;
    double gam[CH], bet[CH], kb[CH];
#pragma unroll
    for (int c = 0; c < CH; ++c) {
      gam[c] = (double)lnwH[lane + 32 * c]; bet[c] = (double)lnbH[lane + 32 * c];
      kb[c] = kbarU.at(j, lane + 32 * c, gam[c], bet[c]);
    }
    double score = -INFINITY, best = -INFINITY;
    int barg = -1;
    for (int64_t i = 0; i < m; ++i) {
      const double acc = warp_sim<CH>(kb, p.sumK + (rowBase + i) * D, p.kmu[rowBase + i], p.krstd[rowBase + i], gam, bet, lane);
      if (acc > score) score = acc;
      if (i >= p.S && acc > best) { best = acc; barg = (int)i; }
    }
    if (lane == 0) { s_lo[j] = score; s_hi[j] = best; s_barg[j] = barg; }
  }
  __syncthreads();
  // ---- 4: append selection: the certain ones, then the unsure ones by exact score (ties: smaller token) ----
  {
    const bool have = tid < C;
    const int cls = have ? s_cls[tid] : SURE_MERGE;
    const int n_sure = __syncthreads_count(have && cls == SURE_APPEND);
    if (have && cls == UNSURE) s_ulist[atomicAdd(&s_nunc, 1)] = tid;
    __syncthreads();
    bool ap = have && cls == SURE_APPEND;
    if (have && cls == UNSURE) {
      const double sj = s_lo[tid];
      int rank = 0;
      const int nu = s_nunc;
      for (int k = 0; k < nu; ++k) {
        const int i = s_ulist[k];
        const double si = s_lo[i];
        rank += (si < sj || (si == sj && i < tid)) ? 1 : 0;
      }
      ap = rank < n_a - n_sure;
    }
    s_app[tid] = ap ? 1 : 0;
    // rows are laid down in ascending token order: position of an appended token = appended tokens before it
    const unsigned bal = __ballot_sync(0xffffffffu, ap);
    const int before_w = __popc(bal & ((1u << lane) - 1u));
    __syncthreads();
    if (lane == 0) s_wsum[warp] = __popc(bal);
    __syncthreads();
    if (ap) {
      int before = before_w;
      for (int wq = 0; wq < warp; ++wq) before += s_wsum[wq];
      s_creator[before] = tid;
    }
    __syncthreads();
  }
  // ---- 5: the new rows in reach of every merged token.  best_old below is the exact best old similarity of a
  //      scored token, a lower bound of it for the others; products are within eps_j of the exact values, so a
  //      new row can only win when its product reaches max(best_old, best product - eps_j) - eps_j. ----
  if (otf) {
    for (int e = tid; e < kGramOnTheFly * HS / 8; e += kPrunedThreads) reinterpret_cast<uint4*>(s_hat)[e] = make_uint4(0u, 0u, 0u, 0u);
    {   // the memory-key kernel skipped these for such folds: eight lanes per creator, its arithmetic and order
      constexpr int NI = D / 32, NC = 4 * NI;
      constexpr double inv_d = 1.0 / D;
      const int a = warp * 4 + (lane >> 3), sub = lane & 7;
      const int jc = s_creator[min(a, n_a - 1)];   // (groups past the last creator compute a copy and store nothing)
      double kb[NC];
#pragma unroll
      for (int i = 0; i < NI; ++i) {
        double k4[4];
        kbar_run4<D, RK>(kbarU, jc, 32 * i + 4 * sub, lnwH, lnbH, k4);
        kb[4 * i] = k4[0]; kb[4 * i + 1] = k4[1]; kb[4 * i + 2] = k4[2]; kb[4 * i + 3] = k4[3];
      }
      double sum = 0.0;
#pragma unroll
      for (int c = 0; c < NC; ++c) sum += kb[c];
      const double mu2 = group8_sum_d(sum) * inv_d;
      double dev = 0.0;
#pragma unroll
      for (int c = 0; c < NC; ++c) dev += (kb[c] - mu2) * (kb[c] - mu2);
      const double rs2 = 1.0 / sqrt(group8_sum_d(dev) * inv_d + p.ln_eps);
      if (sub == 0 && a < n_a) s_hs[a] = make_double2(mu2, rs2);
    }
    __syncthreads();
    double gam[CH], bet[CH];
#pragma unroll
    for (int c = 0; c < CH; ++c) { gam[c] = (double)lnwH[lane + 32 * c]; bet[c] = (double)lnbH[lane + 32 * c]; }
    for (int a = warp; a < n_a; a += kPrunedWarps) {
      const int jc = s_creator[a];
      const double2 hs = s_hs[a];
#pragma unroll
      for (int c = 0; c < CH; ++c)
        s_hat[a * HS + lane + 32 * c] =
            __float2half_rn((float)(gam[c] * ((kbarU.at(jc, lane + 32 * c, gam[c], bet[c]) - hs.x) * hs.y) + bet[c]));
    }
    __syncthreads();
    // 16 tokens x 8 new rows per instruction; lane (g, t) = (lane / 4, lane % 4) holds tokens g and g + 8 of the
    // tile and new rows 8 nt + 2 t, + 1.  The channels are dealt to the instruction's k index in runs of eight per
    // lane (the same permutation on both operands leaves the sums unchanged), so that both operands are read
    // 16 bytes at a time.
    const int g = lane >> 2, t = lane & 3;
    const int NT = (n_a + 7) / 8;
    const __half* kU = p.kbarH + (int64_t)u * p.CbarRows * D;
    for (int mt = warp; mt * 16 < C; mt += kPrunedWarps) {
      const int j0 = mt * 16 + g, j1 = j0 + 8;
      const __half* r0 = kU + (int64_t)min(j0, C - 1) * D + 8 * t;
      const __half* r1 = kU + (int64_t)min(j1, C - 1) * D + 8 * t;
      float acc[4][4];
#pragma unroll
      for (int nt = 0; nt < 4; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[nt][e] = 0.f;
#pragma unroll
      for (int ks = 0; ks < D / 32; ++ks) {
        const uint4 a0 = *reinterpret_cast<const uint4*>(r0 + 32 * ks), a1 = *reinterpret_cast<const uint4*>(r1 + 32 * ks);
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
          if (nt < NT) {
            const uint4 b = *reinterpret_cast<const uint4*>(&s_hat[(nt * 8 + g) * HS + 32 * ks + 8 * t]);
            mma_m16n8k16(acc[nt], a0.x, a1.x, a0.y, a1.y, b.x, b.y);
            mma_m16n8k16(acc[nt], a0.z, a1.z, a0.w, a1.w, b.z, b.w);
          }
        }
      }
      // per token: best product over the new rows, then the rows in reach as a bit mask
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int j = h ? j1 : j0;
        float gm = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < 4; ++nt)
#pragma unroll
          for (int e = 0; e < 2; ++e)
            if (nt * 8 + 2 * t + e < n_a) gm = fmaxf(gm, acc[nt][2 * h + e]);
        gm = fmaxf(gm, __shfl_xor_sync(0xffffffffu, gm, 1));
        gm = fmaxf(gm, __shfl_xor_sync(0xffffffffu, gm, 2));
        unsigned mask = 0;
        if (j < C && !s_app[j]) {
          const double eps = 0.5 * (double)s_thr[j];
          const double best_old = s_cls[j] == UNSURE ? s_hi[j] : s_lo[j];
          const double bar = fmax(best_old, (double)gm - eps) - eps;
#pragma unroll
          for (int nt = 0; nt < 4; ++nt)
#pragma unroll
            for (int e = 0; e < 2; ++e)
              if (nt * 8 + 2 * t + e < n_a && (double)acc[nt][2 * h + e] >= bar) mask |= 1u << (nt * 8 + 2 * t + e);
        }
        mask |= __shfl_xor_sync(0xffffffffu, mask, 1);
        mask |= __shfl_xor_sync(0xffffffffu, mask, 2);
        if (t == 0 && j < C) s_fill[j] = (int)mask;
      }
    }
    __syncthreads();
    if (tid < C && !s_app[tid]) {
      unsigned mask = (unsigned)s_fill[tid];
      const int n = __popc(mask);
      s_ccnt[tid] = (unsigned char)min(n, 5);
      if (n <= 4) {
        for (int k = 0; k < n; ++k) {   // ascending new-row index
          const int a = __ffs(mask) - 1;
          mask &= mask - 1;
          s_cont[4 * tid + k] = (unsigned char)a;
        }
      }
    }
  } else if (tid < C && !s_app[tid]) {
    const int j = tid;
    const double eps = 0.5 * (double)s_thr[j];
    const double best_old = s_cls[j] == UNSURE ? s_hi[j] : s_lo[j];
    // one pass over the batched products with the new rows, ascending a: rows are kept while they reach the
    // running bar (which only rises: a superset) and pruned against the final bar afterwards
    float gm = -INFINITY;
    int cntc = 0, ca[4] = {0, 0, 0, 0};
    float cp[4] = {0.f, 0.f, 0.f, 0.f};
    const float* gcol = p.gramT + (int64_t)u * p.Cmax * p.Cmax + j;
#pragma unroll 8
    for (int a = 0; a < n_a; ++a) {
      const float pv = gcol[(int64_t)s_creator[a] * p.Cmax];
      gm = fmaxf(gm, pv);
      if ((double)pv >= fmax(best_old, (double)gm - eps) - eps) {
#pragma unroll
        for (int k = 0; k < 4; ++k)
          if (k == cntc) { ca[k] = a; cp[k] = pv; }
        ++cntc;
      }
    }
    int kept = cntc;
    if (cntc <= 4) {
      const double bar = fmax(best_old, (double)gm - eps) - eps;
      kept = 0;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        if (k < cntc && (double)cp[k] >= bar) {
          s_cont[4 * j + kept] = (unsigned char)ca[k];
          ++kept;
        }
      }
    }
    s_ccnt[j] = (unsigned char)min(kept, 5);
  }
  __syncthreads();
  // ---- 6: second exact pass: merged tokens whose target is still open: the old candidates of a token without an exact best
  //      (unless it has one candidate and no new row in reach), and the new rows in reach ----
  if (tid == 0) s_np = 0;
  {
    const bool mg = tid < C && !s_app[tid];
    const bool scored = mg && s_cls[tid] == UNSURE;
    const int nnew = mg ? s_ccnt[tid] : 0;
    const int nold = (mg && !scored) ? s_nold[tid] : 0;
    bool exh = mg && (nnew > 4 || (!scored && nold == 0));   // (no old candidate cannot happen; scanned if it does)
    int c = 0;
    bool single = false;
    if (mg && !exh) {
      if (!scored && nold == 1 && nnew == 0) single = true;
      else c = nold + nnew;
      if (c > kPairPerTok) { exh = true; c = 0; }
    }
    const int start = block_scan(c);
    if (start + c > kPairCap2) { exh = mg; c = 0; single = false; }
    s_pstart[tid] = start; s_pcnt[tid] = c;
    s_fill[tid] = single ? -1 : ((mg && !scored && !exh && c > 0) ? 0 : -2);   // -1: take the only candidate; 0: list the old candidates; -2: none
    s_exh[tid] = exh ? 1 : 0;
    if (mg && !exh && c > 0) {   // the new rows go behind the old candidates
      for (int k = 0; k < nnew; ++k) {
        s_prow[start + nold + k] = (int)m + s_cont[4 * tid + k];
        s_ptok[start + nold + k] = (unsigned short)tid;
      }
    }
    const unsigned wend = __reduce_max_sync(0xffffffffu, (unsigned)(c > 0 ? start + c : 0));
    if (lane == 0 && wend > 0) atomicMax(&s_np, (int)wend);
    const int ne = __syncthreads_count(exh);
    if (tid == 0) s_nexh += ne;
  }
  __syncthreads();
  for (int it = tid; it < nitems; it += kPrunedThreads) {
    const int sp = it / C, j = it % C;
    const int mode = s_fill[j];
    if (mode == -2) continue;
    const int gi = s_gmaxi[j];
    const float gmax = __int_as_float(gi >= 0 ? gi : gi ^ 0x7fffffff);
    const int64_t o = obase + sp * ostep + (int64_t)j * kTopK;
    if (!(p.candV[o] >= gmax - s_thr[j])) continue;
    int i[kTopK];
    load_cand_rows(p.candI, o, i);
    if (mode == -1) {
#pragma unroll
      for (int k = 0; k < kTopK; ++k)
        if (i[k] >= p.S) s_barg[j] = i[k];
      continue;
    }
    int c = 0;
#pragma unroll
    for (int k = 0; k < kTopK; ++k)
      if (i[k] >= p.S) ++c;
    if (c == 0) continue;
    int w = s_pstart[j] + atomicAdd(&s_fill[j], c);   // (stays >= 0: a list mode)
#pragma unroll
    for (int k = 0; k < kTopK; ++k) {
      if (i[k] >= p.S) {
        s_prow[w] = i[k];
        s_ptok[w] = (unsigned short)j;
        ++w;
      }
    }
  }
  __syncthreads();
  {
    const int np2 = min(s_np, kPairCap2);
    exact_pairs(np2);
    if (tid == 0) s_npairs += np2;
  }
  for (int j = warp; j < C; j += kPrunedWarps) {   // lists that did not fit: every row in question exactly
    if (!s_exh[j] || s_app[j]) continue;
    double gam[CH], bet[CH], kb[CH];
#pragma unroll
    for (int c = 0; c < CH; ++c) {
      gam[c] = (double)lnwH[lane + 32 * c]; bet[c] = (double)lnbH[lane + 32 * c];
      kb[c] = kbarU.at(j, lane + 32 * c, gam[c], bet[c]);
    }
    double best = -INFINITY;
    int arg = -1;
    if (s_cls[j] == UNSURE) { best = s_hi[j]; arg = s_barg[j]; }
    else {
      for (int64_t i = p.S; i < m; ++i) {
        const double acc = warp_sim<CH>(kb, p.sumK + (rowBase + i) * D, p.kmu[rowBase + i], p.krstd[rowBase + i], gam, bet, lane);
        if (acc > best) { best = acc; arg = (int)i; }
      }
    }
    for (int a = 0; a < n_a; ++a) {
      const int jc = s_creator[a];
      const double2 hs = hat_stat(a, jc);
      double acc = 0.0;
#pragma unroll
      for (int c = 0; c < CH; ++c) {
        const double hat = gam[c] * ((kbarU.at(jc, lane + 32 * c, gam[c], bet[c]) - hs.x) * hs.y) + bet[c];
        acc += kb[c] * hat;
      }
      acc = warp_sum_d(acc);
      if (acc > best) { best = acc; arg = (int)m + a; }
    }
    if (lane == 0) { s_hi[j] = best; s_barg[j] = arg; }
  }
  __syncthreads();
  const bool merged = tid < C && !s_app[tid];
  if (merged) {
    double best = -INFINITY;
    int arg = s_barg[tid];   // (a token with one candidate and no new row in reach: that candidate)
    if (s_cls[tid] == UNSURE || s_exh[tid]) best = s_hi[tid];
    if (!s_exh[tid]) {
      const int st0 = s_pstart[tid];
      for (int q = st0; q < st0 + s_pcnt[tid]; ++q) {   // ties: the lowest row (old rows before new ones)
        const double v = s_pval[q];
        const int i = s_prow[q];
        if (v > best || (v == best && i < arg)) { best = v; arg = i; }
      }
    }
    s_pi[tid] = arg;
  }
  const int nm = __syncthreads_count(merged);
  // ---- 7: order merged tokens by (row, token); publish ----
  {
    unsigned* ekey = reinterpret_cast<unsigned*>(s_prow);   // (the pair list is idle here)
    if (tid < nsort) {
      const int pj = tid < C ? s_pi[tid] : -1;
      unsigned kq = pj >= 0 ? (((unsigned)pj << 9) | (unsigned)tid) : 0xffffffffu;   // rows < 2^23, tokens < 2^9
      if (tid < C) {
        p.pi[tokBase + tid] = pj;
        p.creator[tokBase + tid] = s_creator[tid];
      }
      int zero = 0;
      if (nsort == 128) sort_n<unsigned, 128>(kq, zero, ekey + 256, reinterpret_cast<int*>(s_pval), tid);
      else sort_n<unsigned, 256>(kq, zero, ekey + 256, reinterpret_cast<int*>(s_pval), tid);
      ekey[tid] = kq;
      asm volatile("bar.sync 2, %0;" ::"r"(nsort) : "memory");
      if (kq != 0xffffffffu) {
        const int rowq = (int)(kq >> 9);
        p.sorted[tokBase + tid] = (int)(kq & 511u);
        const bool head = tid == 0 || (int)(ekey[tid - 1] >> 9) != rowq;
        if (head && rowq >= m) p.segnew[tokBase + (rowq - (int)m)] = tid;
      }
    }
  }
  if (tid == 0) {
    p.nmerge[u] = nm;
    atomicAdd(&p.counters[0], s_nexh);
    atomicAdd(&p.counters[1], s_npairs);
    atomicAdd(&p.counters[2], C);
  }
}

// ------------------------------------------------------------------------------------------
// 4. application: one warp per touched row

struct FoldApplyParams {
  const __half* ok;          // (RK) keys of the folded block, laid out like ov
  const double2* kbarStat;   // (RK) [U, Cmax] (mean, rstd) of zero_r(k_j)
  int r;
  const __half* ov;
  const float* og;
  int64_t unit_stride, gate_stride;
  const double* kbar64;
  const float *ln_w, *ln_b;
  const int32_t *pi, *sorted, *creator, *segnew, *nmerge;
  double* sumK; float* sumV; float* rho; double* wsum; int32_t* cnt; double *kmu, *krstd;
  __half *Khat, *Vhat;
  int32_t* slotTok; uint8_t* appTok;
  int64_t Mcap, Tassign, m, b;
  int C, Cmax, Hkv, n_append, all_append, radius_on;
  double ln_eps, norm_eps;
};

// One touched row per warp: the shorter chain per row; used when a launch has too few rows to fill the
// GPU, where the latency of a row is what counts.
template <int D>
__global__ void __launch_bounds__(256, 4) fold_apply_kernel(FoldApplyParams p) {
  constexpr int CH = D / 32;
  __shared__ int s_pi[kMaxBlock], s_sorted[kMaxBlock], s_creator[kMaxBlock], s_segnew[kMaxBlock];
  // the routing filter of the next fold may start its set-up now; it waits for this grid to finish
  // before it reads the readout keys written here
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int u = blockIdx.y, hk = u % p.Hkv;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int q = blockIdx.x * 8 + warp;
  const int64_t tokBase = (int64_t)u * p.Cmax;
  if (!p.all_append) {   // the decisions of this unit, read once per CTA instead of chased per warp
    for (int i = threadIdx.x; i < p.C; i += 256) {
      s_pi[i] = p.pi[tokBase + i];
      s_sorted[i] = p.sorted[tokBase + i];
      s_creator[i] = p.creator[tokBase + i];
      s_segnew[i] = p.segnew[tokBase + i];
    }
    __syncthreads();
  }
  if (q >= p.C) return;
  const int64_t rowBase = (int64_t)u * p.Mcap;
  const double* kbarU = p.kbar64 + tokBase * D;
  const __half* ovU = p.ov + (int64_t)u * p.unit_stride;
  const float* ogU = p.og + (int64_t)u * p.gate_stride;
  const int nmerge = p.all_append ? 0 : p.nmerge[u];
  const int m = (int)p.m;

  // task 0: the q-th appended row; task 1: the segment of an old row whose head sits at sorted[q]
  for (int task = 0; task < 2; ++task) {
    int rowi, seg, jc = -1;
    if (task == 0) {
      if (q >= p.n_append) continue;
      rowi = m + q;
      jc = p.all_append ? q : s_creator[q];
      seg = p.all_append ? -1 : s_segnew[q];
    } else {
      if (q >= nmerge) continue;
      const int j0 = s_sorted[q];
      rowi = s_pi[j0];
      if (rowi >= m) continue;                                 // new rows are task 0
      if (q > 0 && s_pi[s_sorted[q - 1]] == rowi) continue;    // not a head
      seg = q;
    }
    const int64_t row = rowBase + rowi;
    double kx[CH];
    float vx[CH];
    double wacc, rad;
    int nacc;
    if (task == 0) {
      const double* kb = kbarU + (int64_t)jc * D;
      const __half* vr = ovU + (int64_t)jc * D;
      double v2 = 0.0;
#pragma unroll
      for (int i = 0; i < CH; ++i) {
        const int x = lane + 32 * i;
        kx[i] = kb[x];
        vx[i] = __half2float(vr[x]);
        v2 += (double)vx[i] * (double)vx[i];
      }
      rad = (double)(float)sqrt(warp_sum_d(v2));   // the radius is kept in fp32
      wacc = 1.0;
      nacc = 1;
      if (lane == 0 && p.slotTok && p.b + jc < p.Tassign) {
        p.slotTok[(int64_t)u * p.Tassign + p.b + jc] = rowi;
        p.appTok[(int64_t)u * p.Tassign + p.b + jc] = 1;
      }
    } else {
#pragma unroll
      for (int i = 0; i < CH; ++i) {
        const int x = lane + 32 * i;
        kx[i] = p.sumK[row * D + x];
        vx[i] = p.sumV[row * D + x];
      }
      wacc = p.wsum[row];
      nacc = p.cnt[row];
      rad = (double)p.rho[row];
    }
    if (seg >= 0) {
      for (int qq = seg; qq < nmerge; ++qq) {
        const int j = s_sorted[qq];
        if (s_pi[j] != rowi) break;
        const float g = ogU[j];
        const double* kb = kbarU + (int64_t)j * D;
        const __half* vr = ovU + (int64_t)j * D;
#pragma unroll
        for (int i = 0; i < CH; ++i) {
          const int x = lane + 32 * i;
          kx[i] += (double)g * kb[x];
          vx[i] = fmaf(g, __half2float(vr[x]), vx[i]);
        }
        wacc += (double)g;
        nacc += 1;
        if (lane == 0 && p.slotTok && p.b + j < p.Tassign) {
          p.slotTok[(int64_t)u * p.Tassign + p.b + j] = rowi;
          p.appTok[(int64_t)u * p.Tassign + p.b + j] = 0;
        }
      }
    }
    double mu, rs;
    row_stats<CH>(kx, D, p.ln_eps, mu, rs);
    double v2 = 0.0;
#pragma unroll
    for (int i = 0; i < CH; ++i) v2 += (double)vx[i] * (double)vx[i];
    const double vnorm = sqrt(warp_sum_d(v2));
    const double den = vnorm > p.norm_eps ? vnorm : p.norm_eps;
    // one fp64 divide per row instead of one per channel (the readout values are rounded to fp16)
    const double vscale = p.radius_on ? rad / den : 1.0 / wacc;
#pragma unroll
    for (int i = 0; i < CH; ++i) {
      const int x = lane + 32 * i;
      const double hat = (double)p.ln_w[hk * D + x] * ((kx[i] - mu) * rs) + (double)p.ln_b[hk * D + x];
      p.sumK[row * D + x] = kx[i];
      p.sumV[row * D + x] = vx[i];
      p.Khat[row * D + x] = __float2half_rn((float)hat);
      const double vo = (double)vx[i] * vscale;
      p.Vhat[row * D + x] = __float2half_rn((float)vo);
    }
    if (lane == 0) {
      p.rho[row] = (float)rad;
      p.wsum[row] = wacc;
      p.cnt[row] = nacc;
      p.kmu[row] = mu;
      p.krstd[row] = rs;
    }
  }
}

// 32-byte accesses to the fp64 key sums (a lane's four consecutive channels): one instruction instead of two,
// streaming (the rows are touched once per fold)
__device__ __forceinline__ void ld4d_cs(const double* p, double (&v)[4]) {
  asm volatile("ld.global.cs.v4.f64 {%0,%1,%2,%3}, [%4];" : "=d"(v[0]), "=d"(v[1]), "=d"(v[2]), "=d"(v[3]) : "l"(p));
}
__device__ __forceinline__ void st4d_cs(double* p, double a, double b, double c, double d) {
  asm volatile("st.global.cs.v4.f64 [%0], {%1,%2,%3,%4};" ::"l"(p), "d"(a), "d"(b), "d"(c), "d"(d) : "memory");
}

// Four touched rows per warp, eight lanes per row (lane `sub` of a group holds channels
// 32 i + 4 sub .. + 3, as in the memory-key kernel): the fp64 reductions, square roots and divides of
// a row are instructions of the whole warp, so one row per warp spent most of its instructions on
// them, and four rows per warp also put four times the loads in flight.  The member loop of a group
// runs without exchanges between lanes (each lane sums its own channels, members in ascending token
// order: reproducible); all lanes meet again for the reductions.
constexpr int kApplyRowsPerWarp = 4;
constexpr int kApplyRowsPerCta = 8 * kApplyRowsPerWarp;

template <int D, bool RK>
__global__ void __launch_bounds__(256, 2) fold_apply_rows4_kernel(FoldApplyParams p) {
  constexpr int NI = D / 32;          // runs of four channels per lane
  constexpr int NC = 4 * NI;          // channels per lane
  constexpr double inv_d = 1.0 / D;   // D is a power of two: multiplying is dividing, exactly
  __shared__ int s_pi[kMaxBlock], s_sorted[kMaxBlock], s_creator[kMaxBlock], s_segnew[kMaxBlock];
  __shared__ int s_nmerge;
  // the routing filter of the next fold may start its set-up now; it waits for this grid to finish
  // before it reads the readout keys written here
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int u = blockIdx.y, hk = u % p.Hkv;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, sub = lane & 7;
  const int64_t tokBase = (int64_t)u * p.Cmax;
  if (!p.all_append) {   // the decisions of this unit, read once per CTA instead of chased per warp
    if (threadIdx.x == 0) s_nmerge = p.nmerge[u];
    for (int i = threadIdx.x; i < p.C; i += 256) {
      s_pi[i] = p.pi[tokBase + i];
      s_sorted[i] = p.sorted[tokBase + i];
      s_creator[i] = p.creator[tokBase + i];
      s_segnew[i] = p.segnew[tokBase + i];
    }
    __syncthreads();
  }
  const int64_t rowBase = (int64_t)u * p.Mcap;
  KbarRows<D, RK> kbarU;
  kbarU.k64 = p.kbar64 + tokBase * D; kbarU.k16 = p.ok + (int64_t)u * p.unit_stride;
  kbarU.stat = p.kbarStat + tokBase; kbarU.r = p.r;
  const float* lnwH = p.ln_w + hk * D;
  const float* lnbH = p.ln_b + hk * D;
  const __half* ovU = p.ov + (int64_t)u * p.unit_stride;
  const float* ogU = p.og + (int64_t)u * p.gate_stride;
  const int nmerge = p.all_append ? 0 : s_nmerge;
  const int m = (int)p.m;

  // A warp takes groups of four row slots in turn (with few CTAs per unit the stores of one group drain
  // while the next group's rows are fetched, and the decisions are read once for more work).
  // task 0: the q-th appended row; task 1: the segment of an old row whose head sits at sorted[q]
  for (int qg = blockIdx.x * 8 + warp; qg * kApplyRowsPerWarp < p.C; qg += gridDim.x * 8)
  for (int task = 0; task < 2; ++task) {
    const int q = qg * kApplyRowsPerWarp + (lane >> 3);
    bool act = q < p.C;
    int rowi = 0, seg = -1, jc = -1;
    if (act) {
      if (task == 0) {
        if (q >= p.n_append) act = false;
        else {
          rowi = m + q;
          jc = p.all_append ? q : s_creator[q];
          seg = p.all_append ? -1 : s_segnew[q];
        }
      } else {
        if (q >= nmerge) act = false;
        else {
          const int j0 = s_sorted[q];
          rowi = s_pi[j0];
          if (rowi >= m) act = false;                                          // new rows are task 0
          else if (q > 0 && s_pi[s_sorted[q - 1]] == rowi) act = false;        // not a head
          seg = q;
        }
      }
    }
    if (!__any_sync(0xffffffffu, act)) continue;
    const int64_t row = rowBase + rowi;
    double kx[NC];
    float vx[NC];
    double wacc = 1.0, rad = 0.0, v2 = 0.0;
    int nacc = 1;
#pragma unroll
    for (int c = 0; c < NC; ++c) { kx[c] = 0.0; vx[c] = 0.f; }
    if (act) {
      if (task == 0) {
        const __half* vr = ovU + (int64_t)jc * D;
#pragma unroll
        for (int i = 0; i < NI; ++i) {
          const int x = 32 * i + 4 * sub;
          double k4[4];
          kbar_run4<D, RK>(kbarU, jc, x, lnwH, lnbH, k4);
          kx[4 * i] = k4[0]; kx[4 * i + 1] = k4[1]; kx[4 * i + 2] = k4[2]; kx[4 * i + 3] = k4[3];
          alignas(8) __half hv[4];
          *reinterpret_cast<uint2*>(hv) = *reinterpret_cast<const uint2*>(vr + x);
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            vx[4 * i + e] = __half2float(hv[e]);
            v2 += (double)vx[4 * i + e] * (double)vx[4 * i + e];
          }
        }
        if (sub == 0 && p.slotTok && p.b + jc < p.Tassign) {
          p.slotTok[(int64_t)u * p.Tassign + p.b + jc] = rowi;
          p.appTok[(int64_t)u * p.Tassign + p.b + jc] = 1;
        }
      } else {
#pragma unroll
        for (int i = 0; i < NI; ++i) {
          const int x = 32 * i + 4 * sub;
          double k4[4];
          ld4d_cs(p.sumK + row * D + x, k4);
          kx[4 * i] = k4[0]; kx[4 * i + 1] = k4[1]; kx[4 * i + 2] = k4[2]; kx[4 * i + 3] = k4[3];
          const float4 v4 = __ldcs(reinterpret_cast<const float4*>(p.sumV + row * D + x));
          vx[4 * i] = v4.x; vx[4 * i + 1] = v4.y; vx[4 * i + 2] = v4.z; vx[4 * i + 3] = v4.w;
        }
        wacc = p.wsum[row];
        nacc = p.cnt[row];
        rad = (double)p.rho[row];
      }
    }
    // radius of a new row = the norm of its creator's value, kept in fp32 (all lanes: group reduction)
    v2 = group8_sum_d(v2);
    if (task == 0) rad = (double)(float)sqrt(v2);
    if (act && seg >= 0) {
      for (int qq = seg; qq < nmerge; ++qq) {
        const int j = s_sorted[qq];
        if (s_pi[j] != rowi) break;
        const float g = ogU[j];
        const __half* vr = ovU + (int64_t)j * D;
#pragma unroll
        for (int i = 0; i < NI; ++i) {
          const int x = 32 * i + 4 * sub;
          double k4[4];
          kbar_run4<D, RK>(kbarU, j, x, lnwH, lnbH, k4);
          kx[4 * i] += (double)g * k4[0]; kx[4 * i + 1] += (double)g * k4[1];
          kx[4 * i + 2] += (double)g * k4[2]; kx[4 * i + 3] += (double)g * k4[3];
          alignas(8) __half hv[4];
          *reinterpret_cast<uint2*>(hv) = *reinterpret_cast<const uint2*>(vr + x);
#pragma unroll
          for (int e = 0; e < 4; ++e) vx[4 * i + e] = fmaf(g, __half2float(hv[e]), vx[4 * i + e]);
        }
        wacc += (double)g;
        nacc += 1;
        if (sub == 0 && p.slotTok && p.b + j < p.Tassign) {
          p.slotTok[(int64_t)u * p.Tassign + p.b + j] = rowi;
          p.appTok[(int64_t)u * p.Tassign + p.b + j] = 0;
        }
      }
    }
    // all lanes again: LayerNorm statistics of the key sum, norm of the value sum
    double sum = 0.0;
#pragma unroll
    for (int c = 0; c < NC; ++c) sum += kx[c];
    const double mu = group8_sum_d(sum) * inv_d;
    double dev = 0.0, vv = 0.0;
#pragma unroll
    for (int c = 0; c < NC; ++c) {
      dev += (kx[c] - mu) * (kx[c] - mu);
      vv += (double)vx[c] * (double)vx[c];
    }
    const double rs = 1.0 / sqrt(group8_sum_d(dev) * inv_d + p.ln_eps);
    const double vnorm = sqrt(group8_sum_d(vv));
    const double den = vnorm > p.norm_eps ? vnorm : p.norm_eps;
    // one fp64 divide per row instead of one per channel (the readout values are rounded to fp16)
    const double vscale = p.radius_on ? rad / den : 1.0 / wacc;
    if (!act) continue;
#pragma unroll
    for (int i = 0; i < NI; ++i) {
      const int x = 32 * i + 4 * sub;
      const float4 w4 = *reinterpret_cast<const float4*>(p.ln_w + hk * D + x), b4 = *reinterpret_cast<const float4*>(p.ln_b + hk * D + x);
      const float wv[4] = {w4.x, w4.y, w4.z, w4.w}, bv[4] = {b4.x, b4.y, b4.z, b4.w};
      alignas(8) __half kh[4], vh[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const double hat = (double)wv[e] * ((kx[4 * i + e] - mu) * rs) + (double)bv[e];
        kh[e] = __float2half_rn((float)hat);
        vh[e] = __float2half_rn((float)((double)vx[4 * i + e] * vscale));
      }
      st4d_cs(p.sumK + row * D + x, kx[4 * i], kx[4 * i + 1], kx[4 * i + 2], kx[4 * i + 3]);
      __stcs(reinterpret_cast<float4*>(p.sumV + row * D + x), make_float4(vx[4 * i], vx[4 * i + 1], vx[4 * i + 2], vx[4 * i + 3]));
      __stcs(reinterpret_cast<uint2*>(p.Khat + row * D + x), *reinterpret_cast<const uint2*>(kh));
      __stcs(reinterpret_cast<uint2*>(p.Vhat + row * D + x), *reinterpret_cast<const uint2*>(vh));
    }
    if (sub == 0) {
      p.rho[row] = (float)rad;
      p.wsum[row] = wacc;
      p.cnt[row] = nacc;
      p.kmu[row] = mu;
      p.krstd[row] = rs;
    }
  }
}

// Row statistics and readout rows (both copies) of rows [0, m) recomputed from the stored sums, for a
// state whose sums were loaded from a snapshot.  The arithmetic and the reduction order are those of
// the apply kernel that this state's folds run (ROWS4: four rows per warp, eight lanes per row; else
// one row per warp), so the refreshed values equal bit for bit what the folds had left.
struct RefreshParams {
  const double* sumK; const float* sumV; const float* rho; const double* wsum;
  const float *ln_w, *ln_b;
  double *kmu, *krstd;
  __half *Khat0, *Vhat0, *Khat1, *Vhat1;
  int64_t Mcap, m;
  int Hkv, radius_on;
  double ln_eps, norm_eps;
};

template <int D, bool ROWS4>
__global__ void __launch_bounds__(256) refresh_rows_kernel(RefreshParams p) {
  const int u = blockIdx.y, hk = u % p.Hkv;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (ROWS4) {
    constexpr int NI = D / 32, NC = 4 * NI;
    constexpr double inv_d = 1.0 / D;
    const int sub = lane & 7;
    const int64_t q = ((int64_t)blockIdx.x * 8 + warp) * kApplyRowsPerWarp + (lane >> 3);
    const bool act = q < p.m;
    const int64_t row = (int64_t)u * p.Mcap + (act ? q : 0);
    double kx[NC];
    float vx[NC];
#pragma unroll
    for (int i = 0; i < NI; ++i) {
      const int x = 32 * i + 4 * sub;
      const double2 k01 = *reinterpret_cast<const double2*>(p.sumK + row * D + x), k23 = *reinterpret_cast<const double2*>(p.sumK + row * D + x + 2);
      kx[4 * i] = k01.x; kx[4 * i + 1] = k01.y; kx[4 * i + 2] = k23.x; kx[4 * i + 3] = k23.y;
      const float4 v4 = *reinterpret_cast<const float4*>(p.sumV + row * D + x);
      vx[4 * i] = v4.x; vx[4 * i + 1] = v4.y; vx[4 * i + 2] = v4.z; vx[4 * i + 3] = v4.w;
    }
    const double wacc = p.wsum[row], rad = (double)p.rho[row];
    double sum = 0.0;
#pragma unroll
    for (int c = 0; c < NC; ++c) sum += kx[c];
    const double mu = group8_sum_d(sum) * inv_d;
    double dev = 0.0, vv = 0.0;
#pragma unroll
    for (int c = 0; c < NC; ++c) {
      dev += (kx[c] - mu) * (kx[c] - mu);
      vv += (double)vx[c] * (double)vx[c];
    }
    const double rs = 1.0 / sqrt(group8_sum_d(dev) * inv_d + p.ln_eps);
    const double vnorm = sqrt(group8_sum_d(vv));
    const double den = vnorm > p.norm_eps ? vnorm : p.norm_eps;
    const double vscale = p.radius_on ? rad / den : 1.0 / wacc;
    if (!act) return;
#pragma unroll
    for (int i = 0; i < NI; ++i) {
      const int x = 32 * i + 4 * sub;
      const float4 w4 = *reinterpret_cast<const float4*>(p.ln_w + hk * D + x), b4 = *reinterpret_cast<const float4*>(p.ln_b + hk * D + x);
      const float wv[4] = {w4.x, w4.y, w4.z, w4.w}, bv[4] = {b4.x, b4.y, b4.z, b4.w};
      alignas(8) __half kh[4], vh[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const double hat = (double)wv[e] * ((kx[4 * i + e] - mu) * rs) + (double)bv[e];
        kh[e] = __float2half_rn((float)hat);
        vh[e] = __float2half_rn((float)((double)vx[4 * i + e] * vscale));
      }
      *reinterpret_cast<uint2*>(p.Khat0 + row * D + x) = *reinterpret_cast<const uint2*>(kh);
      *reinterpret_cast<uint2*>(p.Vhat0 + row * D + x) = *reinterpret_cast<const uint2*>(vh);
      *reinterpret_cast<uint2*>(p.Khat1 + row * D + x) = *reinterpret_cast<const uint2*>(kh);
      *reinterpret_cast<uint2*>(p.Vhat1 + row * D + x) = *reinterpret_cast<const uint2*>(vh);
    }
    if (sub == 0) { p.kmu[row] = mu; p.krstd[row] = rs; }
  } else {
    constexpr int CH = D / 32;
    const int64_t q = (int64_t)blockIdx.x * 8 + warp;
    if (q >= p.m) return;
    const int64_t row = (int64_t)u * p.Mcap + q;
    double kx[CH];
    float vx[CH];
#pragma unroll
    for (int i = 0; i < CH; ++i) {
      kx[i] = p.sumK[row * D + lane + 32 * i];
      vx[i] = p.sumV[row * D + lane + 32 * i];
    }
    const double wacc = p.wsum[row], rad = (double)p.rho[row];
    double mu, rs;
    row_stats<CH>(kx, D, p.ln_eps, mu, rs);
    double v2 = 0.0;
#pragma unroll
    for (int i = 0; i < CH; ++i) v2 += (double)vx[i] * (double)vx[i];
    const double vnorm = sqrt(warp_sum_d(v2));
    const double den = vnorm > p.norm_eps ? vnorm : p.norm_eps;
    const double vscale = p.radius_on ? rad / den : 1.0 / wacc;
#pragma unroll
    for (int i = 0; i < CH; ++i) {
      const int x = lane + 32 * i;
      const double hat = (double)p.ln_w[hk * D + x] * ((kx[i] - mu) * rs) + (double)p.ln_b[hk * D + x];
      const __half kh = __float2half_rn((float)hat);
      const __half vh = __float2half_rn((float)((double)vx[i] * vscale));
      p.Khat0[row * D + x] = kh; p.Vhat0[row * D + x] = vh;
      p.Khat1[row * D + x] = kh; p.Vhat1[row * D + x] = vh;
    }
    if (lane == 0) { p.kmu[row] = mu; p.krstd[row] = rs; }
  }
}

// which apply kernel the folds of this state run (fixed per state and block): four rows per warp when
// the launch is bound by throughput (measured: better from 8192 rows on: U = 32, C = 256; worse at
// 4096 and 2048 rows, where the longer chain per row shows)
static bool apply_uses_rows4(const State* st) { return (int64_t)st->C * st->U >= 8192; }

int launch_refresh_rows(State* st, int64_t m, cudaStream_t s) {
  if (m <= 0) return 0;
  RefreshParams p;
  p.sumK = st->sumK; p.sumV = st->sumV; p.rho = st->rho; p.wsum = st->wsum; p.ln_w = st->ln_w; p.ln_b = st->ln_b;
  p.kmu = st->kmu; p.krstd = st->krstd;
  p.Khat0 = st->KhatBuf[0]; p.Vhat0 = st->VhatBuf[0]; p.Khat1 = st->KhatBuf[1]; p.Vhat1 = st->VhatBuf[1];
  p.Mcap = st->Mcap; p.m = m; p.Hkv = st->Hkv; p.radius_on = (st->flags & KVM_FLAG_NO_RADIUS) ? 0 : 1;
  p.ln_eps = (double)st->ln_eps; p.norm_eps = (double)st->norm_eps;
  if (apply_uses_rows4(st)) {
    dim3 grid((unsigned)((m + kApplyRowsPerCta - 1) / kApplyRowsPerCta), st->U);
    if (st->d == 128) refresh_rows_kernel<128, true><<<grid, 256, 0, s>>>(p);
    else refresh_rows_kernel<64, true><<<grid, 256, 0, s>>>(p);
  } else {
    dim3 grid((unsigned)((m + 7) / 8), st->U);
    if (st->d == 128) refresh_rows_kernel<128, false><<<grid, 256, 0, s>>>(p);
    else refresh_rows_kernel<64, false><<<grid, 256, 0, s>>>(p);
  }
  return 1;
}

int launch_route_filter_tc(State* st, int64_t m, int nsplit, int slot, bool early_start, cudaStream_t s);
int launch_gram_tc(State* st, int slot0, int nblk, cudaStream_t s);

// Folds that compute their new-row products themselves (no batched product: want_gram false) and run the
// decision kernel for many units take the statistics of LN_s(kbar_c) there, for the creators only.
static bool hat_stats_in_decide(const State* st) { return st->U > 148 && gram_from(st) > 0; }

int launch_kbar(State* st, const __half* ok, int64_t unit_stride, int nblk, int slot0, bool want_gram, cudaStream_t s) {
  KernelTimer kt(st, 2, s);
  const int C = st->C, D = st->d;
  const int64_t U = st->U;
  dim3 grid((C + kKbarRowsPerCta - 1) / kKbarRowsPerCta, st->U, nblk);
  double* k64 = st->kbar64 + (int64_t)slot0 * U * st->Cmax * D;
  __half* kh = st->kbarH + (int64_t)slot0 * U * st->CbarRows * D;
  float* kn = st->kbarNorm + (int64_t)slot0 * U * st->Cmax;
  double2* khat = st->kbarHatStat + (int64_t)slot0 * U * st->Cmax;
  __half* khh = st->kbarHatH + (int64_t)slot0 * U * st->CbarRows * D;
  double2* kst = st->kbarStat + (int64_t)slot0 * U * st->Cmax;
#define KVM_KBAR(DD, RR)                                                                                                   \
  kbar_kernel<DD, RR><<<grid, 256, 0, s>>>(ok, unit_stride, st->ln_w, st->ln_b, k64, kh, kn, khat, khh, C, st->Cmax,        \
                                           st->CbarRows, st->U, st->Hkv, st->r, (double)st->ln_eps,                         \
                                           want_gram ? 1 : (hat_stats_in_decide(st) ? -1 : 0), kst)
  if (D == 128) { if (st->recomputeK) KVM_KBAR(128, true); else KVM_KBAR(128, false); }
  else { if (st->recomputeK) KVM_KBAR(64, true); else KVM_KBAR(64, false); }
#undef KVM_KBAR
  int launches = 1;
  // the new-row filter is only read by folds that append some but not all of their tokens
  if (want_gram) launches += launch_gram_tc(st, slot0, nblk, s);
  return launches;
}

int launch_prev_copy(State* st, cudaStream_t s) {
  if (!st->prevValid) return 0;
  st->prevValid = false;
  if (st->serial) return 0;   // one readout copy: nothing to bring over
  // the last fold (number nfolds) wrote copy nfolds & 1; the other copy lacks the rows it touched
  const int src = (int)(st->nfolds & 1), dst = src ^ 1;
  PrevFoldCopy pc;
  pc.all_append = st->prevAllAppend ? 1 : 0; pc.n_append = st->prevNAppend; pc.C = st->C; pc.Cmax = st->Cmax;
  pc.m = st->prevM; pc.Mcap = st->Mcap;
  pc.pi = st->foldPi[src]; pc.sorted = st->foldSorted[src]; pc.nmerge = st->foldNMerge[src];
  pc.Ksrc = st->KhatBuf[src]; pc.Vsrc = st->VhatBuf[src]; pc.Kdst = st->KhatBuf[dst]; pc.Vdst = st->VhatBuf[dst];
  KernelTimer kt(st, 2, s);
  dim3 grid((st->C + 7) / 8, st->U);
  if (st->d == 128) prev_copy_kernel<128><<<grid, 256, 0, s>>>(pc);
  else prev_copy_kernel<64><<<grid, 256, 0, s>>>(pc);
  return 1;
}

int launch_fold(State* st, const FoldArgs& a, cudaStream_t s) {
  int launches = 0;
  const int C = st->C, D = st->d;
  // the state after nfolds folds is read from readout copy `src`; this fold writes copy `dst`
  const int src = (int)(st->nfolds & 1), dst = src ^ 1;
  const int64_t U = st->U;
  const double* kbar64 = st->kbar64 + (int64_t)a.slot * U * st->Cmax * D;
  const __half* kbarH = st->kbarH + (int64_t)a.slot * U * st->CbarRows * D;
  const float* kbarNorm = st->kbarNorm + (int64_t)a.slot * U * st->Cmax;
  const double2* kbarHatStat = st->kbarHatStat + (int64_t)a.slot * U * st->Cmax;
  const bool all_append = a.first || a.n_append >= C;
  if (!all_append) {
    // enough CTAs to fill the GPU, at least 256 rows per split
    int64_t want = 148 / st->U;   // rounded down: a few CTAs in a second wave would double the kernel's time
    int64_t maxs = (a.m + 255) / 256;
    int nsplit = (int)(want < maxs ? want : maxs);
    if (nsplit < 1) nsplit = 1;
    if (nsplit > st->nsplitRoute) nsplit = st->nsplitRoute;
    if (st->flags & KVM_FLAG_SIMT_ROUTING) {
      KernelTimer kt(st, 3, s);
      dim3 grid(nsplit, st->U);
      if (D == 128)
        route_filter_simt_kernel<128><<<grid, 256, 0, s>>>(kbarH, st->KhatBuf[src], st->candV, st->candI, C, st->Cmax,
                                                           st->CbarRows, st->Mcap, a.m, nsplit, kbarNorm,
                                                           route_thr_coeff(st), st->S);
      else
        route_filter_simt_kernel<64><<<grid, 256, 0, s>>>(kbarH, st->KhatBuf[src], st->candV, st->candI, C, st->Cmax,
                                                          st->CbarRows, st->Mcap, a.m, nsplit, kbarNorm,
                                                          route_thr_coeff(st), st->S);
      ++launches;
    } else {
      KernelTimer kt(st, 3, s);
      launches += launch_route_filter_tc(st, a.m, nsplit, a.slot, a.early_start, s);
    }
    FoldDecideParams p;
    p.kbar64 = kbar64; p.kbarNorm = kbarNorm; p.kbarHatStat = kbarHatStat;
    p.ok = a.ok; p.unit_stride = a.unit_stride; p.kbarStat = st->kbarStat + (int64_t)a.slot * U * st->Cmax; p.r = st->r;
    p.gramT = st->gramT + (int64_t)a.slot * U * st->Cmax * st->Cmax;
    p.kbarH = kbarH; p.CbarRows = st->CbarRows; p.otf_max = gram_from(st);
    p.candV = st->candV; p.candI = st->candI; p.ln_w = st->ln_w; p.ln_b = st->ln_b;
    p.sumK = st->sumK; p.kmu = st->kmu; p.krstd = st->krstd;
    p.pi = st->foldPi[dst]; p.sorted = st->foldSorted[dst]; p.creator = st->foldCreator[dst];
    p.segnew = st->foldSegNew[dst]; p.nmerge = st->foldNMerge[dst];
    p.counters = st->status + 1;
    p.xScore = st->xScore; p.xBest = st->xBest; p.xArg = st->xArg; p.xCount = st->xCount;
    p.Mcap = st->Mcap; p.m = a.m;
    p.C = C; p.Cmax = st->Cmax; p.Hkv = st->Hkv; p.S = st->S; p.n_append = a.n_append; p.nsplit = nsplit;
    p.thr_coeff = route_thr_coeff(st);
    p.ln_eps = (double)st->ln_eps;
    KernelTimer kt(st, 4, s);
    // CTAs per unit (measured on U = 1, 8, 32, 256): about 64 CTAs in all, at least two per unit while
    // 2U CTAs fit the GPU in one wave, at most eight, at least 16 tokens each - beyond that the
    // hand-over costs more than the shorter slices save.  A fold that appends nothing has few pairs
    // to refine (most tokens have one candidate and need no exact similarity): one CTA per unit.
    int R = 64 / st->U;
    if (R < 2 && 2 * st->U <= 2 * 148) R = 2;
    if (R > 8) R = 8;
    if (R > C / 16) R = C / 16;
    if (R < 1 || a.n_append == 0) R = 1;
    dim3 dgrid(R, st->U);
    // programmatic dependent launch: the CTAs may start (and set up their shared memory) while the
    // routing filter is still running; they wait for it before the first read of its output
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dgrid; lc.blockDim = dim3(kDecideThreads); lc.dynamicSmemBytes = 0; lc.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    // Measured: the early start pays when the filter, these CTAs and the attention CTAs of a block
    // all find room on the GPU at once (or when every kernel fills it anyway); in between, CTAs
    // that sit waiting keep the attention kernel, which needs whole SMs, off them.
    const int sms_wanted = nsplit * st->U + (R * st->U + 1) / 2 + st->B * st->Hq * ((C + 127) / 128);
    const bool pdl = st->prof_hook == nullptr && !(st->flags & KVM_FLAG_SIMT_ROUTING) &&
                     (sms_wanted <= 148 || st->U >= 148);
    lc.attrs = at; lc.numAttrs = pdl ? 1 : 0;
    const bool roomy = R * st->U <= 148;
#define KVM_DECIDE(DD, PP, RR) cudaLaunchKernelEx(&lc, fold_decide_kernel<DD, PP, RR>, p)
    const bool rk = st->recomputeK;
    if (st->U > 148 && a.n_append > 0) {   // (R == 1 here) more units than SMs: bounds first, few exact pairs
      lc.blockDim = dim3(kPrunedThreads);
      if (D == 128) { if (rk) cudaLaunchKernelEx(&lc, fold_decide_pruned_kernel<128, true>, p); else cudaLaunchKernelEx(&lc, fold_decide_pruned_kernel<128, false>, p); }
      else { if (rk) cudaLaunchKernelEx(&lc, fold_decide_pruned_kernel<64, true>, p); else cudaLaunchKernelEx(&lc, fold_decide_pruned_kernel<64, false>, p); }
    } else if (D == 128) {
      if (roomy) { if (rk) KVM_DECIDE(128, 1, true); else KVM_DECIDE(128, 1, false); }
      else { if (rk) KVM_DECIDE(128, 2, true); else KVM_DECIDE(128, 2, false); }
    } else {
      if (roomy) { if (rk) KVM_DECIDE(64, 1, true); else KVM_DECIDE(64, 1, false); }
      else { if (rk) KVM_DECIDE(64, 2, true); else KVM_DECIDE(64, 2, false); }
    }
#undef KVM_DECIDE
    ++launches;
  }
  FoldApplyParams q;
  q.ov = a.ov; q.og = a.og; q.unit_stride = a.unit_stride; q.gate_stride = a.gate_stride;
  q.kbar64 = kbar64; q.ln_w = st->ln_w; q.ln_b = st->ln_b;
  q.ok = a.ok; q.kbarStat = st->kbarStat + (int64_t)a.slot * U * st->Cmax; q.r = st->r;
  q.pi = st->foldPi[dst]; q.sorted = st->foldSorted[dst]; q.creator = st->foldCreator[dst];
  q.segnew = st->foldSegNew[dst]; q.nmerge = st->foldNMerge[dst];
  q.sumK = st->sumK; q.sumV = st->sumV; q.rho = st->rho; q.wsum = st->wsum; q.cnt = st->cnt;
  q.kmu = st->kmu; q.krstd = st->krstd; q.Khat = st->KhatBuf[dst]; q.Vhat = st->VhatBuf[dst];
  q.slotTok = st->slotTok; q.appTok = st->appTok;
  q.Mcap = st->Mcap; q.Tassign = st->Tassign; q.m = a.m; q.b = a.b;
  q.C = C; q.Cmax = st->Cmax; q.Hkv = st->Hkv; q.n_append = a.n_append; q.all_append = all_append ? 1 : 0;
  q.radius_on = (st->flags & KVM_FLAG_NO_RADIUS) ? 0 : 1;
  q.ln_eps = (double)st->ln_eps; q.norm_eps = (double)st->norm_eps;
  if (a.before_apply && cudaStreamWaitEvent(s, a.before_apply, 0) != cudaSuccess) return -1000000;
  KernelTimer kt(st, 5, s);
  if (apply_uses_rows4(st)) {
    // CTAs per unit: one when the units alone fill the GPU's CTA slots (measured at 256 and 2048 units: 1 beats
    // 2, 4 and 8), else enough to fill them, at most one per 32 row slots
    const int R = std::max(1, std::min(2 * 148 / st->U, (C + kApplyRowsPerCta - 1) / kApplyRowsPerCta));
    dim3 grid(R, st->U);
    if (D == 128) { if (st->recomputeK) fold_apply_rows4_kernel<128, true><<<grid, 256, 0, s>>>(q); else fold_apply_rows4_kernel<128, false><<<grid, 256, 0, s>>>(q); }
    else { if (st->recomputeK) fold_apply_rows4_kernel<64, true><<<grid, 256, 0, s>>>(q); else fold_apply_rows4_kernel<64, false><<<grid, 256, 0, s>>>(q); }
  } else {
    dim3 grid((C + 7) / 8, st->U);
    if (D == 128) fold_apply_kernel<128><<<grid, 256, 0, s>>>(q);
    else fold_apply_kernel<64><<<grid, 256, 0, s>>>(q);
  }
  ++launches;
  st->prevValid = true; st->prevAllAppend = all_append; st->prevM = a.m; st->prevNAppend = a.n_append;
  return launches;
}

}  // namespace kvm
