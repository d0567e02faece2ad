// The fold of one overflow block into the state (Section 3.2 "Append", "Merge", budget rule,
// value-radius preservation) for every unit:
//   1. kbar_kernel          memory keys kbar_j = LN_s(zero_r(k_j))            (Eq. 1) in fp64
//   2. route filter         approximate similarities kbar_j . LN_s(s^K_i) in fp16 x fp16 -> fp32,
//                           K best per token and per row split (candidates only)
//   3. fold_update_kernel   exact fp64 similarities for the candidates, append selection,
//                           merge routing against s_+, deterministic per-row accumulation,
//                           refresh of the readout caches of the touched rows
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

// ------------------------------------------------------------------------------------------
// 1. memory keys

template <int D>
__global__ void __launch_bounds__(256) kbar_kernel(const __half* __restrict__ ok, int64_t unit_stride,
                                                   const float* __restrict__ ln_w, const float* __restrict__ ln_b,
                                                   double* __restrict__ kbar64, __half* __restrict__ kbarH,
                                                   float* __restrict__ kbarNorm, int C, int Cmax, int Hkv, int r,
                                                   double ln_eps) {
  constexpr int CH = D / 32;
  const int u = blockIdx.y, hk = u % Hkv;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int j = blockIdx.x * 8 + warp;
  if (j >= C) return;
  const __half* row = ok + (int64_t)u * unit_stride + (int64_t)j * D;
  double val[CH];
  double sum = 0.0;
#pragma unroll
  for (int i = 0; i < CH; ++i) {
    const int x = lane + 32 * i;
    val[i] = (x < r) ? 0.0 : (double)__half2float(row[x]);
    sum += val[i];
  }
  const double mean = warp_sum_d(sum) / D;
  double sq = 0.0;
#pragma unroll
  for (int i = 0; i < CH; ++i) sq += (val[i] - mean) * (val[i] - mean);
  const double var = warp_sum_d(sq) / D;
  const double rstd = 1.0 / sqrt(var + ln_eps);
  double n2 = 0.0;
  const int64_t o = ((int64_t)u * Cmax + j) * D;
#pragma unroll
  for (int i = 0; i < CH; ++i) {
    const int x = lane + 32 * i;
    const double kb = (double)ln_w[hk * D + x] * ((val[i] - mean) * rstd) + (double)ln_b[hk * D + x];
    kbar64[o + x] = kb;
    kbarH[o + x] = __float2half_rn((float)kb);
    n2 += kb * kb;
  }
  n2 = warp_sum_d(n2);
  if (lane == 0) kbarNorm[(int64_t)u * Cmax + j] = (float)sqrt(n2) * 1.000001f;
}

// ------------------------------------------------------------------------------------------
// 2. routing filter on the scalar cores (cross-check path; the default filter runs on tcgen05)

template <int D>
__global__ void __launch_bounds__(256) route_filter_simt_kernel(const __half* __restrict__ kbarH,
                                                                const __half* __restrict__ KhatH,
                                                                float* __restrict__ candV,
                                                                int32_t* __restrict__ candI, int C, int Cmax,
                                                                int64_t Mcap, int64_t m, int nsplit) {
  __shared__ __half2 sH[32 * (D / 2)];
  const int split = blockIdx.x, u = blockIdx.y;
  const int j = threadIdx.x;
  const bool active = j < C;
  int64_t per = (m + nsplit - 1) / nsplit;
  per = (per + 31) / 32 * 32;
  const int64_t i0 = (int64_t)split * per;
  const int64_t i1 = min(m, i0 + per);

  __half2 kb[D / 2];
  if (active) {
    const __half2* src = reinterpret_cast<const __half2*>(kbarH + ((int64_t)u * Cmax + j) * D);
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
      sH[wd] = (i < i1) ? reinterpret_cast<const __half2*>(KhatH + ((int64_t)u * Mcap + i) * D)[cw]
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
    const int64_t o = (((int64_t)u * nsplit + split) * Cmax + j) * kTopK;
#pragma unroll
    for (int k = 0; k < kTopK; ++k) { candV[o + k] = tv[k]; candI[o + k] = ti[k]; }
  }
}

// ------------------------------------------------------------------------------------------
// 3. exact refine, append selection, routing, accumulation, readout refresh

struct FoldUpdateParams {
  const __half* ov;          // overflow values
  const float* og;           // overflow gates
  int64_t unit_stride, gate_stride;
  const double* kbar64;
  const float* kbarNorm;
  double* newhat64;
  const float* candV;
  const int32_t* candI;
  const float *ln_w, *ln_b;
  double* sumK; float* sumV; float* rho; double* wsum; int32_t* cnt; double *kmu, *krstd;
  __half *Khat, *Vhat;
  int32_t* slotTok; uint8_t* appTok;
  int64_t Mcap, Tassign, m, b;
  int C, Cmax, Hkv, S, n_append, nsplit, first, radius_on;
  double ln_eps, norm_eps;
  float thr_coeff;   // 2 * (fp16 error coefficient) * bound of ||LN_s(.)||
};

constexpr int kPairCap = 1536;
constexpr int kPairPerTok = 24;

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

template <int D>
__global__ void __launch_bounds__(256) fold_update_kernel(FoldUpdateParams p) {
  constexpr int CH = D / 32;
  __shared__ double s_gamma[D], s_beta[D];
  __shared__ double s_score[kMaxBlock], s_best[kMaxBlock];
  __shared__ int s_barg[kMaxBlock], s_pi[kMaxBlock], s_newrow[kMaxBlock], s_sorted[kMaxBlock];
  __shared__ int s_pstart[kMaxBlock], s_pcnt[kMaxBlock];
  __shared__ unsigned char s_app[kMaxBlock], s_exh[kMaxBlock];
  __shared__ int s_prow[kPairCap];
  __shared__ unsigned short s_ptok[kPairCap];
  __shared__ double s_pval[kPairCap];
  __shared__ int s_np, s_nmerge;

  const int u = blockIdx.x, hk = u % p.Hkv;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int C = p.C;
  const int64_t m = p.m;
  const int n_a = p.n_append;
  const bool all_append = p.first || n_a >= C;
  const double* kbarU = p.kbar64 + (int64_t)u * p.Cmax * D;
  const __half* ovU = p.ov + (int64_t)u * p.unit_stride;
  const float* ogU = p.og + (int64_t)u * p.gate_stride;
  const int64_t rowBase = (int64_t)u * p.Mcap;

  for (int x = tid; x < D; x += 256) {
    s_gamma[x] = (double)p.ln_w[hk * D + x];
    s_beta[x] = (double)p.ln_b[hk * D + x];
  }
  if (tid == 0) { s_np = 0; s_nmerge = 0; }
  if (tid < kMaxBlock) {
    s_app[tid] = (all_append && tid < C) ? 1 : 0;
    s_exh[tid] = 0;
    s_pcnt[tid] = 0;
    s_pstart[tid] = 0;
    s_pi[tid] = -1;
    s_best[tid] = -INFINITY;
    s_barg[tid] = -1;
    s_score[tid] = -INFINITY;
    s_newrow[tid] = all_append ? (int)m + tid : -1;   // first fold: m == 0
  }
  __syncthreads();

  if (!all_append) {
    // ---- A1/A2: candidate pairs from the filter lists ----
    if (tid < C) {
      const int j = tid;
      const float thr = p.thr_coeff * p.kbarNorm[(int64_t)u * p.Cmax + j] + 1e-5f;
      float vmax_all = -INFINITY, vmax_ns = -INFINITY;
      for (int sp = 0; sp < p.nsplit; ++sp) {
        const int64_t o = (((int64_t)u * p.nsplit + sp) * p.Cmax + j) * kTopK;
        for (int k = 0; k < kTopK; ++k) {
          const int i = p.candI[o + k];
          if (i < 0) break;
          const float v = p.candV[o + k];
          vmax_all = fmaxf(vmax_all, v);
          if (i >= p.S) vmax_ns = fmaxf(vmax_ns, v);
        }
      }
      const float cut_ns = vmax_ns - thr;     // merge candidates (rows >= S)
      const float cut_all = vmax_all - thr;   // append-score candidates (all rows)
      bool exh = !(vmax_ns > -INFINITY);
      int cntc = 0;
      for (int sp = 0; sp < p.nsplit && !exh; ++sp) {
        const int64_t o = (((int64_t)u * p.nsplit + sp) * p.Cmax + j) * kTopK;
        if (p.candI[o + kTopK - 1] >= 0 && p.candV[o + kTopK - 1] >= fminf(cut_ns, cut_all)) exh = true;
        for (int k = 0; k < kTopK; ++k) {
          const int i = p.candI[o + k];
          if (i < 0) break;
          const float v = p.candV[o + k];
          if ((i >= p.S && v >= cut_ns) || (n_a > 0 && v >= cut_all)) ++cntc;
        }
      }
      if (cntc > kPairPerTok) exh = true;
      int start = 0;
      if (!exh) {
        start = atomicAdd(&s_np, cntc);
        if (start + cntc > kPairCap) exh = true;
      }
      if (!exh) {
        int w = start;
        for (int sp = 0; sp < p.nsplit; ++sp) {
          const int64_t o = (((int64_t)u * p.nsplit + sp) * p.Cmax + j) * kTopK;
          for (int k = 0; k < kTopK; ++k) {
            const int i = p.candI[o + k];
            if (i < 0) break;
            const float v = p.candV[o + k];
            if ((i >= p.S && v >= cut_ns) || (n_a > 0 && v >= cut_all)) {
              s_prow[w] = i;
              s_ptok[w] = (unsigned short)j;
              ++w;
            }
          }
        }
        s_pstart[j] = start;
        s_pcnt[j] = cntc;
      }
      s_exh[j] = exh ? 1 : 0;
    }
    __syncthreads();
    // ---- A3: exact fp64 similarity of every candidate pair ----
    const int np = min(s_np, kPairCap);
    for (int q = tid; q < np; q += 256) {
      const int j = s_ptok[q];
      const int i = s_prow[q];
      // pairs of tokens that fell back to the exhaustive path are skipped (their slots are unused)
      if (s_exh[j]) continue;
      const double* kb = kbarU + (int64_t)j * D;
      const double* sk = p.sumK + (rowBase + i) * D;
      const double mu = p.kmu[rowBase + i], rs = p.krstd[rowBase + i];
      double acc = 0.0;
#pragma unroll 8
      for (int x = 0; x < D; ++x) acc += kb[x] * (s_gamma[x] * ((sk[x] - mu) * rs) + s_beta[x]);
      s_pval[q] = acc;
    }
    __syncthreads();
    // ---- A4: per-token reduction (ties: lowest row) ----
    if (tid < C && !s_exh[tid]) {
      double score = -INFINITY, best = -INFINITY;
      int barg = -1;
      const int st0 = s_pstart[tid];
      for (int q = st0; q < st0 + s_pcnt[tid]; ++q) {
        const double v = s_pval[q];
        const int i = s_prow[q];
        if (v > score) score = v;
        if (i >= p.S && (v > best || (v == best && i < barg))) { best = v; barg = i; }
      }
      s_score[tid] = score;
      s_best[tid] = best;
      s_barg[tid] = barg;
    }
    // ---- A5: exhaustive path: one warp per flagged token, one lane per row ----
    for (int j = warp; j < C; j += 8) {
      if (!s_exh[j]) continue;
      const double* kb = kbarU + (int64_t)j * D;
      double score = -INFINITY, best = -INFINITY;
      int barg = 0x7fffffff;
      for (int64_t i = lane; i < m; i += 32) {
        const double* sk = p.sumK + (rowBase + i) * D;
        const double mu = p.kmu[rowBase + i], rs = p.krstd[rowBase + i];
        double acc = 0.0;
        for (int x = 0; x < D; ++x) acc += kb[x] * (s_gamma[x] * ((sk[x] - mu) * rs) + s_beta[x]);
        if (acc > score) score = acc;
        if (i >= p.S && acc > best) { best = acc; barg = (int)i; }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const double os = __shfl_xor_sync(0xffffffffu, score, o);
        const double ob = __shfl_xor_sync(0xffffffffu, best, o);
        const int oa = __shfl_xor_sync(0xffffffffu, barg, o);
        if (os > score) score = os;
        if (ob > best || (ob == best && oa < barg)) { best = ob; barg = oa; }
      }
      if (lane == 0) { s_score[j] = score; s_best[j] = best; s_barg[j] = barg; }
    }
    __syncthreads();
    // ---- B: append selection: the n_a smallest scores, ties to the smaller token index ----
    if (n_a > 0) {
      int rank = 0;
      if (tid < C) {
        const double sj = s_score[tid];
        for (int jj = 0; jj < C; ++jj) {
          const double so = s_score[jj];
          rank += (so < sj || (so == sj && jj < tid)) ? 1 : 0;
        }
      }
      __syncthreads();
      if (tid < C) s_app[tid] = rank < n_a ? 1 : 0;
      __syncthreads();
      if (tid < C && s_app[tid]) {
        int before = 0;
        for (int jj = 0; jj < tid; ++jj) before += s_app[jj];
        s_newrow[tid] = (int)m + before;
      }
      __syncthreads();
    }
  }

  // ---- C: create the appended rows ----
  for (int j = warp; j < C; j += 8) {
    if (!s_app[j]) continue;
    const int64_t row = rowBase + s_newrow[j];
    const double* kb = kbarU + (int64_t)j * D;
    const __half* vr = ovU + (int64_t)j * D;
    double kx[CH];
    float vx[CH];
    double v2 = 0.0;
#pragma unroll
    for (int i = 0; i < CH; ++i) {
      const int x = lane + 32 * i;
      kx[i] = kb[x];
      vx[i] = __half2float(vr[x]);
      v2 += (double)vx[i] * (double)vx[i];
    }
    double mu, rs;
    row_stats<CH>(kx, D, p.ln_eps, mu, rs);
    const double vnorm = sqrt(warp_sum_d(v2));
    const double den = vnorm > p.norm_eps ? vnorm : p.norm_eps;
#pragma unroll
    for (int i = 0; i < CH; ++i) {
      const int x = lane + 32 * i;
      const double hat = s_gamma[x] * ((kx[i] - mu) * rs) + s_beta[x];
      p.sumK[row * D + x] = kx[i];
      p.sumV[row * D + x] = vx[i];
      p.newhat64[((int64_t)u * p.Cmax + (s_newrow[j] - (int)m)) * D + x] = hat;
      p.Khat[row * D + x] = __float2half_rn((float)hat);
      const double vo = p.radius_on ? (vnorm * (double)vx[i] / den) : (double)vx[i];
      p.Vhat[row * D + x] = __float2half_rn((float)vo);
    }
    if (lane == 0) {
      p.rho[row] = (float)vnorm;
      p.wsum[row] = 1.0;
      p.cnt[row] = 1;
      p.kmu[row] = mu;
      p.krstd[row] = rs;
      if (p.slotTok && p.b + j < p.Tassign) {
        p.slotTok[(int64_t)u * p.Tassign + p.b + j] = s_newrow[j];
        p.appTok[(int64_t)u * p.Tassign + p.b + j] = 1;
      }
    }
  }
  if (all_append) return;
  __syncthreads();

  // ---- D: merge target against s_+ (old rows: refined candidates; new rows: exact) ----
  if (tid < C && !s_app[tid]) {
    const double* kb = kbarU + (int64_t)tid * D;
    double best = s_best[tid];
    int arg = s_barg[tid];
    for (int a = 0; a < n_a; ++a) {
      const double* nh = p.newhat64 + ((int64_t)u * p.Cmax + a) * D;
      double acc = 0.0;
#pragma unroll 8
      for (int x = 0; x < D; ++x) acc += kb[x] * nh[x];
      if (acc > best) { best = acc; arg = (int)m + a; }
    }
    s_pi[tid] = arg;
    atomicAdd(&s_nmerge, 1);
  }
  __syncthreads();
  // ---- E: order merged tokens by (row, token) ----
  if (tid < C && s_pi[tid] >= 0) {
    const int pj = s_pi[tid];
    int ord = 0;
    for (int jj = 0; jj < C; ++jj) {
      const int po = s_pi[jj];
      ord += (po >= 0 && (po < pj || (po == pj && jj < tid))) ? 1 : 0;
    }
    s_sorted[ord] = tid;
  }
  __syncthreads();
  // ---- F: per-row accumulation in ascending token order, then readout refresh ----
  const int nmerge = s_nmerge;
  for (int q = warp; q < nmerge; q += 8) {
    const int j0 = s_sorted[q];
    const int rowi = s_pi[j0];
    if (q > 0 && s_pi[s_sorted[q - 1]] == rowi) continue;   // not the head of its segment
    const int64_t row = rowBase + rowi;
    double kx[CH];
    float vx[CH];
#pragma unroll
    for (int i = 0; i < CH; ++i) {
      const int x = lane + 32 * i;
      kx[i] = p.sumK[row * D + x];
      vx[i] = p.sumV[row * D + x];
    }
    double wacc = p.wsum[row];
    int nacc = p.cnt[row];
    for (int qq = q; qq < nmerge; ++qq) {
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
    double mu, rs;
    row_stats<CH>(kx, D, p.ln_eps, mu, rs);
    double v2 = 0.0;
#pragma unroll
    for (int i = 0; i < CH; ++i) v2 += (double)vx[i] * (double)vx[i];
    const double vnorm = sqrt(warp_sum_d(v2));
    const double den = vnorm > p.norm_eps ? vnorm : p.norm_eps;
    const double rad = (double)p.rho[row];
#pragma unroll
    for (int i = 0; i < CH; ++i) {
      const int x = lane + 32 * i;
      const double hat = s_gamma[x] * ((kx[i] - mu) * rs) + s_beta[x];
      p.sumK[row * D + x] = kx[i];
      p.sumV[row * D + x] = vx[i];
      p.Khat[row * D + x] = __float2half_rn((float)hat);
      const double vo = p.radius_on ? (rad * (double)vx[i] / den) : ((double)vx[i] / wacc);
      p.Vhat[row * D + x] = __float2half_rn((float)vo);
    }
    if (lane == 0) {
      p.wsum[row] = wacc;
      p.cnt[row] = nacc;
      p.kmu[row] = mu;
      p.krstd[row] = rs;
    }
  }
}

int launch_route_filter_tc(State* st, const FoldArgs& a, int nsplit, cudaStream_t s);

int launch_fold(State* st, const FoldArgs& a, cudaStream_t s) {
  int launches = 0;
  const int C = st->C, D = st->d;
  {
    dim3 grid((C + 7) / 8, st->U);
    if (D == 128)
      kbar_kernel<128><<<grid, 256, 0, s>>>(a.ok, a.unit_stride, st->ln_w, st->ln_b, st->kbar64, st->kbarH,
                                            st->kbarNorm, C, st->Cmax, st->Hkv, st->r, (double)st->ln_eps);
    else
      kbar_kernel<64><<<grid, 256, 0, s>>>(a.ok, a.unit_stride, st->ln_w, st->ln_b, st->kbar64, st->kbarH,
                                           st->kbarNorm, C, st->Cmax, st->Hkv, st->r, (double)st->ln_eps);
    ++launches;
  }
  const bool all_append = a.first || a.n_append >= C;
  int nsplit = 1;
  if (!all_append) {
    // enough CTAs to fill the GPU, at least 128 rows per split
    int64_t want = (2 * 148 + st->U - 1) / st->U;
    int64_t maxs = (a.m + 127) / 128;
    nsplit = (int)(want < maxs ? want : maxs);
    if (nsplit < 1) nsplit = 1;
    if (nsplit > st->nsplitRoute) nsplit = st->nsplitRoute;
    dim3 grid(nsplit, st->U);
    if (D == 128)
      route_filter_simt_kernel<128><<<grid, 256, 0, s>>>(st->kbarH, st->Khat, st->candV, st->candI, C, st->Cmax,
                                                         st->Mcap, a.m, nsplit);
    else
      route_filter_simt_kernel<64><<<grid, 256, 0, s>>>(st->kbarH, st->Khat, st->candV, st->candI, C, st->Cmax,
                                                        st->Mcap, a.m, nsplit);
    ++launches;
  }
  FoldUpdateParams p;
  p.ov = a.ov; p.og = a.og; p.unit_stride = a.unit_stride; p.gate_stride = a.gate_stride;
  p.kbar64 = st->kbar64; p.kbarNorm = st->kbarNorm; p.newhat64 = st->newhat64;
  p.candV = st->candV; p.candI = st->candI; p.ln_w = st->ln_w; p.ln_b = st->ln_b;
  p.sumK = st->sumK; p.sumV = st->sumV; p.rho = st->rho; p.wsum = st->wsum; p.cnt = st->cnt;
  p.kmu = st->kmu; p.krstd = st->krstd; p.Khat = st->Khat; p.Vhat = st->Vhat;
  p.slotTok = st->slotTok; p.appTok = st->appTok;
  p.Mcap = st->Mcap; p.Tassign = st->Tassign; p.m = a.m; p.b = a.b;
  p.C = C; p.Cmax = st->Cmax; p.Hkv = st->Hkv; p.S = st->S; p.n_append = a.n_append; p.nsplit = nsplit;
  p.first = a.first ? 1 : 0; p.radius_on = (st->flags & KVM_FLAG_NO_RADIUS) ? 0 : 1;
  p.ln_eps = (double)st->ln_eps; p.norm_eps = (double)st->norm_eps;
  // fp16 rounding of both operands: |err| <= (2u + u^2) |a|.|b| with u = 2^-11, plus subnormal
  // and fp32 accumulation slack; candidates lie within twice that of the approximate maximum.
  p.thr_coeff = 2.0f * (1.0f / 1024.0f + 1.0f / 65536.0f) * st->sim_norm_bound;
  if (D == 128) fold_update_kernel<128><<<st->U, 256, 0, s>>>(p);
  else fold_update_kernel<64><<<st->U, 256, 0, s>>>(p);
  ++launches;
  return launches;
}

}  // namespace kvm
