/*
 * kvm_oracle.c -- slow, plain fp64 CPU statement of the Key-Value Means (KVM) layer.
 *
 * THIS IS TEST INFRASTRUCTURE.  It exists to check the CUDA library and to be timed
 * as a CPU baseline; nothing in the product path may call it.  It shares no code with
 * the CUDA path.  Every step follows the paper "Key-Value Means: Transformers with
 * Expandable Block-Recurrent Compressed Memory", Section 3.2 ("KVM Formulation") in
 * the paper's order and notation; the passage each function follows is cited at the
 * function.  No blocking, fusion or reordering: each query token is attended by the
 * definition (one softmax over [state rows ; visible window tokens]) and each fold is
 * the append / merge rule written out.
 *
 * Readings of points the paper leaves open (all are also what the CUDA library does):
 *   - RoPE (Section 3.1 "Positional Encoding", Appendix C/D): first r channels, pairs
 *     (i, i + r/2), angle t * base^(-2 i / r), absolute position t from 0.
 *   - Memory key (Eq. 1): LayerNorm over all d channels AFTER zeroing the r rotary
 *     channels, biased variance, eps = ln_eps.
 *   - Budget B(e): FIXED = constant, SQRT = floor(coeff * sqrt(e)) computed in integers,
 *     UNBOUNDED = infinity; e = end of the chunk just attended.
 *   - Ties: arg max -> lowest row index; "smallest scores" -> lowest token index;
 *     appended rows are laid down in ascending token order.
 *   - The append score (max over ALL rows, sinks included) and the merge target
 *     (arg max over rows i >= S) are taken literally.
 *   - Rows created by initialisation or append are not gated; merged tokens are (Eq. 2-4,
 *     merge update).  A per-row weight (1 + sum of gates) and a count are kept as
 *     by-products so that "means" = sums / weight can be checked.
 *   - Folds are eager: the overflow block is folded right after the chunk ending at e
 *     has been attended.
 *
 * Parity pins (tests/test_oracle_*.py): state-size closed forms, the T <= L and the
 * never-compress limits against brute-force causal softmax, weighted-mean / radius /
 * sink invariants from the emitted member lists, brute-force routing on tiny inputs,
 * constructed tie and duplicate cases, token-at-a-time == chunked.  The choices listed
 * above (RoPE pairing, LN epsilon, budget rounding, tie rules) are fixed by this file
 * only: for those, parity is unpinned by the paper.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#else
static int omp_in_parallel(void) { return 0; }
#endif

typedef struct {
  int32_t B, Hq, Hkv, d;
  int32_t C, w, S, r;
  int32_t growth_kind; /* 0 fixed, 1 sqrt, 2 unbounded, 3 power, 4 saturating */
  int32_t sqrt_coeff;
  int64_t fixed_slots;
  double rope_base, ln_eps, norm_eps;
  int32_t radius_on; /* 1: rho * s^V / max(||s^V||, eps) ; 0: s^V / weight (ablation) */
  int32_t reserved;
  int32_t pow_num, pow_den; /* power:      B(e) = floor(sqrt_coeff * e^(pow_num/pow_den)) */
  int64_t sat_half;         /* saturating: B(e) = floor(fixed_slots * e / (e + sat_half)) */
} kvm_oracle_cfg;

typedef struct {
  int64_t m;      /* rows */
  int64_t cap;    /* allocated rows */
  double *sumK, *sumV, *rho, *wsum;
  int32_t* cnt;
  int64_t hist_len, hist_cap; /* tokens stored */
  double *khist, *vhist;      /* rotated keys / values of every token so far [t, d] */
  double* ghist;              /* merge gate of every token */
  int32_t* slot;              /* per token: row merged into / appended as; -1 not folded */
  uint8_t* appended;          /* per token */
  double* margin;             /* per merged token: best - second best similarity */
} unit_t;

typedef struct {
  kvm_oracle_cfg c;
  double *ln_w, *ln_b;   /* [Hkv, d] */
  double *tau_s, *tau_b; /* [Hq] */
  int64_t pos;
  int64_t nfolds;
  int64_t m; /* same for every unit */
  int64_t* m_after_fold; /* [nfolds] */
  int64_t* e_of_fold;
  int64_t* nappend_of_fold;
  int64_t fold_cap;
  unit_t* u; /* [B*Hkv] */
} kvm_oracle;

/* ------------------------------------------------------------------------------------ */

/* LN_s of Eq. 1 / "Readout": gamma * (x - mean) / sqrt(var + eps) + beta over d channels. */
static void layer_norm(const double* x, const double* gamma, const double* beta, double eps, int d,
                       double* out) {
  double mean = 0.0;
  for (int i = 0; i < d; ++i) mean += x[i];
  mean /= d;
  double var = 0.0;
  for (int i = 0; i < d; ++i) var += (x[i] - mean) * (x[i] - mean);
  var /= d;
  double rstd = 1.0 / sqrt(var + eps);
  for (int i = 0; i < d; ++i) out[i] = gamma[i] * ((x[i] - mean) * rstd) + beta[i];
}

/* Partial RoPE on the first r channels (Section 3.1 "Positional Encoding"). */
static void rope(const double* x, int d, int r, double base, int64_t t, double* out) {
  memcpy(out, x, sizeof(double) * d);
  int h = r / 2;
  for (int i = 0; i < h; ++i) {
    double theta = (double)t * pow(base, -2.0 * (double)i / (double)r);
    double cs = cos(theta), sn = sin(theta);
    double a = x[i], b = x[i + h];
    out[i] = a * cs - b * sn;
    out[i + h] = a * sn + b * cs;
  }
}

/* Memory key, Eq. 1: LN_s(k * diag(0_r, 1_{d-r})). */
static void memory_key(const double* k, const kvm_oracle* o, int hk, double* out) {
  int d = o->c.d;
  double* z = (double*)malloc(sizeof(double) * d);
  for (int i = 0; i < d; ++i) z[i] = (i < o->c.r) ? 0.0 : k[i];
  layer_norm(z, o->ln_w + (size_t)hk * d, o->ln_b + (size_t)hk * d, o->c.ln_eps, d, out);
  free(z);
}

static double dot(const double* a, const double* b, int d) {
  double s = 0.0;
  for (int i = 0; i < d; ++i) s += a[i] * b[i];
  return s;
}

static uint64_t isqrt_u64(uint64_t x) {
  uint64_t r = (uint64_t)sqrt((double)x);
  while (r * r > x) --r;
  while ((r + 1) * (r + 1) <= x) ++r;
  return r;
}

/* State budget B(e) (Section 3.2, budget paragraph; "16 sqrt(N)" in Section 4). */
static int64_t budget(const kvm_oracle_cfg* c, int64_t e) {
  if (c->growth_kind == 0) return c->fixed_slots;
  if (c->growth_kind == 1)
    return (int64_t)isqrt_u64((uint64_t)c->sqrt_coeff * (uint64_t)c->sqrt_coeff * (uint64_t)e);
  if (c->growth_kind == 3) {
    /* Power law (the paper names the shape, Section 3.2 and the schedule figure, without a formula;
     * reading: floor(a e^(p/q)), the integer n with n^q <= a^q e^p < (n+1)^q).  A floating-point
     * estimate, then corrected in exact 128-bit integer arithmetic. */
    unsigned __int128 rhs = 1;
    for (int i = 0; i < c->pow_den; ++i) rhs *= (unsigned __int128)c->sqrt_coeff;
    for (int i = 0; i < c->pow_num; ++i) rhs *= (unsigned __int128)e;
    int64_t n = (int64_t)((double)c->sqrt_coeff * pow((double)e, (double)c->pow_num / (double)c->pow_den));
    if (n < 0) n = 0;
    for (;;) {
      unsigned __int128 lo = 1, hi = 1;
      for (int i = 0; i < c->pow_den; ++i) { lo *= (unsigned __int128)n; hi *= (unsigned __int128)(n + 1); }
      if (lo > rhs) --n;
      else if (hi <= rhs) ++n;
      else break;
    }
    return n;
  }
  if (c->growth_kind == 4) /* saturating: rational reading, exact */
    return (int64_t)(((unsigned __int128)c->fixed_slots * (unsigned __int128)e) / (unsigned __int128)(e + c->sat_half));
  return INT64_MAX / 4;
}

static int ensure_rows(unit_t* u, int64_t rows, int d) {
  if (rows <= u->cap) return 0;
  int64_t nc = u->cap ? u->cap : 64;
  while (nc < rows) nc *= 2;
  u->sumK = (double*)realloc(u->sumK, sizeof(double) * nc * d);
  u->sumV = (double*)realloc(u->sumV, sizeof(double) * nc * d);
  u->rho = (double*)realloc(u->rho, sizeof(double) * nc);
  u->wsum = (double*)realloc(u->wsum, sizeof(double) * nc);
  u->cnt = (int32_t*)realloc(u->cnt, sizeof(int32_t) * nc);
  if (!u->sumK || !u->sumV || !u->rho || !u->wsum || !u->cnt) return -1;
  u->cap = nc;
  return 0;
}

static int ensure_hist(unit_t* u, int64_t tokens, int d) {
  if (tokens <= u->hist_cap) return 0;
  int64_t nc = u->hist_cap ? u->hist_cap : 256;
  while (nc < tokens) nc *= 2;
  u->khist = (double*)realloc(u->khist, sizeof(double) * nc * d);
  u->vhist = (double*)realloc(u->vhist, sizeof(double) * nc * d);
  u->ghist = (double*)realloc(u->ghist, sizeof(double) * nc);
  u->slot = (int32_t*)realloc(u->slot, sizeof(int32_t) * nc);
  u->appended = (uint8_t*)realloc(u->appended, nc);
  u->margin = (double*)realloc(u->margin, sizeof(double) * nc);
  if (!u->khist || !u->vhist || !u->ghist || !u->slot || !u->appended || !u->margin) return -1;
  for (int64_t t = u->hist_cap; t < nc; ++t) {
    u->slot[t] = -1;
    u->appended[t] = 0;
    u->margin[t] = INFINITY;
  }
  u->hist_cap = nc;
  return 0;
}

/* Creates a row from token j: s^K = kbar_j, s^V = v_j, rho = ||v_j||_2 (state
 * initialisation and "Append"). */
static void create_row(unit_t* u, int64_t row, const double* kbar, const double* v, int d) {
  memcpy(u->sumK + row * d, kbar, sizeof(double) * d);
  memcpy(u->sumV + row * d, v, sizeof(double) * d);
  u->rho[row] = sqrt(dot(v, v, d));
  u->wsum[row] = 1.0;
  u->cnt[row] = 1;
}

/* The fold of overflow block Omega = [b, b + C) into the state of one unit, after the
 * chunk ending at e was attended (Section 3.2 "Append", "Merge", budget rule). */
static int fold_unit(kvm_oracle* o, int unit, int64_t b, int64_t e, int64_t* n_append_out) {
  const kvm_oracle_cfg* c = &o->c;
  const int d = c->d, C = c->C;
  const int hk = unit % c->Hkv;
  unit_t* u = &o->u[unit];
  const double* gamma = o->ln_w + (size_t)hk * d;
  const double* beta = o->ln_b + (size_t)hk * d;

  double* kbar = (double*)malloc(sizeof(double) * (size_t)C * d);
  for (int j = 0; j < C; ++j) memory_key(u->khist + (b + j) * d, o, hk, kbar + (size_t)j * d);

  if (u->m == 0) { /* first state-creation step: copy the block */
    if (ensure_rows(u, C, d)) { free(kbar); return -1; }
    for (int j = 0; j < C; ++j) {
      create_row(u, j, kbar + (size_t)j * d, u->vhist + (b + j) * d, d);
      u->slot[b + j] = j;
      u->appended[b + j] = 1;
    }
    u->m = C;
    *n_append_out = C;
    free(kbar);
    return 0;
  }

  const int64_t m = u->m;
  /* normalised state keys LN_s(s^K_i) */
  double* shat = (double*)malloc(sizeof(double) * (size_t)(m + C) * d);
  #pragma omp parallel for if (!omp_in_parallel())
  for (int64_t i = 0; i < m; ++i) layer_norm(u->sumK + i * d, gamma, beta, c->ln_eps, d, shat + i * d);

  /* n_append from the budget rule */
  int64_t Bud = budget(c, e);
  int64_t lim = (Bud < m + C) ? Bud : m + C;
  int64_t Mstar = (m > lim) ? m : lim;
  int64_t n_a = Mstar - m;
  if (n_a > C) n_a = C;

  /* append score s_j = max_i kbar_j . LN_s(s^K_i) over all rows */
  double* score = (double*)malloc(sizeof(double) * C);
  #pragma omp parallel for if (!omp_in_parallel())
  for (int j = 0; j < C; ++j) {
    double best = -INFINITY;
    for (int64_t i = 0; i < m; ++i) {
      double s = dot(kbar + (size_t)j * d, shat + i * d, d);
      if (s > best) best = s;
    }
    score[j] = best;
  }
  /* A_e: the n_a tokens with the smallest scores (ties: smaller j) */
  uint8_t* inA = (uint8_t*)calloc(C, 1);
  for (int64_t a = 0; a < n_a; ++a) {
    int pick = -1;
    for (int j = 0; j < C; ++j) {
      if (inA[j]) continue;
      if (pick < 0 || score[j] < score[pick]) pick = j;
    }
    inA[pick] = 1;
  }
  if (ensure_rows(u, m + n_a, d)) { free(kbar); free(shat); free(score); free(inA); return -1; }
  int64_t mp = m;
  for (int j = 0; j < C; ++j) {
    if (!inA[j]) continue;
    create_row(u, mp, kbar + (size_t)j * d, u->vhist + (b + j) * d, d);
    layer_norm(u->sumK + mp * d, gamma, beta, c->ln_eps, d, shat + mp * d);
    u->slot[b + j] = (int32_t)mp;
    u->appended[b + j] = 1;
    ++mp;
  }
  /* merge targets pi(j) = arg max_{i >= S} kbar_j . LN_s(s^K_{+,i}), all against s_+ */
  int32_t* pi = (int32_t*)malloc(sizeof(int32_t) * C);
  #pragma omp parallel for if (!omp_in_parallel())
  for (int j = 0; j < C; ++j) {
    pi[j] = -1;
    if (inA[j]) continue;
    double best = -INFINITY, second = -INFINITY;
    int64_t arg = -1;
    for (int64_t i = c->S; i < mp; ++i) {
      double s = dot(kbar + (size_t)j * d, shat + i * d, d);
      if (s > best) { second = best; best = s; arg = i; }
      else if (s > second) second = s;
    }
    pi[j] = (int32_t)arg;
    u->margin[b + j] = best - second;
  }
  /* merge update: s^K_i += g_j kbar_j, s^V_i += g_j v_j */
  for (int j = 0; j < C; ++j) {
    if (inA[j] || pi[j] < 0) continue;
    int64_t i = pi[j];
    double g = u->ghist[b + j];
    const double* v = u->vhist + (b + j) * d;
    for (int x = 0; x < d; ++x) {
      u->sumK[i * d + x] += g * kbar[(size_t)j * d + x];
      u->sumV[i * d + x] += g * v[x];
    }
    u->wsum[i] += g;
    u->cnt[i] += 1;
    u->slot[b + j] = (int32_t)i;
    u->appended[b + j] = 0;
  }
  u->m = mp;
  *n_append_out = n_a;
  free(kbar); free(shat); free(score); free(inA); free(pi);
  return 0;
}

/* Output y_t of one query token (Section 3.2 "Readout"): softmax over all m state rows
 * (keys tau_state * LN_s(s^K), values by value-radius readout) and the window tokens
 * j in [b, t] (keys tau_bswa * k_j, values v_j), logits scaled by 1/sqrt(d).
 * khat / vhat are the readout-normalised state of this unit ([m, d] each). */
static void attend_token(const kvm_oracle* o, int unit, int qh, const double* q_rot, int64_t t,
                         int64_t b, const double* khat, const double* vhat, double* y) {
  const int d = o->c.d;
  const unit_t* u = &o->u[unit];
  const int64_t m = u->m;
  const int64_t nwin = t - b + 1;
  const int64_t n = m + nwin;
  const double ts = o->tau_s[qh], tb = o->tau_b[qh];
  const double inv = 1.0 / sqrt((double)d);
  double* logit = (double*)malloc(sizeof(double) * n);
  double mx = -INFINITY;
  for (int64_t i = 0; i < m; ++i) {
    double s = 0.0;
    for (int x = 0; x < d; ++x) s += q_rot[x] * (ts * khat[i * d + x]);
    logit[i] = s * inv;
    if (logit[i] > mx) mx = logit[i];
  }
  for (int64_t j = 0; j < nwin; ++j) {
    const double* kj = u->khist + (b + j) * d;
    double s = 0.0;
    for (int x = 0; x < d; ++x) s += q_rot[x] * (tb * kj[x]);
    logit[m + j] = s * inv;
    if (logit[m + j] > mx) mx = logit[m + j];
  }
  double den = 0.0;
  for (int64_t i = 0; i < n; ++i) { logit[i] = exp(logit[i] - mx); den += logit[i]; }
  for (int x = 0; x < d; ++x) y[x] = 0.0;
  for (int64_t i = 0; i < m; ++i) {
    double p = logit[i] / den;
    for (int x = 0; x < d; ++x) y[x] += p * vhat[i * d + x];
  }
  for (int64_t j = 0; j < nwin; ++j) {
    double p = logit[m + j] / den;
    const double* vj = u->vhist + (b + j) * d;
    for (int x = 0; x < d; ++x) y[x] += p * vj[x];
  }
  free(logit);
}

/* "Readout": s^K_hat = LN_s(s^K), s^V_hat = rho * s^V / max(||s^V||_2, eps_norm). */
static void readout_state(const kvm_oracle* o, int unit, double* khat, double* vhat) {
  const int d = o->c.d;
  const int hk = unit % o->c.Hkv;
  const unit_t* u = &o->u[unit];
  #pragma omp parallel for if (!omp_in_parallel())
  for (int64_t i = 0; i < u->m; ++i) {
    layer_norm(u->sumK + i * d, o->ln_w + (size_t)hk * d, o->ln_b + (size_t)hk * d, o->c.ln_eps, d,
               khat + i * d);
    const double* sv = u->sumV + i * d;
    if (o->c.radius_on) {
      double nrm = sqrt(dot(sv, sv, d));
      double den = nrm > o->c.norm_eps ? nrm : o->c.norm_eps;
      for (int x = 0; x < d; ++x) vhat[i * d + x] = u->rho[i] * sv[x] / den;
    } else {
      for (int x = 0; x < d; ++x) vhat[i * d + x] = sv[x] / u->wsum[i];
    }
  }
}

/* ------------------------------------------------------------------------------------ */
/* exported API (called through ctypes from tests and from the benchmark's CPU leg)      */

kvm_oracle* kvm_oracle_create(const kvm_oracle_cfg* cfg, const double* ln_w, const double* ln_b,
                              const double* tau_s, const double* tau_b) {
  if (!cfg || cfg->B < 1 || cfg->Hkv < 1 || cfg->Hq % cfg->Hkv || cfg->d < 1 || cfg->C < 1 ||
      cfg->w < 1 || cfg->S < 0 || cfg->r < 0 || cfg->r > cfg->d || (cfg->r & 1) || cfg->S >= cfg->C)
    return NULL;
  kvm_oracle* o = (kvm_oracle*)calloc(1, sizeof(kvm_oracle));
  o->c = *cfg;
  const int d = cfg->d;
  o->ln_w = (double*)malloc(sizeof(double) * cfg->Hkv * d);
  o->ln_b = (double*)malloc(sizeof(double) * cfg->Hkv * d);
  o->tau_s = (double*)malloc(sizeof(double) * cfg->Hq);
  o->tau_b = (double*)malloc(sizeof(double) * cfg->Hq);
  for (int i = 0; i < cfg->Hkv * d; ++i) {
    o->ln_w[i] = ln_w ? ln_w[i] : 1.0;
    o->ln_b[i] = ln_b ? ln_b[i] : 0.0;
  }
  for (int i = 0; i < cfg->Hq; ++i) {
    o->tau_s[i] = tau_s ? tau_s[i] : 1.0;
    o->tau_b[i] = tau_b ? tau_b[i] : 1.0;
  }
  o->u = (unit_t*)calloc((size_t)cfg->B * cfg->Hkv, sizeof(unit_t));
  return o;
}

void kvm_oracle_free(kvm_oracle* o) {
  if (!o) return;
  for (int i = 0; i < o->c.B * o->c.Hkv; ++i) {
    unit_t* u = &o->u[i];
    free(u->sumK); free(u->sumV); free(u->rho); free(u->wsum); free(u->cnt);
    free(u->khist); free(u->vhist); free(u->ghist); free(u->slot); free(u->appended); free(u->margin);
  }
  free(o->u); free(o->ln_w); free(o->ln_b); free(o->tau_s); free(o->tau_b);
  free(o->m_after_fold); free(o->e_of_fold); free(o->nappend_of_fold);
  free(o);
}

/* Consumes n further tokens.  q [B,Hq,n,d], k,v [B,Hkv,n,d], gate [B,Hkv,n] or NULL,
 * y [B,Hq,n,d] (all contiguous doubles).  Tokens are taken chunk by chunk
 * (Section 3.2 "Chunks and attention regions"): every query of the part of a chunk that
 * lies in this call is attended against the state as it stands, then, if the chunk is
 * complete and at least w chunks have been seen, the overflow block is folded.
 * Returns 0, or -1 on allocation failure. */
int kvm_oracle_forward(kvm_oracle* o, const double* q, const double* k, const double* v,
                       const double* gate, int64_t n, double* y) {
  const kvm_oracle_cfg* c = &o->c;
  const int d = c->d, C = c->C, G = c->Hq / c->Hkv;
  const int64_t L = (int64_t)c->w * C;
  const int U = c->B * c->Hkv;
  const int64_t pos0 = o->pos;
  int fail = 0;
#ifdef _OPENMP
  const int nthreads = omp_get_max_threads();
#else
  const int nthreads = 1;
#endif

  int64_t t0 = pos0;
  while (t0 < pos0 + n) {
    const int64_t cidx = t0 / C;
    const int64_t e = (cidx + 1) * C;
    const int64_t t1 = (e < pos0 + n) ? e : pos0 + n; /* tokens [t0, t1) of chunk cidx */
    const int64_t b = (e - L > 0) ? e - L : 0;
    int64_t n_append = 0;
    int do_fold = (t1 == e) && (cidx >= c->w - 1);

    #pragma omp parallel for schedule(dynamic) if (U >= nthreads)
    for (int unit = 0; unit < U; ++unit) {
      unit_t* u = &o->u[unit];
      const int bb = unit / c->Hkv, hk = unit % c->Hkv;
      if (ensure_hist(u, t1, d)) { fail = 1; continue; }
      /* store rotated keys, values and gates of the new tokens */
      for (int64_t t = t0; t < t1; ++t) {
        const size_t src = (((size_t)bb * c->Hkv + hk) * n + (t - pos0)) * d;
        rope(k + src, d, c->r, c->rope_base, t, u->khist + t * d);
        memcpy(u->vhist + t * d, v + src, sizeof(double) * d);
        u->ghist[t] = gate ? gate[((size_t)bb * c->Hkv + hk) * n + (t - pos0)] : 1.0;
      }
      u->hist_len = t1;
      /* just-in-time readout normalisation of the state */
      double* khat = (double*)malloc(sizeof(double) * (size_t)(u->m + 1) * d);
      double* vhat = (double*)malloc(sizeof(double) * (size_t)(u->m + 1) * d);
      readout_state(o, unit, khat, vhat);
      #pragma omp parallel for schedule(dynamic) if (!omp_in_parallel())
      for (int64_t idx = 0; idx < (t1 - t0) * G; ++idx) {
        const int64_t t = t0 + idx / G;
        const int qh = hk * G + (int)(idx % G);
        const size_t qoff = (((size_t)bb * c->Hq + qh) * n + (t - pos0)) * d;
        double* qr = (double*)malloc(sizeof(double) * d);
        rope(q + qoff, d, c->r, c->rope_base, t, qr);
        attend_token(o, unit, qh, qr, t, b, khat, vhat, y + qoff);
        free(qr);
      }
      free(khat); free(vhat);
      if (do_fold) {
        int64_t na = 0;
        if (fold_unit(o, unit, b, e, &na)) fail = 1;
        if (unit == 0) n_append = na;
      }
    }
    if (fail) return -1;
    if (do_fold) {
      if (o->nfolds == o->fold_cap) {
        o->fold_cap = o->fold_cap ? 2 * o->fold_cap : 64;
        o->m_after_fold = (int64_t*)realloc(o->m_after_fold, sizeof(int64_t) * o->fold_cap);
        o->e_of_fold = (int64_t*)realloc(o->e_of_fold, sizeof(int64_t) * o->fold_cap);
        o->nappend_of_fold = (int64_t*)realloc(o->nappend_of_fold, sizeof(int64_t) * o->fold_cap);
      }
      o->m = o->u[0].m;
      o->m_after_fold[o->nfolds] = o->m;
      o->e_of_fold[o->nfolds] = e;
      o->nappend_of_fold[o->nfolds] = n_append;
      o->nfolds++;
    }
    t0 = t1;
  }
  o->pos = pos0 + n;
  return 0;
}

int64_t kvm_oracle_position(const kvm_oracle* o) { return o->pos; }
int64_t kvm_oracle_rows(const kvm_oracle* o) { return o->m; }
int64_t kvm_oracle_nfolds(const kvm_oracle* o) { return o->nfolds; }

/* Fold log: e, rows after the fold, n_append; each [nfolds]. */
void kvm_oracle_fold_log(const kvm_oracle* o, int64_t* e, int64_t* m_after, int64_t* n_append) {
  for (int64_t i = 0; i < o->nfolds; ++i) {
    e[i] = o->e_of_fold[i];
    m_after[i] = o->m_after_fold[i];
    n_append[i] = o->nappend_of_fold[i];
  }
}

/* State rows: sum_k, sum_v [U,m,d]; rho, weight [U,m]; count [U,m] (any may be NULL). */
void kvm_oracle_export(const kvm_oracle* o, double* sum_k, double* sum_v, double* rho,
                       double* weight, int32_t* count) {
  const int d = o->c.d;
  const int U = o->c.B * o->c.Hkv;
  const int64_t m = o->m;
  for (int unit = 0; unit < U; ++unit) {
    const unit_t* u = &o->u[unit];
    if (sum_k) memcpy(sum_k + (size_t)unit * m * d, u->sumK, sizeof(double) * m * d);
    if (sum_v) memcpy(sum_v + (size_t)unit * m * d, u->sumV, sizeof(double) * m * d);
    if (rho) memcpy(rho + (size_t)unit * m, u->rho, sizeof(double) * m);
    if (weight) memcpy(weight + (size_t)unit * m, u->wsum, sizeof(double) * m);
    if (count) memcpy(count + (size_t)unit * m, u->cnt, sizeof(int32_t) * m);
  }
}

/* Readout-normalised state [U,m,d] each: LN_s(s^K) (no temperature) and the value readout. */
void kvm_oracle_readout(const kvm_oracle* o, double* khat, double* vhat) {
  const int d = o->c.d;
  const int U = o->c.B * o->c.Hkv;
  for (int unit = 0; unit < U; ++unit)
    readout_state(o, unit, khat + (size_t)unit * o->m * d, vhat + (size_t)unit * o->m * d);
}

/* Per-token records for tokens [0, pos): slot [U,pos], appended [U,pos], margin [U,pos]. */
void kvm_oracle_assignments(const kvm_oracle* o, int32_t* slot, uint8_t* appended, double* margin) {
  const int U = o->c.B * o->c.Hkv;
  for (int unit = 0; unit < U; ++unit) {
    const unit_t* u = &o->u[unit];
    for (int64_t t = 0; t < o->pos; ++t) {
      if (slot) slot[(size_t)unit * o->pos + t] = u->slot[t];
      if (appended) appended[(size_t)unit * o->pos + t] = u->appended[t];
      if (margin) margin[(size_t)unit * o->pos + t] = u->margin[t];
    }
  }
}

/* Memory keys kbar_t (Eq. 1) of tokens [0, pos): [U,pos,d].  Lets tests recompute row sums
 * from member lists without retyping the layer norm. */
void kvm_oracle_memory_keys(const kvm_oracle* o, double* kbar) {
  const int d = o->c.d;
  const int U = o->c.B * o->c.Hkv;
  for (int unit = 0; unit < U; ++unit)
    for (int64_t t = 0; t < o->pos; ++t)
      memory_key(o->u[unit].khist + t * d, o, unit % o->c.Hkv, kbar + ((size_t)unit * o->pos + t) * d);
}

int kvm_oracle_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}
