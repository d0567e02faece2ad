// extern "C" entry points of libkvm (declared in include/kvm.h) and the host-side chunk loop.
#include <math.h>
#include <stdio.h>
#include <string.h>

#include <new>
#include <vector>

#include "kvm_internal.h"

using namespace kvm;

struct ProfBracket { cudaEvent_t a, b; int phase; };

struct kvm_state {
  State s;
  std::vector<void*> allocs;
  bool host_staging = false;
  bool prof_on = false;
  bool prof_open = false;
  ProfBracket prof_cur{};
  std::vector<ProfBracket> prof_free, prof_used;
};

namespace {
constexpr size_t kProfMaxBrackets = 16384;
// Timing hook installed in State::prof_hook: brackets the launches of one phase with two events.
void prof_hook_fn(void* ctx, int phase, int begin, cudaStream_t stream) {
  kvm_state* ks = static_cast<kvm_state*>(ctx);
  if (begin) {
    if (ks->prof_open || ks->prof_used.size() >= kProfMaxBrackets) return;
    ProfBracket br{};
    if (!ks->prof_free.empty()) { br = ks->prof_free.back(); ks->prof_free.pop_back(); }
    else if (cudaEventCreate(&br.a) != cudaSuccess || cudaEventCreate(&br.b) != cudaSuccess) { cudaGetLastError(); return; }
    br.phase = phase;
    if (cudaEventRecord(br.a, stream) != cudaSuccess) { cudaGetLastError(); ks->prof_free.push_back(br); return; }
    ks->prof_cur = br;
    ks->prof_open = true;
  } else {
    if (!ks->prof_open || ks->prof_cur.phase != phase) return;
    cudaEventRecord(ks->prof_cur.b, stream);
    ks->prof_used.push_back(ks->prof_cur);
    ks->prof_open = false;
  }
}
}  // namespace

namespace {

uint64_t isqrt_u64(uint64_t x) {
  uint64_t r = (uint64_t)sqrt((double)x);
  while (r * r > x) --r;
  while ((r + 1) * (r + 1) <= x) ++r;
  return r;
}

// State budget B(e) (Section 3.2, budget rule; "16 sqrt(N)" and "KVM 256" of Section 4).
int64_t budget(const kvm_growth_t& g, int64_t e) {
  if (g.kind == KVM_GROWTH_FIXED) return g.fixed_slots;
  if (g.kind == KVM_GROWTH_SQRT) return (int64_t)isqrt_u64((uint64_t)g.sqrt_coeff * (uint64_t)g.sqrt_coeff * (uint64_t)e);
  if (g.kind == KVM_GROWTH_POWER) {
    // floor(a * e^(p/q)) = the largest n with n^q <= a^q * e^p, by bisection in 128-bit integers
    // (a <= 2^10, q <= 4, e < 2^26: the right-hand side stays below 2^118)
    typedef unsigned __int128 u128;
    u128 rhs = 1;
    for (int i = 0; i < g.pow_den; ++i) rhs *= (u128)g.sqrt_coeff;
    for (int i = 0; i < g.pow_num; ++i) rhs *= (u128)e;
    int64_t lo = 0, hi = (int64_t)g.sqrt_coeff * e;   // p <= q: the budget is at most a * e
    while (lo < hi) {
      const int64_t mid = lo + (hi - lo + 1) / 2;
      u128 pw = 1;
      for (int i = 0; i < g.pow_den; ++i) pw *= (u128)mid;
      if (pw <= rhs) lo = mid; else hi = mid - 1;
    }
    return lo;
  }
  if (g.kind == KVM_GROWTH_SATURATING)
    return (int64_t)(((unsigned __int128)g.fixed_slots * (unsigned __int128)e) / (unsigned __int128)(e + g.sat_half));
  return INT64_MAX / 4;
}

// n_append = min(M* - m, |Omega|), M* = max(m, min(B(e), m + C)).
int64_t n_append_of(const kvm_growth_t& g, int64_t e, int64_t m, int C) {
  const int64_t bud = budget(g, e);
  const int64_t lim = bud < m + C ? bud : m + C;
  const int64_t mstar = m > lim ? m : lim;
  const int64_t na = mstar - m;
  return na < C ? na : C;
}

bool growth_valid(const kvm_growth_t& g) {
  if (g.kind == KVM_GROWTH_FIXED) return g.fixed_slots >= 1;
  if (g.kind == KVM_GROWTH_SQRT) return g.sqrt_coeff >= 1 && g.sqrt_coeff <= 65535;
  if (g.kind == KVM_GROWTH_POWER)
    return g.sqrt_coeff >= 1 && g.sqrt_coeff <= 1024 && g.pow_num >= 1 && g.pow_num <= g.pow_den && g.pow_den <= 4;
  if (g.kind == KVM_GROWTH_SATURATING) return g.fixed_slots >= 1 && g.sat_half >= 1;
  return g.kind == KVM_GROWTH_UNBOUNDED;
}
constexpr int64_t kPowerMaxPos = (int64_t)1 << 26;   // positions the POWER budget is defined for

bool growth_equal(const kvm_growth_t& a, const kvm_growth_t& b) {
  if (a.kind != b.kind) return false;
  if (a.kind == KVM_GROWTH_FIXED) return a.fixed_slots == b.fixed_slots;
  if (a.kind == KVM_GROWTH_SQRT) return a.sqrt_coeff == b.sqrt_coeff;
  if (a.kind == KVM_GROWTH_POWER) return a.sqrt_coeff == b.sqrt_coeff && a.pow_num == b.pow_num && a.pow_den == b.pow_den;
  if (a.kind == KVM_GROWTH_SATURATING) return a.fixed_slots == b.fixed_slots && a.sat_half == b.sat_half;
  return true;
}

template <typename T>
kvm_status_t dev_alloc(kvm_state* ks, T** p, size_t count, bool zero = true) {
  void* ptr = nullptr;
  size_t bytes = count * sizeof(T);
  if (bytes == 0) bytes = sizeof(T);
  cudaError_t e = cudaMalloc(&ptr, bytes);
  if (e != cudaSuccess) {
    cudaGetLastError();
    return e == cudaErrorMemoryAllocation ? KVM_ERR_OOM : KVM_ERR_CUDA;
  }
  ks->allocs.push_back(ptr);
  if (zero && cudaMemset(ptr, 0, bytes) != cudaSuccess) return KVM_ERR_CUDA;
  *p = reinterpret_cast<T*>(ptr);
  return KVM_OK;
}

void free_all(kvm_state* ks) {
  for (void* p : ks->allocs) cudaFree(p);
  ks->allocs.clear();
  State& s = ks->s;
  if (s.foldStream) { cudaStreamDestroy(s.foldStream); s.foldStream = nullptr; }
  if (s.kbStream) { cudaStreamDestroy(s.kbStream); s.kbStream = nullptr; }
  if (s.hinStream) { cudaStreamDestroy(s.hinStream); s.hinStream = nullptr; }
  if (s.houtStream) { cudaStreamDestroy(s.houtStream); s.houtStream = nullptr; }
  for (cudaEvent_t* e : {&s.evHostStart, &s.evHostOut}) if (*e) { cudaEventDestroy(*e); *e = nullptr; }
  for (int i = 0; i < 8; ++i) {
    if (s.evIn[i]) { cudaEventDestroy(s.evIn[i]); s.evIn[i] = nullptr; }
    if (s.evComp[i]) { cudaEventDestroy(s.evComp[i]); s.evComp[i] = nullptr; }
  }
  for (cudaEvent_t* e : {&s.evJoin, &s.evPre[0], &s.evPre[1], &s.evFold[0], &s.evFold[1], &s.evKb[0], &s.evKb[1], &s.evBatchDone[0], &s.evBatchDone[1]})
    if (*e) { cudaEventDestroy(*e); *e = nullptr; }
}

struct DeviceGuard {
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; cudaGetLastError(); return; }
    if (prev != dev && cudaSetDevice(dev) != cudaSuccess) { ok = false; cudaGetLastError(); }
  }
  ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

// Everything a prefill of n further tokens can fail on, checked on the host without touching the
// state: block / growth / rope_dims (against the state's when it is bound), the positions the POWER
// budget is defined for, and the row capacity - the row count after the call follows from the budget
// rule alone.  (n_tokens against max_call_tokens is the caller's check: the host-buffer entry point
// cuts a long call into segments.)
kvm_status_t validate_prefill(const State& s, int32_t block, const kvm_growth_t& growth, int32_t r, int64_t n) {
  if (n < 1) return KVM_ERR_INVALID_ARG;
  if (!s.bound) {
    if (block < 8 || block > s.Cmax || (block % 8) != 0 || s.S >= block) return KVM_ERR_INVALID_ARG;
    if (r < 0 || r > s.d || (r & 1)) return KVM_ERR_INVALID_ARG;
    if (!growth_valid(growth)) return KVM_ERR_INVALID_ARG;
  } else if (block != s.C || r != s.r || !growth_equal(growth, s.growth)) {
    return KVM_ERR_STATE_MISMATCH;
  }
  const int C = block;
  const int64_t pos0 = s.bound ? s.pos : 0, pos1 = pos0 + n;
  if (growth.kind == KVM_GROWTH_POWER && pos1 >= kPowerMaxPos) return KVM_ERR_UNSUPPORTED;
  int64_t m_sim = s.bound ? s.m : 0;
  for (int64_t c = pos0 / C; c <= (pos1 - 1) / C; ++c) {
    const int64_t e = (c + 1) * C;
    if (e <= pos1 && c >= s.w - 1) m_sim += (m_sim == 0) ? C : n_append_of(growth, e, m_sim, C);
  }
  if (m_sim > s.Mcap) return KVM_ERR_CAPACITY;
  return KVM_OK;
}

// Binds block / growth / rope_dims (host bookkeeping only; called once the call can no longer fail).
void bind_state(State& s, int32_t block, const kvm_growth_t& growth, int32_t r) {
  s.C = block; s.r = r; s.growth = growth; s.ringLen = (int64_t)s.w * block;
  const int k = r / 2;
  s.inv_freq = s.inv_freq_all + (int64_t)k * (k - 1) / 2;
  s.recomputeK = s.serial && (int64_t)block * s.U >= 8192;   // (the threshold of the four-rows-per-warp apply kernel)
  s.bound = true;
}

kvm_status_t ensure_host_staging(kvm_state* ks) {
  if (ks->host_staging) return KVM_OK;
  State& s = ks->s;
  const size_t nq = (size_t)s.B * s.Hq * s.Tcall * s.d, nk = (size_t)s.U * s.Tcall * s.d;
  __nv_bfloat16 *a, *b, *c, *o;
  kvm_status_t rc;
  if ((rc = dev_alloc(ks, &a, nq, false)) != KVM_OK) return rc;
  if ((rc = dev_alloc(ks, &b, nk, false)) != KVM_OK) return rc;
  if ((rc = dev_alloc(ks, &c, nk, false)) != KVM_OK) return rc;
  if ((rc = dev_alloc(ks, &o, nq, false)) != KVM_OK) return rc;
  if ((rc = dev_alloc(ks, &s.hG, (size_t)s.U * s.Tcall, false)) != KVM_OK) return rc;
  s.hQ = a; s.hK = b; s.hV = c; s.hOut = o;
  bool ok = cudaStreamCreateWithFlags(&s.hinStream, cudaStreamNonBlocking) == cudaSuccess;
  ok = ok && cudaStreamCreateWithFlags(&s.houtStream, cudaStreamNonBlocking) == cudaSuccess;
  ok = ok && cudaEventCreateWithFlags(&s.evHostStart, cudaEventDisableTiming) == cudaSuccess;
  ok = ok && cudaEventCreateWithFlags(&s.evHostOut, cudaEventDisableTiming) == cudaSuccess;
  for (int i = 0; i < 8; ++i) {
    ok = ok && cudaEventCreateWithFlags(&s.evIn[i], cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&s.evComp[i], cudaEventDisableTiming) == cudaSuccess;
  }
  if (!ok) { cudaGetLastError(); return KVM_ERR_CUDA; }
  ks->host_staging = true;
  return KVM_OK;
}

bool launch_ok() { return cudaGetLastError() == cudaSuccess; }

}  // namespace

namespace {
// Window tokens [wb, wb + len) <-> host arrays [U, len, ...]: the ring holds token t in slot t mod ringLen,
// so the range is one or two runs of consecutive slots.
template <typename F>
bool for_ring_runs(const State& s, int64_t wb, int64_t len, F&& f) {
  int64_t done = 0;
  while (done < len) {
    const int64_t slot = (wb + done) % s.ringLen;
    int64_t run = s.ringLen - slot;
    if (run > len - done) run = len - done;
    if (!f(done, slot, run)) return false;
    done += run;
  }
  return true;
}
}  // namespace

#define KVM_API __attribute__((visibility("default")))

extern "C" {

KVM_API const char* kvm_status_string(kvm_status_t s) {
  switch (s) {
    case KVM_OK: return "ok";
    case KVM_ERR_INVALID_ARG: return "invalid argument";
    case KVM_ERR_UNSUPPORTED: return "unsupported configuration";
    case KVM_ERR_OOM: return "out of device memory";
    case KVM_ERR_CUDA: return "CUDA error";
    case KVM_ERR_STATE_MISMATCH: return "block/growth/rope_dims differ from the state's";
    case KVM_ERR_CAPACITY: return "state or call capacity exceeded";
    case KVM_ERR_TIMEOUT: return "device-side wait expired";
  }
  return "unknown status";
}

KVM_API int64_t kvm_plan_capacity(int32_t block, int32_t n_bswa_chunks, kvm_growth_t growth, int64_t seq_len) {
  if (block < 1 || n_bswa_chunks < 1 || seq_len < 0 || !growth_valid(growth)) return -1;
  if (growth.kind == KVM_GROWTH_POWER && seq_len >= kPowerMaxPos) return -1;
  int64_t m = 0;
  for (int64_t c = n_bswa_chunks - 1; (c + 1) * block <= seq_len; ++c) {
    const int64_t e = (c + 1) * block;
    m += (m == 0) ? block : n_append_of(growth, e, m, block);
  }
  return m;
}

KVM_API kvm_status_t kvm_state_create(const kvm_config_t* cfg, kvm_state_t** out) {
  if (!cfg || !out) return KVM_ERR_INVALID_ARG;
  if (cfg->batch < 1 || cfg->n_q_heads < 1 || cfg->n_kv_heads < 1 || cfg->n_q_heads % cfg->n_kv_heads) return KVM_ERR_INVALID_ARG;
  if (cfg->n_bswa_chunks < 1 || cfg->sink_len < 0) return KVM_ERR_INVALID_ARG;
  if (cfg->max_block < 8 || (cfg->max_block % 8) || cfg->sink_len >= cfg->max_block) return KVM_ERR_INVALID_ARG;
  if (cfg->max_state_slots < cfg->max_block || cfg->max_call_tokens < 1) return KVM_ERR_INVALID_ARG;
  if (!(cfg->rope_base > 0.f) || !(cfg->ln_eps >= 0.f) || !(cfg->norm_eps >= 0.f)) return KVM_ERR_INVALID_ARG;
  if ((cfg->flags & KVM_FLAG_RECORD_ASSIGN) && cfg->max_seq_len < 1) return KVM_ERR_INVALID_ARG;
  if (cfg->head_dim != 64 && cfg->head_dim != 128) return KVM_ERR_UNSUPPORTED;
  if (cfg->max_block > kMaxBlock) return KVM_ERR_UNSUPPORTED;
  if (cfg->max_state_slots >= (1 << 23)) return KVM_ERR_UNSUPPORTED;   // sort keys of the fold hold a row in 23 bits

  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev < 1 || cfg->device < 0 || cfg->device >= ndev) {
    cudaGetLastError();
    return KVM_ERR_CUDA;
  }
  DeviceGuard guard(cfg->device);
  if (!guard.ok) return KVM_ERR_CUDA;

  kvm_state* ks = new (std::nothrow) kvm_state();
  if (!ks) return KVM_ERR_OOM;
  State& s = ks->s;
  memset(&s, 0, sizeof(State));
  s.B = cfg->batch; s.Hq = cfg->n_q_heads; s.Hkv = cfg->n_kv_heads; s.d = cfg->head_dim;
  s.G = s.Hq / s.Hkv; s.U = s.B * s.Hkv; s.w = cfg->n_bswa_chunks; s.S = cfg->sink_len;
  s.Cmax = cfg->max_block;
  s.Mcap = (cfg->max_state_slots + kRowAlign - 1) / kRowAlign * kRowAlign;
  s.Tcall = cfg->max_call_tokens;
  s.Tassign = (cfg->flags & KVM_FLAG_RECORD_ASSIGN) ? cfg->max_seq_len : 0;
  s.rope_base = cfg->rope_base; s.ln_eps = cfg->ln_eps; s.norm_eps = cfg->norm_eps;
  s.flags = cfg->flags; s.device = cfg->device;
  s.stRows = (int64_t)s.w * s.Cmax + s.Tcall;

  const int d = s.d;
  std::vector<float> lw((size_t)s.Hkv * d, 1.f), lb((size_t)s.Hkv * d, 0.f), ts(s.Hq, 1.f), tb(s.Hq, 1.f);
  if (cfg->ln_weight) memcpy(lw.data(), cfg->ln_weight, sizeof(float) * lw.size());
  if (cfg->ln_bias) memcpy(lb.data(), cfg->ln_bias, sizeof(float) * lb.size());
  if (cfg->tau_state) memcpy(ts.data(), cfg->tau_state, sizeof(float) * ts.size());
  if (cfg->tau_bswa) memcpy(tb.data(), cfg->tau_bswa, sizeof(float) * tb.size());
  double bound = 0.0;
  for (int h = 0; h < s.Hkv; ++h) {
    double gmax = 0.0, b2 = 0.0;
    for (int x = 0; x < d; ++x) {
      gmax = fmax(gmax, fabs((double)lw[(size_t)h * d + x]));
      b2 += (double)lb[(size_t)h * d + x] * lb[(size_t)h * d + x];
    }
    bound = fmax(bound, sqrt((double)d) * gmax + sqrt(b2));
  }
  if (!(bound < 3.0e4)) { delete ks; return KVM_ERR_UNSUPPORTED; }   // fp16 routing copies must not overflow
  s.sim_norm_bound = (float)(bound * 1.0001);

  const size_t U = s.U, M = s.Mcap, ringCap = (size_t)s.w * s.Cmax, Cm = s.Cmax;
  s.nsplitRoute = (int)((2 * 148 + U - 1) / U);
  if (s.nsplitRoute > kMaxSplits) s.nsplitRoute = kMaxSplits;
  if (s.nsplitRoute < 1) s.nsplitRoute = 1;
  {
    // decode CTAs serve up to eight query heads of a kv group; the row splits fill the GPU about four times
    const int gq = (s.G % 8 == 0) ? 8 : (s.G % 4 == 0) ? 4 : (s.G % 2 == 0) ? 2 : 1;
    const size_t ncta = (size_t)s.B * s.Hq / gq;
    s.nsplitDec = (int)((4 * 148 + ncta - 1) / ncta);
  }
  if (s.nsplitDec > kMaxSplits) s.nsplitDec = kMaxSplits;
  if (s.nsplitDec < 1) s.nsplitDec = 1;

  kvm_status_t rc = KVM_OK;
#define A(ptr, count) if (rc == KVM_OK) rc = dev_alloc(ks, &(ptr), (count))
  A(s.ln_w, (size_t)s.Hkv * d); A(s.ln_b, (size_t)s.Hkv * d); A(s.tau_s, (size_t)s.Hq); A(s.tau_b, (size_t)s.Hq);
  A(s.inv_freq_all, (size_t)(d / 2) * (d / 2 + 1) / 2);
  s.fusedLn = (cfg->flags & KVM_FLAG_FUSED_QK_LN) != 0;
  s.qk_ln_eps = cfg->qk_ln_eps;
  if (s.fusedLn) {
    if (!(cfg->qk_ln_eps >= 0.f)) rc = KVM_ERR_INVALID_ARG;
    auto up = [&](float** dst, const float* src, size_t n) {   // optional host array -> device (NULL stays NULL)
      *dst = nullptr;
      if (!src || rc != KVM_OK) return;
      rc = dev_alloc(ks, dst, n, false);
      if (rc == KVM_OK && cudaMemcpy(*dst, src, n * sizeof(float), cudaMemcpyHostToDevice) != cudaSuccess) rc = KVM_ERR_CUDA;
    };
    up(&s.lnq_w, cfg->ln_q_weight, (size_t)s.Hq * d); up(&s.lnq_b, cfg->ln_q_bias, (size_t)s.Hq * d);
    up(&s.lnk_w, cfg->ln_k_weight, (size_t)s.Hkv * d); up(&s.lnk_b, cfg->ln_k_bias, (size_t)s.Hkv * d);
  }
  A(s.sumK, U * M * d); A(s.sumV, U * M * d); A(s.rho, U * M); A(s.wsum, U * M); A(s.cnt, U * M);
  A(s.kmu, U * M); A(s.krstd, U * M);
  // with enough units every kernel of a fold fills the GPU by itself and nothing is gained by running the
  // folds beside the attention: such a state keeps ONE readout copy (both names refer to it)
  s.serial = s.U >= kSerialUnits || (cfg->flags & KVM_FLAG_SERIAL_FOLDS);
  A(s.KhatBuf[0], U * M * d); A(s.VhatBuf[0], U * M * d);
  if (s.serial) { s.KhatBuf[1] = s.KhatBuf[0]; s.VhatBuf[1] = s.VhatBuf[0]; }
  else { A(s.KhatBuf[1], U * M * d); A(s.VhatBuf[1], U * M * d); }
  A(s.ringK, U * ringCap * d); A(s.ringV, U * ringCap * d); A(s.ringG, U * ringCap);
  A(s.stQ, (size_t)s.B * s.Hq * s.Tcall * d);
  A(s.stK, U * (size_t)s.stRows * d); A(s.stV, U * (size_t)s.stRows * d); A(s.stG, U * (size_t)s.stRows);
  A(s.ropeCS, (size_t)s.Tcall * (d / 2));
  s.CbarRows = (s.Cmax + 127) / 128 * 128;
  {
    // memory-key slots: as many blocks per batched launch as fit in 2 GiB (at most 64, never more than
    // a call can hold) and at least two, one per half: a prefill computes the keys of one batch of
    // blocks while the folds consume the batch before it, so the two must never share a slot
    const size_t per_slot = U * Cm * d * 8 + U * (size_t)s.CbarRows * d * 4 + U * Cm * 20 + U * Cm * Cm * 4;
    size_t slots = ((size_t)2 << 30) / per_slot;
    const size_t call_blocks = (size_t)(s.Tcall / s.Cmax) + 2;
    if (slots > call_blocks) slots = call_blocks;
    if (slots > 64) slots = 64;
    if (slots < 2 || (cfg->flags & KVM_FLAG_MIN_KEY_SLOTS)) slots = 2;
    s.kbSlots = (int)slots;
  }
  {
    const size_t G = (size_t)s.kbSlots;
    A(s.kbarStat, G * U * Cm); A(s.kbar64, G * U * Cm * d); A(s.kbarH, G * U * (size_t)s.CbarRows * d); A(s.kbarNorm, G * U * Cm);
    A(s.kbarHatStat, G * U * Cm); A(s.kbarHatH, G * U * (size_t)s.CbarRows * d);
    A(s.gramT, G * U * Cm * Cm);
  }
  for (int i = 0; i < 2; ++i) {
    A(s.foldPi[i], U * Cm); A(s.foldSorted[i], U * Cm); A(s.foldCreator[i], U * Cm); A(s.foldSegNew[i], U * Cm);
    A(s.foldNMerge[i], U);
  }
  A(s.xScore, U * Cm); A(s.xBest, U * Cm); A(s.xArg, U * Cm); A(s.xCount, U);
  if (rc == KVM_OK && cudaMemset(s.xCount, 0, U * sizeof(int32_t)) != cudaSuccess) rc = KVM_ERR_CUDA;
  A(s.candV, U * (size_t)s.nsplitRoute * Cm * kTopK); A(s.candI, U * (size_t)s.nsplitRoute * Cm * kTopK);
  A(s.chunkMeta, U * (size_t)s.nsplitRoute * Cm * kChunkCap); A(s.chunkMax, U * (size_t)s.nsplitRoute * Cm * kChunkCap);
  if (rc == KVM_OK) rc = dev_alloc(ks, &s.chunkVal, U * (size_t)s.nsplitRoute * Cm * kChunkCap * 32, false);
  A(s.decPart, (size_t)s.B * s.Hq * s.nsplitDec * (d + 2)); A(s.decQ, (size_t)s.B * s.Hq * d);
  // (tiles x splits: up to kAttnSplitTiles x kAttnMaxSplits, or 2 kAttnSplitTiles tiles of two splits)
  A(s.attnPart, (size_t)kAttnSplitTiles * kAttnMaxSplits * (d + 2) * 128); A(s.attnCnt, (size_t)2 * kAttnSplitTiles);
  if (rc == KVM_OK && cudaMemset(s.attnCnt, 0, 2 * kAttnSplitTiles * sizeof(int32_t)) != cudaSuccess) rc = KVM_ERR_CUDA;
  A(s.status, (size_t)16);   // [0] status word, [1..3] fold debug counters
  if (s.Tassign > 0) { A(s.slotTok, U * (size_t)s.Tassign); A(s.appTok, U * (size_t)s.Tassign); }
#undef A
  if (rc == KVM_OK && s.Tassign > 0 && cudaMemset(s.slotTok, 0xff, U * (size_t)s.Tassign * sizeof(int32_t)) != cudaSuccess) rc = KVM_ERR_CUDA;
  if (rc == KVM_OK) {
    bool ok = cudaMemcpy(s.ln_w, lw.data(), sizeof(float) * lw.size(), cudaMemcpyHostToDevice) == cudaSuccess;
    ok = ok && cudaMemcpy(s.ln_b, lb.data(), sizeof(float) * lb.size(), cudaMemcpyHostToDevice) == cudaSuccess;
    ok = ok && cudaMemcpy(s.tau_s, ts.data(), sizeof(float) * ts.size(), cudaMemcpyHostToDevice) == cudaSuccess;
    ok = ok && cudaMemcpy(s.tau_b, tb.data(), sizeof(float) * tb.size(), cudaMemcpyHostToDevice) == cudaSuccess;
    // RoPE frequencies base^(-2i/r) for every even r <= d, so that binding rope_dims later needs no copy
    std::vector<double> fr;
    for (int k = 1; k <= d / 2; ++k)
      for (int i = 0; i < k; ++i) fr.push_back(pow((double)s.rope_base, -2.0 * (double)i / (double)(2 * k)));
    ok = ok && cudaMemcpy(s.inv_freq_all, fr.data(), sizeof(double) * fr.size(), cudaMemcpyHostToDevice) == cudaSuccess;
    ok = ok && cudaDeviceSynchronize() == cudaSuccess;
    if (!ok) rc = KVM_ERR_CUDA;
  }
  if (rc == KVM_OK && !(setup_attn_tc(&s) && setup_route_tc(&s))) rc = KVM_ERR_CUDA;
  if (rc == KVM_OK) {
    bool ok = cudaStreamCreateWithFlags(&s.foldStream, cudaStreamNonBlocking) == cudaSuccess;
    ok = ok && cudaStreamCreateWithFlags(&s.kbStream, cudaStreamNonBlocking) == cudaSuccess;
    for (cudaEvent_t* e : {&s.evJoin, &s.evPre[0], &s.evPre[1], &s.evFold[0], &s.evFold[1], &s.evKb[0], &s.evKb[1], &s.evBatchDone[0], &s.evBatchDone[1]})
      ok = ok && cudaEventCreateWithFlags(e, cudaEventDisableTiming) == cudaSuccess;
    if (!ok) rc = KVM_ERR_CUDA;
  }
  if (rc != KVM_OK) {
    cudaGetLastError();
    free_all(ks);
    delete ks;
    return rc;
  }
  *out = ks;
  return KVM_OK;
}

KVM_API kvm_status_t kvm_state_free(kvm_state_t* ks) {
  if (!ks) return KVM_OK;
  DeviceGuard guard(ks->s.device);
  cudaDeviceSynchronize();
  for (auto& v : {&ks->prof_free, &ks->prof_used})
    for (const ProfBracket& br : *v) { cudaEventDestroy(br.a); cudaEventDestroy(br.b); }
  free_all(ks);
  delete ks;
  return KVM_OK;
}

KVM_API kvm_status_t kvm_debug_counters(kvm_state_t* ks, int64_t* out, void* cuda_stream) {
  if (!ks || !out) return KVM_ERR_INVALID_ARG;
  DeviceGuard guard(ks->s.device);
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  int32_t w[16];
  if (cudaMemcpyAsync(w, ks->s.status, sizeof(w), cudaMemcpyDeviceToHost, stream) != cudaSuccess) return KVM_ERR_CUDA;
  if (cudaStreamSynchronize(stream) != cudaSuccess) return KVM_ERR_CUDA;
  for (int i = 0; i < 4; ++i) out[i] = w[1 + i];
  return KVM_OK;
}

KVM_API kvm_status_t kvm_state_reset(kvm_state_t* ks) {
  if (!ks) return KVM_ERR_INVALID_ARG;
  State& s = ks->s;
  s.bound = false; s.pos = 0; s.m = 0; s.nfolds = 0; s.prevValid = false;
  if (s.slotTok) s.assignDirty = true;   // debug recording only: the next prefill forgets the old assignments, on its stream
  return KVM_OK;
}

KVM_API kvm_status_t kvm_profile_enable(kvm_state_t* ks, int32_t on) {
  if (!ks) return KVM_ERR_INVALID_ARG;
  ks->prof_on = on != 0;
  ks->s.prof_hook = ks->prof_on ? prof_hook_fn : nullptr;
  ks->s.prof_ctx = ks;
  return KVM_OK;
}

KVM_API kvm_status_t kvm_profile_read(kvm_state_t* ks, double* ms, int64_t* groups) {
  if (!ks || !ms || !groups) return KVM_ERR_INVALID_ARG;
  DeviceGuard guard(ks->s.device);
  if (cudaDeviceSynchronize() != cudaSuccess) return KVM_ERR_CUDA;
  for (const ProfBracket& br : ks->prof_used) {
    float t = 0.f;
    if (cudaEventElapsedTime(&t, br.a, br.b) == cudaSuccess) { ms[br.phase] += t; groups[br.phase] += 1; }
    else cudaGetLastError();
    ks->prof_free.push_back(br);
  }
  ks->prof_used.clear();
  return KVM_OK;
}

KVM_API kvm_status_t kvm_state_info(const kvm_state_t* ks, int64_t* n_slots, int64_t* position, int64_t* n_folds) {
  if (!ks) return KVM_ERR_INVALID_ARG;
  if (n_slots) *n_slots = ks->s.m;
  if (position) *position = ks->s.pos;
  if (n_folds) *n_folds = ks->s.nfolds;
  return KVM_OK;
}

KVM_API int64_t kvm_launch_count(const kvm_state_t* ks) { return ks ? ks->s.launches : -1; }

KVM_API kvm_status_t kvm_state_check(kvm_state_t* ks, void* cuda_stream) {
  if (!ks) return KVM_ERR_INVALID_ARG;
  DeviceGuard guard(ks->s.device);
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  int32_t w = 0;
  if (cudaMemcpyAsync(&w, ks->s.status, sizeof(w), cudaMemcpyDeviceToHost, stream) != cudaSuccess) return KVM_ERR_CUDA;
  if (cudaStreamSynchronize(stream) != cudaSuccess) return KVM_ERR_CUDA;
  if (w == 0) return KVM_OK;
  if (cudaMemsetAsync(ks->s.status, 0, sizeof(w), stream) != cudaSuccess) return KVM_ERR_CUDA;   // reported once
  return w == KVM_ERR_TIMEOUT ? KVM_ERR_TIMEOUT : KVM_ERR_CUDA;
}

KVM_API kvm_status_t kvm_debug_expire_wait(kvm_state_t* ks, int32_t spins, void* cuda_stream) {
  if (!ks || spins < 1 || spins > (1 << 20)) return KVM_ERR_INVALID_ARG;
  DeviceGuard guard(ks->s.device);
  if (!guard.ok) return KVM_ERR_CUDA;
  launch_expire_wait(&ks->s, spins, (cudaStream_t)cuda_stream);
  ks->s.launches += 1;
  return launch_ok() ? KVM_OK : KVM_ERR_CUDA;
}

KVM_API kvm_status_t kvm_prefill(const void* q, const void* k, const void* v, kvm_state_t* ks, int32_t block,
                         kvm_growth_t growth, int32_t rope_dims, int64_t n_tokens, const float* gate, void* out,
                         const kvm_strides_t* strides, void* cuda_stream) {
  if (!q || !k || !v || !ks || !out) return KVM_ERR_INVALID_ARG;
  State& s = ks->s;
  if (n_tokens < 1) return KVM_ERR_INVALID_ARG;
  if (n_tokens > s.Tcall) return KVM_ERR_CAPACITY;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  DeviceGuard guard(s.device);
  if (!guard.ok) return KVM_ERR_CUDA;

  const int d = s.d;
  const int64_t n = n_tokens;
  IngestArgs ia;
  AttnArgs aa;
  if (strides) {
    for (int i = 0; i < 4; ++i) { ia.sq[i] = strides->q[i]; ia.sk[i] = strides->k[i]; ia.sv[i] = strides->v[i]; aa.so[i] = strides->out[i]; }
    if (ia.sq[3] != 1 || ia.sk[3] != 1 || ia.sv[3] != 1 || aa.so[3] != 1) return KVM_ERR_INVALID_ARG;
    // rows are read and written as pairs of bf16
    for (int i = 0; i < 3; ++i)
      if ((ia.sq[i] & 1) || (ia.sk[i] & 1) || (ia.sv[i] & 1) || (aa.so[i] & 1)) return KVM_ERR_INVALID_ARG;
  } else {
    ia.sq[0] = (int64_t)s.Hq * n * d; ia.sq[1] = n * d; ia.sq[2] = d; ia.sq[3] = 1;
    ia.sk[0] = (int64_t)s.Hkv * n * d; ia.sk[1] = n * d; ia.sk[2] = d; ia.sk[3] = 1;
    for (int i = 0; i < 4; ++i) { ia.sv[i] = ia.sk[i]; aa.so[i] = ia.sq[i]; }
  }
  if (((uintptr_t)q & 3) || ((uintptr_t)k & 3) || ((uintptr_t)v & 3) || ((uintptr_t)out & 3)) return KVM_ERR_INVALID_ARG;
  ia.sg[0] = (int64_t)s.Hkv * n; ia.sg[1] = n; ia.sg[2] = 1;

  {
    const kvm_status_t rc = validate_prefill(s, block, growth, rope_dims, n);
    if (rc != KVM_OK) return rc;
  }
  ia.q = (const __nv_bfloat16*)q; ia.k = (const __nv_bfloat16*)k; ia.v = (const __nv_bfloat16*)v;
  // the fused front end works on whole 16-byte chunks of every row
  if (s.fusedLn && !ingest_rows_aligned(rope_dims, ia)) return KVM_ERR_INVALID_ARG;
  if (!s.bound) bind_state(s, block, growth, rope_dims);
  const int C = s.C;
  const int64_t L = (int64_t)s.w * C;
  const int64_t pos0 = s.pos, pos1 = pos0 + n;
  const int64_t c0 = pos0 / C, c_last = (pos1 - 1) / C;
  if (s.assignDirty) {
    s.assignDirty = false;
    if (cudaMemsetAsync(s.slotTok, 0xff, (size_t)s.U * s.Tassign * sizeof(int32_t), stream) != cudaSuccess) return KVM_ERR_CUDA;
  }

  ia.q = (const __nv_bfloat16*)q; ia.k = (const __nv_bfloat16*)k; ia.v = (const __nv_bfloat16*)v; ia.gate = gate;
  ia.pos0 = pos0; ia.n = n;
  ia.hist_start = (c0 + 1) * C - L; if (ia.hist_start < 0) ia.hist_start = 0;
  ia.nhist = pos0 - ia.hist_start;
  {
    const int64_t c_next = pos1 / C;
    ia.tail_start = (c_next + 1) * C - L; if (ia.tail_start < 0) ia.tail_start = 0;
  }
  { KernelTimer pt(&s, 0, stream); s.launches += launch_ingest(&s, ia, stream); }

  // Two streams: attention runs on the caller's stream, folds on the state's own stream.  The fold
  // that ends block c needs the state after the fold before it and block c-w+1's keys, not block c's
  // attention, so the two overlap.  Orderings kept by events:
  //   the fold stream waits for the ingest (and with it for everything earlier on the caller's stream);
  //   attention(c+1) waits for the fold that ends block c (it reads the readout copy that fold wrote);
  //   before attention(c) the caller's stream brings the rows the last fold touched over to the other
  //   readout copy (attention(c-1), the last reader of that copy, is earlier on the same stream) and
  //   records evPre; the last kernel of the fold that ends block c, which writes that copy, waits for evPre;
  //   the caller's stream waits for the last fold before the call returns.
  // With the per-kernel timing hook on, everything stays on the caller's stream so that the
  // measured durations are those of kernels running alone.
  // A state with so many units that every kernel fills the GPU by itself (State::serial) keeps one
  // readout copy and runs its folds on the caller's stream between the attention launches; only the
  // memory keys are still computed ahead on their own stream.
  const bool ovk = s.prof_hook == nullptr;     // memory keys ahead of the folds on their own stream
  const bool ovf = ovk && !s.serial;           // folds on their own stream beside the attention
  cudaStream_t fstream = ovf ? s.foldStream : stream;
  bool ev_ok = true;
  if (ovk) ev_ok = ev_ok && cudaEventRecord(s.evJoin, stream) == cudaSuccess;
  if (ovf) ev_ok = ev_ok && cudaStreamWaitEvent(fstream, s.evJoin, 0) == cudaSuccess;
  int fold_pending = -1;               // evFold index the next attention must wait for
  // The folds of this call, planned ahead from the budget rule: fold i ends block cf0 + i, folds the
  // block that starts at bf0 + i*C and appends fold_na[i] rows.  Their memory keys (and new-row
  // filters) need the ingested keys only, so they are computed in batches on a third stream, one
  // batch ahead of the folds; a batch fills one half of the slots.
  std::vector<int> fold_na;
  int64_t cf0 = -1;
  int n_done_folds = 0;                // folds of this call launched so far
  {
    int64_t m_sim = s.m;
    for (int64_t c = c0; c <= c_last; ++c) {
      const int64_t e = (c + 1) * C;
      if (e > pos1 || c < s.w - 1) continue;
      if (cf0 < 0) cf0 = c;
      const int64_t na = m_sim == 0 ? C : n_append_of(s.growth, e, m_sim, C);
      fold_na.push_back((int)na);
      m_sim += na;
    }
  }
  const int n_call_folds = (int)fold_na.size();
  const int halves = 2;
  const int per_batch = s.kbSlots / 2;   // (kbSlots >= 2)
  cudaStream_t kstream = ovk ? s.kbStream : stream;
  if (ovk && n_call_folds > 0) ev_ok = ev_ok && cudaStreamWaitEvent(kstream, s.evJoin, 0) == cudaSuccess;
  bool batch_done_rec[2] = {false, false};
  auto launch_batch = [&](int k) {      // batch k = folds [k*per_batch, ...) into slot half k % halves
    const int f0 = k * per_batch;
    if (f0 >= n_call_folds) return;
    const int nf = n_call_folds - f0 < per_batch ? n_call_folds - f0 : per_batch;
    const int h = k % halves;
    bool want_gram = false;              // does a fold of the batch append more than a few, not all, of its tokens?
    int64_t m_sim = s.m;
    for (int i = 0; i < f0 + nf; ++i) {
      // (m_sim restarts from the current rows: folds before f0 that are already launched moved s.m)
      if (i >= n_done_folds) { if (i >= f0 && fold_na[i] > gram_from(&s) && fold_na[i] < C && m_sim > 0) want_gram = true; m_sim += fold_na[i]; }
    }
    if (ovk && batch_done_rec[h]) ev_ok = ev_ok && cudaStreamWaitEvent(kstream, s.evBatchDone[h], 0) == cudaSuccess;
    const int64_t bf = (cf0 + f0 + 1) * C - L;   // first token of the first block of the batch
    s.launches += launch_kbar(&s, s.stK + (bf - ia.hist_start) * d, s.stRows * d, nf, h * per_batch, want_gram, kstream);
    if (ovk) ev_ok = ev_ok && cudaEventRecord(s.evKb[h], kstream) == cudaSuccess;
  };
  for (int64_t c = c0; c <= c_last; ++c) {
    const int64_t e = (c + 1) * C;
    const int64_t qs = c * C > pos0 ? c * C : pos0;
    const int64_t qe = e < pos1 ? e : pos1;
    int64_t b = e - L; if (b < 0) b = 0;
    aa.q_row0 = qs - pos0; aa.nq = (int)(qe - qs); aa.t0 = qs; aa.m = s.m;
    aa.win_row0 = b - ia.hist_start; aa.b = b; aa.out = (__nv_bfloat16*)out; aa.out_t0 = qs - pos0;
    if (ovf && fold_pending >= 0) {
      ev_ok = ev_ok && cudaStreamWaitEvent(stream, s.evFold[fold_pending], 0) == cudaSuccess;
      fold_pending = -1;
    }
    s.launches += launch_prev_copy(&s, stream);
    if (ovf) ev_ok = ev_ok && cudaEventRecord(s.evPre[c & 1], stream) == cudaSuccess;
    {
      KernelTimer pt(&s, 1, stream);
      if (s.flags & KVM_FLAG_SIMT_ATTENTION) s.launches += launch_attn_simt(&s, aa, stream);
      else s.launches += launch_attn_tc(&s, aa, stream);
    }
    if (qe == e && c >= s.w - 1) {
      const int fi = n_done_folds, bk = fi / per_batch;
      if (fi % per_batch == 0) {
        if (!ovk || fi == 0) launch_batch(bk);            // (with one stream: just in time)
        if (ovk) {
          launch_batch(bk + 1);                            // one batch ahead
          ev_ok = ev_ok && cudaStreamWaitEvent(fstream, s.evKb[bk % halves], 0) == cudaSuccess;
        }
      }
      FoldArgs fa;
      fa.ok = s.stK + (b - ia.hist_start) * d; fa.ov = s.stV + (b - ia.hist_start) * d; fa.og = s.stG + (b - ia.hist_start);
      fa.unit_stride = s.stRows * d; fa.gate_stride = s.stRows;
      fa.b = b; fa.m = s.m; fa.first = (s.m == 0);
      fa.n_append = fa.first ? C : (int)n_append_of(s.growth, e, s.m, C);
      fa.slot = (bk % halves) * per_batch + fi % per_batch;
      // only the last kernel of the fold writes the readout copy: the routing filter and the
      // decisions run while the caller's stream still copies the previous fold's rows
      fa.before_apply = ovf ? s.evPre[c & 1] : nullptr;
      fa.early_start = true;
      {
        const int nl = launch_fold(&s, fa, fstream);
        if (nl < 0) ev_ok = false; else s.launches += nl;
      }
      s.m += fa.n_append;
      s.nfolds += 1;
      n_done_folds += 1;
      if (ovk && (n_done_folds % per_batch == 0 || n_done_folds == n_call_folds)) {
        ev_ok = ev_ok && cudaEventRecord(s.evBatchDone[bk % halves], fstream) == cudaSuccess;
        batch_done_rec[bk % halves] = true;
      }
      if (ovf) {
        fold_pending = (int)(s.nfolds & 1);
        ev_ok = ev_ok && cudaEventRecord(s.evFold[fold_pending], fstream) == cudaSuccess;
      }
    }
  }
  if (ovf && fold_pending >= 0) ev_ok = ev_ok && cudaStreamWaitEvent(stream, s.evFold[fold_pending], 0) == cudaSuccess;
  s.pos = pos1;
  if (!ev_ok) { cudaGetLastError(); return KVM_ERR_CUDA; }
  return launch_ok() ? KVM_OK : KVM_ERR_CUDA;
}

KVM_API kvm_status_t kvm_decode_step(const void* q, const void* k, const void* v, kvm_state_t* ks, const float* gate,
                             void* out, void* cuda_stream) {
  if (!q || !k || !v || !ks || !out) return KVM_ERR_INVALID_ARG;
  State& s = ks->s;
  if (!s.bound) return KVM_ERR_STATE_MISMATCH;
  if (((uintptr_t)q & 1) || ((uintptr_t)k & 1) || ((uintptr_t)v & 1) || ((uintptr_t)out & 1)) return KVM_ERR_INVALID_ARG;
  if (s.fusedLn && ((((uintptr_t)q | (uintptr_t)k | (uintptr_t)v) & 15) != 0)) return KVM_ERR_INVALID_ARG;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  DeviceGuard guard(s.device);
  if (!guard.ok) return KVM_ERR_CUDA;
  const int C = s.C, d = s.d;
  const int64_t L = (int64_t)s.w * C;
  const int64_t t = s.pos, c = t / C, e = (c + 1) * C;
  if (s.growth.kind == KVM_GROWTH_POWER && e >= kPowerMaxPos) return KVM_ERR_UNSUPPORTED;
  int64_t b = e - L; if (b < 0) b = 0;
  const bool fold = ((t + 1) % C == 0) && c >= s.w - 1;
  int n_a = 0;
  if (fold) {
    n_a = (s.m == 0) ? C : (int)n_append_of(s.growth, e, s.m, C);
    if (s.m + n_a > s.Mcap) return KVM_ERR_CAPACITY;
  }
  DecodeArgs da;
  da.q = (const __nv_bfloat16*)q; da.k = (const __nv_bfloat16*)k; da.v = (const __nv_bfloat16*)v; da.gate = gate;
  da.out = (__nv_bfloat16*)out; da.t = t; da.b = b; da.m = s.m;
  { KernelTimer pt(&s, 6, stream); s.launches += launch_decode(&s, da, stream); }
  if (fold) {
    const int64_t ringCap = (int64_t)s.w * s.Cmax;
    const int64_t slot = b % s.ringLen;
    FoldArgs fa;
    fa.ok = s.ringK + slot * d; fa.ov = s.ringV + slot * d; fa.og = s.ringG + slot;
    fa.unit_stride = ringCap * d; fa.gate_stride = ringCap;
    fa.b = b; fa.m = s.m; fa.first = (s.m == 0); fa.n_append = n_a; fa.slot = 0; fa.before_apply = nullptr;
    fa.early_start = false;   // the memory-key kernel runs right before the filter on this stream
    s.launches += launch_prev_copy(&s, stream);
    s.launches += launch_kbar(&s, fa.ok, fa.unit_stride, 1, 0, n_a > gram_from(&s) && n_a < C && s.m > 0, stream);
    s.launches += launch_fold(&s, fa, stream);
    s.m += n_a;
    s.nfolds += 1;
  }
  s.pos = t + 1;
  return launch_ok() ? KVM_OK : KVM_ERR_CUDA;
}

KVM_API kvm_status_t kvm_prefill_host(const void* q_host, const void* k_host, const void* v_host, kvm_state_t* ks,
                              int32_t block, kvm_growth_t growth, int32_t rope_dims, int64_t n_tokens,
                              const float* gate_host, void* out_host, void* cuda_stream) {
  if (!q_host || !k_host || !v_host || !ks || !out_host) return KVM_ERR_INVALID_ARG;
  State& s = ks->s;
  if (n_tokens < 1) return KVM_ERR_INVALID_ARG;
  if (n_tokens > s.Tcall) return KVM_ERR_CAPACITY;
  // the whole call is validated before the first copy is enqueued: a call that fails leaves the
  // state and the caller's buffers untouched
  kvm_status_t rc = validate_prefill(s, block, growth, rope_dims, n_tokens);
  if (rc != KVM_OK) return rc;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  DeviceGuard guard(s.device);
  if (!guard.ok) return KVM_ERR_CUDA;
  rc = ensure_host_staging(ks);
  if (rc != KVM_OK) return rc;
  // The call is cut into up to eight segments of at least two whole blocks; segment i+1 is copied in, and segment
  // i-1 copied out, while segment i is computed (three streams, the copies as strided 2-D copies into /
  // out of staging buffers that have the host layout [batch, head, token, channel]).
  const int64_t n = n_tokens;
  const int64_t d = s.d;
  int nseg = (int)(n / (2 * (int64_t)block));   // (the last segment's compute and copy-out are not overlapped: keep it short)
  if (nseg > 8) nseg = 8;
  if (nseg < 1) nseg = 1;
  const int64_t seg_len = ((n + nseg - 1) / nseg + block - 1) / block * block;
  // a failure after the first copy was enqueued (a CUDA error; the arguments were checked above): the
  // caller gets its buffers back only once nothing reads or writes them any more
  auto fail = [&](kvm_status_t code) {
    cudaGetLastError();
    cudaStreamSynchronize(s.hinStream); cudaStreamSynchronize(s.houtStream); cudaStreamSynchronize(stream);
    cudaGetLastError();
    return code;
  };
  bool ok = cudaEventRecord(s.evHostStart, stream) == cudaSuccess;
  ok = ok && cudaStreamWaitEvent(s.hinStream, s.evHostStart, 0) == cudaSuccess;
  ok = ok && cudaStreamWaitEvent(s.houtStream, s.evHostStart, 0) == cudaSuccess;
  if (!ok) return fail(KVM_ERR_CUDA);
  kvm_strides_t st;
  st.q[0] = (int64_t)s.Hq * n * d; st.q[1] = n * d; st.q[2] = d; st.q[3] = 1;
  st.k[0] = (int64_t)s.Hkv * n * d; st.k[1] = n * d; st.k[2] = d; st.k[3] = 1;
  for (int i = 0; i < 4; ++i) { st.v[i] = st.k[i]; st.out[i] = st.q[i]; }
  const size_t pitch = (size_t)n * d * 2;
  int iseg = 0;
  for (int64_t t0 = 0; t0 < n; t0 += seg_len, ++iseg) {
    const int64_t len = t0 + seg_len <= n ? seg_len : n - t0;
    const size_t width = (size_t)len * d * 2;
    const size_t off = (size_t)t0 * d;   // elements
    ok = cudaMemcpy2DAsync((__nv_bfloat16*)s.hQ + off, pitch, (const __nv_bfloat16*)q_host + off, pitch, width,
                           (size_t)s.B * s.Hq, cudaMemcpyHostToDevice, s.hinStream) == cudaSuccess;
    ok = ok && cudaMemcpy2DAsync((__nv_bfloat16*)s.hK + off, pitch, (const __nv_bfloat16*)k_host + off, pitch, width,
                                 (size_t)s.U, cudaMemcpyHostToDevice, s.hinStream) == cudaSuccess;
    ok = ok && cudaMemcpy2DAsync((__nv_bfloat16*)s.hV + off, pitch, (const __nv_bfloat16*)v_host + off, pitch, width,
                                 (size_t)s.U, cudaMemcpyHostToDevice, s.hinStream) == cudaSuccess;
    float* gseg = nullptr;
    if (gate_host) {   // gates of the segment, contiguous [unit, token] as kvm_prefill expects them
      gseg = s.hG + (size_t)s.U * t0;
      ok = ok && cudaMemcpy2DAsync(gseg, (size_t)len * 4, gate_host + t0, (size_t)n * 4, (size_t)len * 4, (size_t)s.U,
                                   cudaMemcpyHostToDevice, s.hinStream) == cudaSuccess;
    }
    ok = ok && cudaEventRecord(s.evIn[iseg], s.hinStream) == cudaSuccess;
    ok = ok && cudaStreamWaitEvent(stream, s.evIn[iseg], 0) == cudaSuccess;
    if (!ok) return fail(KVM_ERR_CUDA);
    rc = kvm_prefill((__nv_bfloat16*)s.hQ + off, (__nv_bfloat16*)s.hK + off, (__nv_bfloat16*)s.hV + off, ks, block, growth,
                     rope_dims, len, gseg, (__nv_bfloat16*)s.hOut + off, &st, cuda_stream);
    if (rc != KVM_OK) return fail(rc);
    ok = cudaEventRecord(s.evComp[iseg], stream) == cudaSuccess;
    ok = ok && cudaStreamWaitEvent(s.houtStream, s.evComp[iseg], 0) == cudaSuccess;
    ok = ok && cudaMemcpy2DAsync((__nv_bfloat16*)out_host + off, pitch, (__nv_bfloat16*)s.hOut + off, pitch, width,
                                 (size_t)s.B * s.Hq, cudaMemcpyDeviceToHost, s.houtStream) == cudaSuccess;
    if (!ok) return fail(KVM_ERR_CUDA);
  }
  ok = cudaEventRecord(s.evHostOut, s.houtStream) == cudaSuccess;
  ok = ok && cudaStreamWaitEvent(stream, s.evHostOut, 0) == cudaSuccess;
  ok = ok && cudaStreamSynchronize(stream) == cudaSuccess;
  if (!ok) return fail(KVM_ERR_CUDA);
  return KVM_OK;
}

KVM_API kvm_status_t kvm_decode_step_host(const void* q_host, const void* k_host, const void* v_host, kvm_state_t* ks,
                                  const float* gate_host, void* out_host, void* cuda_stream) {
  if (!q_host || !k_host || !v_host || !ks || !out_host) return KVM_ERR_INVALID_ARG;
  State& s = ks->s;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  DeviceGuard guard(s.device);
  if (!guard.ok) return KVM_ERR_CUDA;
  kvm_status_t rc = ensure_host_staging(ks);
  if (rc != KVM_OK) return rc;
  const size_t bq = (size_t)s.B * s.Hq * s.d * 2, bk = (size_t)s.U * s.d * 2;
  bool ok = cudaMemcpyAsync(s.hQ, q_host, bq, cudaMemcpyHostToDevice, stream) == cudaSuccess;
  ok = ok && cudaMemcpyAsync(s.hK, k_host, bk, cudaMemcpyHostToDevice, stream) == cudaSuccess;
  ok = ok && cudaMemcpyAsync(s.hV, v_host, bk, cudaMemcpyHostToDevice, stream) == cudaSuccess;
  if (gate_host) ok = ok && cudaMemcpyAsync(s.hG, gate_host, (size_t)s.U * 4, cudaMemcpyHostToDevice, stream) == cudaSuccess;
  if (!ok) { cudaGetLastError(); return KVM_ERR_CUDA; }
  rc = kvm_decode_step(s.hQ, s.hK, s.hV, ks, gate_host ? s.hG : nullptr, s.hOut, cuda_stream);
  if (rc != KVM_OK) return rc;
  if (cudaMemcpyAsync(out_host, s.hOut, bq, cudaMemcpyDeviceToHost, stream) != cudaSuccess) return KVM_ERR_CUDA;
  if (cudaStreamSynchronize(stream) != cudaSuccess) return KVM_ERR_CUDA;
  return KVM_OK;
}

KVM_API kvm_status_t kvm_state_export(kvm_state_t* ks, double* sum_k, float* sum_v, float* radius, double* weight,
                              int32_t* count, void* k_read, void* v_read, void* cuda_stream) {
  if (!ks) return KVM_ERR_INVALID_ARG;
  State& s = ks->s;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  DeviceGuard guard(s.device);
  if (!guard.ok) return KVM_ERR_CUDA;
  const size_t m = (size_t)s.m, M = (size_t)s.Mcap, d = (size_t)s.d, U = (size_t)s.U;
  bool ok = true;
  if (m > 0) {
#define CP(dst, src, elt, width) \
  if (dst) ok = ok && cudaMemcpy2DAsync(dst, m * (width) * (elt), src, M * (width) * (elt), m * (width) * (elt), U, cudaMemcpyDeviceToHost, stream) == cudaSuccess
    CP(sum_k, s.sumK, sizeof(double), d);
    CP(sum_v, s.sumV, sizeof(float), d);
    CP(radius, s.rho, sizeof(float), (size_t)1);
    CP(weight, s.wsum, sizeof(double), (size_t)1);
    CP(count, s.cnt, sizeof(int32_t), (size_t)1);
    CP(k_read, s.KhatBuf[s.nfolds & 1], (size_t)2, d);
    CP(v_read, s.VhatBuf[s.nfolds & 1], (size_t)2, d);
#undef CP
  }
  ok = ok && cudaStreamSynchronize(stream) == cudaSuccess;
  if (!ok) { cudaGetLastError(); return KVM_ERR_CUDA; }
  return KVM_OK;
}

KVM_API kvm_status_t kvm_state_snapshot_info(const kvm_state_t* ks, kvm_snapshot_info_t* out) {
  if (!ks || !out) return KVM_ERR_INVALID_ARG;
  const State& s = ks->s;
  memset(out, 0, sizeof(*out));
  if (!s.bound) return KVM_OK;
  out->block = s.C; out->rope_dims = s.r; out->growth = s.growth;
  out->n_slots = s.m; out->position = s.pos; out->n_folds = s.nfolds;
  int64_t wb = (s.pos / s.C + 1) * s.C - (int64_t)s.w * s.C;   // first token that the next block's window still holds
  if (wb < 0) wb = 0;
  out->window_begin = wb; out->window_len = s.pos - wb;
  return KVM_OK;
}

KVM_API kvm_status_t kvm_state_export_window(kvm_state_t* ks, void* win_k, void* win_v, float* win_gate, void* cuda_stream) {
  if (!ks) return KVM_ERR_INVALID_ARG;
  State& s = ks->s;
  if (!s.bound) return KVM_ERR_STATE_MISMATCH;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  DeviceGuard guard(s.device);
  if (!guard.ok) return KVM_ERR_CUDA;
  kvm_snapshot_info_t info;
  kvm_state_snapshot_info(ks, &info);
  const size_t d = (size_t)s.d, U = (size_t)s.U, ringCap = (size_t)s.w * s.Cmax, len = (size_t)info.window_len;
  bool ok = for_ring_runs(s, info.window_begin, info.window_len, [&](int64_t at, int64_t slot, int64_t run) {
    bool k = true;
    if (win_k) k = k && cudaMemcpy2DAsync((__half*)win_k + at * d, len * d * 2, s.ringK + slot * d, ringCap * d * 2, run * d * 2, U, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    if (win_v) k = k && cudaMemcpy2DAsync((__half*)win_v + at * d, len * d * 2, s.ringV + slot * d, ringCap * d * 2, run * d * 2, U, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    if (win_gate) k = k && cudaMemcpy2DAsync(win_gate + at, len * 4, s.ringG + slot, ringCap * 4, run * 4, U, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    return k;
  });
  ok = ok && cudaStreamSynchronize(stream) == cudaSuccess;
  if (!ok) { cudaGetLastError(); return KVM_ERR_CUDA; }
  return KVM_OK;
}

KVM_API kvm_status_t kvm_state_import(kvm_state_t* ks, const kvm_snapshot_info_t* info, const double* sum_k, const float* sum_v,
                              const float* radius, const double* weight, const int32_t* count, const void* win_k,
                              const void* win_v, const float* win_gate, void* cuda_stream) {
  if (!ks || !info) return KVM_ERR_INVALID_ARG;
  State& s = ks->s;
  // ---- validation on the host; nothing is touched before it has passed ----
  const int C = info->block, r = info->rope_dims;
  if (C < 8 || (C % 8) != 0 || s.S >= C) return KVM_ERR_INVALID_ARG;
  if (C > s.Cmax) return KVM_ERR_CAPACITY;
  if (r < 0 || r > s.d || (r & 1) || !growth_valid(info->growth)) return KVM_ERR_INVALID_ARG;
  if (info->position < 0 || info->n_slots < 0 || info->n_folds < 0) return KVM_ERR_INVALID_ARG;
  if (info->growth.kind == KVM_GROWTH_POWER && info->position >= kPowerMaxPos) return KVM_ERR_UNSUPPORTED;
  {
    // rows and folds follow from the position by the budget rule; the window from the block structure
    int64_t m = 0, nf = 0;
    for (int64_t c = s.w - 1; (c + 1) * C <= info->position; ++c) {
      m += (m == 0) ? C : n_append_of(info->growth, (c + 1) * C, m, C);
      ++nf;
    }
    int64_t wb = (info->position / C + 1) * C - (int64_t)s.w * C;
    if (wb < 0) wb = 0;
    if (m != info->n_slots || nf != info->n_folds || wb != info->window_begin || info->window_len != info->position - wb)
      return KVM_ERR_INVALID_ARG;
    if (m > s.Mcap) return KVM_ERR_CAPACITY;
  }
  if (info->n_slots > 0 && (!sum_k || !sum_v || !radius || !weight || !count)) return KVM_ERR_INVALID_ARG;
  if (info->window_len > 0 && (!win_k || !win_v)) return KVM_ERR_INVALID_ARG;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  DeviceGuard guard(s.device);
  if (!guard.ok) return KVM_ERR_CUDA;

  kvm_state_reset(ks);
  bind_state(s, C, info->growth, r);
  s.pos = info->position; s.m = info->n_slots; s.nfolds = info->n_folds;
  const size_t m = (size_t)s.m, M = (size_t)s.Mcap, d = (size_t)s.d, U = (size_t)s.U;
  bool ok = true;
  if (m > 0) {
#define CP(dst, src, elt, width) \
  ok = ok && cudaMemcpy2DAsync(dst, M * (width) * (elt), src, m * (width) * (elt), m * (width) * (elt), U, cudaMemcpyHostToDevice, stream) == cudaSuccess
    CP(s.sumK, sum_k, sizeof(double), d);
    CP(s.sumV, sum_v, sizeof(float), d);
    CP(s.rho, radius, sizeof(float), (size_t)1);
    CP(s.wsum, weight, sizeof(double), (size_t)1);
    CP(s.cnt, count, sizeof(int32_t), (size_t)1);
#undef CP
    if (ok) s.launches += launch_refresh_rows(&s, s.m, stream);
  }
  const size_t ringCap = (size_t)s.w * s.Cmax, len = (size_t)info->window_len;
  std::vector<float> ones;
  if (len > 0 && !win_gate) ones.assign(U * len, 1.0f);
  const float* wg = win_gate ? win_gate : ones.data();
  ok = ok && for_ring_runs(s, info->window_begin, info->window_len, [&](int64_t at, int64_t slot, int64_t run) {
    bool k = cudaMemcpy2DAsync(s.ringK + slot * d, ringCap * d * 2, (const __half*)win_k + at * d, len * d * 2, run * d * 2, U, cudaMemcpyHostToDevice, stream) == cudaSuccess;
    k = k && cudaMemcpy2DAsync(s.ringV + slot * d, ringCap * d * 2, (const __half*)win_v + at * d, len * d * 2, run * d * 2, U, cudaMemcpyHostToDevice, stream) == cudaSuccess;
    k = k && cudaMemcpy2DAsync(s.ringG + slot, ringCap * 4, wg + at, len * 4, run * 4, U, cudaMemcpyHostToDevice, stream) == cudaSuccess;
    return k;
  });
  ok = ok && cudaStreamSynchronize(stream) == cudaSuccess;
  ok = ok && launch_ok();
  if (!ok) { cudaGetLastError(); kvm_state_reset(ks); return KVM_ERR_CUDA; }
  return KVM_OK;
}

KVM_API kvm_status_t kvm_debug_assignments(kvm_state_t* ks, int64_t n, int32_t* slot_of_token, uint8_t* was_appended,
                                   void* cuda_stream) {
  if (!ks || n < 0) return KVM_ERR_INVALID_ARG;
  State& s = ks->s;
  if (s.Tassign == 0) return KVM_ERR_STATE_MISMATCH;
  if (n > s.pos || n > s.Tassign) return KVM_ERR_INVALID_ARG;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  DeviceGuard guard(s.device);
  if (!guard.ok) return KVM_ERR_CUDA;
  bool ok = true;
  if (n > 0) {
    if (slot_of_token)
      ok = ok && cudaMemcpy2DAsync(slot_of_token, n * 4, s.slotTok, s.Tassign * 4, n * 4, s.U, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    if (was_appended)
      ok = ok && cudaMemcpy2DAsync(was_appended, n, s.appTok, s.Tassign, n, s.U, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
  }
  ok = ok && cudaStreamSynchronize(stream) == cudaSuccess;
  if (!ok) { cudaGetLastError(); return KVM_ERR_CUDA; }
  return KVM_OK;
}

}  // extern "C"
