// Internal declarations shared by the translation units of libkvm (not installed).
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "kvm.h"

namespace kvm {

constexpr int kMaxBlock = 256;      // largest block C (one thread per overflow token in the fold)
constexpr int kTopK = 8;            // routing filter keeps at most K candidate rows per (token, row split)
constexpr int kChunkCap = 16;       // 32-row chunks of approximate similarities the routing filter can record per (token, row split)
constexpr int kMaxSplits = 32;      // routing filter / decode split count upper bound
constexpr int kAttnSplitTiles = 37; // launches with at most this many (batch, head, query tile) CTAs - a quarter of the GPU - are split along the keys
constexpr int kAttnMaxSplits = 8;
constexpr int kRowAlign = 128;      // state capacity is rounded up to the attention key tile
constexpr int kGramOnTheFly = 32;   // in a state with enough units to fill the GPU (State::serial), folds that append at most this
                                    // many rows compute the products of the other tokens with the new rows inside the decision
                                    // kernel; all other folds read them from the batched tensor-core product of all token pairs of
                                    // the block (gramT), computed off the folds' critical path - most of it never read
constexpr int kSerialUnits = 256;   // from this many (batch, kv head) units on, folds run on the caller's stream with one readout copy

// State of one layer: host bookkeeping + device buffers.  U = batch * n_kv_heads "units";
// unit u = b * Hkv + hk owns rows [u*Mcap, (u+1)*Mcap) of every per-row array.
struct State {
  // ---- configuration (host) ----
  int B, Hq, Hkv, d, G, U, w, S;
  int Cmax;            // max block
  int64_t Mcap;        // state rows capacity (multiple of kRowAlign)
  int64_t Tcall;       // max tokens per prefill call
  int64_t Tassign;     // max_seq_len for assignment recording (0 = off)
  float rope_base, ln_eps, norm_eps;
  uint32_t flags;
  int device;
  float sim_norm_bound;  // upper bound of ||LN_s(x)||_2 for any x (per layer)
  // ---- bound by the first prefill ----
  bool bound;
  int C, r;
  kvm_growth_t growth;
  int64_t ringLen;     // w * C
  // ---- progress (host) ----
  int64_t pos, m, nfolds, launches;
  // ---- parameters (device) ----
  float *ln_w, *ln_b;     // [Hkv, d]
  float *tau_s, *tau_b;   // [Hq]
  // fused front end (KVM_FLAG_FUSED_QK_LN): LN_q / LN_k weights and biases, [Hq, d] / [Hkv, d] (NULL = 1 / 0)
  bool fusedLn;
  float qk_ln_eps;
  float *lnq_w, *lnq_b, *lnk_w, *lnk_b;
  double* inv_freq;       // [r/2]: the bound rope_dims' slice of inv_freq_all
  double* inv_freq_all;   // base^(-2i/r), i < r/2, for every even r <= d, r's slice at offset (r/2)(r/2 - 1)/2
  bool assignDirty;       // recorded assignments of an earlier sequence are still in slotTok (cleared by the next prefill)
  // ---- state rows (device) ----
  double* sumK;           // [U, Mcap, d]  running key sums (fp64: routing decisions are taken on them)
  float* sumV;            // [U, Mcap, d]
  float* rho;             // [U, Mcap]
  double* wsum;           // [U, Mcap]
  int32_t* cnt;           // [U, Mcap]
  double *kmu, *krstd;    // [U, Mcap]   mean / rstd of LN_s(s^K_i)
  // Readout cache (fp16): LN_s(s^K) and the value readout, each [U, Mcap, d]; operand of attention,
  // decode and the routing filter.  Two copies: the state after f folds is read from copy f & 1, so
  // fold f+1 can write copy (f+1) & 1 while the attention of the current block still reads copy f & 1.
  __half *KhatBuf[2], *VhatBuf[2];
  bool serial;            // one readout copy (KhatBuf[1] == KhatBuf[0]), folds on the caller's stream
  // what the previous fold touched (host): its rows are copied into the other copy (launch_prev_copy)
  // before the next fold writes there; prevValid = such a copy is still owed
  bool prevValid, prevAllAppend;
  int64_t prevM;
  int prevNAppend;
  // second stream and events that let a block's attention and the fold of the block before it overlap
  cudaStream_t foldStream, kbStream;   // folds; memory keys computed ahead of the folds
  // host-buffer entry points: copy-in / copy-out streams and per-segment events (created on first use)
  cudaStream_t hinStream, houtStream;
  cudaEvent_t evHostStart, evHostOut, evIn[8], evComp[8];
  cudaEvent_t evJoin, evPre[2], evFold[2], evKb[2], evBatchDone[2];
  // ---- window ring (device): slot = t mod ringLen ----
  __half *ringK, *ringV;         // [U, w*Cmax, d]  rotated keys / values (fp16)
  float* ringG;                  // [U, w*Cmax]
  // ---- per-call staging (device) ----
  int64_t stRows;                // w*Cmax + Tcall
  __half* stQ;                   // [B*Hq, Tcall, d] rotated queries (fp16)
  __half *stK, *stV;             // [U, stRows, d]   history + new tokens (rotated keys, fp16)
  float* stG;                    // [U, stRows]
  float2* ropeCS;                // [Tcall, r/2] (cos, sin)
  // ---- fold scratch (device).  The memory keys depend on the block's own keys only, so a prefill
  //      call computes them for up to kbSlots consecutive overflow blocks in one launch; slot g holds
  //      one block's arrays in the layouts below ----
  int kbSlots;
  bool recomputeK;               // (bound with the block) serial && the four-rows-per-warp apply kernel: kbar64 is not kept,
                                 // the fold kernels recompute kbar_j from the fp16 key and kbarStat
  double2* kbarStat;             // [kbSlots][U, Cmax]  (mean, rstd) of zero_r(k_j)
  double* kbar64;                // [kbSlots][U, Cmax, d]
  __half* kbarH;                 // [kbSlots][U, CbarRows, d]
  float* kbarNorm;               // [kbSlots][U, Cmax]
  int CbarRows;                  // rows per unit of kbarH (Cmax rounded up to the 128-row MMA tile)
  double2* kbarHatStat;          // [kbSlots][U, Cmax]  (mean, rstd) of kbar_j: LN_s(kbar_j), the readout key of a row
                                 // created by token j, is recomputed from kbar64 and these where it is needed
  __half* kbarHatH;              // [kbSlots][U, CbarRows, d]  the same in fp16 (operand of the new-row filter)
  float* gramT;                  // [kbSlots][U, Cmax, Cmax]  approximate kbarHat_a . kbar_j at [a][j] (new-row filter)
  // decisions of the fold being computed ([(nfolds+1) & 1]) and of the one before ([nfolds & 1])
  int32_t *foldPi[2], *foldSorted[2], *foldCreator[2], *foldSegNew[2], *foldNMerge[2];
  double *xScore, *xBest;        // [U, Cmax] hand-over between the CTAs of the decide kernel
  int32_t *xArg, *xCount;        // [U, Cmax]; [U]
  int nsplitRoute;               // splits the routing filter may use
  float* candV;                  // [U, nsplitRoute, Cmax, kTopK]  routing filter output: (split maximum, candidate count, ...)
  int32_t* candI;                // [U, nsplitRoute, Cmax, kTopK]  candidate rows
  // scratch of the routing filter's threads: the 32-row chunks of products a token recorded on its way through
  // the split (maximum, first row and mask of valid rows, the 32 products)
  float* chunkMax;               // [U, nsplitRoute, Cmax, kChunkCap]
  int2* chunkMeta;               // [U, nsplitRoute, Cmax, kChunkCap]
  float* chunkVal;               // [U, nsplitRoute, Cmax, kChunkCap, 32]
  // ---- split-KV attention scratch (device) ----
  float* attnPart;               // [kAttnSplitTiles][kAttnMaxSplits][d + 2][128]
  int32_t* attnCnt;              // [2 kAttnSplitTiles] tickets
  // ---- decode scratch (device) ----
  int nsplitDec;
  float* decPart;                // [B*Hq, nsplitDec, d + 2]
  __half* decQ;                  // [B*Hq, d] rotated query
  // ---- optional per-kernel timing hook (set by kvm_profile_enable): phase ids
  //      0 ingest, 1 attention, 2 memory keys, 3 routing filter, 4 decide, 5 apply, 6 decode ----
  void (*prof_hook)(void* ctx, int phase, int begin, cudaStream_t s);
  void* prof_ctx;
  // ---- recording / status ----
  int32_t* slotTok;              // [U, Tassign]
  uint8_t* appTok;               // [U, Tassign]
  int32_t* status;               // device status word [0]; [1..3] fold debug counters; [4] inputs clamped to the fp16 range
  // ---- TMA tensor maps (host copies, passed to kernels by value):
  //      0 stQ, 1 Khat copy 0, 2 Vhat copy 0, 3 stK, 4 stV, 5 kbarH, 6 Khat copy 1, 7 Vhat copy 1,
  //      8 kbarHatH ----
  alignas(64) unsigned char tmaps[9 * 128];
  // ---- device staging for the *_host entry points ----
  void *hQ, *hK, *hV, *hOut;
  float* hG;
};

inline int64_t budget_of(const kvm_growth_t& g, int64_t e);
// folds that append more rows than this (and not the whole block) take the batched product of the block's token pairs
inline int gram_from(const State* st) { return st->serial ? kGramOnTheFly : 0; }

// ---------------- launchers (each returns the number of kernels it launched) ----------------

struct IngestArgs {
  const __nv_bfloat16 *q, *k, *v;
  const float* gate;
  int64_t sq[4], sk[4], sv[4];  // element strides (B, H, T, 1)
  int64_t sg[3];
  int64_t pos0, n, hist_start, nhist, tail_start;
};
int launch_ingest(State* st, const IngestArgs& a, cudaStream_t s);
bool ingest_rows_aligned(int r, const IngestArgs& a);   // rows 16-byte aligned, rotary half whole 8-channel chunks

struct AttnArgs {
  int64_t q_row0;      // first query row in stQ (local token index)
  int nq;              // queries in this launch (<= C)
  int64_t t0;          // absolute position of the first query
  int64_t m;           // visible state rows
  int64_t win_row0;    // row in stK/stV of window begin b
  int64_t b;           // absolute position of window begin
  __nv_bfloat16* out;  // user tensor
  int64_t so[4];       // out strides
  int64_t out_t0;      // token index inside `out` of the first query
};
int launch_attn_simt(State* st, const AttnArgs& a, cudaStream_t s);
int launch_attn_tc(State* st, const AttnArgs& a, cudaStream_t s);
bool setup_attn_tc(State* st);   // encodes the tensor maps, raises the shared-memory limits
bool setup_route_tc(State* st);
// Width of the candidate window of the routing filter per unit of ||kbar_j||: twice the bound on the
// error of an fp16 x fp16 -> fp32 dot product against LN_s rows.  fp16 rounding of both operands
// gives |err| <= (2u + u^2) |a|.|b| with u = 2^-11; 2^-13 |a|.|b| more covers fp16 subnormals and
// 128 truncating fp32 additions.
inline float route_thr_coeff(const State* st) { return 2.0f * (1.0f / 1024.0f + 1.0f / 8192.0f) * st->sim_norm_bound; }

struct FoldArgs {
  const __half *ok, *ov;         // overflow block rows: unit u at ok + u*unit_stride (elements), C rows
  const float* og;               // gates, unit u at og + u*gate_stride
  int64_t unit_stride, gate_stride;
  int64_t b;        // absolute position of the first overflow token
  int64_t m;        // rows before the fold
  int n_append;     // rows to append (== C on the first fold)
  bool first;       // first state-creation step
  int slot;         // memory-key slot that holds this block's keys (launch_kbar)
  cudaEvent_t before_apply;   // if set, the stream waits for it before the kernel that writes the readout copy
  bool early_start;           // the routing filter may start under the kernel before it on the stream (programmatic
                              // dependent launch) and fetch the block's memory keys before it waits: only where that
                              // kernel is not the one that writes those keys
};
int launch_fold(State* st, const FoldArgs& a, cudaStream_t s);
// Memory keys of nblk consecutive blocks (C rows each, starting at ok within every unit) into slots
// slot0 .. slot0 + nblk - 1.
int launch_kbar(State* st, const __half* ok, int64_t unit_stride, int nblk, int slot0, bool want_gram, cudaStream_t s);
// Copies the readout rows that the last fold touched from the current readout copy into the other
// one (no-op when nothing is owed).  Must run after every reader of the other copy has finished and
// before the next fold writes it.
int launch_prev_copy(State* st, cudaStream_t s);
// Recomputes the row statistics and both readout copies of rows [0, m) from the stored sums (snapshot import).
int launch_refresh_rows(State* st, int64_t m, cudaStream_t s);

struct DecodeArgs {
  const __nv_bfloat16 *q, *k, *v;
  const float* gate;
  __nv_bfloat16* out;
  int64_t t;   // absolute position of the token
  int64_t b;   // window begin
  int64_t m;
};
int launch_decode(State* st, const DecodeArgs& a, cudaStream_t s);

// Self test of the bounded waits: one thread waits `spins` iterations on a barrier nobody arrives at and
// records KVM_ERR_TIMEOUT in the status word.
void launch_expire_wait(State* st, int spins, cudaStream_t s);

// Brackets the launches issued during its lifetime with the state's timing hook (no-op when off).
struct KernelTimer {
  State* st; int phase; cudaStream_t s;
  KernelTimer(State* st_, int phase_, cudaStream_t s_) : st(st_), phase(phase_), s(s_) {
    if (st->prof_hook) st->prof_hook(st->prof_ctx, phase, 1, s);
  }
  ~KernelTimer() { if (st->prof_hook) st->prof_hook(st->prof_ctx, phase, 0, s); }
};

}  // namespace kvm
