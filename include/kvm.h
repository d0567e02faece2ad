/*
 * kvm.h -- C ABI of the Key-Value Means (KVM) attention layer for NVIDIA B200 (sm_100a).
 *
 * The library implements the sequence-mixing hot path of the paper
 * "Key-Value Means: Transformers with Expandable Block-Recurrent Compressed
 * Memory" (Section 3 "Method", Appendix B "Pseudocode"): for every block (chunk)
 * of the sequence one softmax attention over [compressed state ; exact block
 * sliding window], then the fold of the block that leaves the window into the
 * state (append / merge / value-radius preservation under a state budget), and
 * the matching single-token decode step.
 *
 * Conventions
 *   - All tensors named "device" are CUDA device pointers owned by the caller;
 *     the library never frees or keeps them beyond the call.  Element type of
 *     q/k/v/out is bfloat16.  Layout is [batch, heads, tokens, head_dim] with
 *     optional element strides (head_dim stride must be 1).
 *   - The state object and every scratch buffer are owned by the library and are
 *     allocated once in kvm_state_create(); no call on the hot path allocates.
 *   - Work is enqueued on the given CUDA stream (a cudaStream_t passed as
 *     void*; NULL = default stream).  No entry point synchronises the host with
 *     the device except those that move data to or from HOST memory: kvm_state_export,
 *     kvm_state_export_window, kvm_state_import, kvm_debug_assignments, kvm_debug_counters,
 *     kvm_state_check, kvm_profile_read and the *_host convenience variants.
 *   - Host-side validation happens before any launch; a failed call leaves the
 *     state untouched.  There is no CPU fallback: without a CUDA device
 *     kvm_state_create() returns KVM_ERR_CUDA.
 *   - Inside the library bf16 inputs are carried as fp16 (tensor-core operands, readout
 *     cache, softmax weights): every bf16 value with 2^-14 <= |x| <= 65504 converts exactly,
 *     larger magnitudes saturate at +-65504.  Accumulation is fp32; routing decisions fp64.
 *   - Results are deterministic (bitwise identical from run to run).
 *
 * Notation (Section 3.2): C = block (chunk_len), w = n_bswa_chunks, L = w*C,
 * r = rope_dims, S = sink_len, m = current number of state rows, d = head_dim.
 */
#ifndef KVM_H_
#define KVM_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct kvm_state kvm_state_t; /* opaque, library-owned */

typedef enum {
  KVM_OK = 0,
  KVM_ERR_INVALID_ARG = 1,    /* null pointer, bad shape, bad stride ...                 */
  KVM_ERR_UNSUPPORTED = 2,    /* legal in the paper, not built (e.g. head_dim 96)         */
  KVM_ERR_OOM = 3,            /* device allocation failed in kvm_state_create             */
  KVM_ERR_CUDA = 4,           /* a CUDA runtime call failed / no device                   */
  KVM_ERR_STATE_MISMATCH = 5, /* block / growth / rope_dims differ from the first call    */
  KVM_ERR_CAPACITY = 6,       /* the call would exceed max_state_slots / max_call_tokens  */
  KVM_ERR_TIMEOUT = 7         /* a bounded device-side wait expired (status word)         */
} kvm_status_t;

/* State budget B(e) of Section 3.2, budget rule (M*, n_append):
 *   FIXED      B(e) = fixed_slots                        ("KVM 256")
 *   SQRT       B(e) = floor(sqrt_coeff * sqrt(e))        ("KVM sqrt", coeff 16), exact integer
 *   UNBOUNDED  B(e) = infinity (every overflow token is appended; test limit in
 *              which the layer never compresses)
 * and the two further shapes the paper names without a formula ("power-law", "saturating";
 * the figure that shows them is all it gives), each with an exact integer definition:
 *   POWER      B(e) = floor(sqrt_coeff * e^(pow_num/pow_den)) = the largest n with
 *              n^pow_den <= sqrt_coeff^pow_den * e^pow_num (SQRT is pow 1/2);
 *              1 <= pow_num <= pow_den <= 4, sqrt_coeff <= 1024, positions below 2^26
 *   SATURATING B(e) = floor(fixed_slots * e / (e + sat_half)): half of fixed_slots at
 *              e = sat_half, approaching fixed_slots from below; sat_half >= 1            */
typedef enum { KVM_GROWTH_FIXED = 0, KVM_GROWTH_SQRT = 1, KVM_GROWTH_UNBOUNDED = 2,
               KVM_GROWTH_POWER = 3, KVM_GROWTH_SATURATING = 4 } kvm_growth_kind_t;

typedef struct {
  int32_t kind;        /* kvm_growth_kind_t */
  int32_t sqrt_coeff;  /* SQRT, POWER: the coefficient; the paper uses 16 */
  int64_t fixed_slots; /* FIXED: the budget (values below the block are clamped up by the rule itself);
                          SATURATING: the limit */
  int32_t pow_num, pow_den; /* POWER only */
  int64_t sat_half;    /* SATURATING only */
} kvm_growth_t;

/* Element strides for dims (batch, head, token, channel); channel stride must be 1. */
typedef struct { int64_t q[4], k[4], v[4], out[4]; } kvm_strides_t;

enum {
  KVM_FLAG_NO_RADIUS = 1u << 0,      /* ablation "no v-len normalization": read s^V out unnormalised */
  KVM_FLAG_RECORD_ASSIGN = 1u << 1,  /* keep per-token slot ids / append flags for kvm_debug_assignments */
  KVM_FLAG_SIMT_ATTENTION = 1u << 2, /* use the scalar-core attention kernel (cross-check path) */
  KVM_FLAG_SIMT_ROUTING = 1u << 3,   /* use the scalar-core routing filter (cross-check path)   */
  KVM_FLAG_MIN_KEY_SLOTS = 1u << 4,  /* debug: keep only the minimum of two memory-key slots (the look-ahead
                                        of one block that very large batches run with), whatever the size */
  KVM_FLAG_SERIAL_FOLDS = 1u << 5,   /* one readout copy and folds on the caller's stream between the attention
                                        launches (what states of 256 or more units do by themselves) */
  KVM_FLAG_FUSED_QK_LN = 1u << 6     /* fused front end: kvm_prefill / kvm_decode_step apply LN_q to q and LN_k to k
                                        (ln_q_* / ln_k_* below) before the RoPE, exactly as kvm_head_layernorm
                                        would have on the bf16 tensors, without its pass over q and k */
};

typedef struct {
  int32_t batch, n_q_heads, n_kv_heads, head_dim; /* head_dim in {64,128}; n_q_heads % n_kv_heads == 0 */
  int32_t n_bswa_chunks;                           /* w, the paper uses 2 (Section 4)                    */
  int32_t sink_len;                                /* S, the paper uses 1 (Section 3.2 "Merge")           */
  float rope_base;                                 /* 10000 (Appendix D)                                  */
  float ln_eps;                                    /* LayerNorm epsilon of LN_s, 1e-5                     */
  float norm_eps;                                  /* epsilon_norm of the value readout, 1e-12            */
  const float* ln_weight;                          /* host [n_kv_heads, head_dim] or NULL = 1 (copied)    */
  const float* ln_bias;                            /* host [n_kv_heads, head_dim] or NULL = 0 (copied)    */
  const float* tau_state;                          /* host [n_q_heads] or NULL = 1 (copied)               */
  const float* tau_bswa;                           /* host [n_q_heads] or NULL = 1 (copied)               */
  int32_t max_block;                               /* largest block C that will be used (<= 256)          */
  int64_t max_state_slots;                         /* capacity in state rows (see kvm_plan_capacity), < 2^23 */
  int64_t max_call_tokens;                         /* largest n_tokens of one kvm_prefill call            */
  int64_t max_seq_len;                             /* only used with KVM_FLAG_RECORD_ASSIGN               */
  int32_t device;                                  /* CUDA device ordinal                                 */
  uint32_t flags;
  /* Fused front end (only read with KVM_FLAG_FUSED_QK_LN; Appendix, time mixer: q <- RoPE_r(LN_q(q)),
   * k <- RoPE_r(LN_k(k))): host arrays, copied; NULL weight = 1, NULL bias = 0.  With the flag, q / k / v
   * rows must be 16-byte aligned (pointers and strides) and rope_dims / 2 a multiple of 8, else
   * kvm_prefill returns KVM_ERR_INVALID_ARG. */
  float qk_ln_eps;                                 /* epsilon of LN_q and LN_k                            */
  const float* ln_q_weight;                        /* host [n_q_heads, head_dim]                          */
  const float* ln_q_bias;
  const float* ln_k_weight;                        /* host [n_kv_heads, head_dim]                         */
  const float* ln_k_bias;
} kvm_config_t;

/* Rows a state needs after `seq_len` tokens under (block, growth): the closed form of
 * the budget rule M* = max(m, min(B(e), m + C)) iterated over the folds.  Pure host
 * arithmetic; returns -1 on invalid arguments. */
int64_t kvm_plan_capacity(int32_t block, int32_t n_bswa_chunks, kvm_growth_t growth, int64_t seq_len);

/* Creates an empty state (position 0, m = 0) and allocates every buffer on
 * cfg->device.  Section 3.2 "Terminology": the state holds, per (batch, kv head), the
 * rows (s^K_i, s^V_i, rho_i) plus the uncompressed BSWA window.
 * Errors: INVALID_ARG, UNSUPPORTED, OOM, CUDA.  *out is set only on KVM_OK. */
kvm_status_t kvm_state_create(const kvm_config_t* cfg, kvm_state_t** out);

/* Chunk-wise prefill of n_tokens further tokens (Section 3.2 "Chunks and attention
 * regions", "Readout", "Append", "Merge"; budget rule; Appendix B).
 *   q      device bf16 [B, Hq,  n_tokens, d]   raw (un-rotated) queries
 *   k, v   device bf16 [B, Hkv, n_tokens, d]   raw keys, values
 *   block  C; growth B(e); rope_dims r (even, <= d; first r channels get RoPE with
 *          half-split pairs (i, i + r/2), angle t * base^(-2i/r), position t absolute)
 *   gate   device fp32 [B, Hkv, n_tokens] merge gate g_t (Eq. 2) or NULL = 1
 *   out    device bf16 [B, Hq, n_tokens, d]    per-head attention outputs y_t
 *   strides NULL = contiguous; otherwise element strides per tensor
 * Resumable: tokens continue at the state's position; block, growth and rope_dims are
 * fixed by the first call (later mismatch -> STATE_MISMATCH).  Any n_tokens in
 * [1, max_call_tokens] is legal; a partial last block waits in the window and is
 * folded once later tokens (prefill or decode) complete it.  A fold happens right
 * after the block ending at e was attended, for every complete block.
 * Errors: INVALID_ARG, UNSUPPORTED, STATE_MISMATCH, CAPACITY, CUDA. */
kvm_status_t kvm_prefill(const void* q, const void* k, const void* v, kvm_state_t* state,
                         int32_t block, kvm_growth_t growth, int32_t rope_dims,
                         int64_t n_tokens, const float* gate, void* out,
                         const kvm_strides_t* strides, void* cuda_stream);

/* One decode token per sequence (Table 1 "Decode time per token"): rotates q,k at the
 * state's position, pushes k,v into the window, attends over [state ; window], and
 * folds the overflow block when the token completes a block.
 *   q device bf16 [B, Hq, d]; k, v device bf16 [B, Hkv, d]; gate device fp32 [B, Hkv] or NULL
 *   out device bf16 [B, Hq, d]
 * Requires a state whose block/growth/rope_dims were fixed by a prefill call.
 * Errors: INVALID_ARG, STATE_MISMATCH, CAPACITY, CUDA. */
kvm_status_t kvm_decode_step(const void* q, const void* k, const void* v, kvm_state_t* state,
                             const float* gate, void* out, void* cuda_stream);

/* Same operations with HOST buffers (contiguous layouts as above): the call copies the
 * inputs to library-owned device staging, runs the path, copies `out` back and
 * synchronises the stream before returning.  n_tokens <= max_call_tokens.  A long prefill is cut
 * into up to eight segments of whole blocks whose host-to-device and device-to-host copies run on
 * the state's own streams beside the computation of the neighbouring segments (pinned host memory
 * is needed for the copies to overlap; pageable memory works, serially).  The result is identical to
 * one kvm_prefill call. */
kvm_status_t kvm_prefill_host(const void* q_host, const void* k_host, const void* v_host,
                              kvm_state_t* state, int32_t block, kvm_growth_t growth,
                              int32_t rope_dims, int64_t n_tokens, const float* gate_host,
                              void* out_host, void* cuda_stream);
kvm_status_t kvm_decode_step_host(const void* q_host, const void* k_host, const void* v_host,
                                  kvm_state_t* state, const float* gate_host, void* out_host,
                                  void* cuda_stream);

/* Frees the state and all device memory it owns.  NULL is accepted. */
kvm_status_t kvm_state_free(kvm_state_t* state);

/* Host-side bookkeeping (no device access): rows m, tokens consumed, folds done.
 * Any output pointer may be NULL.  m depends only on (position, block, growth), never
 * on data (budget rule), so it is the same for every (batch, head). */
kvm_status_t kvm_state_info(const kvm_state_t* state, int64_t* n_slots, int64_t* position,
                            int64_t* n_folds);

/* Reads the device status word (set by bounded device-side waits or debug index checks)
 * after synchronising the stream and clears it: KVM_OK, KVM_ERR_TIMEOUT or KVM_ERR_CUDA.  A kernel
 * whose wait ran out has torn down normally (its outputs are undefined); the state can be reset
 * (kvm_state_reset) or restored (kvm_state_import) and used again. */
kvm_status_t kvm_state_check(kvm_state_t* state, void* cuda_stream);

/* Failure-detection self test (no counterpart in the paper): launches one thread that waits, with the
 * library's bounded wait and a limit of `spins` iterations (1 .. 2^20), on a barrier that nothing ever
 * arrives at, and reports the expiry exactly as the production kernels do: KVM_ERR_TIMEOUT in the
 * state's status word, normal return.  kvm_state_check then returns KVM_ERR_TIMEOUT once.  Touches
 * nothing else of the state. */
kvm_status_t kvm_debug_expire_wait(kvm_state_t* state, int32_t spins, void* cuda_stream);

/* Copies the state rows to HOST arrays (synchronises the stream).  Shapes, with
 * U = batch * n_kv_heads and m = n_slots:
 *   sum_k   double [U, m, d]  running key sums   s^K   (Section 3.2 "Merge")
 *   sum_v   float  [U, m, d]  running value sums s^V
 *   radius  float  [U, m]     rho_i, set when the row was created
 *   weight  double [U, m]     1 + sum of merge gates of the row (means = sum / weight)
 *   count   int32  [U, m]     number of tokens in the row
 *   k_read  fp16   [U, m, d]  readout cache LN_s(s^K)   (may be NULL)
 *   v_read  fp16   [U, m, d]  readout cache rho * s^V / max(||s^V||, eps) (may be NULL)
 * Any pointer may be NULL to skip that array. */
kvm_status_t kvm_state_export(kvm_state_t* state, double* sum_k, float* sum_v, float* radius,
                              double* weight, int32_t* count, void* k_read, void* v_read,
                              void* cuda_stream);

/* Checkpoint / resume (Section 3.2 "Terminology": the state is what is carried from one chunk to the
 * later ones).  A snapshot is kvm_state_snapshot_info + the arrays of kvm_state_export (sums, radii,
 * weights, counts) + the uncompressed window of kvm_state_export_window; kvm_state_import loads it into
 * a state of the same shape (batch, heads, head_dim, n_bswa_chunks, sink_len, LayerNorm parameters and
 * temperatures are the state's own and are not part of a snapshot), after which kvm_prefill /
 * kvm_decode_step continue exactly -- bit for bit -- where the exported state stood. */
typedef struct {
  int32_t block, rope_dims;      /* bound by the first kvm_prefill; 0 / 0 while unbound               */
  kvm_growth_t growth;
  int64_t n_slots, position, n_folds;
  int64_t window_begin;          /* tokens [window_begin, position) are held uncompressed             */
  int64_t window_len;            /* position - window_begin, < (n_bswa_chunks + 1) * block             */
} kvm_snapshot_info_t;

/* Host bookkeeping only.  INVALID_ARG on NULL; a state that no prefill has bound yet reports zeros. */
kvm_status_t kvm_state_snapshot_info(const kvm_state_t* state, kvm_snapshot_info_t* out);

/* Copies the window tokens [window_begin, position) to HOST arrays (synchronises the stream):
 *   win_k  fp16  [U, window_len, d]  keys as the window holds them (rotated by the partial RoPE)
 *   win_v  fp16  [U, window_len, d]  values
 *   win_gate float [U, window_len]   merge gates of those tokens
 * Any pointer may be NULL.  STATE_MISMATCH when no prefill has bound the state yet. */
kvm_status_t kvm_state_export_window(kvm_state_t* state, void* win_k, void* win_v, float* win_gate,
                                     void* cuda_stream);

/* Loads a snapshot (all arrays HOST memory, shapes as exported: [U, n_slots, ...] and
 * [U, window_len, ...]; win_gate may be NULL = 1; the other arrays may be NULL only when their extent
 * is zero).  The state's previous contents are dropped (as by kvm_state_reset) and block / growth /
 * rope_dims are bound from `info`.  Row statistics and both readout caches are recomputed from the
 * sums by the code that a fold uses, so the continuation equals the uninterrupted run bit for bit.
 * With KVM_FLAG_RECORD_ASSIGN the recorded assignments of tokens before `position` are lost (-1).
 * Validation (before anything is copied): info->n_slots and n_folds must be what the budget rule gives
 * for `position`, window_begin / window_len what the block structure gives, block <= max_block,
 * n_slots <= max_state_slots.  Synchronises the stream before returning.
 * Errors: INVALID_ARG, UNSUPPORTED, CAPACITY, CUDA; a failed validation leaves the state untouched. */
kvm_status_t kvm_state_import(kvm_state_t* state, const kvm_snapshot_info_t* info, const double* sum_k,
                              const float* sum_v, const float* radius, const double* weight,
                              const int32_t* count, const void* win_k, const void* win_v,
                              const float* win_gate, void* cuda_stream);

/* With KVM_FLAG_RECORD_ASSIGN: copies, for tokens [0, n) (n <= position, n <= max_seq_len),
 * slot_of_token int32 [U, n] (row merged into / appended as; -1 = not folded yet) and
 * was_appended uint8 [U, n] to HOST arrays (synchronises the stream). */
kvm_status_t kvm_debug_assignments(kvm_state_t* state, int64_t n, int32_t* slot_of_token,
                                   uint8_t* was_appended, void* cuda_stream);

/* Returns the state to "empty" (position 0, no rows, no folds, block/growth/rope_dims unbound)
 * without freeing or clearing device memory, so that one allocation serves many sequences.
 * Host bookkeeping only: nothing is enqueued and pending work is not waited for (the next call is
 * ordered behind it on its own stream; with KVM_FLAG_RECORD_ASSIGN that next kvm_prefill also
 * clears the recorded assignments, on its stream). */
kvm_status_t kvm_state_reset(kvm_state_t* state);

/* Per-kernel device timing for benchmarks.  kvm_profile_enable(state, 1) makes every later
 * call bracket the launches of each phase with CUDA events on the call's stream (phases:
 * 0 ingest, 1 attention, 2 memory keys, 3 routing filter, 4 fold decision, 5 fold application,
 * 6 decode step attention incl. its ingest/combine, 7 unused); kvm_profile_read synchronises
 * the device, adds the elapsed milliseconds and bracket counts into ms[8] / groups[8] and
 * clears the record.  Off by default; at most 16384 brackets are kept between reads (later
 * ones are dropped and not counted). */
kvm_status_t kvm_profile_enable(kvm_state_t* state, int32_t on);
kvm_status_t kvm_profile_read(kvm_state_t* state, double* ms, int64_t* groups);

/* Debug counters since the state was created (synchronises the stream):
 * out[0] overflow tokens whose routing fell back to the exhaustive fp64 scan, out[1] candidate
 * (token, row) pairs refined in fp64, out[2] overflow tokens routed, out[3] input elements of q, k, v
 * whose magnitude exceeded 65504 and was clamped on the way in (bf16 inputs are carried as fp16).
 * `out` has room for four values.  32-bit device counters. */
kvm_status_t kvm_debug_counters(kvm_state_t* state, int64_t* out, void* cuda_stream);

/* Number of kernels the library has launched for this state so far (host counter). */
int64_t kvm_launch_count(const kvm_state_t* state);

/* Single-query attention over caller-held rows, for callers that must not allocate device
 * memory.  (The paper has no counterpart: this is a packaging variant of the decode step's
 * attention kernel.)  Meant for code that cannot call cudaMalloc where it runs -- a serving loop
 * whose memory all belongs to its own pool, a plugin inside another framework's memory plan, a
 * section that must not risk the implicit device synchronisation of cudaMalloc/cudaFree -- and
 * that already holds the rows in its own buffers, e.g. a readout cache from kvm_state_export
 * followed by the window tokens.  For every head h:
 *     out[h] = softmax(scale * q[h] . keys[h]^T) . values[h]
 *   q       device fp16 [n_heads, head_dim]            (16-byte aligned)
 *   keys    device fp16 [n_heads, n_rows, head_dim]    (16-byte aligned)
 *   values  device fp16 [n_heads, n_rows, head_dim]    (16-byte aligned)
 *   out     device bf16 [n_heads, head_dim]
 *   scale   multiplies the dot products (tau / sqrt(head_dim) for the layer's logits)
 * The caller owns all four buffers; the call allocates and frees nothing.  The rows are split
 * over several CTAs per head; the per-split partial results go to a fixed array inside the
 * library image (about 4.3 MB on every GPU that loads the library, held until the process exits)
 * instead of an allocated buffer.  That array bounds the problem: n_heads * n_splits <= 8192,
 * where n_splits = min(32, ceil(n_rows / 256), ceil(592 / n_heads)); larger calls return
 * KVM_ERR_CAPACITY and launch nothing.  head_dim must be 64 or 128 (else KVM_ERR_UNSUPPORTED).
 * All calls share the array and it keeps the previous call's contents; nothing in it needs
 * clearing because each call rewrites every slot it reads.  Calls that overlap on the same GPU
 * (other streams or threads) race on it -- serialise them.  The first call on each device looks
 * up the array's device address (with the calling thread's current device); make that first
 * call before starting any stream capture.  Work is enqueued on cuda_stream on the current
 * device; no synchronisation. */
kvm_status_t kvm_attend_rows_noalloc(const void* q, const void* keys, const void* values, int32_t n_heads,
                                     int64_t n_rows, int32_t head_dim, float scale, void* out,
                                     void* cuda_stream);

/* Front end, merge gate (Section 3.2 "KVM weight preparation", Eq. 2): g_t = 1 + ELU(x_t W_g) with
 * ELU's alpha = 1, i.e. g = 1 + z for z > 0 and exp(z) otherwise, z = x_t . W_g[h]; one scalar per
 * token and kv head (W_g is one d_model-vector per head).  The result is what kvm_prefill and
 * kvm_decode_step take as `gate` (for a decode step: batch rows of one token, n_tokens = 1).
 *   x       device bf16 [batch, n_tokens, d_model]   the layer's input rows; 16-byte aligned,
 *                                                    d_model a multiple of 8
 *   w_gate  device fp32 [n_kv_heads, d_model]
 *   gate    device fp32 [batch, n_kv_heads, n_tokens]   (out)
 *   status  device int32 word or NULL: the tensor-core path waits on barriers with a bounded number of
 *           spins; should such a wait ever run out, the gates of the affected tokens are NaN and
 *           KVM_ERR_TIMEOUT is stored here (the word is never cleared by the library: zero it before)
 * Products and sums in fp32 (inputs bf16 -> fp32 exactly).  n_kv_heads <= 64 and batch <= 65535,
 * else KVM_ERR_UNSUPPORTED; bad pointers, alignment or sizes KVM_ERR_INVALID_ARG; nothing is
 * launched on an error.  The caller owns all three buffers; no allocation, no synchronisation;
 * the work is enqueued on cuda_stream on the current device. */
kvm_status_t kvm_merge_gate(const void* x, const float* w_gate, int32_t batch, int64_t n_tokens, int32_t d_model,
                            int32_t n_kv_heads, float* gate, int32_t* status, void* cuda_stream);

/* Front end, LN_q / LN_k (Appendix, time mixer of the backbone: q_t <- RoPE_r(LN_q(q_t)),
 * k_t <- RoPE_r(LN_k(k_t))): LayerNorm over the head channels of every (batch, head, token) row, in
 * place; call it on q and on k before kvm_prefill / kvm_decode_step, which apply the RoPE.
 *   x       device bf16 [batch, n_heads, n_tokens, head_dim], contiguous, 16-byte aligned (in/out)
 *   weight  device fp32 [n_heads, head_dim] or NULL (= 1); bias likewise or NULL (= 0); 16-byte aligned
 *   eps     added to the biased variance
 * Statistics and the affine map in fp32, result rounded to bf16.  head_dim 64 or 128 (else
 * KVM_ERR_UNSUPPORTED).  The caller owns the buffers; no allocation, no synchronisation; enqueued on
 * cuda_stream on the current device. */
kvm_status_t kvm_head_layernorm(void* x, const float* weight, const float* bias, int32_t batch, int32_t n_heads,
                                int64_t n_tokens, int32_t head_dim, float eps, void* cuda_stream);

const char* kvm_status_string(kvm_status_t s);

#ifdef __cplusplus
}
#endif
#endif /* KVM_H_ */
