// Merge gate of the layer's front end (Section 3.2 "KVM weight preparation", Eq. 2):
//     g_t = 1 + ELU(x_t W_g),   one scalar per token and kv head,
// i.e. g = 1 + z for z > 0 and exp(z) otherwise, z = x_t . W_g[h].  The result is the `gate`
// argument of kvm_prefill / kvm_decode_step.
//
// A skinny product [tokens x d_model] x [d_model x heads] with at most 64 heads: every x element is
// needed once per head, so the kernel is bound by reading x (2 d_model bytes per token) as long as
// the FMA pipe keeps up.  A CTA takes 64 tokens; thread (token, part) owns one token, all heads and
// one quarter of every 128-channel slice: its share of the x row streams through registers, eight
// channels (16 bytes) per load, and is never shared; the W_g rows go through shared memory slice by
// slice and are read as broadcasts (every lane of a warp wants the same weights), so a step of eight
// channels costs 2 HT shared-memory loads for 8 HT FMAs.  The four partial sums of a token meet in
// shared memory at the end (fixed order: reproducible), and the stores run along the token axis of
// gate[B, heads, T].
#include "kvm_internal.h"
#include "tc_common.cuh"

namespace kvm {

bool encode_tmap_rows(CUtensorMap* map, const void* base, int d, int64_t rows, int64_t units, int box_rows);   // kvm_attn_tc.cu

constexpr int kGateTokens = 64;   // tokens per CTA
constexpr int kGateParts = 4;     // threads per token, each a quarter of the channels of a slice
constexpr int kGateThreads = kGateTokens * kGateParts;
constexpr int kGateK = 128;       // channels per shared-memory slice of W_g

template <int HT>                 // heads, padded to 8, 16, 32 or 64
__global__ void __launch_bounds__(kGateThreads) merge_gate_kernel(const __nv_bfloat16* __restrict__ x, const float* __restrict__ w,
                                                                  float* __restrict__ gate, int64_t T, int dm, int H) {
  __shared__ __align__(16) float ws[HT * kGateK];   // W_g slice [HT][128]; afterwards the partial sums
  const int tid = threadIdx.x, tok = tid % kGateTokens, part = tid / kGateTokens;   // a warp shares `part`
  const int b = blockIdx.y;
  const int64_t t = (int64_t)blockIdx.x * kGateTokens + tok;
  const bool valid = t < T;
  const __nv_bfloat16* row = x + ((int64_t)b * T + (valid ? t : 0)) * dm;
  float acc[HT];
#pragma unroll
  for (int h = 0; h < HT; ++h) acc[h] = 0.f;
  for (int k0 = 0; k0 < dm; k0 += kGateK) {
    __syncthreads();   // the previous slice is no longer read
    for (int e = tid; e < HT * kGateK; e += kGateThreads) {
      const int h = e / kGateK, c = e % kGateK;
      ws[e] = (h < H && k0 + c < dm) ? w[(int64_t)h * dm + k0 + c] : 0.f;
    }
    __syncthreads();
#pragma unroll 2
    for (int j = 0; j < kGateK / 8 / kGateParts; ++j) {
      const int c = 8 * (part * (kGateK / 8 / kGateParts) + j);   // first of eight channels inside the slice
      if (k0 + c >= dm) break;                                    // d_model is a multiple of 8
      const uint4 raw = *reinterpret_cast<const uint4*>(row + k0 + c);
      const __nv_bfloat162* p2 = reinterpret_cast<const __nv_bfloat162*>(&raw);
      const float2 f0 = __bfloat1622float2(p2[0]), f1 = __bfloat1622float2(p2[1]);
      const float2 f2 = __bfloat1622float2(p2[2]), f3 = __bfloat1622float2(p2[3]);
#pragma unroll
      for (int h = 0; h < HT; ++h) {
        const float4 wa = *reinterpret_cast<const float4*>(&ws[h * kGateK + c]);       // one address per warp: broadcast
        const float4 wb = *reinterpret_cast<const float4*>(&ws[h * kGateK + c + 4]);
        float a = acc[h];
        a = fmaf(f0.x, wa.x, a); a = fmaf(f0.y, wa.y, a); a = fmaf(f1.x, wa.z, a); a = fmaf(f1.y, wa.w, a);
        a = fmaf(f2.x, wb.x, a); a = fmaf(f2.y, wb.y, a); a = fmaf(f3.x, wb.z, a); a = fmaf(f3.y, wb.w, a);
        acc[h] = a;
      }
    }
  }
  // parts 2, 3 -> parts 0, 1, then part 1 -> part 0, through the slice buffer (2 x 64 x HT floats fit it)
  __syncthreads();
  if (part >= 2) {
#pragma unroll
    for (int h = 0; h < HT; ++h) ws[((part - 2) * HT + h) * kGateTokens + tok] = acc[h];
  }
  __syncthreads();
  if (part < 2) {
#pragma unroll
    for (int h = 0; h < HT; ++h) acc[h] += ws[(part * HT + h) * kGateTokens + tok];
  }
  __syncthreads();
  if (part == 1) {
#pragma unroll
    for (int h = 0; h < HT; ++h) ws[h * kGateTokens + tok] = acc[h];
  }
  __syncthreads();
  if (part == 0 && valid) {
#pragma unroll
    for (int h = 0; h < HT; ++h) {
      const float z = acc[h] + ws[h * kGateTokens + tok];
      if (h < H) gate[((int64_t)b * H + h) * T + t] = z > 0.f ? 1.f + z : expf(z);   // 1 + ELU(z), alpha = 1
    }
  }
}

// ------------------------------------------------------------------------------------------
// Tensor-core version (d_model a multiple of 64, more than 8 heads): with 16 or more heads the product
// above is bound by the FMA pipe and by the shared-memory broadcasts, not by reading x.  Here a CTA
// takes 128 tokens:
//   warp 0      TMA producer: 128-token x 64-channel slices of x (bf16, 128-byte swizzle), 4 stages
//   warps 2-5   weight converters: the same 64 channels of every W_g row, fp32 -> bf16 "hi" plus bf16
//               "lo" = bf16(w - hi) (together 16 mantissa bits; the products hi*x and lo*x are exact in
//               fp32; a third term was measured: same error, which the fp32 accumulation dominates,
//               and 1.8x the time), written into shared memory in the swizzled K-major layout the MMA
//               reads; after the last slice the same warps read the accumulator and store the gates
//   warp 1      one thread issues, per slice, 4 k-steps x (hi, lo) tcgen05.mma (kind::f16, bf16 x bf16,
//               M 128, N = heads padded to 16..64, fp32 accumulator in tensor memory)
// Every wait is bounded; if one expires the CTA stores NaN gates for its tokens and tears down.
constexpr int kGateTcStages = 4;
constexpr int kGateTcXBytes = 128 * 128;   // 128 tokens x 64 bf16

enum { GB_XFULL = 0, GB_WFULL = 4, GB_FREE = 8, GB_DONE = 12, GB_COUNT = 13 };

__host__ __device__ constexpr uint32_t idesc_bf16(int M, int N) {   // as tc::idesc_f16, A and B formats = 1 (bf16), both K-major
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

template <int NP>   // heads padded to a multiple of 16
__global__ void __launch_bounds__(192, 1)
merge_gate_tc_kernel(const __grid_constant__ CUtensorMap mapX, const float* __restrict__ w, float* __restrict__ gate,
                     int64_t T, int dm, int H, int32_t* status) {
  constexpr int WBYTES = 2 * NP * 128;     // hi and lo tiles of one slice
  constexpr uint32_t TMEM_COLS = NP <= 32 ? 32 : 64;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sX = base;
  uint8_t* sW = base + kGateTcStages * kGateTcXBytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(sW + kGateTcStages * WBYTES);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + GB_COUNT);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int b = blockIdx.y;
  const int64_t t0 = (int64_t)blockIdx.x * 128;
  const int nslices = dm / 64;

  if (tid == 0) {
    for (int s = 0; s < kGateTcStages; ++s) {
      tc::mbar_init(&bars[GB_XFULL + s], 1);
      tc::mbar_init(&bars[GB_WFULL + s], 128);
      tc::mbar_init(&bars[GB_FREE + s], 1);
    }
    tc::mbar_init(&bars[GB_DONE], 1);
    *abort_flag = 0;
    tc::fence_barrier_init();
  }
  if (warp == 1) {
    tc::tmem_alloc(tmem_slot, TMEM_COLS);
    tc::tmem_relinquish();
  }
  tc::tc_fence_before();
  __syncthreads();
  tc::tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      tc::prefetch_tmap(&mapX);
      for (int j = 0; j < nslices; ++j) {
        const int s = j % kGateTcStages;
        if (*abort_flag) break;
        if (j >= kGateTcStages && !tc::mbar_wait(&bars[GB_FREE + s], ((j / kGateTcStages) - 1) & 1)) { *abort_flag = 1; break; }
        tc::mbar_expect_tx(&bars[GB_XFULL + s], kGateTcXBytes);
        tc::tma_load_3d(sX + s * kGateTcXBytes, &mapX, &bars[GB_XFULL + s], j * 64, (int)t0, b);   // rows past T read zeros
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t IDESC = idesc_bf16(128, NP);
      const uint32_t aX = tc::smem_u32(sX), aW = tc::smem_u32(sW);
      bool dead = false;
      for (int j = 0; j < nslices && !dead; ++j) {
        const int s = j % kGateTcStages;
        const uint32_t par = (j / kGateTcStages) & 1;
        if (*abort_flag || !tc::mbar_wait(&bars[GB_XFULL + s], par) || !tc::mbar_wait(&bars[GB_WFULL + s], par)) { dead = true; break; }
        tc::tc_fence_after();
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
          const uint64_t da = tc::smem_desc_sw128(aX + s * kGateTcXBytes + ks * 32, 16, 1024);
          tc::mma_f16_ss(tmem, da, tc::smem_desc_sw128(aW + s * WBYTES + ks * 32, 16, 1024), IDESC, (j > 0 || ks > 0) ? 1u : 0u);
          tc::mma_f16_ss(tmem, da, tc::smem_desc_sw128(aW + s * WBYTES + NP * 128 + ks * 32, 16, 1024), IDESC, 1u);
        }
        tc::mma_commit(&bars[GB_FREE + s]);
      }
      if (dead) *abort_flag = 1;
      tc::mma_commit(&bars[GB_DONE]);   // (arrives once everything issued so far has completed)
    }
  } else {
    const int ct = tid - 64;   // 0..127
    bool ok = true;
    // item = (head row r, 16-byte chunk c of the slice's 64 channels); a thread's items of slice j + 1
    // are loaded before it converts those of slice j, so that the loads' latency is off the chain
    constexpr int ITEMS = NP * 8 / 128;
    float4 nxt[ITEMS][2];
    auto load_items = [&](int j) {
#pragma unroll
      for (int q = 0; q < ITEMS; ++q) {
        const int item = ct + 128 * q, r = item >> 3, c = item & 7;
        if (r < H) {
          nxt[q][0] = *reinterpret_cast<const float4*>(w + (int64_t)r * dm + j * 64 + 8 * c);
          nxt[q][1] = *reinterpret_cast<const float4*>(w + (int64_t)r * dm + j * 64 + 8 * c + 4);
        } else {
          nxt[q][0] = nxt[q][1] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
      }
    };
    load_items(0);
    for (int j = 0; j < nslices && ok; ++j) {
      const int s = j % kGateTcStages;
      float4 cur[ITEMS][2];
#pragma unroll
      for (int q = 0; q < ITEMS; ++q) { cur[q][0] = nxt[q][0]; cur[q][1] = nxt[q][1]; }
      if (j + 1 < nslices) load_items(j + 1);
      if (j >= kGateTcStages && !tc::mbar_wait(&bars[GB_FREE + s], ((j / kGateTcStages) - 1) & 1)) { *abort_flag = 1; ok = false; break; }
      uint8_t* hi = sW + s * WBYTES;
      uint8_t* lo = hi + NP * 128;
#pragma unroll
      for (int q = 0; q < ITEMS; ++q) {
        const int item = ct + 128 * q, r = item >> 3, c = item & 7;
        const float v[8] = {cur[q][0].x, cur[q][0].y, cur[q][0].z, cur[q][0].w, cur[q][1].x, cur[q][1].y, cur[q][1].z, cur[q][1].w};
        uint32_t ph[4], pl[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const __nv_bfloat16 h0 = __float2bfloat16_rn(v[2 * i]), h1 = __float2bfloat16_rn(v[2 * i + 1]);
          const __nv_bfloat16 l0 = __float2bfloat16_rn(v[2 * i] - __bfloat162float(h0));
          const __nv_bfloat16 l1 = __float2bfloat16_rn(v[2 * i + 1] - __bfloat162float(h1));
          ph[i] = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
          pl[i] = (uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16);
        }
        // K-major tile with the 128-byte swizzle: row r of 128 bytes, chunk c stored at c ^ (r mod 8)
        const int off = (r >> 3) * 1024 + (r & 7) * 128 + ((c ^ (r & 7)) << 4);
        *reinterpret_cast<uint4*>(hi + off) = make_uint4(ph[0], ph[1], ph[2], ph[3]);
        *reinterpret_cast<uint4*>(lo + off) = make_uint4(pl[0], pl[1], pl[2], pl[3]);
      }
      tc::fence_proxy_async();   // the tensor core reads these tiles through the async proxy
      tc::mbar_arrive(&bars[GB_WFULL + s]);
    }
    // epilogue: thread = token row of the accumulator (TMEM lane quarter = warp mod 4)
    if (ok && !tc::mbar_wait(&bars[GB_DONE], 0)) { *abort_flag = 1; ok = false; }
    tc::tc_fence_after();
    const int quarter = warp & 3;
    const int64_t t = t0 + quarter * 32 + lane;
    const bool good = ok && !*abort_flag;
#pragma unroll
    for (int c = 0; c < (NP + 31) / 32; ++c) {
      uint32_t r[32];
      tc::tmem_ld32(tmem + ((uint32_t)(quarter * 32) << 16) + c * 32, r);
      tc::tmem_wait_ld();
      if (t < T) {
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const int h = c * 32 + i;
          if (h < H) {
            const float z = __uint_as_float(r[i]);
            gate[((int64_t)b * H + h) * T + t] = good ? (z > 0.f ? 1.f + z : expf(z)) : __int_as_float(0x7fc00000);
          }
        }
      }
    }
  }
  // a wait that ran out: the gates of this tile are NaN, and the caller's status word (if any) says why
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag && status) atomicExch(status, (int)KVM_ERR_TIMEOUT);
  tc::tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc::tmem_dealloc(tmem, TMEM_COLS);
  }
}

template <int NP>
static bool launch_gate_tc(const CUtensorMap& map, const float* w, float* gate, int batch, int64_t T, int dm, int H, int32_t* status,
                           cudaStream_t s) {
  const int smem = kGateTcStages * (kGateTcXBytes + 2 * NP * 128) + 256 + 1024;
  static bool attr_set = false;   // (per instantiation; setting it again is harmless)
  if (!attr_set) {
    if (cudaFuncSetAttribute(merge_gate_tc_kernel<NP>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return false;
    attr_set = true;
  }
  const dim3 grid((unsigned)((T + 127) / 128), (unsigned)batch);
  merge_gate_tc_kernel<NP><<<grid, 192, smem, s>>>(map, w, gate, T, dm, H, status);
  return true;
}

}  // namespace kvm

using namespace kvm;

extern "C" __attribute__((visibility("default")))
kvm_status_t kvm_merge_gate(const void* x, const float* w_gate, int32_t batch, int64_t n_tokens, int32_t d_model,
                                    int32_t n_kv_heads, float* gate, int32_t* status, void* cuda_stream) {
  if (!x || !w_gate || !gate || batch < 1 || n_tokens < 1 || d_model < 8 || n_kv_heads < 1) return KVM_ERR_INVALID_ARG;
  if (d_model % 8 || ((uintptr_t)x & 15) || ((uintptr_t)w_gate & 3) || ((uintptr_t)gate & 3) || ((uintptr_t)status & 3)) return KVM_ERR_INVALID_ARG;
  if (n_kv_heads > 64) return KVM_ERR_UNSUPPORTED;
  if (batch > 65535) return KVM_ERR_UNSUPPORTED;
  cudaStream_t s = (cudaStream_t)cuda_stream;
  const dim3 grid((unsigned)((n_tokens + kGateTokens - 1) / kGateTokens), (unsigned)batch);
  const __nv_bfloat16* xp = (const __nv_bfloat16*)x;
  if (d_model % 64 == 0 && n_kv_heads > 8 && n_tokens < ((int64_t)1 << 31)) {
    // tensor-core path (few heads are bound by reading x already on the scalar path)
    CUtensorMap map;
    if (encode_tmap_rows(&map, x, d_model, n_tokens, batch, 128)) {
      bool ok;
      if (n_kv_heads <= 16) ok = launch_gate_tc<16>(map, w_gate, gate, batch, n_tokens, d_model, n_kv_heads, status, s);
      else if (n_kv_heads <= 32) ok = launch_gate_tc<32>(map, w_gate, gate, batch, n_tokens, d_model, n_kv_heads, status, s);
      else if (n_kv_heads <= 48) ok = launch_gate_tc<48>(map, w_gate, gate, batch, n_tokens, d_model, n_kv_heads, status, s);
      else ok = launch_gate_tc<64>(map, w_gate, gate, batch, n_tokens, d_model, n_kv_heads, status, s);
      if (ok) return cudaGetLastError() == cudaSuccess ? KVM_OK : KVM_ERR_CUDA;
    }
    cudaGetLastError();   // fall through to the scalar path
  }
  if (n_kv_heads <= 8) merge_gate_kernel<8><<<grid, kGateThreads, 0, s>>>(xp, w_gate, gate, n_tokens, d_model, n_kv_heads);
  else if (n_kv_heads <= 16) merge_gate_kernel<16><<<grid, kGateThreads, 0, s>>>(xp, w_gate, gate, n_tokens, d_model, n_kv_heads);
  else if (n_kv_heads <= 32) merge_gate_kernel<32><<<grid, kGateThreads, 0, s>>>(xp, w_gate, gate, n_tokens, d_model, n_kv_heads);
  else merge_gate_kernel<64><<<grid, kGateThreads, 0, s>>>(xp, w_gate, gate, n_tokens, d_model, n_kv_heads);
  return cudaGetLastError() == cudaSuccess ? KVM_OK : KVM_ERR_CUDA;
}

// ------------------------------------------------------------------------------------------
// LN_q / LN_k of the layer's front end (Appendix, GPTAlpha-2 time mixer: q_t <- RoPE_r(LN_q(q_t)),
// k_t <- RoPE_r(LN_k(k_t))): a LayerNorm over the head channels of every (batch, head, token) row,
// in place on the bf16 tensor that kvm_prefill / kvm_decode_step then take (they apply the RoPE).
// HBM-bound: every element is read and written once.  d / 8 lanes share a row, 16 bytes each;
// statistics in fp32 through shuffles inside the lane group (biased variance, as LN_s).
#include "ln_rows.cuh"

namespace kvm {

constexpr int kLnRowsPerGroup = 4;   // rows per lane group, loaded up front: enough bytes in flight per SM for the HBM latency

template <int D>
__global__ void __launch_bounds__(256) head_layernorm_kernel(__nv_bfloat16* __restrict__ x, const float* __restrict__ weight,
                                                             const float* __restrict__ bias, int64_t rows, int64_t T, int H,
                                                             float eps) {
  constexpr int LPR = D / 8;                 // lanes per row: 8 (d = 64) or 16 (d = 128)
  constexpr int RPW = 32 / LPR;              // lane groups per warp
  constexpr int NR = kLnRowsPerGroup;
  const int lane = threadIdx.x & 31, sub = lane % LPR;
  const int64_t warp_global = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int64_t row0 = warp_global * (RPW * NR) + lane / LPR;   // this group's rows: row0 + k RPW
  uint4 raw[NR];
#pragma unroll
  for (int k = 0; k < NR; ++k) {
    const int64_t rr = min(row0 + k * RPW, rows - 1);   // (a clamped duplicate is computed and not stored: the shuffles need every lane)
    raw[k] = *reinterpret_cast<const uint4*>(x + rr * D + sub * 8);
  }
  float wv[8], bv[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) { wv[i] = 1.f; bv[i] = 0.f; }
  int h_cur = -1;
#pragma unroll
  for (int k = 0; k < NR; ++k) {
    const int64_t row = row0 + k * RPW;
    const bool live = row < rows;
    const int64_t rr = live ? row : rows - 1;
    const int h = (int)((rr / T) % H);          // rows are [B, H, T]
    const __nv_bfloat162* p2 = reinterpret_cast<const __nv_bfloat162*>(&raw[k]);
    float v[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 f = __bfloat1622float2(p2[i]);
      v[2 * i] = f.x; v[2 * i + 1] = f.y;
    }
    if (h != h_cur) {   // consecutive rows nearly always belong to one head: its weights stay in registers
      h_cur = h;
      ln_load_affine<D>(weight, bias, h, sub, wv, bv);
    }
    ln_chunk8<D>(v, wv, bv, eps);
    uint32_t out[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const __nv_bfloat162 o2 = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);   // (already bf16 values: exact)
      out[i] = *reinterpret_cast<const uint32_t*>(&o2);
    }
    if (live) *reinterpret_cast<uint4*>(x + rr * D + sub * 8) = make_uint4(out[0], out[1], out[2], out[3]);
  }
}

}  // namespace kvm

extern "C" __attribute__((visibility("default")))
kvm_status_t kvm_head_layernorm(void* x, const float* weight, const float* bias, int32_t batch, int32_t n_heads,
                                int64_t n_tokens, int32_t head_dim, float eps, void* cuda_stream) {
  if (!x || batch < 1 || n_heads < 1 || n_tokens < 1 || !(eps >= 0.f)) return KVM_ERR_INVALID_ARG;
  if (((uintptr_t)x & 15) || ((uintptr_t)weight & 15) || ((uintptr_t)bias & 15)) return KVM_ERR_INVALID_ARG;
  if (head_dim != 64 && head_dim != 128) return KVM_ERR_UNSUPPORTED;
  cudaStream_t s = (cudaStream_t)cuda_stream;
  const int64_t rows = (int64_t)batch * n_heads * n_tokens;
  const int rows_per_cta = 8 * (32 / (head_dim / 8)) * kvm::kLnRowsPerGroup;
  const int64_t ctas = (rows + rows_per_cta - 1) / rows_per_cta;
  if (ctas > 0x7fffffff) return KVM_ERR_UNSUPPORTED;
  __nv_bfloat16* xp = (__nv_bfloat16*)x;
  if (head_dim == 128) kvm::head_layernorm_kernel<128><<<(unsigned)ctas, 256, 0, s>>>(xp, weight, bias, rows, n_tokens, n_heads, eps);
  else kvm::head_layernorm_kernel<64><<<(unsigned)ctas, 256, 0, s>>>(xp, weight, bias, rows, n_tokens, n_heads, eps);
  return cudaGetLastError() == cudaSuccess ? KVM_OK : KVM_ERR_CUDA;
}
