// Fused attention of one chunk over [state rows ; window] on the 5th-generation tensor cores
// (Section 3.2 "Readout": one softmax over the concatenation, state fully visible, causal in
// the window, per-region temperatures).
//
// One CTA owns a 128-query tile of one (batch, query head) and walks the key tiles (128 keys:
// first the state's readout cache, then the window) with these warp roles:
//   warp 0      TMA producer: Q once, then K tiles into a 3-stage and V tiles into a 2-stage
//               shared-memory ring (cp.async.bulk.tensor, 128-byte swizzle, mbarrier complete_tx),
//               keys two tiles ahead, values one
//   warp 1      QK^T issuer: S = Q K^T (both operands from shared memory) into one of three TMEM
//               accumulators
//   warp 2      PV issuer: O += P V into a fourth TMEM accumulator; P is read from TMEM (tcgen05.mma
//               with the A operand in tensor memory), V from shared memory
//               (kind::f16, fp32 accumulate; one elected thread each - issuing an MMA takes about as
//               long as executing it, so one thread cannot keep the pipe full and also wait on barriers)
//   warps 4-11  softmax, two warpgroups: warpgroup h owns keys [64h, 64h+64) of every tile and each of
//               its threads one query row (tcgen05.ld 32x32b); it applies the region temperature and
//               masks, agrees with the thread that holds the other half of the row on the tile's row
//               maximum (shared memory + mbarrier), keeps the running max and the sum of its own
//               columns in registers, and writes its half of P as packed fp16 back into tensor memory,
//               over the columns of S it has just read (tcgen05.st) - P never passes through shared
//               memory, and the S accumulator is handed back to the QK^T issuer when the PV product
//               has consumed it.  O is rescaled in TMEM only when the max grew by more than 2^8
//               (each half rescales, and at the end normalises and stores, its share of the channels).
// With few query tiles per launch the key tiles are also split over several CTAs whose partial
// results are merged by the CTA that finishes last; with many, the tiles that would make up a last,
// less than half full wave of CTAs are each split in two, so that the wave is half as long.
// Every mbarrier wait is bounded; on expiry the CTA records KVM_ERR_TIMEOUT and tears down.
#include "kvm_internal.h"
#include "tc_common.cuh"

namespace kvm {

struct AttnTcParams {
  int64_t q_row0, t0, m, win_row0, b, out_t0;
  int64_t so0, so1, so2;
  __nv_bfloat16* out;
  const float *tau_s, *tau_b;
  int32_t* status;
  float* part;       // split-KV partial results, [tile][split][D + 2][128] (see the epilogue)
  int32_t* part_cnt; // [tile] tickets, zero between launches
  int nq, Hq, Hkv, G;
  int qtiles;        // query tiles per (batch, head)
  int n_whole;       // the first n_whole (batch, head, query tile) tiles have one CTA each,
  int nsp_rest;      // the others nsp_rest CTAs each (key splits)
  int out_vec;       // rows of `out` can be written with 16-byte stores (alignment of base and strides)
};

// Output staging: a 128 x D bf16 tile, row-major in shared memory, the 16-byte chunks of a row
// permuted by the row index so that neither the row-per-thread writes nor the row-contiguous reads
// conflict on the banks.
template <int D>
__device__ __forceinline__ uint4* stage_chunk(uint8_t* stage, int row, int k) {
  constexpr int CPR = D / 8;   // chunks per row
  return reinterpret_cast<uint4*>(stage + row * (D * 2) + ((k ^ (row & (CPR - 1))) << 4));
}
// 32 fp32 accumulator values of one row -> four chunks (channels [32 c, 32 c + 32)), scaled
template <int D>
__device__ __forceinline__ void stage_row32(uint8_t* stage, int row, int c, const uint32_t (&r)[32], float inv) {
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(r[8 * q + 2 * i]) * inv, __uint_as_float(r[8 * q + 2 * i + 1]) * inv);
      w[i] = *reinterpret_cast<const uint32_t*>(&h);
    }
    *stage_chunk<D>(stage, row, 4 * c + q) = make_uint4(w[0], w[1], w[2], w[3]);
  }
}
// One warp writes rows [row0, row0 + nrows) of the staged tile to global memory, 32 / (D / 8) rows
// per instruction, every row as one contiguous run of 16-byte stores.
template <int D>
__device__ __forceinline__ void store_staged_rows(uint8_t* stage, __nv_bfloat16* out_row0, int64_t row_stride, int row0, int nrows,
                                                  int rows_valid, int lane) {
  constexpr int CPR = D / 8, RPI = 32 / CPR;
  const int k = lane % CPR;
  for (int r = row0 + lane / CPR; r < row0 + nrows; r += RPI) {
    if (r < rows_valid) {
      const uint4 v = *stage_chunk<D>(stage, r, k);
      *reinterpret_cast<uint4*>(out_row0 + (int64_t)r * row_stride + k * 8) = v;
    }
  }
}

template <int D>
struct AttnTcCfg {
  static constexpr int BM = 128, BN = 128, NS = 3, NSV = 2, NACC = 3;   // K stages, V stages, S/P accumulators
  static constexpr int NKB = D / 64;                 // 64-channel boxes per tile row
  static constexpr int BOX_BYTES = 128 * 128;        // 128 rows x 64 fp16
  static constexpr int TILE_BYTES = NKB * BOX_BYTES; // Q, K or V tile
  static constexpr int OFF_Q = 0;
  static constexpr int OFF_K = OFF_Q + TILE_BYTES;
  static constexpr int OFF_V = OFF_K + NS * TILE_BYTES;
  static constexpr int OFF_XM = OFF_V + NSV * TILE_BYTES;   // float [2][2][128]: row maxima exchanged between the column halves
  static constexpr int OFF_BAR = OFF_XM + 2 * 2 * 128 * 4;
  // + alignment slack; never less than half an SM so that one CTA (and one 512-column TMEM
  // allocation) is resident per SM
  static constexpr int SMEM_BYTES = (OFF_BAR + 256 + 1024) > 120 * 1024 ? (OFF_BAR + 256 + 1024) : 120 * 1024;
  static constexpr uint32_t TMEM_COLS = 512;
  static constexpr uint32_t COL_S = 0, COL_O = 384;   // S/P accumulator i at COL_S + 128 i
};

// K stages and the S / P accumulators cycle with period 3, V stages with period 2.
enum { BAR_QFULL = 0, BAR_KFULL = 1, BAR_KFREE = 4, BAR_VFULL = 7, BAR_VFREE = 9, BAR_SFULL = 11, BAR_PFULL = 14,
       BAR_PVDONE = 17, BAR_XM = 20, BAR_COUNT = 22 };

template <int D>
__global__ void __launch_bounds__(384, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapKs,
               const __grid_constant__ CUtensorMap mapVs, const __grid_constant__ CUtensorMap mapKw,
               const __grid_constant__ CUtensorMap mapVw, const AttnTcParams p) {
  using Cfg = AttnTcCfg<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = base + Cfg::OFF_Q;
  uint8_t* sK = base + Cfg::OFF_K;
  uint8_t* sV = base + Cfg::OFF_V;
  uint64_t* bars = reinterpret_cast<uint64_t*>(base + Cfg::OFF_BAR);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + BAR_COUNT);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // linear CTA index -> (tile, split): whole tiles first, then the split ones
  int tile, sp, nsp;
  if ((int)blockIdx.x < p.n_whole) { tile = blockIdx.x; sp = 0; nsp = 1; }
  else { const int r = (int)blockIdx.x - p.n_whole; tile = p.n_whole + r / p.nsp_rest; sp = r % p.nsp_rest; nsp = p.nsp_rest; }
  const int tile_slot = tile - p.n_whole;   // index among the split tiles (partial results, tickets)
  const int qt = tile % p.qtiles, bh = tile / p.qtiles;
  const int bb = bh / p.Hq, hq = bh % p.Hq, hk = hq / p.G;
  const int u = bb * p.Hkv + hk;
  const int rows_valid = min(128, p.nq - qt * 128);
  const int64_t t_first = p.t0 + (int64_t)qt * 128;
  const int64_t t_last = t_first + rows_valid - 1;
  const int nst = (int)((p.m + 127) / 128);
  const int nwt = (int)((t_last - p.b + 1 + 127) / 128);
  // Split-KV: with few (batch, head, query tile) triples a launch is cut along the keys as well;
  // CTA sp of nsp walks tiles [jbase, jbase + ntiles) of the nst + nwt tiles of its query tile,
  // and the partial results are merged by whichever CTA of the tile finishes last.
  const int ntot = nst + nwt;
  const int per_split = (ntot + nsp - 1) / nsp;
  const int jbase = min(ntot, sp * per_split);
  const int ntiles = min(ntot, jbase + per_split) - jbase;   // tiles of this CTA (0 is possible)

  if (tid == 0) {
    tc::prefetch_tmap(&mapQ); tc::prefetch_tmap(&mapKs); tc::prefetch_tmap(&mapVs);
    tc::prefetch_tmap(&mapKw); tc::prefetch_tmap(&mapVw);
    tc::mbar_init(&bars[BAR_QFULL], 1);
    for (int s = 0; s < 3; ++s) {
      tc::mbar_init(&bars[BAR_KFULL + s], 1);
      tc::mbar_init(&bars[BAR_KFREE + s], 1);
      tc::mbar_init(&bars[BAR_SFULL + s], 1);
      tc::mbar_init(&bars[BAR_PFULL + s], 8);
      tc::mbar_init(&bars[BAR_PVDONE + s], 1);
    }
    for (int s = 0; s < Cfg::NSV; ++s) {
      tc::mbar_init(&bars[BAR_VFULL + s], 1);
      tc::mbar_init(&bars[BAR_VFREE + s], 1);
      tc::mbar_init(&bars[BAR_XM + s], 8);
    }
    *abort_flag = 0;
    tc::fence_barrier_init();
  }
  // Three key stages, two value stages: keys run two tiles ahead of the product that needs them,
  // values one.  A K stage is released as soon as its QK^T product has completed, a V stage after
  // its PV product.  (Called by thread 0 only.)
  auto load_kv = [&](int j, bool keys) -> bool {
    const int ns = keys ? Cfg::NS : Cfg::NSV;
    const int s = j % ns;
    if (j >= ns && !tc::mbar_wait(&bars[(keys ? BAR_KFREE : BAR_VFREE) + s], ((j / ns) - 1) & 1)) return false;
    const int gj = jbase + j;
    const bool st = gj < nst;
    const int row = st ? gj * 128 : (int)(p.win_row0 + (int64_t)(gj - nst) * 128);
    uint64_t* full = &bars[(keys ? BAR_KFULL : BAR_VFULL) + s];
    uint8_t* dst = (keys ? sK : sV) + s * Cfg::TILE_BYTES;
    const CUtensorMap* map = keys ? (st ? &mapKs : &mapKw) : (st ? &mapVs : &mapVw);
    tc::mbar_expect_tx(full, Cfg::TILE_BYTES);
    for (int kb = 0; kb < Cfg::NKB; ++kb)
      tc::tma_load_3d(dst + kb * Cfg::BOX_BYTES, map, full, kb * 64, row, u);
    return true;
  };
  if (tid == 0) {
    // the first loads start before the tensor memory is allocated and the roles split: they need
    // nothing but their own barriers (no stage is waited for yet)
    tc::fence_proxy_async();
    tc::mbar_expect_tx(&bars[BAR_QFULL], Cfg::TILE_BYTES);
    for (int kb = 0; kb < Cfg::NKB; ++kb)
      tc::tma_load_3d(sQ + kb * Cfg::BOX_BYTES, &mapQ, &bars[BAR_QFULL], kb * 64, (int)(p.q_row0 + qt * 128), bh);
    if (ntiles > 0) load_kv(0, true);
    if (ntiles > 1) load_kv(1, true);
    if (ntiles > 0) load_kv(0, false);
  }
  if (warp == 1) {
    tc::tmem_alloc(tmem_slot, Cfg::TMEM_COLS);
    tc::tmem_relinquish();
  }
  tc::tc_fence_before();
  __syncthreads();
  tc::tc_fence_after();
  const uint32_t tmem = *tmem_slot;

#define KVM_WAIT(bar, par)                                   \
  if (!tc::mbar_wait((bar), (par))) {                        \
    atomicExch(p.status, (int)KVM_ERR_TIMEOUT);              \
    *abort_flag = 1;                                         \
    break;                                                   \
  }

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    if (lane == 0) {
      bool okp = true;
      for (int j = 0; j < ntiles && okp; ++j) {
        if (*abort_flag) break;
        if (j + 2 < ntiles && !load_kv(j + 2, true)) { okp = false; break; }
        if (j + 1 < ntiles && !load_kv(j + 1, false)) { okp = false; break; }
      }
      if (!okp) { atomicExch(p.status, (int)KVM_ERR_TIMEOUT); *abort_flag = 1; }
    }
  } else if (warp == 1) {
    // ------------------------------ QK^T issuer ------------------------------
    // Issuing a tcgen05.mma takes about as long as executing it, so the two products of a tile are
    // issued by two threads: the waits, fences and commits of one overlap the issue of the other.
    if (lane == 0) {
      constexpr uint32_t IDESC_QK = tc::idesc_f16(128, 128, false);
      const uint32_t aQ = tc::smem_u32(sQ), aK = tc::smem_u32(sK);
      bool dead = false;
      do {
        if (!tc::mbar_wait(&bars[BAR_QFULL], 0)) { dead = true; break; }
        for (int j = 0; j < ntiles; ++j) {
          const int s = j % Cfg::NS;
          if (*abort_flag) { dead = true; break; }
          // accumulator j % 3 also holds P of tile j-3 (fp16, written over the columns the softmax
          // has read): it is free once the PV product of tile j-3 has consumed it
          const int acc = j % Cfg::NACC;
          if (j >= Cfg::NACC && !tc::mbar_wait(&bars[BAR_PVDONE + acc], ((j / Cfg::NACC) - 1) & 1)) { dead = true; break; }
          if (!tc::mbar_wait(&bars[BAR_KFULL + s], (j / Cfg::NS) & 1)) { dead = true; break; }
          tc::tc_fence_after();
          const uint32_t dS = tmem + Cfg::COL_S + 128 * acc;
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks) {
            const uint32_t off = (ks / 4) * Cfg::BOX_BYTES + (ks % 4) * 32;
            tc::mma_f16_ss(dS, tc::smem_desc_sw128(aQ + off, 16, 1024),
                           tc::smem_desc_sw128(aK + s * Cfg::TILE_BYTES + off, 16, 1024), IDESC_QK, ks > 0);
          }
          tc::mma_commit(&bars[BAR_SFULL + acc]);
          tc::mma_commit(&bars[BAR_KFREE + s]);
        }
      } while (false);
      if (dead) { atomicExch(p.status, (int)KVM_ERR_TIMEOUT); *abort_flag = 1; }
    }
  } else if (warp == 2) {
    // ------------------------------ PV issuer ------------------------------
    if (lane == 0) {
      constexpr uint32_t IDESC_PV = tc::idesc_f16(128, D, true);
      const uint32_t aV = tc::smem_u32(sV);
      bool dead = false;
      for (int j = 0; j < ntiles; ++j) {
        const int s = j % Cfg::NSV, acc = j % Cfg::NACC;
        if (*abort_flag) { dead = true; break; }
        if (!tc::mbar_wait(&bars[BAR_VFULL + s], (j / Cfg::NSV) & 1)) { dead = true; break; }
        if (!tc::mbar_wait(&bars[BAR_PFULL + acc], (j / Cfg::NACC) & 1)) { dead = true; break; }
        tc::tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
          // P comes from TMEM (A operand, one row per lane, two fp16 per column): the column half h
          // of tile j sits in the first 32 columns of that half's share of its S accumulator; a
          // k-step of 16 keys is 8 columns.
          const uint32_t aP = tmem + Cfg::COL_S + 128 * acc + 64 * (kk >> 2) + 8 * (kk & 3);
          const uint32_t offV = kk * 2048;   // 16 key rows x 128 B
          tc::mma_f16_ts(tmem + Cfg::COL_O, aP, tc::smem_desc_sw128(aV + s * Cfg::TILE_BYTES + offV, Cfg::BOX_BYTES, 1024),
                         IDESC_PV, (j > 0 || kk > 0) ? 1u : 0u);
        }
        tc::mma_commit(&bars[BAR_PVDONE + acc]);
        tc::mma_commit(&bars[BAR_VFREE + s]);
      }
      if (dead) { atomicExch(p.status, (int)KVM_ERR_TIMEOUT); *abort_flag = 1; }
    }
  } else if (warp == 3) {
    // spare warp: keeps the softmax warps aligned to the TMEM lane quarters
  } else {
    // ------------------------------ softmax / epilogue ------------------------------
    // Two warpgroups split every key tile by columns: half 0 owns keys 0..63 of the tile, half 1
    // keys 64..127, one thread per (row, half).  The two threads of a row agree on the row maximum
    // of each tile through shared memory (an mbarrier per tile parity, so the wait is bounded), keep
    // the same running maximum, and each keeps the sum of its own columns; all PV products go into
    // one O accumulator, of which each half rescales and finally stores its share of the channels.
    const int half = (warp - 4) >> 2;                 // which 64 columns of every tile
    const int quarter = warp & 3;                     // TMEM lane quarter this warp may access
    const int row = quarter * 32 + lane;              // query row inside the tile
    const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
    constexpr int HD = D / 2;
    const uint32_t to_mine = tmem + lane_base + Cfg::COL_O + half * HD;   // this thread's share of O
    float* xm = reinterpret_cast<float*>(base + Cfg::OFF_XM);             // [parity][half][row]
    const int64_t t_row = t_first + row;
    const float kLog2e = 1.4426950408889634f;
    const float sc_s = p.tau_s[hq] * rsqrtf((float)D) * kLog2e;
    const float sc_b = p.tau_b[hq] * rsqrtf((float)D) * kLog2e;
    float m_run = -INFINITY, l_run = 0.f;
    bool ok = true;
    for (int j = 0; j < ntiles && ok; ++j) {
      do {
        ok = false;
        const int acc = j % Cfg::NACC;
        KVM_WAIT(&bars[BAR_SFULL + acc], (j / Cfg::NACC) & 1);
        tc::tc_fence_after();
        const uint32_t ts = tmem + lane_base + Cfg::COL_S + 128 * acc + half * 64;
        float x[64];
        {
#pragma unroll
          for (int c = 0; c < 2; ++c) {
            uint32_t r[32];
            tc::tmem_ld32(ts + c * 32, r);
#pragma unroll
            for (int i = 0; i < 32; ++i) x[c * 32 + i] = __uint_as_float(r[i]);
          }
          tc::tmem_wait_ld();
        }
        // region scale (folded into the exponent) and masks; the scale is positive, so the row
        // maximum can be taken on the raw products
        const int gj = jbase + j;
        const bool st = gj < nst;
        const float sc = st ? sc_s : sc_b;
        int64_t nvis;   // number of visible columns of this tile for this row
        if (st) nvis = p.m - (int64_t)gj * 128;
        else nvis = t_row - (p.b + (int64_t)(gj - nst) * 128) + 1;
        const int vis = (int)max((int64_t)0, min((int64_t)64, nvis - half * 64));
        if (vis != 64) {
#pragma unroll
          for (int c = 0; c < 64; ++c) x[c] = (c < vis) ? x[c] : -INFINITY;
        }
        float mx;
        {   // four chains: a single chain of 64 dependent maxima is latency bound
          float m4[4] = {x[0], x[1], x[2], x[3]};
#pragma unroll
          for (int c = 4; c < 64; ++c) m4[c & 3] = fmaxf(m4[c & 3], x[c]);
          mx = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
        }
        // the other half's maximum of this row
        xm[((j & 1) * 2 + half) * 128 + row] = mx;
        __syncwarp();
        if (lane == 0) tc::mbar_arrive(&bars[BAR_XM + (j & 1)]);
        KVM_WAIT(&bars[BAR_XM + (j & 1)], (j >> 1) & 1);
        mx = fmaxf(mx, xm[((j & 1) * 2 + (1 - half)) * 128 + row]);
        const float mnew = fmaxf(m_run, mx * sc);
        if (j == 0) {
          m_run = mnew;
        } else {
          const bool need = mnew > m_run + 8.0f;
          if (__any_sync(0xffffffffu, need)) {   // the same decision in both warps that share these rows
            // all earlier PV products must have landed before O is touched (commits complete in order)
            KVM_WAIT(&bars[BAR_PVDONE + (j - 1) % Cfg::NACC], ((j - 1) / Cfg::NACC) & 1);
            tc::tc_fence_after();
            const float corr = (m_run == -INFINITY) ? 0.f : tc::ex2_approx(m_run - mnew);
            l_run *= corr;
            m_run = mnew;
#pragma unroll
            for (int c = 0; c < HD / 32; ++c) {
              uint32_t r[32];
              tc::tmem_ld32(to_mine + c * 32, r);
              tc::tmem_wait_ld();
#pragma unroll
              for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * corr);
              tc::tmem_st32(to_mine + c * 32, r);
            }
            tc::tmem_wait_st();
          }
        }
        const float neg_m = (m_run == -INFINITY) ? 0.f : -m_run;
        float lsum = 0.f, lsum2 = 0.f;
        // P row -> tensor memory, as the A operand of the PV product: this thread's lane, two fp16
        // per column, over the first 32 of the 64 columns of S that it has just read out (the QK^T
        // issuer does not touch this accumulator again before the PV product has consumed it)
        uint32_t w[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const float p0 = tc::ex2_approx(fmaf(x[2 * i], sc, neg_m));
          // every fourth exponential on the FMA pipe instead of the special-function unit, which
          // bounds this loop (P is rounded to fp16 anyway: relative error of the polynomial < 5e-5)
          const float p1 = (i & 1) ? tc::ex2_poly(fmaf(x[2 * i + 1], sc, neg_m)) : tc::ex2_approx(fmaf(x[2 * i + 1], sc, neg_m));
          if (i & 1) lsum += p0 + p1; else lsum2 += p0 + p1;
          const __half2 h = __floats2half2_rn(p0, p1);
          w[i] = *reinterpret_cast<const uint32_t*>(&h);
        }
        lsum += lsum2;
        tc::tmem_st32(ts, w);
        tc::tmem_wait_st();
        l_run += lsum;
        tc::tc_fence_before();
        __syncwarp();
        if (lane == 0) tc::mbar_arrive(&bars[BAR_PFULL + acc]);
        ok = true;
      } while (false);
    }
    // Epilogue: the row sum is the sum of the two halves' sums (exchanged through shared memory, laid
    // over the value stages, which nothing reads any more once the last PV product is done); half h
    // normalises and stores channels [h D/2, (h+1) D/2).
    float* xl = reinterpret_cast<float*>(sV);           // [2][128]
    int* last_flag = reinterpret_cast<int*>(tmem_slot + 2);
    do {
      if (!ok) break;
      if (ntiles > 0) {
        ok = false;
        KVM_WAIT(&bars[BAR_PVDONE + (ntiles - 1) % Cfg::NACC], ((ntiles - 1) / Cfg::NACC) & 1);
        tc::tc_fence_after();
        ok = true;
      }
      xl[half * 128 + row] = l_run;
    } while (false);
    // every softmax thread reaches this barrier, whether or not its waits succeeded
    asm volatile("bar.sync 1, 256;" ::: "memory");
    const bool good = ok && !*abort_flag;
    const float lsum2 = l_run + xl[(1 - half) * 128 + row];
    __nv_bfloat16* orow = p.out + bb * p.so0 + hq * p.so1 + (p.out_t0 + (int64_t)qt * 128 + row) * p.so2 + half * HD;
    if (nsp == 1 && p.out_vec) {
      // rows go through shared memory (the key stages, idle by now) so that the global stores are
      // whole rows of 16-byte pieces instead of one 4-byte piece per row and instruction
      if (good) {
        const float inv = 1.f / lsum2;
#pragma unroll
        for (int c = 0; c < HD / 32; ++c) {
          uint32_t r[32];
          tc::tmem_ld32(to_mine + c * 32, r);
          tc::tmem_wait_ld();
          stage_row32<D>(sK, row, half * (HD / 32) + c, r, inv);
        }
      }
      asm volatile("bar.sync 1, 256;" ::: "memory");
      if (good)
        store_staged_rows<D>(sK, p.out + bb * p.so0 + hq * p.so1 + (p.out_t0 + (int64_t)qt * 128) * p.so2, p.so2,
                             (warp - 4) * 16, 16, rows_valid, lane);
    } else if (nsp == 1) {
      if (good) {
        const float inv = 1.f / lsum2;
#pragma unroll
        for (int c = 0; c < HD / 32; ++c) {
          uint32_t r[32];
          tc::tmem_ld32(to_mine + c * 32, r);
          tc::tmem_wait_ld();
          if (row < rows_valid) {
#pragma unroll
            for (int i = 0; i < 16; ++i)
              reinterpret_cast<__nv_bfloat162*>(orow + c * 32)[i] =
                  __floats2bfloat162_rn(__uint_as_float(r[2 * i]) * inv, __uint_as_float(r[2 * i + 1]) * inv);
          }
        }
      }
    } else {
      // Partial result of this split: unnormalised O (relative to m_run), m_run and the sum, column-major
      // ([channel][row]) so that the rows of a warp are contiguous.
      const int tile_id = tile_slot;
      float* mine = p.part + ((int64_t)tile_id * nsp + sp) * (D + 2) * 128;
      if (good && ntiles > 0) {
#pragma unroll
        for (int c = 0; c < HD / 32; ++c) {
          uint32_t r[32];
          tc::tmem_ld32(to_mine + c * 32, r);
          tc::tmem_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; ++i) mine[(half * HD + c * 32 + i) * 128 + row] = __uint_as_float(r[i]);
        }
      }
      if (half == 0) {
        mine[(D + 0) * 128 + row] = (good && ntiles > 0) ? m_run : -INFINITY;
        mine[(D + 1) * 128 + row] = (good && ntiles > 0) ? lsum2 : 0.f;
      }
      __threadfence();
      asm volatile("bar.sync 1, 256;" ::: "memory");
      if (warp == 4 && lane == 0) *last_flag = atomicAdd(&p.part_cnt[tile_id], 1) == nsp - 1 ? 1 : 0;
      asm volatile("bar.sync 1, 256;" ::: "memory");
      if (*last_flag) {   // the last split of the tile to arrive merges all of them (nobody waits)
        __threadfence();
        if (warp == 4 && lane == 0) p.part_cnt[tile_id] = 0;
        const float* allp = p.part + (int64_t)tile_id * nsp * (D + 2) * 128;
        float mstar = -INFINITY;
        for (int z = 0; z < nsp; ++z) mstar = fmaxf(mstar, __ldcg(allp + ((int64_t)z * (D + 2) + D) * 128 + row));
        float accv[HD];
#pragma unroll
        for (int c = 0; c < HD; ++c) accv[c] = 0.f;
        float den = 0.f;
        for (int z = 0; z < nsp; ++z) {
          const float* pz = allp + (int64_t)z * (D + 2) * 128;
          const float mz = __ldcg(pz + D * 128 + row);
          if (mz == -INFINITY) continue;
          const float wz = tc::ex2_approx(mz - mstar);
          den += __ldcg(pz + (D + 1) * 128 + row) * wz;
#pragma unroll
          for (int c = 0; c < HD; ++c) accv[c] += __ldcg(pz + (half * HD + c) * 128 + row) * wz;
        }
        const float inv = 1.f / den;
        if (p.out_vec) {   // (uniform over the CTA, as is last_flag: every softmax thread reaches the barrier)
#pragma unroll
          for (int c = 0; c < HD / 8; ++c) {
            uint32_t w[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const __nv_bfloat162 h = __floats2bfloat162_rn(accv[8 * c + 2 * i] * inv, accv[8 * c + 2 * i + 1] * inv);
              w[i] = *reinterpret_cast<const uint32_t*>(&h);
            }
            *stage_chunk<D>(sK, row, half * (HD / 8) + c) = make_uint4(w[0], w[1], w[2], w[3]);
          }
          asm volatile("bar.sync 1, 256;" ::: "memory");
          store_staged_rows<D>(sK, p.out + bb * p.so0 + hq * p.so1 + (p.out_t0 + (int64_t)qt * 128) * p.so2, p.so2,
                               (warp - 4) * 16, 16, rows_valid, lane);
        } else if (row < rows_valid) {
#pragma unroll
          for (int c = 0; c < HD / 2; ++c)
            reinterpret_cast<__nv_bfloat162*>(orow)[c] = __floats2bfloat162_rn(accv[2 * c] * inv, accv[2 * c + 1] * inv);
        }
      }
    }
  }
#undef KVM_WAIT
  tc::tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc::tmem_dealloc(tmem, Cfg::TMEM_COLS);
  }
}

// ------------------------------------------------------------------------------------------

bool encode_tmap_rows(CUtensorMap* map, const void* base, int d, int64_t rows, int64_t units, int box_rows) {
  typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                               const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                               CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  static EncodeFn fn = nullptr;
  if (!fn) {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) != cudaSuccess || !ptr) {
      cudaGetLastError();
      return false;
    }
    fn = reinterpret_cast<EncodeFn>(ptr);
  }
  cuuint64_t gdim[3] = {(cuuint64_t)d, (cuuint64_t)rows, (cuuint64_t)units};
  cuuint64_t gstr[2] = {(cuuint64_t)d * 2, (cuuint64_t)rows * d * 2};
  cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<void*>(base), gdim, gstr, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int launch_attn_tc(State* st, const AttnArgs& a, cudaStream_t s) {
  AttnTcParams p;
  p.q_row0 = a.q_row0; p.t0 = a.t0; p.m = a.m; p.win_row0 = a.win_row0; p.b = a.b; p.out_t0 = a.out_t0;
  p.so0 = a.so[0]; p.so1 = a.so[1]; p.so2 = a.so[2];
  p.out = a.out; p.tau_s = st->tau_s; p.tau_b = st->tau_b; p.status = st->status;
  p.nq = a.nq; p.Hq = st->Hq; p.Hkv = st->Hkv; p.G = st->G;
  p.part = st->attnPart; p.part_cnt = st->attnCnt;
  p.out_vec = (reinterpret_cast<uintptr_t>(a.out) % 16 == 0 && a.so[0] % 8 == 0 && a.so[1] % 8 == 0 && a.so[2] % 8 == 0) ? 1 : 0;
  // key splits when there are few query tiles: up to a quarter of the GPU (the folds of the block
  // before run beside this kernel and are usually the longer chain; measured: a wider attention
  // kernel only takes SMs away from them), at least two key tiles per split
  const int qtiles = (a.nq + 127) / 128;
  const int ctas = qtiles * st->B * st->Hq;
  int nsp = 1;
  if (ctas <= kAttnSplitTiles) {
    nsp = kAttnSplitTiles / ctas;
    const int ntot_min = (int)((a.m + 127) / 128) + 1;
    if (nsp > ntot_min / 2) nsp = ntot_min / 2;
    if (nsp > kAttnMaxSplits) nsp = kAttnMaxSplits;
    if (nsp < 1) nsp = 1;
  }
  // Many tiles: when the last wave of one-CTA-per-SM would be less than half full, its tiles are split
  // in two (the partial-result buffer holds 2 * kAttnSplitTiles tiles of two splits).
  const int tiles = qtiles * st->B * st->Hq;
  int n_whole = nsp > 1 ? 0 : tiles, nsp_rest = nsp;
  if (nsp == 1 && tiles > 148) {
    const int rem = tiles % 148;
    const int ntot_min2 = (int)((a.m + 127) / 128) + 1;
    if (rem > 0 && rem <= 2 * kAttnSplitTiles && ntot_min2 >= 4) { n_whole = tiles - rem; nsp_rest = 2; }
  }
  p.qtiles = qtiles; p.n_whole = n_whole; p.nsp_rest = nsp_rest;
  dim3 grid(n_whole + (tiles - n_whole) * nsp_rest);
  const CUtensorMap* tm = reinterpret_cast<const CUtensorMap*>(st->tmaps);
  const int ks = (st->nfolds & 1) ? 6 : 1, vs = (st->nfolds & 1) ? 7 : 2;   // readout copy of the current version
  if (st->d == 128) {
    attn_tc_kernel<128><<<grid, 384, AttnTcCfg<128>::SMEM_BYTES, s>>>(tm[0], tm[ks], tm[vs], tm[3], tm[4], p);
  } else {
    attn_tc_kernel<64><<<grid, 384, AttnTcCfg<64>::SMEM_BYTES, s>>>(tm[0], tm[ks], tm[vs], tm[3], tm[4], p);
  }
  return 1;
}

// Self test of the bounded waits (kvm_debug_expire_wait): the wait below can only run out.
__global__ void expire_wait_kernel(int32_t* status, uint32_t spins) {
  __shared__ uint64_t bar;
  tc::mbar_init(&bar, 1);
  tc::fence_barrier_init();
  if (!tc::mbar_wait(&bar, 0, spins)) atomicExch(status, (int)KVM_ERR_TIMEOUT);
}

void launch_expire_wait(State* st, int spins, cudaStream_t s) { expire_wait_kernel<<<1, 1, 0, s>>>(st->status, (uint32_t)spins); }

bool setup_attn_tc(State* st) {
  CUtensorMap* tm = reinterpret_cast<CUtensorMap*>(st->tmaps);
  bool ok = encode_tmap_rows(&tm[0], st->stQ, st->d, st->Tcall, (int64_t)st->B * st->Hq, 128);
  ok = ok && encode_tmap_rows(&tm[1], st->KhatBuf[0], st->d, st->Mcap, st->U, 128);
  ok = ok && encode_tmap_rows(&tm[2], st->VhatBuf[0], st->d, st->Mcap, st->U, 128);
  ok = ok && encode_tmap_rows(&tm[6], st->KhatBuf[1], st->d, st->Mcap, st->U, 128);
  ok = ok && encode_tmap_rows(&tm[7], st->VhatBuf[1], st->d, st->Mcap, st->U, 128);
  ok = ok && encode_tmap_rows(&tm[3], st->stK, st->d, st->stRows, st->U, 128);
  ok = ok && encode_tmap_rows(&tm[4], st->stV, st->d, st->stRows, st->U, 128);
  if (!ok) return false;
  if (cudaFuncSetAttribute(attn_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttnTcCfg<128>::SMEM_BYTES) != cudaSuccess) return false;
  if (cudaFuncSetAttribute(attn_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttnTcCfg<64>::SMEM_BYTES) != cudaSuccess) return false;
  return true;
}

}  // namespace kvm
