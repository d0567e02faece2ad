// Routing filter on the tensor cores: approximate similarities S = Kbar . LN_s(S^K)^T between
// the overflow block's memory keys (fp16, up to 256 tokens = two 128-row M tiles) and a split of
// the state's readout keys, reduced on the fly to the rows whose similarity lies within the
// rounding bound of the row maximum (Section 3.2 "Append" score and "Merge" arg max; the exact
// decision is taken later in fp64 on these candidates only).  The split is streamed ONCE: per
// 128-row tile a thread (one token) takes the maxima of its four 32-column chunks (three-input
// maxima: half an instruction per element), raises its running maximum, and records every chunk
// whose maximum reaches (running maximum - bound): the chunk's 32 products go to the token's list in
// global memory as they are.  The running maximum only grows, so the recorded chunks are a superset
// of the chunks that hold a row within the bound of the final maximum; after its last tile the thread
// goes back over its own few records (their maxima first: usually one chunk survives) and lists the
// rows above (final maximum - bound).  A token meets a new running maximum about ln(tiles) times,
// and a new maximum nearly always makes the earlier records obsolete, so the list is restarted in
// place and stays a record or two (128 bytes each) long, while the state is read, and multiplied,
// once.
//
//   warp 0      TMA producer: the Kbar tiles once, then 128-row tiles of K_hat in a 3-stage ring
//   warps 1, 10 MMA issuers, one thread per M tile: per key tile one 128x128x(d) product into a
//               double-buffered TMEM accumulator (tcgen05.mma kind::f16)
//   warps 2-9   epilogue: one thread per token row; tcgen05.ld of its 128 similarities, chunk maxima,
//               running maximum, recorded chunks straight to global memory
// Output per (unit, split, token): candI[0..kTopK) candidate rows in the order found (-1 = none),
// candV[0] = the split's maximum over rows >= S, candV[1] = number of candidates found (more than
// kTopK = the list overflowed - or more chunks were met than could be recorded - and the decision
// kernel scans all rows for that token).  chunkMax / chunkMeta / chunkVal are the threads' scratch.
// All waits are bounded (error word + normal teardown on expiry).
#include "kvm_internal.h"
#include "tc_common.cuh"

namespace kvm {

struct RouteTcParams {
  float* candV;
  int32_t* candI;
  float* chunkMax;
  int2* chunkMeta;
  float* chunkVal;
  int32_t* status;
  const float* kbarNorm;   // [U, Cmax] upper bound of ||kbar_j||
  int a_unit0;             // first unit of this block's slot in the memory-key tensor map
  float* gramT;            // [slots][U, Cmax, Cmax]: output of the new-row filter launch (gram_mode), see below
  int gram_mode, U;        // gram_mode: grid (1, U, blocks), block z uses slot a_unit0 / U + z
  float thr_coeff;         // candidate window = thr_coeff * ||kbar_j|| + 1e-5
  int64_t m;
  int C, Cmax, nsplit, S;
};

template <int D>
struct RouteTcCfg {
  static constexpr int NS = 3, MT = 2;
  static constexpr int NKB = D / 64;
  static constexpr int BOX_BYTES = 128 * 128;
  static constexpr int TILE_BYTES = NKB * BOX_BYTES;
  static constexpr int OFF_A = 0;
  static constexpr int OFF_B = OFF_A + MT * TILE_BYTES;
  // the first two records of every token (32 products each), [record][16-byte piece][token]: with the list
  // restarted at nearly every new maximum a token rarely has more, and a record costs eight 16-byte stores
  // that every lane of a warp waits for whenever one of its 32 tokens records
  static constexpr int OFF_REC = OFF_B + NS * TILE_BYTES;
  static constexpr int REC_SLOTS = 2;
  static constexpr int OFF_BAR = OFF_REC + REC_SLOTS * 8 * 256 * 16;
  static constexpr int SMEM_BYTES = (OFF_BAR + 256 + 1024) > 120 * 1024 ? (OFF_BAR + 256 + 1024) : 120 * 1024;
  static constexpr uint32_t TMEM_COLS = 512;   // [buffer][M tile] x 128 columns
};

enum { RB_AFULL = 0, RB_BFULL = 1, RB_BFREE = 4, RB_SFULL = 7, RB_ACCFREE = 9, RB_COUNT = 11 };

template <int D>
__global__ void __launch_bounds__(352, 1)
route_filter_tc_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB,
                       const __grid_constant__ CUtensorMap mapH, const RouteTcParams p) {
  using Cfg = RouteTcCfg<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sA = base + Cfg::OFF_A;
  uint8_t* sB = base + Cfg::OFF_B;
  uint64_t* bars = reinterpret_cast<uint64_t*>(base + Cfg::OFF_BAR);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + RB_COUNT);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int split = blockIdx.x, u = blockIdx.y;
  const int mt_used = (p.C + 127) / 128;
  // New-row filter mode (a launch of its own, ahead of the folds: it needs the block's keys only):
  // the would-be row keys LN_s(kbar_a) are the M operand, the memory keys kbar_j the N operand, one
  // pass, and the products themselves are stored, gramT[a][j]; which rows a exist is known later.
  const bool gram = p.gram_mode != 0;
  const int a_unit = p.a_unit0 + (gram ? (int)blockIdx.z * p.U : 0) + u;
  int64_t per = (p.m + p.nsplit - 1) / p.nsplit;
  per = (per + 127) / 128 * 128;
  const int64_t i0 = gram ? 0 : (int64_t)split * per;
  const int64_t i1 = gram ? (int64_t)p.C : min(p.m, i0 + per);
  const int ntiles = i1 > i0 ? (int)((i1 - i0 + 127) / 128) : 0;
  const int nsteps = ntiles;

  if (tid == 0) {
    tc::mbar_init(&bars[RB_AFULL], 1);
    for (int s = 0; s < Cfg::NS; ++s) {
      tc::mbar_init(&bars[RB_BFULL + s], 1);
      tc::mbar_init(&bars[RB_BFREE + s], mt_used);      // one commit per issuer
    }
    tc::mbar_init(&bars[RB_SFULL + 0], mt_used);
    tc::mbar_init(&bars[RB_SFULL + 1], mt_used);
    tc::mbar_init(&bars[RB_ACCFREE + 0], 4 * mt_used);
    tc::mbar_init(&bars[RB_ACCFREE + 1], 4 * mt_used);
    *abort_flag = 0;
    tc::fence_barrier_init();
  }
  if (warp == 1) {
    tc::tmem_alloc(tmem_slot, Cfg::TMEM_COLS);
    tc::tmem_relinquish();
  }
  tc::tc_fence_before();
  __syncthreads();
  tc::tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  // the kernel launched behind this one may begin its set-up now (it waits for this grid to finish
  // before it reads anything written here)
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  if (warp == 0) {
    if (lane == 0) {
      tc::prefetch_tmap(&mapA); tc::prefetch_tmap(&mapB); tc::prefetch_tmap(&mapH);
      tc::mbar_expect_tx(&bars[RB_AFULL], mt_used * Cfg::TILE_BYTES);
      for (int mt = 0; mt < mt_used; ++mt)
        for (int kb = 0; kb < Cfg::NKB; ++kb)
          tc::tma_load_3d(sA + mt * Cfg::TILE_BYTES + kb * Cfg::BOX_BYTES, gram ? &mapH : &mapA, &bars[RB_AFULL], kb * 64, mt * 128, a_unit);
      // the readout keys are written by the apply kernel of the fold before this one: wait for it here
      // (the set-up above and the load of the block's own keys run beside its tail)
      asm volatile("griddepcontrol.wait;" ::: "memory");
      for (int j = 0; j < nsteps; ++j) {
        const int s = j % Cfg::NS;
        const int jt = j;
        if (*abort_flag) break;
        if (j >= Cfg::NS && !tc::mbar_wait(&bars[RB_BFREE + s], ((j / Cfg::NS) - 1) & 1)) {
          atomicExch(p.status, (int)KVM_ERR_TIMEOUT); *abort_flag = 1; break;
        }
        tc::mbar_expect_tx(&bars[RB_BFULL + s], Cfg::TILE_BYTES);
        for (int kb = 0; kb < Cfg::NKB; ++kb)
          tc::tma_load_3d(sB + s * Cfg::TILE_BYTES + kb * Cfg::BOX_BYTES, gram ? &mapA : &mapB, &bars[RB_BFULL + s], kb * 64,
                          (int)(i0 + (int64_t)jt * 128), gram ? a_unit : u);
      }
    }
  } else if (warp == 1 || warp == 10) {
    // one issuer thread per 128-token M tile: issuing an MMA takes longer than executing it, so one
    // thread cannot keep the pipe busy
    const int mt = warp == 1 ? 0 : 1;
    if (lane == 0 && mt < mt_used) {
      constexpr uint32_t IDESC = tc::idesc_f16(128, 128, false);
      const uint32_t aA = tc::smem_u32(sA), aB = tc::smem_u32(sB);
      bool dead = !tc::mbar_wait(&bars[RB_AFULL], 0);
      for (int j = 0; j < nsteps && !dead; ++j) {
        const int s = j % Cfg::NS, buf = j & 1;
        if (*abort_flag) { dead = true; break; }
        if (!tc::mbar_wait(&bars[RB_BFULL + s], (j / Cfg::NS) & 1)) { dead = true; break; }
        if (j >= 2 && !tc::mbar_wait(&bars[RB_ACCFREE + buf], ((j >> 1) - 1) & 1)) { dead = true; break; }
        tc::tc_fence_after();
        const uint32_t dS = tmem + buf * 256 + mt * 128;
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          const uint32_t off = (ks / 4) * Cfg::BOX_BYTES + (ks % 4) * 32;
          tc::mma_f16_ss(dS, tc::smem_desc_sw128(aA + mt * Cfg::TILE_BYTES + off, 16, 1024),
                         tc::smem_desc_sw128(aB + s * Cfg::TILE_BYTES + off, 16, 1024), IDESC, ks > 0);
        }
        tc::mma_commit(&bars[RB_SFULL + buf]);
        tc::mma_commit(&bars[RB_BFREE + s]);
      }
      if (dead) { atomicExch(p.status, (int)KVM_ERR_TIMEOUT); *abort_flag = 1; }
    }
  } else {
    const int e = warp - 2;
    const int mt = e >> 2;
    if (mt < mt_used) {
      const int quarter = warp & 3;
      const int tok = mt * 128 + quarter * 32 + lane;
      const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
      int nrec = 0;
      int sink_rec = 0;            // 1 once the record of the chunk that holds the sink rows sits in slot 0
      // records 0 and 1: products in shared memory, first row / valid rows / maximum in registers
      uint4* srec = reinterpret_cast<uint4*>(base + Cfg::OFF_REC) + tok;
      int rrow[2] = {0, 0};
      uint32_t rval[2] = {0u, 0u};
      float rmax[2] = {-INFINITY, -INFINITY};
      float mx = -INFINITY;        // running maximum over rows >= S of this split
      const bool live = tok < p.C;   // (rows of the M tile past the block record nothing)
      const float thr = live ? p.thr_coeff * p.kbarNorm[(int64_t)u * p.Cmax + tok] + 1e-5f : 0.f;
      const int64_t o = (((int64_t)u * p.nsplit + split) * p.Cmax + (live ? tok : 0)) * kChunkCap;
      for (int j = 0; j < nsteps; ++j) {
        const int buf = j & 1;
        if (!tc::mbar_wait(&bars[RB_SFULL + buf], (j >> 1) & 1)) {
          atomicExch(p.status, (int)KVM_ERR_TIMEOUT); *abort_flag = 1; break;
        }
        tc::tc_fence_after();
        const uint32_t ts = tmem + lane_base + buf * 256 + mt * 128;
        const int row0 = (int)(i0 + (int64_t)j * 128);
        const int nvalid = (int)min((int64_t)128, i1 - row0);
        // the maximum ignores the sink rows (< S) and the rows past the end of the split; recorded chunks only the latter
        const int lo = max(0, p.S - row0);
        const bool plain = nvalid == 128 && lo == 0;
        // all 128 columns of the row go to registers in one round trip; the accumulator is handed
        // back before they are looked at
        uint32_t rr[4][32];
#pragma unroll
        for (int c4 = 0; c4 < 4; ++c4) tc::tmem_ld32(ts + c4 * 32, rr[c4]);
        tc::tmem_wait_ld();
        tc::tc_fence_before();
        __syncwarp();
        if (lane == 0) tc::mbar_arrive(&bars[RB_ACCFREE + buf]);
        if (gram) {   // row `tok` of gramT: 32 consecutive tokens j = row0 + c4*32 .. (rows past C are never read)
#pragma unroll
          for (int c4 = 0; c4 < 4; ++c4) {
            uint32_t (&r)[32] = rr[c4];
            if (tok < p.C) {
              float* dst = p.gramT + ((int64_t)a_unit * p.Cmax + tok) * p.Cmax + row0 + c4 * 32;
              if (row0 + c4 * 32 + 32 <= p.Cmax) {
#pragma unroll
                for (int i = 0; i < 8; ++i)
                  reinterpret_cast<uint4*>(dst)[i] = make_uint4(r[4 * i], r[4 * i + 1], r[4 * i + 2], r[4 * i + 3]);
              } else {
                for (int i = 0; i < 32; ++i)
                  if (row0 + c4 * 32 + i < p.Cmax) dst[i] = __uint_as_float(r[i]);
              }
            }
          }
          continue;
        }
        // chunk maxima: cm over the rows that count for the maximum, ca over all valid rows
        float cm[4], ca[4];
        uint32_t va[4];   // valid rows of each chunk (bit i = row i of the chunk)
#pragma unroll
        for (int c4 = 0; c4 < 4; ++c4) {
          uint32_t (&r)[32] = rr[c4];
          if (plain) {
            float t4[4] = {__uint_as_float(r[0]), __uint_as_float(r[1]), __uint_as_float(r[2]), __uint_as_float(r[3])};
#pragma unroll
            for (int i = 4; i < 28; i += 8) {
#pragma unroll
              for (int k = 0; k < 4; ++k) t4[k] = tc::fmax3(t4[k], __uint_as_float(r[i + k]), __uint_as_float(r[i + 4 + k]));
            }
#pragma unroll
            for (int k = 0; k < 4; ++k) t4[k] = fmaxf(t4[k], __uint_as_float(r[28 + k]));
            cm[c4] = fmaxf(fmaxf(t4[0], t4[1]), fmaxf(t4[2], t4[3]));
            ca[c4] = cm[c4];
            va[c4] = 0xffffffffu;
          } else {
            const int a = min(32, max(0, lo - c4 * 32)), b = min(32, max(0, nvalid - c4 * 32));
            const uint32_t vall = b == 32 ? 0xffffffffu : ((1u << b) - 1u);
            const uint32_t vns = (b <= a) ? 0u : (vall & ~((1u << a) - 1u));
            float m1 = -INFINITY, m2 = -INFINITY;
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              const float v = __uint_as_float(r[i]);
              m1 = fmaxf(m1, ((vns >> i) & 1u) ? v : -INFINITY);
              m2 = fmaxf(m2, ((vall >> i) & 1u) ? v : -INFINITY);
            }
            cm[c4] = m1; ca[c4] = m2; va[c4] = vall;
          }
        }
        const float tmax = fmaxf(fmaxf(cm[0], cm[1]), fmaxf(cm[2], cm[3]));
        // a maximum that beats the old one by more than the bound makes every earlier record obsolete (all
        // their rows lie below the new line), except the one that may hold sink rows, which the maximum
        // ignores: the list starts over, in place - it stays a record or two long and warm in L2
        if (tmax > mx + thr) nrec = min(nrec, sink_rec);
        mx = fmaxf(mx, tmax);
        const float cut = mx - thr;
#pragma unroll
        for (int c4 = 0; c4 < 4; ++c4) {
          if (live && ca[c4] >= cut) {   // record the chunk: 128 bytes of products, as they are
            uint32_t (&r)[32] = rr[c4];
            if (nrec < Cfg::REC_SLOTS) {
#pragma unroll
              for (int i = 0; i < 8; ++i) srec[(nrec * 8 + i) * 256] = make_uint4(r[4 * i], r[4 * i + 1], r[4 * i + 2], r[4 * i + 3]);
              if (nrec == 0) { rrow[0] = row0 + c4 * 32; rval[0] = va[c4]; rmax[0] = ca[c4]; }
              else { rrow[1] = row0 + c4 * 32; rval[1] = va[c4]; rmax[1] = ca[c4]; }
            } else if (nrec < kChunkCap) {
              uint4* dst = reinterpret_cast<uint4*>(p.chunkVal + (o + nrec) * 32);
#pragma unroll
              for (int i = 0; i < 8; ++i) dst[i] = make_uint4(r[4 * i], r[4 * i + 1], r[4 * i + 2], r[4 * i + 3]);
              p.chunkMeta[o + nrec] = make_int2(row0 + c4 * 32, (int)va[c4]);
              p.chunkMax[o + nrec] = ca[c4];
            }
            if (row0 + c4 * 32 < p.S) sink_rec = (nrec == 0) ? 1 : sink_rec;   // (the first chunk of the state; met first)
            ++nrec;
          }
        }
      }
      if (live && !gram) {
        // back over this thread's own records (written above, read here by the same thread): the chunks
        // whose maximum reaches the final line, and in them the valid rows that do
        static_assert(kChunkCap == 16, "chunk maxima are read as four float4");
        int ci[kTopK];
#pragma unroll
        for (int k = 0; k < kTopK; ++k) ci[k] = -1;
        int ncand = 0;
        const float cut = mx - thr;
        uint32_t kept = 0;
        if (nrec > Cfg::REC_SLOTS) {   // (rare) records past the ones in shared memory
          const float4* cm4 = reinterpret_cast<const float4*>(p.chunkMax + o);
          const float4 c0 = cm4[0], c1 = cm4[1], c2 = cm4[2], c3 = cm4[3];
          const float cmv[16] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w, c2.x, c2.y, c2.z, c2.w, c3.x, c3.y, c3.z, c3.w};
#pragma unroll
          for (int k = Cfg::REC_SLOTS; k < 16; ++k) kept |= (k < nrec && cmv[k] >= cut) ? (1u << k) : 0u;
        }
        if (nrec > 0 && rmax[0] >= cut) kept |= 1u;
        if (nrec > 1 && rmax[1] >= cut) kept |= 2u;
        while (kept) {
          const int k = __ffs(kept) - 1;
          kept &= kept - 1;
          int2 mt;
          uint32_t hit = 0;
          if (k < Cfg::REC_SLOTS) {
            mt = k == 0 ? make_int2(rrow[0], (int)rval[0]) : make_int2(rrow[1], (int)rval[1]);
#pragma unroll
            for (int q = 0; q < 8; ++q) {
              const uint4 w = srec[(k * 8 + q) * 256];
              const float4 v = make_float4(__uint_as_float(w.x), __uint_as_float(w.y), __uint_as_float(w.z), __uint_as_float(w.w));
              hit |= ((v.x >= cut ? 1u : 0u) | (v.y >= cut ? 2u : 0u) | (v.z >= cut ? 4u : 0u) | (v.w >= cut ? 8u : 0u)) << (4 * q);
            }
          } else {
            mt = p.chunkMeta[o + k];
            const float4* v4 = reinterpret_cast<const float4*>(p.chunkVal + (o + k) * 32);
#pragma unroll
            for (int q = 0; q < 8; ++q) {
              const float4 v = v4[q];
              hit |= ((v.x >= cut ? 1u : 0u) | (v.y >= cut ? 2u : 0u) | (v.z >= cut ? 4u : 0u) | (v.w >= cut ? 8u : 0u)) << (4 * q);
            }
          }
          hit &= (uint32_t)mt.y;
          while (hit) {
            const int bit = __ffs(hit) - 1;
            hit &= hit - 1;
            if (ncand < kTopK) {
#pragma unroll
              for (int kk = 0; kk < kTopK; ++kk)
                if (kk == ncand) ci[kk] = mt.x + bit;
            }
            ++ncand;
          }
        }
        if (nrec > kChunkCap) ncand = kTopK + 1;   // records were lost: let the decision kernel scan every row
        const int64_t oc = (((int64_t)u * p.nsplit + split) * p.Cmax + tok) * kTopK;
#pragma unroll
        for (int k = 0; k < kTopK; ++k) p.candI[oc + k] = ci[k];
        // values are not kept: the decision kernel needs the split's maximum and the candidate count
        p.candV[oc] = mx;
        p.candV[oc + 1] = (float)ncand;
      }
    }
  }
  tc::tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc::tmem_dealloc(tmem, Cfg::TMEM_COLS);
  }
}

int launch_route_filter_tc(State* st, int64_t m, int nsplit, int slot, bool early_start, cudaStream_t s) {
  RouteTcParams p;
  p.candV = st->candV; p.candI = st->candI; p.chunkMax = st->chunkMax; p.chunkMeta = st->chunkMeta; p.chunkVal = st->chunkVal; p.status = st->status; p.m = m;
  p.C = st->C; p.Cmax = st->Cmax; p.nsplit = nsplit; p.S = st->S;
  p.kbarNorm = st->kbarNorm + (int64_t)slot * st->U * st->Cmax; p.thr_coeff = route_thr_coeff(st);
  p.a_unit0 = slot * st->U; p.gramT = st->gramT; p.gram_mode = 0; p.U = st->U;
  const CUtensorMap* tm = reinterpret_cast<const CUtensorMap*>(st->tmaps);
  dim3 grid(nsplit, st->U);
  const int ks = (st->nfolds & 1) ? 6 : 1;   // the fold reads the readout copy of the current version
  // programmatic dependent launch behind the apply kernel of the previous fold: the CTAs set up and
  // fetch the block's memory keys while it finishes (not where the kernel before this one on the
  // stream is the one that writes those keys: a decode step's fold)
  cudaLaunchConfig_t lc = {};
  lc.gridDim = grid; lc.blockDim = dim3(352); lc.stream = s;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = at; lc.numAttrs = (early_start && st->prof_hook == nullptr) ? 1 : 0;
  if (st->d == 128) { lc.dynamicSmemBytes = RouteTcCfg<128>::SMEM_BYTES; cudaLaunchKernelEx(&lc, route_filter_tc_kernel<128>, tm[5], tm[ks], tm[8], p); }
  else { lc.dynamicSmemBytes = RouteTcCfg<64>::SMEM_BYTES; cudaLaunchKernelEx(&lc, route_filter_tc_kernel<64>, tm[5], tm[ks], tm[8], p); }
  return 1;
}

// New-row filter of nblk blocks whose memory keys sit in slots slot0 .. slot0 + nblk - 1.
int launch_gram_tc(State* st, int slot0, int nblk, cudaStream_t s) {
  RouteTcParams p;
  p.candV = st->candV; p.candI = st->candI; p.chunkMax = st->chunkMax; p.chunkMeta = st->chunkMeta; p.chunkVal = st->chunkVal; p.status = st->status; p.m = 0;
  p.C = st->C; p.Cmax = st->Cmax; p.nsplit = 1; p.S = st->S;
  p.kbarNorm = st->kbarNorm; p.thr_coeff = 0.f;
  p.a_unit0 = slot0 * st->U; p.gramT = st->gramT; p.gram_mode = 1; p.U = st->U;
  const CUtensorMap* tm = reinterpret_cast<const CUtensorMap*>(st->tmaps);
  dim3 grid(1, st->U, nblk);
  if (st->d == 128) route_filter_tc_kernel<128><<<grid, 352, RouteTcCfg<128>::SMEM_BYTES, s>>>(tm[5], tm[1], tm[8], p);
  else route_filter_tc_kernel<64><<<grid, 352, RouteTcCfg<64>::SMEM_BYTES, s>>>(tm[5], tm[1], tm[8], p);
  return 1;
}

bool setup_route_tc(State* st) {
  CUtensorMap* tm = reinterpret_cast<CUtensorMap*>(st->tmaps);
  if (!encode_tmap_rows(&tm[5], st->kbarH, st->d, st->CbarRows, (int64_t)st->kbSlots * st->U, 128)) return false;
  if (!encode_tmap_rows(&tm[8], st->kbarHatH, st->d, st->CbarRows, (int64_t)st->kbSlots * st->U, 128)) return false;
  if (cudaFuncSetAttribute(route_filter_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, RouteTcCfg<128>::SMEM_BYTES) != cudaSuccess) return false;
  if (cudaFuncSetAttribute(route_filter_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, RouteTcCfg<64>::SMEM_BYTES) != cudaSuccess) return false;
  return true;
}

}  // namespace kvm
