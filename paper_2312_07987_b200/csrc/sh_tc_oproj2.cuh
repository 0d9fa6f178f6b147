// Output-expert projection on CTA pairs with the gates folded into the A operand (the MoE output
// equation of Sec. 2.2):  y[t] = sum_h sum_{e in E_D^h(t)} s_D^h[t,e] * Ahat^h[t] W_O^{h,e}
//                              = sum_h sum_e ( diag(g^{h,e}) Ahat^h )[t] W_O^{h,e},   g^{h,e}[t] = gate or 0.
//
// sh_tc_oproj_kernel multiplies by the gate AFTER the UMMA, in registers, so every expert needs a
// tensor-memory accumulator of its own, and the hand-over of the two accumulators between the
// issuing thread and the epilogue warps (commit -> barrier -> four TMEM loads + FFMA -> arrive ->
// barrier, ~1000 cycles) is as long as the 1024 cycles the tensor pipe needs per expert: the pipe
// waits.  Here "builder" warps scale the token rows by their gates on the way into shared memory
// (rows that did not select the expert become zero), so all experts and heads of a work unit
// accumulate into ONE tensor-memory buffer; the pipe runs without a per-expert hand-over, and the
// other buffer is read out and stored by separate epilogue warps while the next unit accumulates.
// The sum still never leaves the SM, out is written exactly once, and the result does not depend on
// timing (the UMMAs are issued in a fixed order).  The price is one more fp16 rounding (of gate x
// Ahat) than the single-CTA kernel makes.
//
// CTA pair (cluster of two, tcgen05 cta_group::2): work unit = 256 consecutive tokens x 256 output
// features; each CTA owns 128 of the tokens (its scaled tiles, its accumulators, its stores) and
// loads only its half of every expert's 256 weight rows - the pair's tensor cores read both halves.
//
// Roles per CTA (480 threads): warp 0 lane 0 = TMA producer (weights), warp 1 = TMEM allocation; in
// the leader (even CTA) lane 0 of warps 1 and 14 = UMMA issuers for the pair (they alternate, see
// below); warps 2..9 = builders (thread = one token x half of the head's D columns: Ahat row from
// global memory into registers one head ahead, per expert a scaled copy into the stage's
// 128-byte-swizzled K-major tile); warps 10..13 = epilogue (thread = one token, TMEM -> transpose
// in shared memory -> 16-byte coalesced stores).
// Two rings: weights in 64-column blocks of this CTA's 128 feature rows (16 KB, five stages: a TMA
// load from L2 takes ~1 us, two experts' worth of tensor work) and scaled token tiles (128 x D, four
// stages: a tile is rebuilt ~1000 cycles after the UMMAs that read it complete, and those may wait
// in the pipe's queue behind the expert before).  Together with the epilogue's staging that is all
// of the 227 KB; of the splits that fit (7 + 3, 5 + 4, four 32 KB weight stages + 2 tiles) this one
// measured best.  An issuing thread waits for each weight block (leader's barrier: the pair's
// bytes) and once per expert for the tile (leader's barrier: one arrival per builder warp of both
// CTAs), and commits each to the empty barrier of both CTAs (multicast).
#pragma once
#include "sh_tc_oproj.cuh"

namespace shtc {

constexpr int OPAIR_KMAX = 4;                            // selections per (token, head) a builder keeps in registers (the kernel serves k <= 4)

template <int D>
struct OprojPairSmem {
  static constexpr int W_BYTES = 128 * 64 * 2;           // one 64-column block of this CTA's 128 feature rows of an expert
  static constexpr int P_BYTES = 128 * D * 2;            // scaled token tile: this CTA's 128 tokens x D
  static constexpr int WST = 5, PST = 4;                 // ring depths
  static constexpr int STAGING = 4 * 32 * 32 * 4;        // per epilogue warp a 32 x 32 fp32 transpose tile
  static constexpr int TOTAL = WST * W_BYTES + PST * P_BYTES + STAGING + 512 + 1024;
};

// One 32-column chunk of a unit's accumulator: TMEM -> registers -> 32 x 32 transpose in shared
// memory (token-per-lane -> 128-byte row segments) -> 16-byte coalesced stores.  One warp; stg = its
// 4 KB of staging; obase = element index in out of (first of the warp's 32 tokens, the unit's first feature).
__device__ __forceinline__ void oproj_store_chunk(uint32_t taddr, int c, float* stg, float* out, size_t obase, int out_f16, int M, int rows_here, bool cols_live, int lane) {
  uint32_t v[32];
  tmem_ld32(taddr + c * 32, v);
  tmem_ld_wait();
  __syncwarp();
#pragma unroll
  for (int ch = 0; ch < 8; ++ch)                           // 16-byte chunk ch of row `lane` sits at chunk ch ^ (lane & 7)
    *reinterpret_cast<uint4*>(stg + lane * 32 + ((ch ^ (lane & 7)) << 2)) = make_uint4(v[4 * ch], v[4 * ch + 1], v[4 * ch + 2], v[4 * ch + 3]);
  __syncwarp();
  if (cols_live) {
#pragma unroll
    for (int r4 = 0; r4 < 32; r4 += 4) {
      const int r = r4 + (lane >> 3), ch = lane & 7;
      if (r < rows_here)
        oproj_put4(out, obase + (size_t)r * M + c * 32 + 4 * ch, *reinterpret_cast<const float4*>(stg + r * 32 + ((ch ^ (r & 7)) << 2)), out_f16);
    }
  }
}

template <int D>
__global__ void __launch_bounds__(480, 1)
sh_tc_oproj_pair_kernel(const __grid_constant__ CUtensorMap mapWo, TcOprojArgs g, const __half* __restrict__ ahat) {
  using SM = OprojPairSmem<D>;
  constexpr int DB = D / 64;                             // 64-column (128-byte) blocks per row
  constexpr int WST = SM::WST, PST = SM::PST;
  static_assert(WST <= 8 && PST <= 4, "barrier slots");
  constexpr uint32_t TBLK = 128 * 128;                   // one 64-column block of a 128-row tile
  constexpr int CH = D / 16;                             // 16-byte chunks per builder thread (half a row)
  extern __shared__ unsigned char smem_raw[];
  const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* sgen = smem_raw + (sbase - smem_u32(smem_raw));
  const ShDims& d = g.d;
  constexpr uint32_t w_off = 0, p_off = WST * SM::W_BYTES, stg_off = p_off + PST * SM::P_BYTES, misc_off = stg_off + SM::STAGING;
  uint64_t* bars = (uint64_t*)(sgen + misc_off);
  uint64_t* w_full = bars;               // [WST] leader's: the pair's bytes of one weight block
  uint64_t* w_empty = bars + 8;          // [WST] both CTAs (multicast commit)
  uint64_t* p_full = bars + 16;          // [PST] leader's: 16 arrivals (builder warps of both CTAs)
  uint64_t* p_empty = bars + 20;         // [PST] both CTAs (multicast commit)
  uint64_t* d_full = bars + 24;          // [2] both CTAs (multicast commit): a unit's accumulator is complete
  uint64_t* d_empty = bars + 26;         // [2] leader's: 8 arrivals (epilogue warps of both CTAs)
  uint64_t* turn = bars + 28;            // [2] leader's: the token of the two issuing threads
  uint32_t* tmem_slot = (uint32_t*)(bars + 30);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();               // 0 = leader
  const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
  const int nfc = (d.M + 255) / 256;
  const int HD = d.H * D;
  const int nout = sh_out_rows(d);                       // rows of out (= tokens, unless a cache sits in front of every sequence)
  bool dead = false;

  if (threadIdx.x == 0) {
    for (int s = 0; s < WST; ++s) { mbar_init(&w_full[s], 1); mbar_init(&w_empty[s], 1); }
    for (int s = 0; s < PST; ++s) { mbar_init(&p_full[s], 16); mbar_init(&p_empty[s], 1); }
    for (int s = 0; s < 2; ++s) { mbar_init(&d_full[s], 2); mbar_init(&d_empty[s], 8); mbar_init(&turn[s], 1); }
    fence_barrier_init();
    tma_prefetch_desc(&mapWo);
  }
  if (warp == 1) { tmem_alloc_pair(tmem_slot, 512); tmem_relinquish_pair(); }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                                    // the peer's barriers exist before anything signals them
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  pdl_trigger();
  if (threadIdx.x == 0) sh_stamp_resident(d.stamps, SH_K_O);
  pdl_wait();
  if (threadIdx.x == 0) sh_stamp_start(d.stamps, SH_K_O);

  if (warp == 0) {
    if (lane == 0) {
      int s = 0;
      uint32_t wpar = 1;                                    // parity to wait for on w_empty[s]
      for (int w = pair; w < g.nwork && !dead; w += npairs) {
        const int fc = w % nfc;
        for (int he = 0; he < d.H * d.E && !dead; ++he) {
          // this CTA's 128 of the 256 feature rows of expert he = h * E + e, one 64-column block at a
          // time; a box that runs past the expert's rows (M not a multiple of 256) fetches rows whose
          // columns are never stored
          for (int c = 0; c < DB; ++c) {
            if (!mbar_wait(&w_empty[s], wpar, g.status, dead)) break;
            if (rank == 0) mbar_expect_tx(&w_full[s], 2 * SM::W_BYTES);
            tma_load_2d_pair(sbase + w_off + s * SM::W_BYTES, &mapWo, &w_full[s], c * 64, he * d.M + fc * 256 + (int)rank * 128);
            if (++s == WST) { s = 0; wpar ^= 1; }
          }
        }
      }
    }
  } else if (warp == 1 || warp == 14) {
    if (lane == 0 && rank == 0) {
      // Two issuing threads take the experts in turn (even / odd running index): one tcgen05.mma costs
      // the issuing thread ~60 cycles and a barrier wait or a commit about as much, so the 8 UMMAs, 3
      // waits and 3 commits of an expert take one thread longer than the 1024 cycles the tensor pipe
      // needs for them.  A token (turn[]) passes from one to the other after the UMMAs of an expert
      // are issued, so the accumulation order is fixed, and a thread looks at the operand barriers
      // only while it holds the token: every earlier phase of those barriers is then complete, so a
      // barrier it has not watched for a while cannot answer with a stale parity.
      const int me = warp == 1 ? 0 : 1;
      constexpr uint32_t idesc = make_idesc_f16(256, 256, 0, 0, 0);
      const uint32_t w_lo0 = desc_lo_k(sbase + w_off), p_lo0 = desc_lo_k(sbase + p_off);
      int un = 0, s = 0, ps = 0, ge = 0;
      uint32_t wpar = 0, ppar = 0;                          // parities to wait for on w_full[s], p_full[ps]
      for (int w = pair; w < g.nwork && !dead; w += npairs, ++un) {
        const int buf = un & 1;
        for (int he = 0; he < d.H * d.E && !dead; ++he, ++ge) {
          if ((ge & 1) == me) {
            if (ge > 0 && !mbar_wait(&turn[me], (uint32_t)((ge >> 1) - 1 + me) & 1u, g.status, dead)) break;
            if (he == 0 && !mbar_wait(&d_empty[buf], ((un >> 1) & 1) ^ 1, g.status, dead)) break;
            if (!mbar_wait(&p_full[ps], ppar, g.status, dead)) break;
            const uint32_t p_lo = p_lo0 + ps * (SM::P_BYTES >> 4);
            int s2 = s;
            uint32_t wpar2 = wpar;
            for (int c = 0; c < DB; ++c) {
              if (!mbar_wait(&w_full[s2], wpar2, g.status, dead)) break;
              tc_fence_after();
              const uint32_t w_lo = w_lo0 + s2 * (SM::W_BYTES >> 4);
#pragma unroll
              for (int k = 0; k < 4; ++k)
                umma_f16_pair(tmem + buf * 256, desc_pack(p_lo + c * (TBLK >> 4) + 2 * k), desc_pack(w_lo + 2 * k), idesc, (he | c | k) != 0);
              if (++s2 == WST) { s2 = 0; wpar2 ^= 1; }
            }
            if (dead) break;
            mbar_arrive(&turn[me ^ 1]);                     // the other thread may issue the next expert
            s2 = s;
            for (int c = 0; c < DB; ++c) {                  // (both blocks are released when all 8 UMMAs are done)
              umma_commit_pair(&w_empty[s2], 3);
              if (++s2 == WST) s2 = 0;
            }
            umma_commit_pair(&p_empty[ps], 3);
          }
          s += DB;
          if (s >= WST) { s -= WST; wpar ^= 1; }
          if (++ps == PST) { ps = 0; ppar ^= 1; }
        }
        if (dead) break;
        umma_commit_pair(&d_full[buf], 3);                  // one of two arrivals: this thread's UMMAs of the unit are done
      }
    }
  } else if (warp < 10) {
    // ---- builders: thread = token `row` x column half `kh` of the head ----
    const int bt = threadIdx.x - 64;
    const int row = bt & 127, kh = bt >> 7;
    uint4 cur[CH], nxt[CH];
    int ci[OPAIR_KMAX], ni[OPAIR_KMAX];
    float cg[OPAIR_KMAX], ng[OPAIR_KMAX];
    // Ahat half-row and the selections of (token, head), fetched one head ahead (an L2 round trip is
    // ~1 us); (fw, fh) walk the units and heads of this pair in step with the consuming loop
    int fw = pair, fh = 0;
    auto fetch = [&]() {
      const int orow = (fw / nfc) * 256 + (int)rank * 128 + row;    // row of out; its token sits behind the cache, if there is one
      const bool live = fw < g.nwork && orow < nout;
      const int tokn = live ? sh_ctx_tok(d, orow) : 0;
      const uint4* src = reinterpret_cast<const uint4*>(ahat + (size_t)tokn * HD + fh * D + kh * (D / 2));
#pragma unroll
      for (int i = 0; i < CH; ++i) nxt[i] = live ? __ldg(src + i) : make_uint4(0, 0, 0, 0);
      const size_t so = ((size_t)tokn * d.H + fh) * d.k;
#pragma unroll
      for (int j = 0; j < OPAIR_KMAX; ++j) {
        const bool lj = live && j < d.k;
        ni[j] = lj ? __ldg(g.idx + so + j) : -1;
        ng[j] = lj ? __ldg(g.gate + so + j) : 0.f;
        if (lj && !SH_INDEX_OK(ni[j], d.E, g.status, SH_SITE_O_EXPERT)) ni[j] = -1;
      }
      if (++fh == d.H) { fh = 0; fw += npairs; }
    };
    fetch();
    uint32_t toff[CH];                                     // this thread's chunks inside a tile (128-byte swizzle)
#pragma unroll
    for (int i = 0; i < CH; ++i) {
      const int j = kh * CH + i;                           // 16-byte chunk of the row: block j / 8, chunk j % 8
      toff[i] = (j >> 3) * TBLK + row * 128 + (((j & 7) ^ (row & 7)) << 4);
    }
    int ps = 0;
    uint32_t ppar = 1;                                     // parity to wait for on p_empty[ps]
    bool ok = true;
    for (int w = pair; w < g.nwork && ok; w += npairs) {
      for (int h = 0; h < d.H && ok; ++h) {
#pragma unroll
        for (int i = 0; i < CH; ++i) cur[i] = nxt[i];
#pragma unroll
        for (int j = 0; j < OPAIR_KMAX; ++j) { ci[j] = ni[j]; cg[j] = ng[j]; }
        fetch();
        for (int e = 0; e < d.E; ++e) {
          float gv = 0.f;
#pragma unroll
          for (int j = 0; j < OPAIR_KMAX; ++j)
            if (ci[j] == e) gv = cg[j];
          // The gate as the sum of two fp16 values: multiplying by fp16(gate) alone would put one relative
          // error of up to 2^-11 on this expert's WHOLE contribution to the token (the same factor on
          // every feature).  p = a * g_hi rounded; e = the exact rounding error of that product (one
          // fused multiply-add); the result rounds p + (a * g_lo + e): the product a * gate, rounded once.
          const __half gh1 = __float2half_rn(gv);
          const __half2 g_hi = __half2half2(gh1), g_lo = __float2half2_rn(gv - __half2float(gh1));
          // one lane polls for the warp (256 threads polling one barrier word get in each other's way)
          if (lane == 0 && !mbar_wait(&p_empty[ps], ppar, g.status, dead)) ok = false;
          ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
          if (!ok) break;
          unsigned char* tile = sgen + p_off + ps * SM::P_BYTES;
#pragma unroll
          for (int i = 0; i < CH; ++i) {
            uint4 v = cur[i];
            __half2* hv = reinterpret_cast<__half2*>(&v);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const __half2 pq = __hmul2(hv[q], g_hi);
              const __half2 eq = __hfma2(hv[q], g_hi, __hneg2(pq));
              hv[q] = __hadd2(pq, __hfma2(hv[q], g_lo, eq));
            }
            *reinterpret_cast<uint4*>(tile + toff[i]) = v;
          }
          fence_proxy_async_smem();                        // generic-proxy writes -> visible to the UMMA's reads
          __syncwarp();
          if (lane == 0) mbar_arrive_leader(&p_full[ps]);
          if (++ps == PST) { ps = 0; ppar ^= 1; }
        }
      }
    }
  } else if (warp < 14) {
    // ---- epilogue: warp = 32 tokens (TMEM lane quarter warp & 3), all 256 features of the unit ----
    const int q = warp & 3;
    const uint32_t lane_off = (uint32_t)(q * 32) << 16;
    float* stg = reinterpret_cast<float*>(sgen + stg_off) + (warp - 10) * 1024;
    int un = 0;
    for (int w = pair; w < g.nwork; w += npairs, ++un) {
      const int buf = un & 1;
      const int row0 = (w / nfc) * 256 + (int)rank * 128, fc = w % nfc;
      const int rows_here = min(32, nout - row0 - q * 32); // <= 0: these rows are past the end
      if (!mbar_wait(&d_full[buf], (un >> 1) & 1, g.status, dead)) break;
      tc_fence_after();
      const size_t obase = (size_t)(row0 + q * 32) * d.M + fc * 256;
#pragma unroll 1
      for (int c = 0; c < 8; ++c) {
        oproj_store_chunk(tmem + lane_off + buf * 256, c, stg, g.out, obase, g.out_f16, d.M, rows_here, fc * 256 + c * 32 < d.M, lane);
        if (c == 7) {                                      // everything has been read: hand the accumulator back
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_leader(&d_empty[buf]);
        }
      }
    }
  }
  // neither CTA leaves (or frees tensor memory) while the other may still read its shared memory
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (threadIdx.x == 0) sh_stamp_end(d.stamps, SH_K_O);
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem, 512);
  }
}

}  // namespace shtc
