// Output-expert projection on CTA pairs with the expert selection as 2:4 STRUCTURED SPARSITY of the A
// operand (the MoE output equation of Sec. 2.2):
//   y[t] = sum_h sum_{e in E_D^h(t)} s_D^h[t,e] * Ahat^h[t] W_O^{h,e}
//        = sum_h  A_cat^h[t, :] . W_cat^h,      A_cat^h[t, d*E + e] = g^{h,e}[t] * Ahat^h[t, d],
//                                               W_cat^h[d*E + e, f] = W_O^{h,e}[d, f].
// With the experts INNERMOST on the contraction axis, every group of four consecutive K positions of a
// token's row holds the same Ahat value times the gates of four neighbouring experts - of which the token
// selected at most two when k <= 2.  That is exactly the 2:4 pattern the sparse tensor-core instruction
// (tcgen05.mma.sp, kind::f16: K = 32 logical per instruction at the cycles of a dense K = 16) takes in
// compressed form: two values per group and a 4-bit position code.  The masked kernel
// (sh_tc_oproj_pair_kernel) multiplies the E - k zero rows of every token like any other; here the
// tensor pipe skips half of them (all of them at E = 4, k = 2), the builders write k/E... 2/4 of the
// bytes into shared memory, and nothing else changes: one accumulator per work unit, the sum over
// experts and heads never leaves the SM, out is written once, fixed accumulation order.
//
// Served shapes: k <= 2, E = 4 or 8, d_head (padded) = 128, at most 4 heads... see sh_o_sparse_ok().
//
// Compressed row of (token, head): for every d the E/4 groups in turn, two fp16 values each
// (lower expert index first): E*D/2 values.  A ring stage = 128 compressed columns (two 128-byte-swizzled
// K-major blocks of this CTA's 128 tokens, 32 KB) = 8 sparse UMMAs of M = 256, N = 256 = 1024 tensor
// cycles, against four 16 KB weight blocks (this CTA's 128 of the unit's 256 feature rows x 64 logical
// K positions each).  A builder thread (token row x half kh of the head's D columns) fills the row's
// part of E/4 consecutive stages.
//
// Position codes: one 32-bit word per TMEM lane and per head (the code of a token is the same for every
// d: it repeats along K), layout of the instruction's metadata operand for M = 128 rows per CTA: lane
// L = 16*a + 8*b + c (a < 8, b < 2, c < 8) holds in its low half-word the codes of row 16*a + c and in
// its high half-word those of row 16*a + 8 + c, for K positions 16*b .. 16*b + 15 of the instruction
// (four groups x 4 bits; the two positions of a group as 2-bit numbers, lower position in the low bits);
// consecutive instructions' words sit in consecutive TMEM columns and the instruction names the even
// column of the pair plus a selector bit.  All 512 columns belong to the two accumulators, so the words
// of unit u live in the first columns of the accumulator that unit u does NOT use: the epilogue warps,
// which own the TMEM lanes, write them there right after they have read those columns of unit u - 1
// (at the start of the kernel for the first unit) and tell the issuing threads.  Unit u + 1 then
// overwrites them with its accumulator, behind unit u's UMMAs in the pipe's order.
#pragma once
#include "sh_tc_oproj2.cuh"

namespace shtc {

constexpr int OSP_MAXH = 4;                              // heads whose position codes the epilogue keeps in registers

template <int D>
struct OprojSpSmem {
  static constexpr int W_BYTES = 128 * 64 * 2;           // 64 logical K positions of this CTA's 128 feature rows
  static constexpr int P_BYTES = 128 * 128 * 2;          // 128 compressed columns of this CTA's 128 tokens
  static constexpr int WST = 7, PST = 3;                 // ring depths
  static constexpr int STAGING = 4 * 32 * 32 * 4;
  static constexpr int TOTAL = WST * W_BYTES + PST * P_BYTES + STAGING + 512 + 1024;
};

// The two kept positions of one group of four experts (experts 4c .. 4c + 3) for a token that selected
// experts i0, i1 (-1: none) with gates g0, g1: positions lo < hi and their gates (0 for a position that
// only pads the pattern).  Builders (values) and epilogue warps (codes) both go through this function.
__device__ __forceinline__ void osp_group(int i0, float g0, int i1, float g1, int c, int& lo, int& hi, float& glo, float& ghi) {
  int a = (i0 >= 0 && (i0 >> 2) == c) ? (i0 & 3) : -1;
  int b = (i1 >= 0 && (i1 >> 2) == c) ? (i1 & 3) : -1;
  float ga = g0, gb = g1;
  if (a < 0) { a = b; ga = gb; b = -1; }
  if (b >= 0 && b < a) { const int t = a; a = b; b = t; const float tg = ga; ga = gb; gb = tg; }
  if (a < 0) { lo = 0; hi = 1; glo = 0.f; ghi = 0.f; }
  else if (b < 0 || b == a) {
    if (a == 3) { lo = 0; hi = 3; glo = 0.f; ghi = ga; }
    else { lo = a; hi = 3; glo = ga; ghi = 0.f; }
  } else { lo = a; hi = b; glo = ga; ghi = gb; }
}
// 16 bits of position codes of one token row: E = 4: the same group code four times; E = 8: the codes of
// the two groups alternate.
template <int SPT>
__device__ __forceinline__ uint32_t osp_row_codes(int i0, int i1) {
  int lo, hi; float x, y;
  osp_group(i0, 0.f, i1, 0.f, 0, lo, hi, x, y);
  const uint32_t n0 = (uint32_t)(lo | (hi << 2));
  if (SPT == 1) return n0 * 0x1111u;
  osp_group(i0, 0.f, i1, 0.f, 1, lo, hi, x, y);
  const uint32_t n1 = (uint32_t)(lo | (hi << 2));
  return (n0 | (n1 << 4)) * 0x0101u;
}
// a * (g_a, g_b), each product rounded once to fp16: the gates as sums of two fp16 values
// (see sh_tc_oproj_pair_kernel).
__device__ __forceinline__ __half2 osp_scale(__half a, __half2 g_hi, __half2 g_lo) {
  const __half2 a2 = __half2half2(a);
  const __half2 p = __hmul2(a2, g_hi);
  const __half2 e = __hfma2(a2, g_hi, __hneg2(p));
  return __hadd2(p, __hfma2(a2, g_lo, e));
}

// SPT = E / 4: stages a builder thread fills per head (and groups per d).
template <int D, int SPT>
__global__ void __launch_bounds__(480, 1)
sh_tc_oproj_sp_kernel(const __grid_constant__ CUtensorMap mapWos, TcOprojArgs g, const __half* __restrict__ ahat) {
  static_assert(D == 128 && (SPT == 1 || SPT == 2), "served shapes");
  using SM = OprojSpSmem<D>;
  constexpr int WST = SM::WST, PST = SM::PST;
  constexpr int SPH = 2 * SPT;                           // ring stages per head
  constexpr int WPH = 8 * SPT;                           // weight blocks per head (E * D / 64)
  static_assert(WST <= 8 && PST <= 4 && WST > 4, "barrier slots / ring step");
  // A builder group skips the other group's SPT stages of every head: from its last stage of one head to
  // its first of the next it moves SPT + 1 stages on.  With fewer ring slots than that it could arrive two
  // phases ahead of a slot's empty barrier, and a parity wait cannot tell phase p from phase p - 2.
  static_assert(PST >= SPT + 1, "ring depth against the builders' stride");
  constexpr uint32_t TBLK = 128 * 128;
  extern __shared__ unsigned char smem_raw[];
  const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* sgen = smem_raw + (sbase - smem_u32(smem_raw));
  const ShDims& d = g.d;
  constexpr uint32_t w_off = 0, p_off = WST * SM::W_BYTES, stg_off = p_off + PST * SM::P_BYTES, misc_off = stg_off + SM::STAGING;
  uint64_t* bars = (uint64_t*)(sgen + misc_off);
  uint64_t* w_full = bars;               // [WST] leader's: the pair's bytes of one weight block
  uint64_t* w_empty = bars + 8;          // [WST] both CTAs (multicast commit)
  uint64_t* p_full = bars + 16;          // [PST] leader's: 8 arrivals (the four builder warps of a column half, both CTAs)
  uint64_t* p_empty = bars + 20;         // [PST] both CTAs (multicast commit)
  uint64_t* d_full = bars + 24;          // [2] both CTAs (multicast commit): a unit's accumulator is complete
  uint64_t* d_empty = bars + 26;         // [2] leader's: 8 arrivals (epilogue warps of both CTAs)
  uint64_t* turn = bars + 28;            // [2] leader's: the token of the two issuing threads
  uint64_t* m_full = bars + 30;          // [2] leader's: 8 arrivals (epilogue warps): a unit's position codes are in tensor memory
  uint32_t* tmem_slot = (uint32_t*)(bars + 32);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();               // 0 = leader
  const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
  const int nfc = (d.M + 255) / 256;
  const int HD = d.H * D;
  const int nout = sh_out_rows(d);
  bool dead = false;

  if (threadIdx.x == 0) {
    for (int s = 0; s < WST; ++s) { mbar_init(&w_full[s], 1); mbar_init(&w_empty[s], 1); }
    for (int s = 0; s < PST; ++s) { mbar_init(&p_full[s], 8); mbar_init(&p_empty[s], 1); }
    for (int s = 0; s < 2; ++s) { mbar_init(&d_full[s], 2); mbar_init(&d_empty[s], 8); mbar_init(&turn[s], 1); mbar_init(&m_full[s], 8); }
    fence_barrier_init();
    tma_prefetch_desc(&mapWos);
  }
  if (warp == 1) { tmem_alloc_pair(tmem_slot, 512); tmem_relinquish_pair(); }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  pdl_trigger();
  if (threadIdx.x == 0) sh_stamp_resident(d.stamps, SH_K_O);
  // Ahead of the wait for the attention kernel's result (this kernel is launched to become resident while
  // that one drains) everything that does not need Ahat gets under way: the weight stream (weights are
  // constant) and the first unit's position codes (the selections come from the gate kernel, which the
  // attention kernel saw complete before it let this one start).  The roles that read Ahat or write out
  // wait where they need to.

  if (warp == 0) {
    if (lane == 0) {
      int s = 0;
      uint32_t wpar = 1;
      for (int w = pair; w < g.nwork && !dead; w += npairs) {
        const int fc = w % nfc;
        for (int h = 0; h < d.H && !dead; ++h) {
          // this CTA's 128 of the unit's 256 feature rows of W_cat^h, 64 K positions at a time; a box that
          // runs past the head's rows (M not a multiple of 256) fetches rows whose columns are never stored
          for (int c = 0; c < WPH; ++c) {
            if (!mbar_wait(&w_empty[s], wpar, g.status, dead)) break;
            if (rank == 0) mbar_expect_tx(&w_full[s], 2 * SM::W_BYTES);
            tma_load_2d_pair(sbase + w_off + s * SM::W_BYTES, &mapWos, &w_full[s], c * 64, h * d.M + fc * 256 + (int)rank * 128);
            if (++s == WST) { s = 0; wpar ^= 1; }
          }
        }
      }
    }
  } else if (warp == 1 || warp == 14) {
    if (lane == 0 && rank == 0) {
      // two issuing threads take the ring stages in turn and pass a token (see sh_tc_oproj_pair_kernel)
      const int me = warp == 1 ? 0 : 1;
      constexpr uint32_t idesc = make_idesc_f16(256, 256, 0, 0, 0) | (1u << 2);     // sparse A
      const uint32_t w_lo0 = desc_lo_k(sbase + w_off), p_lo0 = desc_lo_k(sbase + p_off);
      int un = 0, s = 0, ps = 0, ge = 0;
      uint32_t wpar = 0, ppar = 0;
      for (int w = pair; w < g.nwork && !dead; w += npairs, ++un) {
        const int buf = un & 1;
        const uint32_t acc = tmem + buf * 256, codes = tmem + (buf ^ 1) * 256;
        for (int st = 0; st < d.H * SPH && !dead; ++st, ++ge) {
          if ((ge & 1) == me) {
            if (ge > 0 && !mbar_wait(&turn[me], (uint32_t)((ge >> 1) - 1 + me) & 1u, g.status, dead)) break;
            if (st == 0) {
              if (!mbar_wait(&d_empty[buf], ((un >> 1) & 1) ^ 1, g.status, dead)) break;
              if (!mbar_wait(&m_full[buf], (un >> 1) & 1, g.status, dead)) break;
            }
            if (!mbar_wait(&p_full[ps], ppar, g.status, dead)) break;
            const int h = st / SPH;
            const uint32_t p_lo = p_lo0 + ps * (SM::P_BYTES >> 4);
            const uint32_t e_addr = codes + (uint32_t)(h & ~1), idh = idesc | (uint32_t)(h & 1);
            int s2 = s;
            uint32_t wpar2 = wpar;
            for (int c = 0; c < 4; ++c) {                   // weight block c = K positions 64c .. 64c + 63 of the stage: two instructions
              if (!mbar_wait(&w_full[s2], wpar2, g.status, dead)) break;
              tc_fence_after();
              const uint32_t w_lo = w_lo0 + s2 * (SM::W_BYTES >> 4);
#pragma unroll
              for (int t = 0; t < 2; ++t) {
                const int i = c * 2 + t;                    // instruction of the stage: 16 compressed columns of A, 32 K positions of B
                umma_sp_f16_pair(acc, desc_pack(p_lo + (i >> 2) * (TBLK >> 4) + 2 * (i & 3)), desc_pack(w_lo + 4 * t), e_addr, idh, (st | i) != 0);
              }
              if (++s2 == WST) { s2 = 0; wpar2 ^= 1; }
            }
            if (dead) break;
            mbar_arrive(&turn[me ^ 1]);
            s2 = s;
            for (int c = 0; c < 4; ++c) {
              umma_commit_pair(&w_empty[s2], 3);
              if (++s2 == WST) s2 = 0;
            }
            umma_commit_pair(&p_empty[ps], 3);
          }
          s += 4;
          if (s >= WST) { s -= WST; wpar ^= 1; }
          if (++ps == PST) { ps = 0; ppar ^= 1; }
        }
        if (dead) break;
        umma_commit_pair(&d_full[buf], 3);
      }
    }
  } else if (warp < 10) {
    // ---- builders: thread = token `row` x column half `kh` of the head: SPT consecutive stages per head ----
    const int bt = threadIdx.x - 64;
    const int row = bt & 127, kh = bt >> 7;
    uint4 cur[8], nxt[8];                                  // 64 fp16: this thread's half of the Ahat row
    int ci[2], ni[2];
    float cg[2], ng[2];
    int fw = pair, fh = 0;
    auto fetch = [&]() {
      const int orow = (fw / nfc) * 256 + (int)rank * 128 + row;
      const bool live = fw < g.nwork && orow < nout;
      const int tokn = live ? sh_ctx_tok(d, orow) : 0;
      const uint4* src = reinterpret_cast<const uint4*>(ahat + (size_t)tokn * HD + fh * D + kh * (D / 2));
#pragma unroll
      for (int i = 0; i < 8; ++i) nxt[i] = live ? __ldg(src + i) : make_uint4(0, 0, 0, 0);
      const size_t so = ((size_t)tokn * d.H + fh) * d.k;
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        const bool lj = live && j < d.k;
        ni[j] = lj ? __ldg(g.idx + so + j) : -1;
        ng[j] = lj ? __ldg(g.gate + so + j) : 0.f;
        if (lj && !SH_INDEX_OK(ni[j], d.E, g.status, SH_SITE_O_EXPERT)) ni[j] = -1;
      }
      if (++fh == d.H) { fh = 0; fw += npairs; }
    };
    pdl_wait();                                            // Ahat is complete
    if (bt == 0) sh_stamp_start(d.stamps, SH_K_O);
    fetch();
    const uint32_t trow = row * 128, tx = row & 7;         // 16-byte chunk j of a stage row: block j / 8, chunk (j % 8) ^ tx (128-byte swizzle)
    int gs = 0;                                            // running stage number of this pair
    bool ok = true;
    for (int w = pair; w < g.nwork && ok; w += npairs) {
      for (int h = 0; h < d.H && ok; ++h, gs += SPH) {
#pragma unroll
        for (int i = 0; i < 8; ++i) cur[i] = nxt[i];
#pragma unroll
        for (int j = 0; j < 2; ++j) { ci[j] = ni[j]; cg[j] = ng[j]; }
        fetch();
        __half2 g_hi[SPT], g_lo[SPT];                      // per group: the gates of its two kept positions, each as hi + lo
#pragma unroll
        for (int c = 0; c < SPT; ++c) {
          int lo, hi; float ga, gb;
          osp_group(ci[0], cg[0], ci[1], cg[1], c, lo, hi, ga, gb);
          const __half ha = __float2half_rn(ga), hb = __float2half_rn(gb);
          g_hi[c] = __halves2half2(ha, hb);
          g_lo[c] = __floats2half2_rn(ga - __half2float(ha), gb - __half2float(hb));
        }
        const __half* av = reinterpret_cast<const __half*>(cur);
#pragma unroll
        for (int s = 0; s < SPT; ++s) {
          const int sn = gs + kh * SPT + s, ps = sn % PST;
          const uint32_t ppar = ((uint32_t)(sn / PST) & 1u) ^ 1u;
          if (lane == 0 && !mbar_wait(&p_empty[ps], ppar, g.status, dead)) ok = false;
          ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
          if (!ok) break;
          unsigned char* tile = sgen + p_off + ps * SM::P_BYTES;
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            uint4 v;
            __half2* hv = reinterpret_cast<__half2*>(&v);
            if (SPT == 1) {                                // four d per chunk, one group each
#pragma unroll
              for (int q = 0; q < 4; ++q) hv[q] = osp_scale(av[4 * j + q], g_hi[0], g_lo[0]);
            } else {                                       // two d per chunk, two groups each
#pragma unroll
              for (int q = 0; q < 2; ++q) {
                const __half a = av[32 * s + 2 * j + q];
                hv[2 * q] = osp_scale(a, g_hi[0], g_lo[0]);
                hv[2 * q + 1] = osp_scale(a, g_hi[SPT - 1], g_lo[SPT - 1]);
              }
            }
            *reinterpret_cast<uint4*>(tile + (j >> 3) * TBLK + trow + (((j & 7) ^ tx) << 4)) = v;
          }
          fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) mbar_arrive_leader(&p_full[ps]);
        }
      }
    }
  } else if (warp < 14) {
    // ---- epilogue: warp = 32 tokens (TMEM lane quarter warp & 3), all 256 features of the unit ----
    const int q = warp & 3;
    const uint32_t lane_off = (uint32_t)(q * 32) << 16;
    float* stg = reinterpret_cast<float*>(sgen + stg_off) + (warp - 10) * 1024;
    // the position-code words of TMEM lane L = q*32 + lane: rows ra and ra + 8 of this CTA's 128 tokens
    const int L = q * 32 + lane, ra = (L & ~15) | (L & 7);
    uint32_t mw[OSP_MAXH];
    auto codes_of = [&](int w) {
#pragma unroll
      for (int h = 0; h < OSP_MAXH; ++h) mw[h] = 0x44444444u;
      if (w >= g.nwork) return;
#pragma unroll
      for (int r2 = 0; r2 < 2; ++r2) {
        const int orow = (w / nfc) * 256 + (int)rank * 128 + ra + 8 * r2;
        if (orow >= nout) continue;
        const size_t so = (size_t)sh_ctx_tok(d, orow) * d.H * d.k;
#pragma unroll
        for (int h = 0; h < OSP_MAXH; ++h) {
          if (h < d.H) {
            int i0 = __ldg(g.idx + so + h * d.k), i1 = d.k > 1 ? __ldg(g.idx + so + h * d.k + 1) : -1;
            if ((unsigned)i0 >= (unsigned)d.E) i0 = -1;
            if ((unsigned)i1 >= (unsigned)d.E) i1 = -1;
            const uint32_t c16 = osp_row_codes<SPT>(i0, i1);
            mw[h] = r2 == 0 ? ((mw[h] & 0xFFFF0000u) | c16) : ((mw[h] & 0x0000FFFFu) | (c16 << 16));
          }
        }
      }
    };
    auto put_codes = [&](int buf_of_codes, int unit_no) {      // unit_no's codes into the first columns of buffer buf_of_codes
#pragma unroll
      for (int h = 0; h < OSP_MAXH; ++h)
        if (h < d.H) tmem_st1(tmem + lane_off + buf_of_codes * 256 + h, mw[h]);
      tmem_st_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_leader(&m_full[unit_no & 1]);
    };
    if (pair < g.nwork) { codes_of(pair); put_codes(1, 0); }
    pdl_wait();                                            // (out is not written before the kernels ahead are done)
    int un = 0;
    for (int w = pair; w < g.nwork; w += npairs, ++un) {
      const int buf = un & 1;
      const int row0 = (w / nfc) * 256 + (int)rank * 128, fc = w % nfc;
      const int rows_here = min(32, nout - row0 - q * 32);
      const bool more = w + npairs < g.nwork;
      if (more) codes_of(w + npairs);                      // (fetched before the wait: an L2 round trip)
      if (!mbar_wait(&d_full[buf], (un >> 1) & 1, g.status, dead)) break;
      tc_fence_after();
      const size_t obase = (size_t)(row0 + q * 32) * d.M + fc * 256;
      const uint32_t taddr = tmem + lane_off + buf * 256;
#pragma unroll 1
      for (int c = 0; c < 8; ++c) {
        uint32_t v[32];
        tmem_ld32(taddr + c * 32, v);
        tmem_ld_wait();
        if (c == 0 && more) put_codes(buf, un + 1);         // these columns are free now: the next unit's codes
        __syncwarp();
#pragma unroll
        for (int ch = 0; ch < 8; ++ch)
          *reinterpret_cast<uint4*>(stg + lane * 32 + ((ch ^ (lane & 7)) << 2)) = make_uint4(v[4 * ch], v[4 * ch + 1], v[4 * ch + 2], v[4 * ch + 3]);
        __syncwarp();
        if (fc * 256 + c * 32 < d.M) {
#pragma unroll
          for (int r4 = 0; r4 < 32; r4 += 4) {
            const int r = r4 + (lane >> 3), ch = lane & 7;
            if (r < rows_here)
              oproj_put4(g.out, obase + (size_t)r * d.M + c * 32 + 4 * ch, *reinterpret_cast<const float4*>(stg + r * 32 + ((ch ^ (r & 7)) << 2)), g.out_f16);
          }
        }
        if (c == 7) {
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_leader(&d_empty[buf]);
        }
      }
    }
  }
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
