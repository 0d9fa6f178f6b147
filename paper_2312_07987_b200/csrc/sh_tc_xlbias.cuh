// Score bias of Transformer-XL's relative-position term on the tensor-core path (the positional
// encoding of the paper's main models; the decomposition is Transformer-XL's):
//   bias[b, h, i, s] = c * ( q_i . r_{p_i - s}  +  v^h . r_{p_i - s}  +  u^h . k_s ),   p_i = Tc + i, s <= p_i
// (c = log2(e)/sqrt(d_head) is already folded into the stored Q; the attention kernel adds bias to its
// S tiles, which are in the same units).  The first term is a GEMM over DISTANCES - Q[b,h] (chunk rows)
// times R16[h]^T - whose result must be shifted, row by row, from distance order to key order (the
// "relative shift" of Transformer-XL).  A warp-uniform TMEM address cannot shift per row, so the shift
// happens in the store: the 32 x 32 chunk of a warp goes through shared memory and every store
// instruction writes 32 consecutive keys of one query row (2-byte elements, coalesced).
//
// CTA = (batch*head, 128-query tile of the chunk): Q tile loaded once, 64-distance tiles of R16[h]
// streamed through a ring of 2 (only distances up to the tile's largest query position exist), UMMA
// N = 64 into two alternating TMEM buffers, eight epilogue warps (two per TMEM lane quarter, one
// 32-column chunk each).  The epilogue is a chain of short latencies, so what helps is warps: the
// CTA is sized (100 KB of shared memory) for two per SM.
// Warp roles (320 threads): warp 0 = TMA producer, warp 1 = TMEM owner + UMMA issuer, warps 2..9 = epilogue.
#pragma once
#include "sh_tc_prims.cuh"

namespace shtc {

struct TcXlBiasArgs {
  ShDims d;
  const float* vr;       // [H, T]     c * v^h . r_dist
  const float* uk;       // [B, H, T]  c * u^h . k_s
  __half* bias;          // [B, H, T - Tc, T]
  int* status;
};

template <int D>
struct XlBiasSmem {
  static constexpr int T_BYTES = 128 * D * 2;            // the query tile
  static constexpr int R_BYTES = 64 * D * 2;             // one tile of 64 distances
  static constexpr int RST = 2;
  static constexpr int Q_OFF = 0;
  static constexpr int R_OFF = T_BYTES;
  static constexpr int STG_OFF = R_OFF + RST * R_BYTES;
  static constexpr int STG_WARP = (32 * 33 + 64) * 4;   // the 32 x 32 chunk (padded rows) + the 63 u.k values it meets
  static constexpr int BAR_OFF = STG_OFF + 8 * STG_WARP;
  static constexpr int TOTAL = BAR_OFF + 256 + 1024;
};

template <int D>
__global__ void __launch_bounds__(320, 2)
sh_tc_xlbias_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapR, TcXlBiasArgs g) {
  using SM = XlBiasSmem<D>;
  constexpr int DB = D / 64, RST = SM::RST;
  constexpr uint32_t BLK = 128 * 128;                    // a 64-column block of the query tile
  constexpr uint32_t RBLK = 64 * 128;                    // a 64-column block of a distance tile
  extern __shared__ unsigned char smem_raw[];
  const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* sgen = smem_raw + (sbase - smem_u32(smem_raw));
  uint64_t* bars = (uint64_t*)(sgen + SM::BAR_OFF);
  uint64_t* q_full = bars;
  uint64_t* r_full = bars + 1;       // [RST]
  uint64_t* r_empty = bars + 5;      // [RST]
  uint64_t* acc_full = bars + 9;     // [2]
  uint64_t* acc_empty = bars + 11;   // [2] eight arrivals (epilogue warps)
  uint32_t* tmem_slot = (uint32_t*)(bars + 13);

  const ShDims& d = g.d;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int Tq = d.T - d.Tc, tiles_q = Tq / 128;
  const int nbh = d.B * d.H;
  const int bh = blockIdx.x % nbh, it = tiles_q - 1 - blockIdx.x / nbh, h = bh % d.H;   // longest tiles (most distances) first
  const int ncol = 2 * (d.Tc / 128 + it + 1);            // 64-distance tiles that hold a visible distance for some row of this tile
  bool dead = false;

  if (threadIdx.x == 0) {
    mbar_init(q_full, 1);
    for (int s = 0; s < RST; ++s) { mbar_init(&r_full[s], 1); mbar_init(&r_empty[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], 8); }
    fence_barrier_init();
    tma_prefetch_desc(&mapQ); tma_prefetch_desc(&mapR);
  }
  if (warp == 1) { tmem_alloc(tmem_slot, 128); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  pdl_trigger();
  pdl_wait();                                            // Q, K (hence u.k) of this pass are complete

  if (warp == 0) {
    if (lane == 0) {
      mbar_expect_tx(q_full, SM::T_BYTES);
#pragma unroll
      for (int c = 0; c < DB; ++c) tma_load_2d(sbase + SM::Q_OFF + c * BLK, &mapQ, q_full, c * 64, bh * d.T + d.Tc + it * 128);
      for (int ct = 0; ct < ncol; ++ct) {
        const int s = ct % RST;
        if (!mbar_wait(&r_empty[s], ((ct / RST) & 1) ^ 1, g.status, dead)) break;
        mbar_expect_tx(&r_full[s], SM::R_BYTES);
#pragma unroll
        for (int c = 0; c < DB; ++c) tma_load_2d(sbase + SM::R_OFF + s * SM::R_BYTES + c * RBLK, &mapR, &r_full[s], c * 64, h * d.T + ct * 64);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc_f16(128, 64, 0, 0, 0);
      const uint32_t q_lo = desc_lo_k(sbase + SM::Q_OFF), r_lo0 = desc_lo_k(sbase + SM::R_OFF);
      if (mbar_wait(q_full, 0, g.status, dead)) {
        for (int ct = 0; ct < ncol; ++ct) {
          const int s = ct % RST, b = ct & 1;
          if (!mbar_wait(&r_full[s], (ct / RST) & 1, g.status, dead)) break;
          if (!mbar_wait(&acc_empty[b], ((ct >> 1) & 1) ^ 1, g.status, dead)) break;
          tc_fence_after();
          const uint32_t r_lo = r_lo0 + s * (SM::R_BYTES >> 4);
#pragma unroll
          for (int k = 0; k < D / 16; ++k)
            umma_f16(tmem + b * 64, desc_pack(q_lo + (k / 4) * (BLK >> 4) + 2 * (k % 4)), desc_pack(r_lo + (k / 4) * (RBLK >> 4) + 2 * (k % 4)), idesc, k != 0);
          umma_commit(&r_empty[s]);
          umma_commit(&acc_full[b]);
        }
      }
    }
  } else {
    // ---- epilogue: warp = 32 query rows (TMEM lane quarter), thread = query row while reading TMEM ----
    const int q = warp & 3, half = (warp - 2) >> 2;
    const uint32_t lane_off = (uint32_t)(q * 32) << 16;
    float* stg = reinterpret_cast<float*>(sgen + SM::STG_OFF + (warp - 2) * SM::STG_WARP);
    float* suk = stg + 32 * 33;
    const int qi0 = it * 128 + q * 32;                     // first query row (inside the chunk) of this warp
    __half* out_bh = g.bias + (size_t)bh * Tq * d.T;
    const float* vr = g.vr + (size_t)h * d.T;
    const float* ukr = g.uk + (size_t)bh * d.T;
    for (int ct = 0; ct < ncol; ++ct) {
      const int b = ct & 1;
      if (!mbar_wait(&acc_full[b], (ct >> 1) & 1, g.status, dead)) break;
      tc_fence_after();
      {
        const int dist0 = ct * 64 + half * 32;             // this warp's 32 distances of the tile
        const int s_lo = d.Tc + qi0 - dist0 - 31;          // keys this chunk meets: s_lo .. s_lo + 62
        const float vrd = vr[dist0 + lane];
        const float uk0 = (s_lo + lane >= 0) ? ukr[s_lo + lane] : 0.f;
        const float uk1 = (s_lo + 32 + lane >= 0 && s_lo + 32 + lane < d.T) ? ukr[s_lo + 32 + lane] : 0.f;
        uint32_t v[32];
        tmem_ld32(tmem + lane_off + b * 64 + half * 32, v);
        tmem_ld_wait();
        tc_fence_before();                                 // this warp's share of the accumulator is in registers
        __syncwarp();
        if (lane == 0) mbar_arrive(&acc_empty[b]);
#pragma unroll
        for (int i = 0; i < 32; ++i) stg[lane * 33 + i] = __uint_as_float(v[i]);
        suk[lane] = uk0;
        suk[32 + lane] = uk1;
        __syncwarp();
        __half* op = out_bh + ((long)qi0 * d.T + (s_lo + 31 - lane));   // row qi0 + rr, key s_lo + 31 + rr - lane: += T + 1 per row
        const int s0 = s_lo + 31 - lane;
#pragma unroll 8
        for (int rr = 0; rr < 32; ++rr) {
          if (s0 + rr >= 0) op[(long)rr * (d.T + 1)] = __float2half_rn(stg[rr * 33 + lane] + vrd + suk[31 + rr - lane]);
        }
        __syncwarp();
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, 128);
  }
}

}  // namespace shtc
