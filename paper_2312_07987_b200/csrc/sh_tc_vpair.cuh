// Value-expert projection of a k = 2 layer on CTA pairs, tiled by (head, PAIR of selected experts)
// (Sec. 2.2, the value equation):  V^h[t] = s^h[t,a] * x[t] W_V^{h,a} + s^h[t,b] * x[t] W_V^{h,b},  {a, b} = E_S^h(t).
//
// The expert-tiled kernel (sh_tc_pgemm_kernel<PG_V>) gathers every token row once per selected expert -
// H*k times per token - and adds the k gate-scaled results with reductions in global memory.  With k = 2
// every (token, head) has exactly one pair {a < b}; sorting the tokens of a head by their pair instead of
// by expert gives tiles whose rows ALL want the same two experts:  one gather of the row (H times per
// token), one UMMA of N = 256 against [W^{h,a} | W^{h,b}], and the gate-weighted sum of the two halves of
// the accumulator row in the epilogue, stored once - no reductions, no cleared buffer, no dependence on
// arrival order.  On a CTA pair (tcgen05 cta_group::2, M = 256) each CTA gathers its own 128 rows and
// loads ONE of the two experts' 128 weight rows; the pair's tensor cores read both.  L2 -> shared memory
// per (token, head): 2 rows' worth of x + 2 of weights per 128 rows... 4 KB at d_model 1024 against 6 KB.
//
// Tile table and lists come from the same bucket sort, run over (head, pair) buckets: lists[h][...] holds
// the tokens of head h ordered by pair number, a tile = up to 256 consecutive entries of one pair.
//
// Warp roles per CTA (320 threads): warp 0 lane 0 = weight producer (TMA), warp 1 = TMEM allocation and,
// in the leader, the UMMA issuer, warps 2..5 = epilogue (thread = accumulator row), warps 6..9 = row
// gatherers (cp.async, 16 bytes per thread and row, manual 128-byte swizzle).
// Barriers: operand-full in the leader (its producer arrives with the pair's weight bytes, every gather
// warp of both CTAs arrives when its rows have landed), operand-empty and accumulator-full in both CTAs
// (multicast tcgen05.commit), accumulator-empty in the leader (epilogue warps of both CTAs).
#pragma once
#include "sh_tc_gemm.cuh"

namespace shtc {

#ifndef VPAIR_LAG
#define VPAIR_LAG 2                                        // gather rounds in flight per thread before it waits for the oldest
#endif

struct TcVPairArgs {
  ShDims d;
  const void* x;             // [N, M] bf16
  const int* lists;          // [H][N]: tokens of head h ordered by pair
  const ShTile* tiles;       // (h, pair, row0, nrows <= 256)
  const int* ntiles;
  const int* idx;            // source side [N, H, 2]
  const float* gate;         // source side [N, H, 2]
  __half* v;                 // [B, H, T, D]: the projection's result (V; K or Q of a layer with key / query experts)
  float scale;               // extra factor on the result (the queries' log2(e)/sqrt(d_head)); 0 = none
  int stamp_id;              // SH_K_V, or -1: no stamps (the key / query launches)
  const int* ready;          // nullptr, or a counter that reaches ready_count when lists, tiles, idx and gate are complete:
  int ready_count;           //   the kernel then waits for the counter at its start and for the grid before it only at its end
  int* status;
};

template <int STAGES>
struct VPairSmem {
  static constexpr int A_BYTES = 128 * 64 * 2;             // this CTA's 128 gathered rows, 64 columns
  static constexpr int B_BYTES = 128 * 64 * 2;             // this CTA's expert: 128 feature rows, 64 columns
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int BAR_OFF = STAGES * STAGE_BYTES;
  static constexpr int TOTAL = BAR_OFF + 256 + 1024;
};

template <int STAGES>
__global__ void __launch_bounds__(320, 1)
sh_tc_vpair_kernel(const __grid_constant__ CUtensorMap mapW, TcVPairArgs g) {
  using SM = VPairSmem<STAGES>;
  extern __shared__ unsigned char smem_raw[];
  const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* sgen = smem_raw + (sbase - smem_u32(smem_raw));
  uint64_t* full_bar = (uint64_t*)(sgen + SM::BAR_OFF);    // [STAGES] leader's: 1 + 8 arrivals
  uint64_t* empty_bar = full_bar + STAGES;                 // [STAGES] both CTAs
  uint64_t* acc_full = empty_bar + STAGES;                 // [2] both CTAs
  uint64_t* acc_empty = acc_full + 2;                      // [2] leader's: 8 arrivals
  uint32_t* tmem_slot = (uint32_t*)(acc_empty + 2);
  static_assert((2 * STAGES + 4) * 8 + 4 <= 256, "barrier area");

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
  const ShDims& d = g.d;
  const int KB = d.M / 64;
  bool dead = false;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full_bar[s], 9); mbar_init(&empty_bar[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], 8); }
    fence_barrier_init();
    tma_prefetch_desc(&mapW);
  }
  if (warp == 1) { tmem_alloc_pair(tmem_slot, 512); tmem_relinquish_pair(); }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  pdl_trigger();
  if (threadIdx.x == 0 && g.stamp_id >= 0) sh_stamp_resident(d.stamps, g.stamp_id);
  if (g.ready) {
    // The kernel before this one (the one-grid front) is wholly resident before any CTA of this one
    // exists, so waiting for its counter cannot starve it.  Bounded like every wait.
    if (threadIdx.x == 0) {
      const uint64_t t0 = global_timer_ns();
      int seen;
      do {
        asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(seen) : "l"(g.ready) : "memory");
        if (seen >= g.ready_count) break;
        if (global_timer_ns() - t0 > SH_WAIT_LIMIT_NS || *(volatile int*)g.status != 0) {
          if (atomicCAS(g.status, 0, SH_ERR_TIMEOUT) == 0) {
            g.status[1] = (int)blockIdx.x; g.status[2] = 0; g.status[3] = -1;
            g.status[4] = seen; g.status[5] = (int)gridDim.x; g.status[6] = (int)blockDim.x;
          }
          break;
        }
      } while (true);
    }
    __syncthreads();
    if (*(volatile int*)g.status != 0) dead = true;
  } else {
    pdl_wait();                                            // the sorted lists and the tile table
  }
  if (threadIdx.x == 0 && g.stamp_id >= 0) sh_stamp_start(d.stamps, g.stamp_id);
  // (the first tile's entry is fetched beside the tile count, not behind it: every dependent trip to L2
  //  costs this kernel's start 2-3 us while the Q/K projection's operand traffic keeps L2 busy)
  const ShTile tile_first = g.tiles[pair];                // (the table has room for every pair's index)
  const int ntiles = dead ? 0 : *g.ntiles;
  const int NP = sh_pair_count(d.E);
  auto tile_of = [&](int t) -> ShTile {
    ShTile tl = t == pair ? tile_first : g.tiles[t];
#ifdef SH_DEBUG
    const bool ok = SH_INDEX_OK(tl.h, d.H, g.status, SH_SITE_V_TILE) && SH_INDEX_OK(tl.e, NP, g.status, SH_SITE_V_TILE) &&
                    SH_INDEX_OK(tl.nrows, 257, g.status, SH_SITE_V_TILE) &&
                    SH_INDEX_OK((long long)tl.row0 + tl.nrows, (long long)d.N + 1, g.status, SH_SITE_V_TILE);
    if (!ok) { tl.h = 0; tl.e = 0; tl.row0 = 0; tl.nrows = 0; }
#endif
    return tl;
  };

  if (warp == 0) {
    if (lane == 0) {
      int s = 0;
      uint32_t par = 1;
      for (int t = pair; t < ntiles && !dead; t += npairs) {
        const ShTile tl = tile_of(t);
        int ea, eb;
        sh_pair_decode(tl.e, d.E, ea, eb);
        const int brow = (tl.h * d.E + (rank == 0 ? ea : eb)) * d.D;     // this CTA's expert: its D = 128 feature rows
        for (int kb = 0; kb < KB; ++kb) {
          if (!mbar_wait(&empty_bar[s], par, g.status, dead)) break;
          if (rank == 0) mbar_expect_tx(&full_bar[s], 2 * SM::B_BYTES);
          tma_load_2d_pair(sbase + s * SM::STAGE_BYTES + SM::A_BYTES, &mapW, &full_bar[s], kb * 64, brow);
          if (++s == STAGES) { s = 0; par ^= 1; }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = make_idesc_f16(256, 256, 1, 1, 0);
      const uint32_t a_lo0 = desc_lo_k(sbase), b_lo0 = desc_lo_k(sbase + SM::A_BYTES);
      int s = 0, it = 0;
      uint32_t par = 0;
      for (int t = pair; t < ntiles && !dead; t += npairs, ++it) {
        const int b = it & 1;
        if (!mbar_wait(&acc_empty[b], ((it >> 1) & 1) ^ 1, g.status, dead)) break;
        const uint32_t td = tmem + b * 256;
        for (int kb = 0; kb < KB; ++kb) {
          if (!mbar_wait(&full_bar[s], par, g.status, dead)) break;
          tc_fence_after();
          const uint32_t a_lo = a_lo0 + s * (SM::STAGE_BYTES >> 4), b_lo = b_lo0 + s * (SM::STAGE_BYTES >> 4);
#pragma unroll
          for (int k = 0; k < 4; ++k)
            umma_f16_pair(td, desc_pack(a_lo + 2 * k), desc_pack(b_lo + 2 * k), idesc, (kb | k) != 0);
          umma_commit_pair(&empty_bar[s], 3);
          if (++s == STAGES) { s = 0; par ^= 1; }
        }
        if (dead) break;
        umma_commit_pair(&acc_full[b], 3);
      }
    }
  } else if (warp >= 6) {
    // ---- gatherers: thread -> 16-byte chunk c of rows rb, rb + 16, ... of this CTA's 128 rows ----
    const int et = threadIdx.x - 192;                      // 0..127
    const int c = et & 7, rb = et >> 3;
    const uint32_t dsw = (uint32_t)((c ^ (rb & 7)) << 4);
    int s = 0, issued = 0, n_arr = 0, s_arr = 0;
    uint32_t par = 1;
    auto landed = [&]() {                                  // this warp's copies of stage s_arr are in shared memory
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive_leader(&full_bar[s_arr]);
      ++n_arr;
      if (++s_arr == STAGES) s_arr = 0;
    };
    for (int t = pair; t < ntiles && !dead; t += npairs) {
      const ShTile tl = tile_of(t);
      const char* src[8];
      uint32_t ok[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int r = (int)rank * 128 + rb + 16 * i;       // row of the tile
        int tok = 0;
        ok[i] = 0;
        if (r < tl.nrows) { tok = g.lists[(size_t)tl.h * d.N + tl.row0 + r]; ok[i] = 16; }
        if (!SH_INDEX_OK(tok, d.N, g.status, SH_SITE_V_LIST)) { tok = 0; ok[i] = 0; }
        src[i] = (const char*)g.x + ((long)tok * d.M + c * 8) * 2;
      }
      for (int kb = 0; kb < KB; ++kb) {
        bool okw = true;
        if (lane == 0) okw = mbar_wait(&empty_bar[s], par, g.status, dead);
        okw = __shfl_sync(0xffffffffu, (int)okw, 0) != 0;
        if (!okw) { dead = true; break; }
        const uint32_t sa = sbase + s * SM::STAGE_BYTES;
#pragma unroll
        for (int i = 0; i < 8; ++i)
          cp_async_16(sa + (rb + 16 * i) * 128 + dsw, src[i] + (long)kb * 128, ok[i]);
        cp_async_commit();
        ++issued;
        if (issued - n_arr > VPAIR_LAG) {                  // the copies of the stage issued VPAIR_LAG rounds ago have landed
          cp_async_wait<VPAIR_LAG>();
          landed();
        }
        if (++s == STAGES) { s = 0; par ^= 1; }
      }
    }
    cp_async_wait<0>();
    if (!dead)
      while (n_arr < issued) landed();
  } else {
    // ---- epilogue: thread = accumulator row = TMEM lane: gate-weighted sum of the two experts' halves ----
    const int q = warp & 3;
    const uint32_t lane_off = (uint32_t)(q * 32) << 16;
    int it = 0;
    for (int t = pair; t < ntiles; t += npairs, ++it) {
      const int b = it & 1;
      const ShTile tl = tile_of(t);
      const int r = (int)rank * 128 + q * 32 + lane;
      int tok = -1;
      float ga = 0.f, gb = 0.f;
      if (r < tl.nrows) {                                  // fetched before the wait: hides the list latency
        tok = g.lists[(size_t)tl.h * d.N + tl.row0 + r];
        if (!SH_INDEX_OK(tok, d.N, g.status, SH_SITE_V_TOKEN)) tok = -1;
      }
      if (tok >= 0) {
        const size_t so = ((size_t)tok * d.H + tl.h) * 2;
        const int i0 = g.idx[so], i1 = g.idx[so + 1];
        const float g0 = g.gate[so], g1 = g.gate[so + 1];
        ga = i0 < i1 ? g0 : g1;                            // a = the lower expert index of the pair
        gb = i0 < i1 ? g1 : g0;
        if (g.scale != 0.f) { ga *= g.scale; gb *= g.scale; }
      }
      if (!mbar_wait(&acc_full[b], (it >> 1) & 1, g.status, dead)) break;
      tc_fence_after();
      const uint32_t trow = tmem + lane_off + b * 256;
      const int bb = tok >= 0 ? tok / d.T : 0, tt = tok >= 0 ? tok % d.T : 0;
      __half* dst = g.v + (((size_t)bb * d.H + tl.h) * d.T + tt) * d.D;
#pragma unroll 1
      for (int c0 = 0; c0 < 128; c0 += 32) {
        uint32_t va[32], vb[32];
        tmem_ld32(trow + c0, va);
        tmem_ld32(trow + 128 + c0, vb);
        tmem_ld_wait();
        if (c0 == 96) {                                    // the accumulator is in registers: hand the buffer back
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_leader(&acc_empty[b]);
        }
        if (tok < 0) continue;
        uint32_t p[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const float y0 = fmaf(ga, __uint_as_float(va[2 * i]), gb * __uint_as_float(vb[2 * i]));
          const float y1 = fmaf(ga, __uint_as_float(va[2 * i + 1]), gb * __uint_as_float(vb[2 * i + 1]));
          __half2 hv = __floats2half2_rn(y0, y1);
          p[i] = *reinterpret_cast<uint32_t*>(&hv);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i)
          *reinterpret_cast<uint4*>(dst + c0 + 8 * i) = make_uint4(p[4 * i], p[4 * i + 1], p[4 * i + 2], p[4 * i + 3]);
      }
    }
  }
  pdl_wait();                                              // (the next kernel's wait for this grid then covers the grid before it)
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (threadIdx.x == 0 && g.stamp_id >= 0) sh_stamp_end(d.stamps, g.stamp_id);
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem, 512);
  }
}

}  // namespace shtc
