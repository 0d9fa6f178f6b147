// Persistent tcgen05 GEMMs for the two projections that dominate the front of the layer: the
// dense Q/K projection (PG_QKV) and the grouped value-expert projection (PG_V).
//
// One CTA per SM walks tiles: blockIdx.x, blockIdx.x + gridDim.x, ... for the value experts; for
// the dense projection, which starts while the gate kernel still holds part of the GPU (so its
// CTAs start at different times), tiles are claimed one at a time from a global counter by the
// producer thread and handed to the other roles through a small shared-memory ring.  The operand ring (TMA for
// B and for dense A; cp.async row gathers for the value experts' A) and the two TMEM
// accumulator buffers run on across tiles, so the ~3 us a CTA needs to set itself up and
// the first ~0.9 us TMA round trip are paid once per SM instead of once per tile, and the
// epilogue of tile i overlaps the main loop of tile i + 1.
//
// Warp roles (320 threads): warp 0 = TMA producer, warp 1 = TMEM owner + UMMA issuer,
// warps 2..5 = epilogue (thread = accumulator row = TMEM lane), warps 6..9 = A-row gatherers
// (PG_V); in PG_QKV warp 6 is a second TMA producer and warps 7..9 idle.
// Tile = (MT * 128) rows x BN columns, MT * BN <= 256 so that two accumulators fit TMEM.
#pragma once
#include "sh_tc_gemm.cuh"

namespace shtc {

enum { PG_QKV = 0, PG_V = 1 };

template <int BN, int STAGES, int MT>
struct PGemmSmem {
  static constexpr int A_BYTES = MT * 128 * 64 * 2;
  static constexpr int B_BYTES = BN * 64 * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int BAR_OFF = STAGES * STAGE_BYTES;
  static constexpr int TOTAL = BAR_OFF + 256 + 1024;
};

template <int BN, int STAGES, int MODE, int MT>
__global__ void __launch_bounds__(352, 1)
sh_tc_pgemm_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB, TcGemmArgs g) {
  using SM = PGemmSmem<BN, STAGES, MT>;
  static_assert(MT * BN <= 256, "two accumulators must fit the 512 TMEM columns");
  constexpr bool GATHER = MODE == PG_V;
  constexpr int ROWS = MT * 128;
  constexpr int ACC_COLS = 256;                            // TMEM columns per accumulator buffer
  extern __shared__ unsigned char smem_raw[];
  const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* sgen = smem_raw + (sbase - smem_u32(smem_raw));
  uint64_t* full_bar = (uint64_t*)(sgen + SM::BAR_OFF);
  uint64_t* empty_bar = full_bar + STAGES;
  uint64_t* acc_full = empty_bar + STAGES;     // [2]
  uint64_t* acc_empty = acc_full + 2;          // [2]
  uint32_t* tmem_slot = (uint32_t*)(acc_empty + 2);
  constexpr int TQ = 4;                                    // claimed-tile ring (dense mode)
  uint64_t* tq_full = (uint64_t*)(sgen + SM::BAR_OFF + 128);
  uint64_t* tq_empty = tq_full + TQ;
  int* tq_tile = (int*)(tq_empty + TQ);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const ShDims& d = g.d;
  const int KB = g.K / 64;
  const int ncol = (g.ncols + BN - 1) / BN;                // column tiles (dense mode)
  bool dead = false;

  if (threadIdx.x == 0) {
    // (MT == 2: one issuing thread per 128-row half of the tile, each committing on its own)
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full_bar[s], GATHER ? 129 : 2); mbar_init(&empty_bar[s], MT); }
    for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], MT); mbar_init(&acc_empty[b], 128); }
    for (int j = 0; j < TQ; ++j) { mbar_init(&tq_full[j], 1); mbar_init(&tq_empty[j], 130); }   // A producer + issuer + 128 epilogue threads
    fence_barrier_init();
    tma_prefetch_desc(&mapB);
    if (!GATHER) tma_prefetch_desc(&mapA);
  }
  if (warp == 1) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  // Programmatic dependent launch: the next kernel in the stream may become resident from here on.
  // The value experts need the sorted lists (kernel before this one) now.  The dense projection
  // reads nothing an earlier kernel of the same forward pass wrote, so it only waits at its end
  // (which makes "this grid completed" imply "everything before it completed") -- but measured on
  // B200, the TMA loads of a grid launched this way do not return before the grid ahead of it has
  // completed (plain loads do), so the layer launches this projection the ordinary way on a
  // second stream instead when it wants it to run beside the gate and sort kernels.
  pdl_trigger();
  if (threadIdx.x == 0) sh_stamp_resident(d.stamps, g.stamp_id);
  if (GATHER) pdl_wait();
  if (threadIdx.x == 0) sh_stamp_start(d.stamps, g.stamp_id);
  const int ntiles = GATHER ? *g.ntiles : ((g.nrows + ROWS - 1) / ROWS) * ncol;
  // the qi-th tile of this CTA for every role but the claiming producer, or -1 when there is none
  auto next_tile = [&](int qi) -> int {
    if (GATHER) {
      const int t = blockIdx.x + qi * gridDim.x;
      return t < ntiles ? t : -1;
    }
    const int j = qi & (TQ - 1);
    if (!mbar_wait(&tq_full[j], (qi / TQ) & 1, g.status, dead)) return -1;
    const int t = tq_tile[j];
    mbar_arrive(&tq_empty[j]);
    return t;
  };

  if (warp == 0 || (!GATHER && warp == 6)) {
    // one thread issues a TMA box only every ~150 ns, so in the dense mode the A and the B boxes
    // of a stage come from two threads (warp 0: B, warp 6: A), each arriving with its own bytes
    if (lane == 0) {
      const bool do_b = warp == 0, do_a = !GATHER && warp == 6;
      int s = 0;
      uint32_t par = 1;
      for (int qi = 0; !dead; ++qi) {
        int t;
        if (!GATHER && do_b) {
          // claim the next tile only now, when the loads of the previous one are all issued
          const int j = qi & (TQ - 1);
          if (!mbar_wait(&tq_empty[j], ((qi / TQ) & 1) ^ 1, g.status, dead)) break;
          t = atomicAdd(g.sched, 1);
          if (t >= ntiles) t = -1;
          tq_tile[j] = t;
          mbar_arrive(&tq_full[j]);
          if (t < 0) {
            // the CTA whose final claim comes last puts both counters back for the next launch
            if (atomicAdd(g.sched + 1, 1) == (int)gridDim.x - 1) { g.sched[0] = 0; g.sched[1] = 0; }
          }
        } else {
          t = next_tile(qi);
        }
        if (t < 0) break;
        int row0, brow;
        if (GATHER) {
          const ShTile tl = tile_checked(g.tiles[t], d, g.status);
          row0 = 0;
          brow = (tl.h * d.E + tl.e) * g.b_rows_per_group;
        } else {
          row0 = (t / ncol) * ROWS;
          brow = (t % ncol) * BN;
        }
        for (int kb = 0; kb < KB; ++kb) {
          if (!mbar_wait(&empty_bar[s], par, g.status, dead)) break;
          const uint32_t sa = sbase + s * SM::STAGE_BYTES, sb = sa + SM::A_BYTES;
          if (do_a) {
            mbar_expect_tx(&full_bar[s], SM::A_BYTES);
#pragma unroll
            for (int mt = 0; mt < MT; ++mt)
              tma_load_2d(sa + mt * (128 * 64 * 2), &mapA, &full_bar[s], kb * 64, row0 + mt * 128);
          }
          if (do_b) {
            mbar_expect_tx(&full_bar[s], SM::B_BYTES);
            tma_load_2d(sb, &mapB, &full_bar[s], kb * 64, brow);
          }
          if (++s == STAGES) { s = 0; par ^= 1; }
        }
      }
    }
  } else if (warp == 1 || (MT == 2 && warp == 10)) {
    // With two 128-row halves per tile (MT == 2, N = 128) a stage is eight UMMAs of 64 cycles, and
    // issuing one costs a thread about as long: each half has its own issuing thread (warp 1 / 10),
    // its own accumulator columns and its own commits.
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc_f16(128, BN, 1, 1, 0);
      const int mt = warp == 1 ? 0 : 1;
      const uint32_t a_lo0 = desc_lo_k(sbase) + mt * (128 * 64 * 2 >> 4), b_lo0 = desc_lo_k(sbase + SM::A_BYTES);
      int s = 0, it = 0;
      uint32_t par = 0;
      for (; !dead; ++it) {
        if (next_tile(it) < 0) break;
        const int b = it & 1;
        if (!mbar_wait(&acc_empty[b], ((it >> 1) & 1) ^ 1, g.status, dead)) break;
        const uint32_t td = tmem + b * ACC_COLS + mt * BN;
        for (int kb = 0; kb < KB; ++kb) {
          if (!mbar_wait(&full_bar[s], par, g.status, dead)) break;
          tc_fence_after();
          const uint32_t a_lo = a_lo0 + s * (SM::STAGE_BYTES >> 4), b_lo = b_lo0 + s * (SM::STAGE_BYTES >> 4);
#pragma unroll
          for (int k = 0; k < 4; ++k)
            umma_f16(td, desc_pack(a_lo + 2 * k), desc_pack(b_lo + 2 * k), idesc, (kb | k) != 0);
          umma_commit(&empty_bar[s]);
          if (++s == STAGES) { s = 0; par ^= 1; }
        }
        if (dead) break;
        umma_commit(&acc_full[b]);
      }
    }
  } else if (warp >= 6 && warp < 10) {
    if (GATHER) {
      // thread -> 16-byte chunk c of rows rb, rb + 16, ... (8 threads cover one 128-byte row)
      const int et = threadIdx.x - 192;                    // 0..127
      const int c = et & 7, rb = et >> 3;
      const uint32_t dsw = (uint32_t)((c ^ (rb & 7)) << 4);
      int s = 0, issued = 0, n_arr = 0, s_arr = 0;
      uint32_t par = 1;
      for (int qi = 0; !dead; ++qi) {
        const int t = next_tile(qi);
        if (t < 0) break;
        const ShTile tl = tile_checked(g.tiles[t], d, g.status);
        const char* src[8 * MT];
        uint32_t ok[8 * MT];
#pragma unroll
        for (int i = 0; i < 8 * MT; ++i) {
          const int r = rb + 16 * i;
          int tok = 0;
          ok[i] = 0;
          if (r < tl.nrows) { tok = g.lists[(size_t)tl.h * d.N * d.k + tl.row0 + r]; ok[i] = 16; }
          if (!SH_INDEX_OK(tok, d.N, g.status, SH_SITE_V_LIST)) { tok = 0; ok[i] = 0; }
          src[i] = (const char*)g.A + ((long)tok * g.lda + c * 8) * 2;
        }
        for (int kb = 0; kb < KB; ++kb) {
          if (!mbar_wait(&empty_bar[s], par, g.status, dead)) break;
          const uint32_t sa = sbase + s * SM::STAGE_BYTES;
#pragma unroll
          for (int i = 0; i < 8 * MT; ++i)
            cp_async_16(sa + (rb + 16 * i) * 128 + dsw, src[i] + (long)kb * 128, ok[i]);
          cp_async_commit();
          ++issued;
          if (issued - n_arr > 2) {                        // the copies of the stage issued two rounds ago have landed
            cp_async_wait<2>();
            fence_proxy_async_smem();
            mbar_arrive(&full_bar[s_arr]);
            ++n_arr;
            if (++s_arr == STAGES) s_arr = 0;
          }
          if (++s == STAGES) { s = 0; par ^= 1; }
        }
      }
      cp_async_wait<0>();
      fence_proxy_async_smem();
      if (!dead)
        for (; n_arr < issued; ++n_arr) {
          mbar_arrive(&full_bar[s_arr]);
          if (++s_arr == STAGES) s_arr = 0;
        }
    }
  } else if (warp < 6) {
    // ---- epilogue: thread = accumulator row = TMEM lane -----------------------------------------
    const int q = warp & 3;
    const uint32_t lane_off = (uint32_t)(q * 32) << 16;
    int it = 0;
    for (;; ++it) {
      const int t = next_tile(it);
      if (t < 0) break;
      const int b = it & 1;
      int th = 0, row0, nrows, col0 = 0;
      if (GATHER) {
        const ShTile tl = tile_checked(g.tiles[t], d, g.status);
        th = tl.h; row0 = tl.row0; nrows = tl.nrows;
      } else {
        row0 = (t / ncol) * ROWS;
        nrows = min(ROWS, g.nrows - row0);
        col0 = (t % ncol) * BN;
      }
      int tok[MT];
      float gate[MT];
#pragma unroll
      for (int mt = 0; mt < MT; ++mt) {                    // fetched before the wait: hides the list latency
        const int r = mt * 128 + q * 32 + lane;
        tok[mt] = -1; gate[mt] = 0.f;
        if (r < nrows) {
          if (GATHER) {
            const size_t li = (size_t)th * d.N * d.k + row0 + r;
            tok[mt] = g.lists[li];
            gate[mt] = g.lgate[li];
            if (!SH_INDEX_OK(tok[mt], d.N, g.status, SH_SITE_V_TOKEN)) tok[mt] = -1;
          } else {
            tok[mt] = row0 + r;
          }
        }
      }
      if (!mbar_wait(&acc_full[b], (it >> 1) & 1, g.status, dead)) break;
      tc_fence_after();
#pragma unroll
      for (int mt = 0; mt < MT; ++mt) {
        const uint32_t trow = tmem + lane_off + b * ACC_COLS + mt * BN;
        const bool live = tok[mt] >= 0;
        const int bb = live ? tok[mt] / d.T : 0, tt = live ? tok[mt] % d.T : 0;
        const bool early = MODE == PG_V && live && g.v_early && tt < d.early_rows;
#pragma unroll 1
        for (int c00 = 0; c00 < BN; c00 += 64) {
          uint32_t vv[64];
          tmem_ld32(trow + c00, *reinterpret_cast<uint32_t(*)[32]>(&vv[0]));
          tmem_ld32(trow + c00 + 32, *reinterpret_cast<uint32_t(*)[32]>(&vv[32]));
          tmem_ld_wait();
          if (mt == MT - 1 && c00 + 64 >= BN) {            // the accumulator is in registers: hand the buffer back
            tc_fence_before();
            mbar_arrive(&acc_empty[b]);
          }
#pragma unroll
          for (int hh2 = 0; hh2 < 2; ++hh2) {
            const int c0 = c00 + hh2 * 32;
            uint32_t* v = &vv[hh2 * 32];
            const int n0 = col0 + c0;
            if (!live || n0 >= g.ncols) continue;
            uint32_t p[16];
            if (MODE == PG_QKV) {
              const int HD = d.H * d.D;
              const int which = n0 / HD, hd = (n0 % HD) / d.D, dd = n0 % d.D;
              __half* dst = (__half*)(which == 0 ? g.out0 : which == 1 ? g.out1 : g.out2) +
                            (((size_t)bb * d.H + hd) * d.T + tt) * d.D + dd;
              const float sc = which == 0 ? g.qscale : 1.f;
              if (g.rope && which < 2) rope_pairs16(v, g.rope + tt, dd >> 1, d.T);
#pragma unroll
              for (int i = 0; i < 16; ++i) {
                __half2 hv = __floats2half2_rn(__uint_as_float(v[2 * i]) * sc, __uint_as_float(v[2 * i + 1]) * sc);
                p[i] = *reinterpret_cast<uint32_t*>(&hv);
              }
#pragma unroll
              for (int i = 0; i < 4; ++i)
                *reinterpret_cast<uint4*>(dst + 8 * i) = make_uint4(p[4 * i], p[4 * i + 1], p[4 * i + 2], p[4 * i + 3]);
            } else {
              __half* dst = (__half*)g.out0 + (((size_t)bb * d.H + th) * d.T + tt) * d.D + n0;
              const float gt = gate[mt];
#pragma unroll
              for (int i = 0; i < 16; ++i) {
                __half2 hv = __floats2half2_rn(__uint_as_float(v[2 * i]) * gt, __uint_as_float(v[2 * i + 1]) * gt);
                p[i] = *reinterpret_cast<uint32_t*>(&hv);
              }
              if (early) {
                float* d32 = g.v_early + (((size_t)bb * d.H + th) * SH_EARLY_ROWS + tt) * d.D + n0;
#pragma unroll
                for (int i = 0; i < 8; ++i)
                  red_add_v4_f32(d32 + 4 * i, __uint_as_float(v[4 * i]) * gt, __uint_as_float(v[4 * i + 1]) * gt,
                                 __uint_as_float(v[4 * i + 2]) * gt, __uint_as_float(v[4 * i + 3]) * gt);
              } else {
#pragma unroll
                for (int i = 0; i < 4; ++i) red_add_v4_f16x2(dst + 8 * i, p[4 * i], p[4 * i + 1], p[4 * i + 2], p[4 * i + 3]);
              }
            }
          }
        }
        if (early)
          v_early_finish(g.v_early + (((size_t)bb * d.H + th) * SH_EARLY_ROWS + tt) * d.D, g.v_early_cnt + ((size_t)bb * d.H + th) * SH_EARLY_ROWS + tt,
                         (__half*)g.out0 + (((size_t)bb * d.H + th) * d.T + tt) * d.D, d.D, d.k);
      }
    }
  }
  if (!GATHER) pdl_wait();
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0) sh_stamp_end(d.stamps, g.stamp_id);
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

}  // namespace shtc
