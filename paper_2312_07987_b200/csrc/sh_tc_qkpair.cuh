// Dense Q/K projection (Sec. 2.2: the query and key projections are plain per-head matrices) on CTA
// pairs: [Q | K] = x [W_Q | W_K], one persistent cluster of two CTAs per SM pair.
//
// A single CTA computing a 128 x 256 tile pulls 48 KB per 64-deep stage (16 KB of x, 32 KB of
// weights) for 512 cycles of UMMA: 96 B/cycle, more than the ~64-68 B/cycle one SM gets from L2, so
// the single-CTA kernel (sh_tc_pgemm_kernel<PG_QKV>) runs the tensor pipe at under half its rate.
// With tcgen05 cta_group::2 the pair computes 256 x 256: each CTA loads its own 128 rows of x and
// only HALF of the 256 weight rows (32 KB per stage, 64 B/cycle), keeps its 128 x 256 accumulator in
// its own tensor memory and runs its own epilogue; the leader (even CTA) issues the UMMAs.
//
// Tiles are claimed one at a time from a global counter (the projection runs beside the gate and
// sort kernels and may be launched as two grids that share the counter: one sized for the SMs the
// gate kernel leaves free, one that takes over the gate kernel's SMs when it is done - see
// sh_tc_forward - so clusters start at different times): the leader's weight
// producer claims, writes the tile number into the claimed-tile ring of both CTAs and arrives on
// both rings' barriers; all roles of both CTAs hand a ring slot back on the leader's barrier.
// Barriers: operand-full in the leader (the leader's two producers arrive with the pair's bytes),
// operand-empty and accumulator-full in both CTAs (multicast tcgen05.commit), accumulator-empty in
// the leader (the epilogue threads of both CTAs arrive).
//
// Warp roles per CTA (320 threads): warp 0 lane 0 = weight producer (in the leader also the tile
// claimer), warp 6 lane 0 = x producer, warp 1 = TMEM allocation and (leader) UMMA issuer,
// warps 2..5 = epilogue (thread = accumulator row: scale, optional rotary embedding, fp16, store
// into the [B, H, T, D] layouts).
#pragma once
#include "sh_tc_gemm.cuh"

namespace shtc {

template <int STAGES>
struct QkPairSmem {
  static constexpr int A_BYTES = 128 * 64 * 2;             // this CTA's 128 rows of x, 64 columns
  static constexpr int B_BYTES = 128 * 64 * 2;             // this CTA's 128 of the tile's 256 weight rows
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int BAR_OFF = STAGES * STAGE_BYTES;
  static constexpr int TOTAL = BAR_OFF + 512 + 1024;
};

// MODE 0: the Q/K(/V) projection (bf16 operands, epilogue above).  MODE 1: a plain product of fp16 operands
// with an fp32 row-major result, out0[row, col] (the dense comparator's output projection).
template <int STAGES, int MODE = 0>
__global__ void __launch_bounds__(320, 1)
sh_tc_qk_pair_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB, TcGemmArgs g) {
  using SM = QkPairSmem<STAGES>;
  constexpr int BN = 256, TQ = 4;
  extern __shared__ unsigned char smem_raw[];
  const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* sgen = smem_raw + (sbase - smem_u32(smem_raw));
  uint64_t* full_bar = (uint64_t*)(sgen + SM::BAR_OFF);    // [STAGES] leader's
  uint64_t* empty_bar = full_bar + STAGES;                 // [STAGES] both CTAs
  uint64_t* acc_full = empty_bar + STAGES;                 // [2] both CTAs
  uint64_t* acc_empty = acc_full + 2;                      // [2] leader's: 256 arrivals
  uint64_t* tq_full = acc_empty + 2;                       // [TQ] both CTAs
  uint64_t* tq_empty = tq_full + TQ;                       // [TQ] leader's: 260 arrivals
  int* tq_tile = (int*)(tq_empty + TQ);                    // [TQ] both CTAs
  uint32_t* tmem_slot = (uint32_t*)(tq_tile + TQ);
  static_assert((2 * STAGES + 4 + 2 * TQ) * 8 + TQ * 4 + 4 <= 512, "barrier area");

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const ShDims& d = g.d;
  const int KB = g.K / 64;
  const int ncol = (g.ncols + BN - 1) / BN;
  const int ntiles = ((g.nrows + 255) / 256) * ncol;
  bool dead = false;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full_bar[s], 2); mbar_init(&empty_bar[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], 256); }
    for (int j = 0; j < TQ; ++j) { mbar_init(&tq_full[j], 1); mbar_init(&tq_empty[j], 260); }
    fence_barrier_init();
    tma_prefetch_desc(&mapA); tma_prefetch_desc(&mapB);
  }
  if (warp == 1) { tmem_alloc_pair(tmem_slot, 512); tmem_relinquish_pair(); }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  pdl_trigger();
  if (threadIdx.x == 0) sh_stamp_resident(d.stamps, g.stamp_id);
  if (MODE == 1) pdl_wait();                             // its A operand is the attention kernel's result
  if (threadIdx.x == 0) sh_stamp_start(d.stamps, g.stamp_id);
  // the qi-th tile of this pair, for every role but the claimer, or -1 when there is none
  auto next_tile = [&](int qi) -> int {
    const int j = qi & (TQ - 1);
    if (!mbar_wait_cluster(&tq_full[j], (qi / TQ) & 1, g.status, dead)) return -1;
    const int t = tq_tile[j];
    mbar_arrive_leader(&tq_empty[j]);
    return t;
  };

  if (warp == 0 || warp == 6) {
    if (lane == 0) {
      const bool do_b = warp == 0, do_a = warp == 6;
      int s = 0;
      uint32_t par = 1;
      for (int qi = 0; !dead; ++qi) {
        int t;
        if (do_b && rank == 0) {
          // claim the next tile only now, when the loads of the previous one are all issued
          const int j = qi & (TQ - 1);
          if (!mbar_wait(&tq_empty[j], ((qi / TQ) & 1) ^ 1, g.status, dead)) break;
          t = atomicAdd(g.sched, 1);
          if (t >= ntiles) t = -1;
          tq_tile[j] = t;
          st_cluster_u32(cluster_map(&tq_tile[j], 1), (uint32_t)t);
          mbar_arrive(&tq_full[j]);
          mbar_arrive_cluster_release(cluster_map(&tq_full[j], 1));
          if (t < 0) {
            // the pair whose final claim comes last puts both counters back for the next launch
            if (atomicAdd(g.sched + 1, 1) == (g.claimers ? g.claimers : (int)(gridDim.x >> 1)) - 1) { g.sched[0] = 0; g.sched[1] = 0; }
          }
        } else {
          t = next_tile(qi);
        }
        if (t < 0) break;
        const int row0 = (t / ncol) * 256 + (int)rank * 128;
        const int brow = g.b_row0 + (t % ncol) * BN + (int)rank * 128;
        for (int kb = 0; kb < KB; ++kb) {
          if (!mbar_wait(&empty_bar[s], par, g.status, dead)) break;
          const uint32_t sa = sbase + s * SM::STAGE_BYTES, sb = sa + SM::A_BYTES;
          if (do_a) {
            if (rank == 0) mbar_expect_tx(&full_bar[s], 2 * SM::A_BYTES);
            tma_load_2d_pair(sa, &mapA, &full_bar[s], kb * 64, row0);
          } else {
            if (rank == 0) mbar_expect_tx(&full_bar[s], 2 * SM::B_BYTES);
            tma_load_2d_pair(sb, &mapB, &full_bar[s], kb * 64, brow);
          }
          if (++s == STAGES) { s = 0; par ^= 1; }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = MODE == 0 ? make_idesc_f16(256, BN, 1, 1, 0) : make_idesc_f16(256, BN, 0, 0, 0);
      const uint32_t a_lo0 = desc_lo_k(sbase), b_lo0 = desc_lo_k(sbase + SM::A_BYTES);
      int s = 0, it = 0;
      uint32_t par = 0;
      for (; !dead; ++it) {
        if (next_tile(it) < 0) break;
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
  } else if (warp < 6) {
    // ---- epilogue: thread = accumulator row = TMEM lane ----------------------------------------
    const int q = warp & 3;
    const uint32_t lane_off = (uint32_t)(q * 32) << 16;
    const int HD = d.H * d.D;
    for (int it = 0;; ++it) {
      const int t = next_tile(it);
      if (t < 0) break;
      const int b = it & 1;
      const int row0 = (t / ncol) * 256 + (int)rank * 128, col0 = (t % ncol) * BN;
      const int r = q * 32 + lane;
      const bool live = row0 + r < g.nrows;
      const int tokn = row0 + r;
      const int bb = live ? tokn / d.T : 0, tt = live ? tokn % d.T : 0;
      if (!mbar_wait(&acc_full[b], (it >> 1) & 1, g.status, dead)) break;
      tc_fence_after();
      const uint32_t trow = tmem + lane_off + b * 256;
#pragma unroll 1
      for (int c00 = 0; c00 < BN; c00 += 64) {
        uint32_t vv[64];
        tmem_ld32(trow + c00, *reinterpret_cast<uint32_t(*)[32]>(&vv[0]));
        tmem_ld32(trow + c00 + 32, *reinterpret_cast<uint32_t(*)[32]>(&vv[32]));
        tmem_ld_wait();
        if (c00 + 64 >= BN) {                              // the accumulator is in registers: hand the buffer back
          tc_fence_before();
          mbar_arrive_leader(&acc_empty[b]);
        }
#pragma unroll
        for (int hh2 = 0; hh2 < 2; ++hh2) {
          const int c0 = c00 + hh2 * 32;
          uint32_t* v = &vv[hh2 * 32];
          const int n0 = col0 + c0;
          if (!live || n0 >= g.ncols) continue;
          if (MODE == 1) {
            float* dstf = (float*)g.out0 + (size_t)tokn * g.ncols + n0;
#pragma unroll
            for (int i = 0; i < 8; ++i)
              *reinterpret_cast<uint4*>(dstf + 4 * i) = make_uint4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
            continue;
          }
          const int which = n0 / HD, hd = (n0 % HD) / d.D, dd = n0 % d.D;
          __half* dst = (__half*)(which == 0 ? g.out0 : which == 1 ? g.out1 : g.out2) +
                        (((size_t)bb * d.H + hd) * d.T + tt) * d.D + dd;
          const float sc = which == 0 ? g.qscale : 1.f;
          if (g.rope && which < 2) rope_pairs16(v, g.rope + tt, dd >> 1, d.T);
          uint32_t p[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            __half2 hv = __floats2half2_rn(__uint_as_float(v[2 * i]) * sc, __uint_as_float(v[2 * i + 1]) * sc);
            p[i] = *reinterpret_cast<uint32_t*>(&hv);
          }
#pragma unroll
          for (int i = 0; i < 4; ++i)
            *reinterpret_cast<uint4*>(dst + 8 * i) = make_uint4(p[4 * i], p[4 * i + 1], p[4 * i + 2], p[4 * i + 3]);
        }
      }
    }
  }
  pdl_wait();
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (threadIdx.x == 0) sh_stamp_end(d.stamps, g.stamp_id);
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem, 512);
  }
}

}  // namespace shtc
