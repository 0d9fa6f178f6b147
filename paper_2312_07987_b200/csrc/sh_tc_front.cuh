// The front of a forward pass as ONE persistent grid of CTA pairs that owns every SM from the first
// cycle: gate logits, top-k selection, bucket sort and tile table (Sec. 2.2: s = sigmoid(x W_S),
// arg top-k) together with the dense query / key projections (Sec. 2.2: Q^h = x W_Q^h, K^h = x W_K^h).
//
// As separate kernels the gate kernel holds its SMs for ~25 us of mostly latency (x cold from HBM for
// 32 columns of product, then selection, a grid-wide barrier and the placement), the projection runs
// beside it on what is left, and the attention kernel is launched behind an event join of two streams.
// Here the gate logits are the FIRST TILE of the projection's own pipeline - the same operand ring,
// the same issuing thread, an accumulator of G columns - and the selection and the sort run on warps of
// their own in the shadow of the projection tiles that follow:
//
//   * gate tile: a pair takes one 128-token block, 64 tokens per CTA (R = 64: up to 74 blocks; every
//     SM pulls x from HBM), or two blocks, one per CTA (R = 128: up to 148 blocks).  cta_group::2 UMMA
//     with M = 256, N = Gp: each CTA loads its rows of x and half of the gate weights.  With R = 64 the
//     upper half of a CTA's operand tile is whatever the ring held: those accumulator rows are never read.
//   * the projection's epilogue warps move the logits, column by column, into the shared memory of the
//     CTA that selects (R = 64: the leader, for the other CTA's rows across the cluster) and hand the
//     accumulator back; the selection threads add the bias, which they staged while they waited;
//   * 512 selection threads of that CTA pick the top k per (token, side, head), publish the block's
//     histogram, meet the other selecting CTAs at a grid-wide barrier (a counter in global memory,
//     bounded wait; the launch is cooperative, so all CTAs are resident) and place the block's tokens
//     (sh_sort_block); block 0 also writes offsets and the tile table;
//   * meanwhile producers, issuer and epilogue go on with 256 x 256 projection tiles claimed from a
//     global counter, as in sh_tc_qk_pair_kernel - on a ring of five stages (six measure the same; the
//     sixth's shared memory holds the selection's scratch), and with an epilogue that stores through
//     2 KB shared-memory tiles and TMA: row-by-row 16-byte stores kept the load / store unit busy a third
//     of the time, and the selection warps beside them ran microseconds longer.
//
// Warp roles (736 threads): warp 0 lane 0 = weight producer (leader: also tile claimer), warp 6 lane 0
// = x producer, warp 1 = TMEM allocation and (leader) UMMA issuer, warps 2..5 = epilogue, warps 7..22 =
// selection and sort.
#pragma once
#include "sh_tc_gate.cuh"
#include "sh_tc_qkpair.cuh"

namespace shtc {

constexpr int FRONT_NSEL = 512;
constexpr int FRONT_THREADS = 224 + FRONT_NSEL;

struct TcFrontArgs {
  TcGemmArgs q;              // the projection (as for sh_tc_qk_pair_kernel)
  TcGateArgs g;              // gate, selection and sort (as for sh_tc_gate_kernel with the fused sort)
  int R;                     // rows of x per CTA in the gate tile: 64 or 128
  int gate_pairs;            // pairs that have a gate tile: nblk (R = 64) or ceil(nblk / 2) (R = 128)
  int sort_bytes;            // shared memory of sh_sort_block behind the logits rows
  int tma_epi;               // 1: the projection's epilogue stores through shared memory and TMA (T a multiple of 32)
};

template <int STAGES>
struct FrontSmem {
  static constexpr int BAR_OFF = QkPairSmem<STAGES>::BAR_OFF;
  static constexpr int STG_OFF = BAR_OFF;                  // epilogue staging: 2 KB per epilogue warp, two buffers each
  static constexpr int STG_BYTES = 4 * 2 * 2048;
  static constexpr int BARS = STG_OFF + STG_BYTES;         // 512 bytes of projection barriers, then logits_ready
  static constexpr int GATE_OFF = BARS + 640;
  // logits rows, the sort's scratch, the histogram (3 GH words and the barrier flag), alignment slack
  static int total(int Gp, int GH, int sort_bytes) {
    return GATE_OFF + 128 * Gp * 4 + ((sort_bytes + 15) & ~15) + (3 * GH + 8) * 4 + ((Gp + 3) & ~3) * 4 + 1024;
  }
};

__device__ __forceinline__ void st_cluster_f32(uint32_t cluster_addr, float v) {
  asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(cluster_addr), "f"(v) : "memory");
}

template <int STAGES>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(FRONT_THREADS, 1)
sh_tc_front_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapAg,
                   const __grid_constant__ CUtensorMap mapB, const __grid_constant__ CUtensorMap mapWg,
                   const __grid_constant__ CUtensorMap mapQo, const __grid_constant__ CUtensorMap mapKo, TcFrontArgs fa) {
  using SM = QkPairSmem<STAGES>;
  using FS = FrontSmem<STAGES>;
  constexpr int BN = 256, TQ = 4;
  constexpr int NSEL = FRONT_NSEL;
  extern __shared__ unsigned char smem_raw[];
  const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* sgen = smem_raw + (sbase - smem_u32(smem_raw));
  uint64_t* full_bar = (uint64_t*)(sgen + FS::BARS);       // [STAGES] leader's
  uint64_t* empty_bar = full_bar + STAGES;                 // [STAGES] both CTAs
  uint64_t* acc_full = empty_bar + STAGES;                 // [2] both CTAs
  uint64_t* acc_empty = acc_full + 2;                      // [2] leader's: 256 arrivals
  uint64_t* tq_full = acc_empty + 2;                       // [TQ] both CTAs
  uint64_t* tq_empty = tq_full + TQ;                       // [TQ] leader's: 260 arrivals
  int* tq_tile = (int*)(tq_empty + TQ);                    // [TQ] both CTAs
  uint32_t* tmem_slot = (uint32_t*)(tq_tile + TQ);
  static_assert((2 * STAGES + 4 + 2 * TQ) * 8 + TQ * 4 + 4 <= 512, "barrier area");
  uint64_t* logits_ready = (uint64_t*)(sgen + FS::BARS + 512);   // in the selecting CTA: one arrival per epilogue warp that feeds it

  const TcGemmArgs& g = fa.q;
  const TcGateArgs& gg = fa.g;
  const ShDims& d = g.d;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int pair = (int)(blockIdx.x >> 1);
  const int KB = g.K / 64;
  const int ncol = (g.ncols + BN - 1) / BN;
  const int ntiles = ((g.nrows + 255) / 256) * ncol;
  const int R = fa.R, Gp = gg.Gp;
  const bool has_gate = pair < fa.gate_pairs;
  const int blk = R == 64 ? pair : 2 * pair + (int)rank;  // the 128-token block this CTA selects for
  const bool selects = has_gate && (R == 64 ? rank == 0 : blk < d.nblk);
  const uint32_t sel_rank = R == 64 ? 0u : rank;          // the CTA of the pair that gets this CTA's logits
  const int stag_bytes = 128 * Gp * 4;                   // logits, column by column: [Gp][128 tokens]
  float* s_logits = reinterpret_cast<float*>(sgen + FS::GATE_OFF);
  int* s_sort = reinterpret_cast<int*>(sgen + FS::GATE_OFF + stag_bytes);
  int* s_hist = reinterpret_cast<int*>(sgen + FS::GATE_OFF + stag_bytes + ((fa.sort_bytes + 15) & ~15));   // [3 GH + 8]
  float* s_bias = reinterpret_cast<float*>(s_hist + 3 * gg.GH + 8);   // [G] gate bias, staged by the selection threads while they wait
  bool dead = false;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full_bar[s], 2); mbar_init(&empty_bar[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], 256); }
    for (int j = 0; j < TQ; ++j) { mbar_init(&tq_full[j], 1); mbar_init(&tq_empty[j], 260); }
    mbar_init(logits_ready, R == 64 ? 8 : 4);
    fence_barrier_init();
    tma_prefetch_desc(&mapA); tma_prefetch_desc(&mapB); tma_prefetch_desc(&mapAg); tma_prefetch_desc(&mapWg);
    tma_prefetch_desc(&mapQo); tma_prefetch_desc(&mapKo);
  }
  for (int i = threadIdx.x; i < gg.GH; i += blockDim.x) s_hist[i] = 0;
  if (blockIdx.x == 0 && threadIdx.x == 0) {              // (no block counts itself in before the grid barrier, which this CTA joins later)
    g.status[SH_ST_SORTED] = 0;
    __threadfence();
  }
  if (warp == 1) { tmem_alloc_pair(tmem_slot, 512); tmem_relinquish_pair(); }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  pdl_trigger();
  if (threadIdx.x == 0) {
    sh_stamp_resident(d.stamps, SH_K_QK_A); sh_stamp_start(d.stamps, SH_K_QK_A);
    if (has_gate) { sh_stamp_resident(d.stamps, SH_K_GATE); sh_stamp_start(d.stamps, SH_K_GATE); }
  }
  // the qi-th claimed tile of this pair, for every role but the claimer, or -1 when there is none
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
      if (has_gate) {
        // ---- gate tile: R rows of x per CTA, Gp / 2 rows of the gate weights per CTA --------------
        const int grow0 = R == 64 ? pair * 128 + (int)rank * 64 : blk * 128;
        for (int kb = 0; kb < KB; ++kb) {
          if (!mbar_wait(&empty_bar[s], par, g.status, dead)) break;
          const uint32_t sa = sbase + s * SM::STAGE_BYTES, sb = sa + SM::A_BYTES;
          if (do_a) {
            if (rank == 0) mbar_expect_tx(&full_bar[s], 2 * R * 128);
            tma_load_2d_pair(sa, &mapAg, &full_bar[s], kb * 64, grow0);
          } else {
            if (rank == 0) mbar_expect_tx(&full_bar[s], Gp * 128);
            tma_load_2d_pair(sb, &mapWg, &full_bar[s], kb * 64, (int)rank * (Gp / 2));
          }
          if (++s == STAGES) { s = 0; par ^= 1; }
        }
      }
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
            if (atomicAdd(g.sched + 1, 1) == (int)(gridDim.x >> 1) - 1) { g.sched[0] = 0; g.sched[1] = 0; }
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
      constexpr uint32_t idesc = make_idesc_f16(256, BN, 1, 1, 0);
      const uint32_t a_lo0 = desc_lo_k(sbase), b_lo0 = desc_lo_k(sbase + SM::A_BYTES);
      int s = 0, ai = 0;                                   // ai: accumulator uses so far (the gate tile is the first)
      uint32_t par = 0;
      if (has_gate) {
        const uint32_t idesc_g = make_idesc_f16(256, Gp, 1, 1, 0);
        for (int kb = 0; kb < KB; ++kb) {
          if (!mbar_wait(&full_bar[s], par, g.status, dead)) break;
          tc_fence_after();
          const uint32_t a_lo = a_lo0 + s * (SM::STAGE_BYTES >> 4), b_lo = b_lo0 + s * (SM::STAGE_BYTES >> 4);
#pragma unroll
          for (int k = 0; k < 4; ++k)
            umma_f16_pair(tmem, desc_pack(a_lo + 2 * k), desc_pack(b_lo + 2 * k), idesc_g, (kb | k) != 0);
          umma_commit_pair(&empty_bar[s], 3);
          if (++s == STAGES) { s = 0; par ^= 1; }
        }
        if (!dead) umma_commit_pair(&acc_full[0], 3);
        ai = 1;
      }
      for (int it = 0; !dead; ++it, ++ai) {
        if (next_tile(it) < 0) break;
        const int b = ai & 1;
        if (!mbar_wait(&acc_empty[b], ((ai >> 1) & 1) ^ 1, g.status, dead)) break;
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
    int ai = 0, nst = 0;                                   // nst: TMA stores issued by this warp
    if (has_gate) {
      // ---- gate tile: logits (+ bias) to the selecting CTA's shared memory ----------------------
      if (mbar_wait(&acc_full[0], 0, g.status, dead)) {
        tc_fence_after();
        const int r = q * 32 + lane;
        if (R == 128 || q < 2) {
          const int srow = R == 64 ? (int)rank * 64 + r : r;
          // (a warp's 32 rows of one column are 128 contiguous bytes: one packet across the cluster; the
          //  selecting CTA's own warps use plain shared-memory stores - the cluster path costs microseconds)
          const bool remote = sel_rank != rank;
          float* dst_l = s_logits + srow;
          const uint32_t dst = cluster_map(dst_l, sel_rank);
          const uint32_t trow = tmem + lane_off;
          // (16 columns per trip of a rolled loop, all Gp columns without a test: this code runs once per
          //  CTA, and under the projection's operand traffic every instruction line it needs costs a
          //  slow fetch - unrolled over the columns it took 3.8 us)
#pragma unroll 1
          for (int c0 = 0; c0 < Gp; c0 += 16) {
            uint32_t w[16];
            asm volatile(
                "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
                : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]), "=r"(w[4]), "=r"(w[5]), "=r"(w[6]), "=r"(w[7]),
                  "=r"(w[8]), "=r"(w[9]), "=r"(w[10]), "=r"(w[11]), "=r"(w[12]), "=r"(w[13]), "=r"(w[14]), "=r"(w[15])
                : "r"(trow + c0)
                : "memory");
            tmem_ld_wait();
            if (remote) {
#pragma unroll
              for (int i = 0; i < 16; ++i) st_cluster_f32(dst + 512 * (c0 + i), __uint_as_float(w[i]));
            } else {
#pragma unroll
              for (int i = 0; i < 16; ++i) dst_l[128 * (c0 + i)] = __uint_as_float(w[i]);
            }
          }
        }
        tc_fence_before();
        mbar_arrive_leader(&acc_empty[0]);
        __syncwarp();                                      // (orders the lanes' stores before lane 0's releasing arrival)
        if (lane == 0) {
          if (sel_rank != rank) mbar_arrive_cluster_release(cluster_map(logits_ready, sel_rank));
          else mbar_arrive(logits_ready);
        }
      }
      ai = 1;
    }
    for (int it = 0;; ++it, ++ai) {
      const int t = next_tile(it);
      if (t < 0) break;
      const int b = ai & 1;
      const int row0 = (t / ncol) * 256 + (int)rank * 128, col0 = (t % ncol) * BN;
      const int r = q * 32 + lane;
      const bool live = row0 + r < g.nrows;
      const int tokn = row0 + r;
      const int bb = live ? tokn / d.T : 0, tt = live ? tokn % d.T : 0;
      if (!mbar_wait(&acc_full[b], (ai >> 1) & 1, g.status, dead)) break;
      tc_fence_after();
      const uint32_t trow = tmem + lane_off + b * 256;
#pragma unroll 1
      for (int c0 = 0; c0 < BN; c0 += 32) {             // (32 columns at a time: 736 threads leave 88 registers each)
        uint32_t v[32];
        tmem_ld32(trow + c0, v);
        tmem_ld_wait();
        if (c0 + 32 >= BN) {                               // the accumulator is in registers: hand the buffer back
          tc_fence_before();
          mbar_arrive_leader(&acc_empty[b]);
        }
        {
          const int n0 = col0 + c0;
          if (n0 >= g.ncols || row0 + q * 32 >= g.nrows) continue;     // (warp-uniform)
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
          if (fa.tma_epi) {
            // The warp's 32 rows x 32 columns go through a 2 KB tile of shared memory (64-byte swizzle: the
            // lanes' 16-byte pieces of one instruction fall on distinct banks) and one TMA store.  Stored
            // row by row - 16 bytes per lane, a cache line per lane and instruction - the epilogue kept the
            // SM's load / store unit busy a third of the time, and the selection and sort warps beside it
            // ran 5-9 us longer.
            unsigned char* stg = sgen + FS::STG_OFF + (q * 2 + (nst & 1)) * 2048;
            if (nst >= 2) {                                // the store before last out of this buffer has read it
              if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
              __syncwarp();
            }
            ++nst;
#pragma unroll
            for (int i = 0; i < 4; ++i)
              *reinterpret_cast<uint4*>(stg + lane * 64 + ((i ^ ((lane >> 1) & 3)) << 4)) = make_uint4(p[4 * i], p[4 * i + 1], p[4 * i + 2], p[4 * i + 3]);
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) {
              const int tok0 = row0 + q * 32;
              tma_store_3d(which == 0 ? &mapQo : &mapKo, smem_u32(stg), dd, tok0 % d.T, (tok0 / d.T) * d.H + hd);
              bulk_commit();
            }
          } else if (live) {
#pragma unroll
            for (int i = 0; i < 4; ++i)
              *reinterpret_cast<uint4*>(dst + 8 * i) = make_uint4(p[4 * i], p[4 * i + 1], p[4 * i + 2], p[4 * i + 3]);
          }
        }
      }
    }
    if (lane == 0) bulk_wait_all();                        // the staging tiles are read and the rows written
  } else if (warp >= 7 && selects) {
    // ---- selection and sort for block blk: 512 threads --------------------------------------------
    const int et = (int)threadIdx.x - 224;
    auto sel_sync = [] { asm volatile("bar.sync 1, 512;" ::: "memory"); };
    const int row0 = blk * 128;
    const int nrows = min(128, d.N - row0);
    if (gg.zero_v) {                                       // value rows that are accumulated into later
      const int row_bytes = d.D * 2;                       // one (token, head) row
      const int cpr = row_bytes / 16;                      // 16-byte chunks per row (a power of two: 8..32)
      const int ch = et & (cpr - 1);
      for (int tl = et / cpr; tl < nrows; tl += NSEL / cpr) {
        const int tok = row0 + tl;
        const int bb = tok / d.T, tt = tok % d.T;
        char* p = (char*)gg.zero_v + ((size_t)bb * d.H * d.T + tt) * row_bytes + ch * 16;
        for (int hh = 0; hh < d.H; ++hh)
          *reinterpret_cast<uint4*>(p + (size_t)hh * d.T * row_bytes) = make_uint4(0, 0, 0, 0);
      }
    }
    const int per_tok = d.H * d.k;
    int* s_idx = s_sort + 8 * gg.GH;                      // [2][128 * per_tok], as sh_sort_block lays it out
    float* s_gt = reinterpret_cast<float*>(s_idx + 2 * 128 * per_tok);     // (pair mode: [128 * H] pair numbers; gates unused)
    for (int i = et; i < d.G; i += NSEL) s_bias[i] = gg.gbias[i];
    sel_sync();
    // (one polling lane per warp: the acquire is the lane's, the warp barrier hands it on)
    bool sel_ok = true;
    if (lane == 0) sel_ok = mbar_wait_cluster(logits_ready, 0, g.status, dead);
    sel_ok = __shfl_sync(0xffffffffu, sel_ok, 0);
    if (sel_ok) {
      const int r = et & 127, sub = et >> 7;
      const float* srow = s_logits + r;
      const int t = row0 + r;
      if (r < nrows) {
        for (int grp = sub; grp < d.sides * d.H; grp += NSEL / 128) {
          const float* z = srow + grp * d.E * 128;
          const float* zb = s_bias + grp * d.E;
          const int side = grp / d.H, h = grp % d.H;
          const size_t o = (((size_t)side * d.N + t) * d.H + h) * d.k;
          unsigned taken = 0;
          int first = 0;
          for (int j = 0; j < d.k; ++j) {
            int best = -1;
            float bz = 0.f;
            for (int e = 0; e < d.E; ++e) {
              if ((taken >> e) & 1u) continue;
              const float ze = z[e * 128] + zb[e];
              if (best < 0 || ze > bz) { best = e; bz = ze; }
            }
            taken |= 1u << best;
            const float gv = 1.f / (1.f + expf(-bz));
            gg.idx[o + j] = best;
            gg.gate[o + j] = gv;
            if (gg.vpairs) {
              if (j == 0) first = best;
              else if (side < gg.vpairs) {
                const int pid = sh_pair_id(min(first, best), max(first, best), d.E);
                gg.gid[((size_t)side * d.N + t) * d.H + h] = pid;
                s_idx[side * 128 * d.H + r * d.H + h] = pid;
                atomicAdd(&s_hist[(side * d.H + h) * gg.NP + pid], 1);
              }
              continue;
            }
            s_idx[side * 128 * per_tok + (r * d.H + h) * d.k + j] = best;
            s_gt[side * 128 * per_tok + (r * d.H + h) * d.k + j] = gv;
            atomicAdd(&s_hist[grp * d.E + best], 1);
          }
        }
      }
    }
    // ---- publish the histogram, meet the other selecting CTAs, place this block's tokens ------------
    sel_sync();                                             // s_hist, s_idx, s_gt complete
    for (int i = et; i < gg.GH; i += NSEL) gg.blockcnt[(size_t)blk * gg.GH + i] = s_hist[i];
    __threadfence();
    sel_sync();
    int* s_flag = s_hist + gg.GH;
    if (et == 0) {
      bool ok = sel_ok;
      atomicAdd(gg.gridbar, 1);
      const uint64_t t0 = global_timer_ns();
      while (ok && *(volatile int*)gg.gridbar < d.nblk) {
        if (global_timer_ns() - t0 > SH_WAIT_LIMIT_NS || *(volatile int*)g.status != 0) {
          atomicCAS(g.status, 0, SH_ERR_TIMEOUT);
          ok = false;
        }
      }
      __threadfence();
      // the CTA that leaves last puts the counters back for the next launch
      if (atomicAdd(gg.gridbar + 1, 1) == d.nblk - 1) { gg.gridbar[0] = 0; gg.gridbar[1] = 0; }
      *s_flag = ok ? 1 : 0;
    }
    sel_sync();
    if (*(volatile int*)s_flag) {
      ShDims ds = d;
      ds.sides = gg.sort_sides;
      if (gg.vpairs) { ds.sides = gg.vpairs; ds.E = gg.NP; ds.k = 1; ds.G = gg.GH; }   // buckets (side, head, pair), one entry per (token, head)
      ds.tile_rows_src = gg.tile_rows_src;
      sh_sort_block(gg.idx, gg.gate, gg.blockcnt, gg.offsets, gg.lists, gg.lgate, gg.tiles, gg.ntiles, ds, s_sort, et, NSEL, blk, true, sel_sync);
    }
    // The value-expert kernel needs the selections, the lists and the tile table - not Q and K: it waits
    // for this count, not for the grid (its CTAs arrive on the SMs of pairs that are done, while other
    // pairs still run their last projection tiles).
    sel_sync();
    if (et == 0) {
      __threadfence();
      atomicAdd(g.status + SH_ST_SORTED, 1);
    }
    if (d.stamps) {
      sel_sync();
      if (et == 0) sh_stamp_end(d.stamps, SH_K_GATE);
    }
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (threadIdx.x == 0) sh_stamp_end(d.stamps, SH_K_QK_A);
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem, 512);
  }
}

}  // namespace shtc
