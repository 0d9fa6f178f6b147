// Fused gate kernel of the bf16 configuration (Sec. 2.2: s = sigmoid(x W), arg top-k):
// the logits tile z[128 tokens, G] = x W_gate^T runs on the tensor pipe (TMA-fed, fp32 in
// TMEM), then each thread owns one token: adds the bias, picks the k largest logits of every
// (side, head) group (strictly-greater scan, so the lower index wins ties), applies the
// sigmoid, writes idx / gate and adds to the CTA's selection histogram.  While the main loop
// runs, the otherwise idle epilogue warps clear the V and out rows of the CTA's tokens (both
// are accumulated into later).
//
// Fused sort (g.fused, cooperative launch): when the whole grid is resident at once, the CTAs meet
// at a grid-wide barrier (a counter in global memory, bounded wait) once their histograms are
// published, and each then places its own tokens in the sorted lists (sh_sort_block, the body of the
// stand-alone sort kernel, run by the 512 selection threads on the selections still in shared
// memory): no second kernel, no second trip of the selections through L2.
//
// Warp roles (608 threads): warps 0 and 6 = TMA producers (x boxes / gate-weight boxes), warp 1 = TMEM owner + UMMA issuer, warps 2..5 and
// 7..18 = zero-fill, then selection: warps 2..5 (one per TMEM lane quarter) move the logits to
// shared memory, then four threads share a token's (side, head) groups - the selection is a
// chain of dependent compares, exp and stores per group (~600 cycles), and with one thread per
// token it alone took 5.6 us of the kernel's 14.
#pragma once
#include "sh_tc_prims.cuh"
#include "sh_simt.cuh"

namespace shtc {

struct TcGateArgs {
  ShDims d;
  int Gp;                    // G rounded up to a multiple of 16 (UMMA N)
  const float* gbias;        // [G]
  int* idx; float* gate;     // [2, N, H, k]
  int* blockcnt;             // [nblk, G] per-CTA selection histogram
  void* zero_v;              // [B, H, T, D] fp16, or nullptr
  float* zero_out;           // [N, M] or nullptr
  int* status;
  // fused sort (cooperative launch only)
  int fused;                 // 1: place the tokens in the sorted lists at the end of this kernel
  int sort_sides;            // sides the sort covers (1: source side only)
  int tile_rows_src;         // rows per tile of the source-side tile table
  int max_tiles;
  int* offsets; int* lists; float* lgate; ShTile* tiles; int* ntiles;
  int* gridbar;              // {arrived, departed}, both 0 between launches
  // value projection tiled by expert PAIRS (k = 2, forward pass only): the source side is bucketed by
  // (head, pair number) - histogram, sort and tile table run over H * NP buckets with one entry per
  // (token, head) - and the destination side is not bucketed at all
  int vpairs;                // 0, or the number of sides bucketed by pair: 1 = the source side, 2 = both (query experts)
  int NP;                    // pairs per head: E (E - 1) / 2
  int GH;                    // histogram width: vpairs ? vpairs * H * NP : G
  int* gid;                  // [vpairs, N, H] pair number of every (token, head)
};

constexpr int GATE_THREADS = 608;

template <int STAGES>
__global__ void __launch_bounds__(GATE_THREADS)
sh_tc_gate_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapW, TcGateArgs g) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* sgen = smem_raw + (sbase - smem_u32(smem_raw));
  const ShDims& d = g.d;
  const int Gp = g.Gp;
  const int a_bytes = 128 * 64 * 2, b_bytes = Gp * 128, stage_bytes = a_bytes + ((b_bytes + 1023) & ~1023);
  const int pipe_bytes = STAGES * stage_bytes;
  const int stag_bytes = 128 * (Gp + 1) * 4;
  const int bar_off = ((pipe_bytes > stag_bytes ? pipe_bytes : stag_bytes) + 1023) & ~1023;
  uint64_t* full_bar = (uint64_t*)(sgen + bar_off);
  uint64_t* empty_bar = full_bar + STAGES;
  uint64_t* tmem_full = empty_bar + STAGES;
  uint64_t* logits_ready = tmem_full + 1;               // the logits tile is in shared memory (4 warp arrivals)
  uint32_t* tmem_slot = (uint32_t*)(logits_ready + 1);
  int* s_hist = (int*)(sgen + bar_off + 256);           // [G]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row0 = blockIdx.x * 128;
  const int nrows = min(128, d.N - row0);
  const int KB = d.M / 64;
  bool dead = false;
  uint32_t tmem_cols = 32;
  while ((int)tmem_cols < Gp) tmem_cols <<= 1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full_bar[s], 2); mbar_init(&empty_bar[s], 1); }
    mbar_init(tmem_full, 1);
    mbar_init(logits_ready, 4);
    fence_barrier_init();
    tma_prefetch_desc(&mapX); tma_prefetch_desc(&mapW);
  }
  for (int i = threadIdx.x; i < g.GH; i += blockDim.x) s_hist[i] = 0;
  if (warp == 1) { tmem_alloc(tmem_slot, tmem_cols); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_d = *tmem_slot;
  pdl_trigger();                                        // the sort kernel may become resident (it waits for this grid)
  if (threadIdx.x == 0) { sh_stamp_resident(d.stamps, SH_K_GATE); sh_stamp_start(d.stamps, SH_K_GATE); }

  if (warp == 0 || warp == 6) {
    // (the boxes of consecutive stages arrive ~290 ns apart however many lanes issue them: with x
    //  coming from HBM, 8 stages x 20 KB in flight over a ~2 us round trip is ~70 GB/s per SM)
    if (lane == 0) {
      for (int kb = 0; kb < KB; ++kb) {
        const int s = kb % STAGES;
        if (!mbar_wait(&empty_bar[s], ((kb / STAGES) & 1) ^ 1, g.status, dead)) break;
        const uint32_t sa = sbase + s * stage_bytes, sb = sa + a_bytes;
        if (warp == 0) {
          mbar_expect_tx(&full_bar[s], a_bytes);
          tma_load_2d(sa, &mapX, &full_bar[s], kb * 64, row0);
        } else {
          mbar_expect_tx(&full_bar[s], b_bytes);
          tma_load_2d(sb, &mapW, &full_bar[s], kb * 64, 0);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = make_idesc_f16(128, Gp, 1, 1, 0);
      for (int kb = 0; kb < KB; ++kb) {
        const int s = kb % STAGES;
        if (!mbar_wait(&full_bar[s], (kb / STAGES) & 1, g.status, dead)) break;
        tc_fence_after();
        const uint32_t sa = sbase + s * stage_bytes, sb = sa + a_bytes;
        const uint64_t adesc = make_desc_k_sw128(sa), bdesc = make_desc_k_sw128(sb);
#pragma unroll
        for (int k = 0; k < 4; ++k) umma_f16(tmem_d, adesc + 2 * k, bdesc + 2 * k, idesc, (kb | k) != 0);
        umma_commit(&empty_bar[s]);
      }
      umma_commit(tmem_full);
    }
  } else {
    // selection threads: 0..127 = warps 2..5, 128..511 = warps 7..18
    const int et = warp < 6 ? threadIdx.x - 64 : threadIdx.x - 96;
    constexpr int NSEL = GATE_THREADS - 96;             // 512
    // ---- clear the rows this CTA's tokens own in V and out (accumulated into later) -----------
    if (g.zero_out) {
      const int n4 = d.M / 4;                           // float4 per row
      float4* base = reinterpret_cast<float4*>(g.zero_out + (size_t)row0 * d.M);
      const long total = (long)nrows * n4;
      for (long i = et; i < total; i += NSEL) base[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    if (g.zero_v) {
      const int row_bytes = d.D * 2;                       // one (token, head) row
      const int cpr = row_bytes / 16;                      // 16-byte chunks per row (a power of two: 8..32)
      const int ch = et & (cpr - 1);
      for (int tl = et / cpr; tl < nrows; tl += NSEL / cpr) {
        const int tok = row0 + tl;
        const int bb = tok / d.T, tt = tok % d.T;
        char* p = (char*)g.zero_v + ((size_t)bb * d.H * d.T + tt) * row_bytes + ch * 16;
        for (int hh = 0; hh < d.H; ++hh)
          *reinterpret_cast<uint4*>(p + (size_t)hh * d.T * row_bytes) = make_uint4(0, 0, 0, 0);
      }
    }
    // ---- logits tile -> shared memory: warps 2..5, thread = token = TMEM lane -----------------
    if (warp < 6) {
      const int q = warp & 3;
      const int r = q * 32 + lane;
      float* srow = reinterpret_cast<float*>(sgen) + (size_t)r * (Gp + 1);
      if (mbar_wait(tmem_full, 0, g.status, dead)) {
        tc_fence_after();
        const uint32_t trow = tmem_d + ((uint32_t)(q * 32) << 16);
        // (the pipeline buffers are idle now); up to four TMEM loads are issued per wait because
        // the load latency, not its bandwidth, bounds this loop
        for (int c0 = 0; c0 < Gp; c0 += 64) {
          uint32_t v[64];
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            if (c0 + 16 * u < Gp) {
              uint32_t* w = &v[16 * u];
              asm volatile(
                  "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
                  : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]), "=r"(w[4]), "=r"(w[5]), "=r"(w[6]), "=r"(w[7]),
                    "=r"(w[8]), "=r"(w[9]), "=r"(w[10]), "=r"(w[11]), "=r"(w[12]), "=r"(w[13]), "=r"(w[14]), "=r"(w[15])
                  : "r"(trow + c0 + 16 * u)
                  : "memory");
            }
          }
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 64; ++i)
            if (c0 + i < d.G) srow[c0 + i] = __uint_as_float(v[i]) + g.gbias[c0 + i];
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(logits_ready);
      }
    }
    // ---- selection: thread = (token r, group slice sub): groups sub, sub + 4, ... ----------------
    // fused sort: its scratch sits behind the logits rows; the selections go there as well
    int* s_sort = reinterpret_cast<int*>(sgen + ((stag_bytes + 15) & ~15));
    const int per_tok = d.H * d.k;
    int* s_idx = s_sort + 8 * g.GH;                       // [2][128 * per_tok], as sh_sort_block lays it out
    float* s_gt = reinterpret_cast<float*>(s_idx + 2 * 128 * per_tok);     // (pair mode: [128 * H] pair numbers; gates unused)
    const bool sel_ok = mbar_wait(logits_ready, 0, g.status, dead);
    if (sel_ok) {
      const int r = et & 127, sub = et >> 7;
      const float* srow = reinterpret_cast<const float*>(sgen) + (size_t)r * (Gp + 1);
      const int t = row0 + r;
      if (r < nrows) {
        for (int grp = sub; grp < d.sides * d.H; grp += NSEL / 128) {
          const float* z = srow + grp * d.E;
          const int side = grp / d.H, h = grp % d.H;
          const size_t o = (((size_t)side * d.N + t) * d.H + h) * d.k;
          unsigned taken = 0;
          int first = 0;
          for (int j = 0; j < d.k; ++j) {
            int best = -1;
            float bz = 0.f;
            for (int e = 0; e < d.E; ++e) {
              if ((taken >> e) & 1u) continue;
              const float ze = z[e];
              if (best < 0 || ze > bz) { best = e; bz = ze; }
            }
            taken |= 1u << best;
            const float gv = 1.f / (1.f + expf(-bz));
            g.idx[o + j] = best;
            g.gate[o + j] = gv;
            if (g.vpairs) {
              if (j == 0) first = best;
              else if (side < g.vpairs) {
                const int pid = sh_pair_id(min(first, best), max(first, best), d.E);
                g.gid[((size_t)side * d.N + t) * d.H + h] = pid;
                if (g.fused) s_idx[side * 128 * d.H + r * d.H + h] = pid;
                atomicAdd(&s_hist[(side * d.H + h) * g.NP + pid], 1);
              }
              continue;
            }
            if (g.fused) {
              s_idx[side * 128 * per_tok + (r * d.H + h) * d.k + j] = best;
              s_gt[side * 128 * per_tok + (r * d.H + h) * d.k + j] = gv;
            }
            atomicAdd(&s_hist[grp * d.E + best], 1);
          }
        }
      }
    }
    if (g.fused) {
      // ---- publish the histogram, meet the other CTAs, place this CTA's tokens ----------------------
      auto sel_sync = [] { asm volatile("bar.sync 1, 512;" ::: "memory"); };
      sel_sync();                                           // s_hist, s_idx, s_gt complete
      for (int i = et; i < g.GH; i += NSEL) g.blockcnt[(size_t)blockIdx.x * g.GH + i] = s_hist[i];
      __threadfence();
      sel_sync();
      int* s_flag = s_hist + g.GH;                          // (the histogram area is 3 GH words)
      if (et == 0) {
        bool ok = sel_ok;
        atomicAdd(g.gridbar, 1);
        const uint64_t t0 = global_timer_ns();
        while (ok && *(volatile int*)g.gridbar < (int)gridDim.x) {
          if (global_timer_ns() - t0 > SH_WAIT_LIMIT_NS || *(volatile int*)g.status != 0) {
            atomicCAS(g.status, 0, SH_ERR_TIMEOUT);
            ok = false;
          }
        }
        __threadfence();
        // the CTA that leaves last puts the counters back for the next launch
        if (atomicAdd(g.gridbar + 1, 1) == (int)gridDim.x - 1) { g.gridbar[0] = 0; g.gridbar[1] = 0; }
        *s_flag = ok ? 1 : 0;
      }
      sel_sync();
      if (*(volatile int*)s_flag) {
        ShDims ds = d;
        ds.sides = g.sort_sides;
        if (g.vpairs) { ds.sides = g.vpairs; ds.E = g.NP; ds.k = 1; ds.G = g.GH; }   // buckets (side, head, pair), one entry per (token, head)
        sh_sort_block(g.idx, g.gate, g.blockcnt, g.offsets, g.lists, g.lgate, g.tiles, g.ntiles, ds, s_sort, et, NSEL, (int)blockIdx.x, true, sel_sync);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_d, tmem_cols);
  }
  // ---- publish this CTA's selection histogram (the sort kernel scans them) ------------------
  if (!g.fused)
    for (int i = threadIdx.x; i < g.GH; i += blockDim.x) g.blockcnt[(size_t)blockIdx.x * g.GH + i] = s_hist[i];
  if (threadIdx.x == 0) sh_stamp_end(d.stamps, SH_K_GATE);
}

}  // namespace shtc
