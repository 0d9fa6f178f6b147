// One-CTA-per-tile tcgen05 GEMM of the bf16 configuration, for the shapes the persistent kernels do
// not take: the dense Q/K projection when 2*H*D is not a multiple of 256, the grouped value-expert
// projection on small workloads (128-row tiles) or with d_head 64, and the dense comparator's
// projections.  One (MT*128) x BN output tile per CTA (MT = 1 or 2 row tiles that
// share the B operand, halving its L2 traffic), accumulators in TMEM, operands
// staged in 128-byte-swizzled shared memory: B always by TMA, A by TMA (dense rows) or by
// cp.async row gathers (rows addressed through a per-expert token list).
//
// Warp roles (192 threads): warp 0 = TMA producer, warp 1 = TMEM owner + UMMA issuer,
// warps 2..5 = A-row gatherers during the main loop (grouped modes) and the epilogue.
#pragma once
#include "sh_tc_prims.cuh"

namespace shtc {

enum { GEMM_QKV = 0, GEMM_V = 1, GEMM_PLAIN = 3 };

struct TcGemmArgs {
  ShDims d;
  int K;                 // reduction length (multiple of 64)
  int ncols;             // output columns (per group in grouped modes)
  int nrows;             // dense modes: rows of A
  // grouped modes
  const void* A;         // gathered operand base (bf16 x or fp16 Ahat)
  long lda;              // elements per A row
  const int* lists;      // [H, N*k] token ids of this side
  const float* lgate;    // gates aligned with lists
  const ShTile* tiles;
  const int* ntiles;
  int b_rows_per_group;  // rows of the B tensor map per (h*E + e)
  void* out0; void* out1; void* out2;
  float qscale;
  const float2* rope;    // dense Q/K mode: (cos, sin) table [D/2, T] of the rotary embedding, or nullptr
  int* status;
  int* sched;            // persistent dense mode: {next tile, CTAs that made their final claim}, both 0 between launches
  float* v_early;        // value experts: fp32 sums [B, H, SH_EARLY_ROWS, D] of the first rows of every sequence, or nullptr
  int* v_early_cnt;      // ... and their arrival counters [B, H, SH_EARLY_ROWS]
  int claimers;          // claiming CTAs (or CTA pairs) over all grids that share sched; 0: this grid's own
  int b_row0;            // CTA-pair dense projection: first weight row (a layer with query experts projects the keys alone: row H*D)
  int stamp_id;          // SH_K_* slot of this launch in the stamp block (sh_forward_stamped)
};

// Rotary embedding of the 16 adjacent feature pairs held in v[0..31] (fp32 bit patterns): pair i of
// the chunk is pair pair0 + i of its head; cs = the (cos, sin) table [D/2][T] at the token's position.
__device__ __forceinline__ void rope_pairs16(uint32_t* v, const float2* cs, int pair0, int T) {
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    const float2 c = cs[(size_t)(pair0 + i) * T];
    const float a0 = __uint_as_float(v[2 * i]), a1 = __uint_as_float(v[2 * i + 1]);
    v[2 * i] = __float_as_uint(a0 * c.x - a1 * c.y);
    v[2 * i + 1] = __float_as_uint(a0 * c.y + a1 * c.x);
  }
}

// Early-row value sums (see SH_EARLY_ROWS).  A thread that has added its gate-weighted contribution
// to the fp32 row `sum` (vector reductions) calls this: the arrival that completes the row's k
// contributions reads the sum back from L2, rounds it to fp16 once into the V row, and clears the
// sum and the counter for the next pass.  (Reductions, fence, counter: the pattern of a last-block
// reduction; the loads bypass L1.)
__device__ __noinline__ void v_early_finish(float* sum, int* cnt, __half* vrow, int D, int k) {
  __threadfence();
  if (atomicAdd(cnt, 1) != k - 1) return;
  __threadfence();
  for (int i0 = 0; i0 < D; i0 += 32) {                   // eight 16-byte loads in flight per trip to L2
    float4 v[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) v[j] = __ldcg(reinterpret_cast<const float4*>(sum + i0) + j);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const __half2 a = __floats2half2_rn(v[j].x, v[j].y), b = __floats2half2_rn(v[j].z, v[j].w);
      *reinterpret_cast<uint2*>(vrow + i0 + 4 * j) = make_uint2(*reinterpret_cast<const uint32_t*>(&a), *reinterpret_cast<const uint32_t*>(&b));
      __stcg(reinterpret_cast<float4*>(sum + i0) + j, make_float4(0.f, 0.f, 0.f, 0.f));
    }
  }
  *cnt = 0;
}

// A row tile of the table the sort wrote, as the grouped kernels use it.  The debug library checks
// its fields first (head, expert, rows inside the side's lists) and turns a bad entry into an empty tile.
__device__ __forceinline__ ShTile tile_checked(ShTile tl, const ShDims& d, int* status) {
#ifdef SH_DEBUG
  const bool ok = SH_INDEX_OK(tl.h, d.H, status, SH_SITE_V_TILE) && SH_INDEX_OK(tl.e, d.E, status, SH_SITE_V_TILE) &&
                  SH_INDEX_OK(tl.nrows, 257, status, SH_SITE_V_TILE) &&
                  SH_INDEX_OK((long long)tl.row0 + tl.nrows, (long long)d.N * d.k + 1, status, SH_SITE_V_TILE);
  if (!ok) { tl.h = 0; tl.e = 0; tl.row0 = 0; tl.nrows = 0; }
#endif
  return tl;
}

constexpr int GEMM_BM = 128;
constexpr int GEMM_BK = 64;

template <int BN, int STAGES, int MT = 1>
struct GemmSmem {
  static constexpr int A_BYTES = MT * GEMM_BM * GEMM_BK * 2;
  static constexpr int B_BYTES = BN * GEMM_BK * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int BAR_OFF = STAGES * STAGE_BYTES;
  static constexpr int TOTAL = BAR_OFF + 256 + 1024;   // + barriers + alignment slack
};

template <int BN, int STAGES, int MODE, int A_BF16, int B_BF16, int MT = 1>
__global__ void __launch_bounds__(192)
sh_tc_gemm_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB, TcGemmArgs g) {
  using SM = GemmSmem<BN, STAGES, MT>;
  static_assert(MT * BN <= 512, "accumulators must fit the 512 TMEM columns");
  constexpr int ROWS = MT * GEMM_BM;
  constexpr bool GATHER = MODE == GEMM_V;
  extern __shared__ unsigned char smem_raw[];
  const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* sgen = smem_raw + (sbase - smem_u32(smem_raw));
  uint64_t* full_bar = (uint64_t*)(sgen + SM::BAR_OFF);
  uint64_t* empty_bar = full_bar + STAGES;
  uint64_t* tmem_full = empty_bar + STAGES;
  uint32_t* tmem_slot = (uint32_t*)(tmem_full + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const ShDims& d = g.d;
  int th = 0, te = 0, row0, nrows;
  if (GATHER) {
    pdl_wait();                                        // (a no-op in an ordinary launch) the tile table and the lists are the kernel's before this one
    if ((int)blockIdx.x >= *g.ntiles) return;          // whole CTA leaves before any barrier
    const ShTile tl = tile_checked(g.tiles[blockIdx.x], d, g.status);
    th = tl.h; te = tl.e; row0 = tl.row0; nrows = tl.nrows;
  } else {
    row0 = blockIdx.x * ROWS;
    nrows = min(ROWS, g.nrows - row0);
  }
  const int col0 = blockIdx.y * BN;
  const int KB = g.K / GEMM_BK;
  bool dead = false;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(&full_bar[s], GATHER ? 129 : 1);
      mbar_init(&empty_bar[s], 1);
    }
    mbar_init(tmem_full, 1);
    fence_barrier_init();
    tma_prefetch_desc(&mapB);
    if (!GATHER) tma_prefetch_desc(&mapA);
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, MT * BN);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_d = *tmem_slot;
  if (threadIdx.x == 0) { sh_stamp_resident(d.stamps, g.stamp_id); sh_stamp_start(d.stamps, g.stamp_id); }

  if (warp == 0) {
    if (lane == 0) {
      const int brow = (GATHER ? (th * d.E + te) * g.b_rows_per_group : 0) + col0;
      for (int kb = 0; kb < KB; ++kb) {
        const int s = kb % STAGES;
        if (!mbar_wait(&empty_bar[s], ((kb / STAGES) & 1) ^ 1, g.status, dead)) break;
        const uint32_t sa = sbase + s * SM::STAGE_BYTES, sb = sa + SM::A_BYTES;
        mbar_expect_tx(&full_bar[s], GATHER ? SM::B_BYTES : SM::STAGE_BYTES);
        if (!GATHER) {
#pragma unroll
          for (int mt = 0; mt < MT; ++mt)
            tma_load_2d(sa + mt * (GEMM_BM * GEMM_BK * 2), &mapA, &full_bar[s], kb * GEMM_BK, row0 + mt * GEMM_BM);
        }
        tma_load_2d(sb, &mapB, &full_bar[s], kb * GEMM_BK, brow);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc_f16(GEMM_BM, BN, A_BF16, B_BF16, 0);
      const uint32_t a_lo0 = desc_lo_k(sbase), b_lo0 = desc_lo_k(sbase + SM::A_BYTES);
      int s = 0;
      uint32_t par = 0;
      for (int kb = 0; kb < KB; ++kb) {
        if (!mbar_wait(&full_bar[s], par, g.status, dead)) break;
        tc_fence_after();
        const uint32_t a_lo = a_lo0 + s * (SM::STAGE_BYTES >> 4), b_lo = b_lo0 + s * (SM::STAGE_BYTES >> 4);
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
#pragma unroll
          for (int k = 0; k < GEMM_BK / 16; ++k)
            umma_f16(tmem_d + mt * BN, desc_pack(a_lo + mt * (GEMM_BM * GEMM_BK * 2 >> 4) + 2 * k), desc_pack(b_lo + 2 * k),
                     idesc, (kb | k) != 0);
        }
        umma_commit(&empty_bar[s]);
        if (++s == STAGES) { s = 0; par ^= 1; }
      }
      umma_commit(tmem_full);
    }
  } else {
    const int et = threadIdx.x - 64;                   // 0..127
    if (GATHER) {
      // thread -> 16-byte chunk c of rows rb, rb+16, ... (8 threads cover one 128-byte row)
      const int c = et & 7, rb = et >> 3;
      const char* src[8 * MT];
      uint32_t ok[8 * MT];
      constexpr int abytes = 2;
#pragma unroll
      for (int i = 0; i < 8 * MT; ++i) {
        const int r = rb + 16 * i;
        int tok = 0;
        ok[i] = 0;
        if (r < nrows) { tok = g.lists[(size_t)th * d.N * d.k + row0 + r]; ok[i] = 16; }
        if (!SH_INDEX_OK(tok, d.N, g.status, SH_SITE_V_LIST)) { tok = 0; ok[i] = 0; }
        src[i] = (const char*)g.A + ((long)tok * g.lda + c * 8) * abytes;
      }
      const uint32_t dsw = (uint32_t)((c ^ (rb & 7)) << 4);
      int arrived = 0;
      for (int kb = 0; kb < KB; ++kb) {
        const int s = kb % STAGES;
        if (!mbar_wait(&empty_bar[s], ((kb / STAGES) & 1) ^ 1, g.status, dead)) break;
        const uint32_t sa = sbase + s * SM::STAGE_BYTES;
#pragma unroll
        for (int i = 0; i < 8 * MT; ++i)
          cp_async_16(sa + (rb + 16 * i) * 128 + dsw, src[i] + (long)kb * GEMM_BK * abytes, ok[i]);
        cp_async_commit();
        if (kb >= 2) {
          cp_async_wait<2>();
          fence_proxy_async_smem();
          mbar_arrive(&full_bar[arrived % STAGES]);
          ++arrived;
        }
      }
      cp_async_wait<0>();
      fence_proxy_async_smem();
      if (!dead)
        for (; arrived < KB; ++arrived) mbar_arrive(&full_bar[arrived % STAGES]);
    }
    // ---- epilogue: thread = accumulator row = TMEM lane (one pass per row tile) ---------------
    const int q = warp & 3;
    const bool tm_ok = mbar_wait(tmem_full, 0, g.status, dead);
    if (tm_ok) tc_fence_after();
#pragma unroll 1
    for (int mt = 0; mt < MT; ++mt) {
    const int r = mt * GEMM_BM + q * 32 + lane;
    bool live = r < nrows;
    int tok = 0;
    float gate = 0.f;
    if (live) {
      if (GATHER) {
        const size_t li = (size_t)th * d.N * d.k + row0 + r;
        tok = g.lists[li];
        gate = g.lgate[li];
        if (!SH_INDEX_OK(tok, d.N, g.status, SH_SITE_V_TOKEN)) tok = -1;
      } else {
        tok = row0 + r;
      }
    }
    if (tok < 0) { live = false; tok = 0; }
    if (tm_ok) {
      const uint32_t trow = tmem_d + ((uint32_t)(q * 32) << 16) + mt * BN;
      const int bb = tok / d.T, tt = tok % d.T;
      const bool early = MODE == GEMM_V && live && g.v_early && tt < d.early_rows;
#pragma unroll 1
      for (int c00 = 0; c00 < BN; c00 += 64) {
        // two TMEM loads in flight per wait: the load latency, not its bandwidth, bounds this loop
        uint32_t vv[64];
        tmem_ld32(trow + c00, *reinterpret_cast<uint32_t(*)[32]>(&vv[0]));
        tmem_ld32(trow + c00 + 32, *reinterpret_cast<uint32_t(*)[32]>(&vv[32]));
        tmem_ld_wait();
#pragma unroll
        for (int hh2 = 0; hh2 < 2; ++hh2) {
        const int c0 = c00 + hh2 * 32;
        uint32_t* v = &vv[hh2 * 32];
        const int n0 = col0 + c0;
        if (!live || n0 >= g.ncols) continue;
        if (MODE == GEMM_QKV) {
          const int HD = d.H * d.D;
          const int which = n0 / HD, hh = (n0 % HD) / d.D, dd = n0 % d.D;
          __half* dst = (__half*)(which == 0 ? g.out0 : which == 1 ? g.out1 : g.out2) +
                        (((size_t)bb * d.H + hh) * d.T + tt) * d.D + dd;
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
        } else if (MODE == GEMM_V) {
          __half* dst = (__half*)g.out0 + (((size_t)bb * d.H + th) * d.T + tt) * d.D + n0;
          uint32_t p[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            __half2 hv = __floats2half2_rn(__uint_as_float(v[2 * i]) * gate, __uint_as_float(v[2 * i + 1]) * gate);
            p[i] = *reinterpret_cast<uint32_t*>(&hv);
          }
          if (early) {
            float* d32 = g.v_early + (((size_t)bb * d.H + th) * SH_EARLY_ROWS + tt) * d.D + n0;
#pragma unroll
            for (int i = 0; i < 8; ++i)
              red_add_v4_f32(d32 + 4 * i, __uint_as_float(v[4 * i]) * gate, __uint_as_float(v[4 * i + 1]) * gate,
                             __uint_as_float(v[4 * i + 2]) * gate, __uint_as_float(v[4 * i + 3]) * gate);
          } else {
#pragma unroll
          for (int i = 0; i < 4; ++i) red_add_v4_f16x2(dst + 8 * i, p[4 * i], p[4 * i + 1], p[4 * i + 2], p[4 * i + 3]);
          }
        } else {
          float* dst = (float*)g.out0 + (size_t)tok * g.ncols + n0;
#pragma unroll
          for (int i = 0; i < 8; ++i)
            *reinterpret_cast<float4*>(dst + 4 * i) =
                make_float4(__uint_as_float(v[4 * i]), __uint_as_float(v[4 * i + 1]), __uint_as_float(v[4 * i + 2]),
                            __uint_as_float(v[4 * i + 3]));
        }
        }
      }
      if (early)
        v_early_finish(g.v_early + (((size_t)bb * d.H + th) * SH_EARLY_ROWS + tt) * d.D, g.v_early_cnt + ((size_t)bb * d.H + th) * SH_EARLY_ROWS + tt,
                       (__half*)g.out0 + (((size_t)bb * d.H + th) * d.T + tt) * d.D, d.D, d.k);
    }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0) sh_stamp_end(d.stamps, g.stamp_id);
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_d, MT * BN);
  }
}

}  // namespace shtc
