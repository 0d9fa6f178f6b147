// Fused gate kernel of the bf16 configuration (Sec. 2.2: s = sigmoid(x W), arg top-k):
// the logits tile z[128 tokens, G] = x W_gate^T runs on the tensor pipe (TMA-fed, fp32 in
// TMEM), then each thread owns one token: adds the bias, picks the k largest logits of every
// (side, head) group (strictly-greater scan, so the lower index wins ties), applies the
// sigmoid, writes idx / gate and adds to the CTA's selection histogram.  While the main loop
// runs, the otherwise idle epilogue warps clear the V and out rows of the CTA's tokens (both
// are accumulated into later).  The last CTA to finish turns the per-CTA histograms into
// block offsets, per-head expert offsets and the row-tile table of the grouped GEMMs.
//
// Warp roles (192 threads): warp 0 = TMA producer, warp 1 = TMEM owner + UMMA issuer,
// warps 2..5 = zero-fill, then selection epilogue.
#pragma once
#include "sh_tc_prims.cuh"

namespace shtc {

struct TcGateArgs {
  ShDims d;
  int Gp;                    // G rounded up to a multiple of 16 (UMMA N)
  const float* gbias;        // [G]
  int* idx; float* gate;     // [2, N, H, k]
  int* blockcnt; int* blockoff; int* offsets; ShTile* tiles; int* ntiles;
  unsigned int* done_counter;
  __half* zero_v;            // [B, H, T, D] or nullptr
  float* zero_out;           // [N, M] or nullptr
  int* status;
};

template <int STAGES>
__global__ void __launch_bounds__(192)
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
  uint32_t* tmem_slot = (uint32_t*)(tmem_full + 1);
  int* s_flag = (int*)(tmem_slot + 1);
  int* s_hist = (int*)(sgen + bar_off + 256);           // [G]
  int* s_total = s_hist + d.G;                          // [G]   (last CTA only)
  int* s_tbase = s_total + d.G;                         // [G]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row0 = blockIdx.x * 128;
  const int nrows = min(128, d.N - row0);
  const int KB = d.M / 64;
  bool dead = false;
  uint32_t tmem_cols = 32;
  while ((int)tmem_cols < Gp) tmem_cols <<= 1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
    mbar_init(tmem_full, 1);
    fence_barrier_init();
    tma_prefetch_desc(&mapX); tma_prefetch_desc(&mapW);
  }
  for (int i = threadIdx.x; i < d.G; i += blockDim.x) s_hist[i] = 0;
  if (warp == 1) { tmem_alloc(tmem_slot, tmem_cols); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_d = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      for (int kb = 0; kb < KB; ++kb) {
        const int s = kb % STAGES;
        if (!mbar_wait(&empty_bar[s], ((kb / STAGES) & 1) ^ 1, g.status, dead)) break;
        const uint32_t sa = sbase + s * stage_bytes, sb = sa + a_bytes;
        mbar_expect_tx(&full_bar[s], a_bytes + b_bytes);
        tma_load_2d(sa, &mapX, &full_bar[s], kb * 64, row0);
        tma_load_2d(sb, &mapW, &full_bar[s], kb * 64, 0);
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
    const int et = threadIdx.x - 64;                    // 0..127
    // ---- clear the rows this CTA's tokens own in V and out (accumulated into later) -----------
    if (g.zero_out) {
      const int n4 = d.M / 4;                           // float4 per row
      float4* base = reinterpret_cast<float4*>(g.zero_out + (size_t)row0 * d.M);
      const long total = (long)nrows * n4;
      for (long i = et; i < total; i += 128) base[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    if (g.zero_v) {
      const int c16 = d.D / 8;                          // 16-byte chunks per (token, head) row
      const long total = (long)nrows * d.H * c16;
      for (long i = et; i < total; i += 128) {
        const int ch = (int)(i % c16);
        const long th = i / c16;
        const int hh = (int)(th % d.H);
        const int tok = row0 + (int)(th / d.H);
        const int bb = tok / d.T, tt = tok % d.T;
        *reinterpret_cast<uint4*>(g.zero_v + (((size_t)bb * d.H + hh) * d.T + tt) * d.D + ch * 8) = make_uint4(0, 0, 0, 0);
      }
    }
    // ---- selection epilogue: thread = token = TMEM lane ---------------------------------------
    const int q = warp & 3;
    const int r = q * 32 + lane;
    float* srow = reinterpret_cast<float*>(sgen) + (size_t)r * (Gp + 1);
    if (mbar_wait(tmem_full, 0, g.status, dead)) {
      tc_fence_after();
      const uint32_t trow = tmem_d + ((uint32_t)(q * 32) << 16);
      for (int c0 = 0; c0 < Gp; c0 += 16) {             // logits row -> shared memory (pipeline buffers are idle now)
        uint32_t v[16];
        asm volatile(
            "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
            : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
              "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
            : "r"(trow + c0)
            : "memory");
        tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 16; ++i)
          if (c0 + i < d.G) srow[c0 + i] = __uint_as_float(v[i]) + g.gbias[c0 + i];
      }
      const int t = row0 + r;
      if (r < nrows) {
        for (int grp = 0; grp < 2 * d.H; ++grp) {
          const float* z = srow + grp * d.E;
          const int side = grp / d.H, h = grp % d.H;
          const size_t o = (((size_t)side * d.N + t) * d.H + h) * d.k;
          unsigned taken = 0;
          for (int j = 0; j < d.k; ++j) {
            int best = -1;
            float bz = 0.f;
            for (int e = 0; e < d.E; ++e) {
              if ((taken >> e) & 1u) continue;
              const float ze = z[e];
              if (best < 0 || ze > bz) { best = e; bz = ze; }
            }
            taken |= 1u << best;
            g.idx[o + j] = best;
            g.gate[o + j] = 1.f / (1.f + expf(-bz));
            atomicAdd(&s_hist[grp * d.E + best], 1);
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_d, tmem_cols);
  }
  // ---- publish the histogram; the last CTA builds offsets and the tile table -----------------
  const int nb = d.G;
  for (int i = threadIdx.x; i < nb; i += blockDim.x) g.blockcnt[(size_t)blockIdx.x * nb + i] = s_hist[i];
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const unsigned prev = atomicAdd(g.done_counter, 1u);
    *s_flag = (prev == gridDim.x - 1);
  }
  __syncthreads();
  if (!*s_flag) return;
  __threadfence();
  // warp per bucket: exclusive scan over the CTAs' counts
  for (int b = warp; b < nb; b += 6) {
    int run = 0;
    for (int blk0 = 0; blk0 < d.nblk; blk0 += 32) {
      const int blk = blk0 + lane;
      const int c = blk < d.nblk ? __ldcg(&g.blockcnt[(size_t)blk * nb + b]) : 0;
      int inc = c;
#pragma unroll
      for (int s = 1; s < 32; s <<= 1) {
        const int n = __shfl_up_sync(0xffffffffu, inc, s);
        if (lane >= s) inc += n;
      }
      if (blk < d.nblk) g.blockoff[(size_t)blk * nb + b] = run + inc - c;
      run += __shfl_sync(0xffffffffu, inc, 31);
    }
    if (lane == 0) s_total[b] = run;
  }
  __syncthreads();
  for (int grp = threadIdx.x; grp < 2 * d.H; grp += blockDim.x) {
    int run = 0;
    for (int e = 0; e < d.E; ++e) {
      g.offsets[grp * (d.E + 1) + e] = run;
      run += s_total[grp * d.E + e];
    }
    g.offsets[grp * (d.E + 1) + d.E] = run;
  }
  if (threadIdx.x < 2) {
    const int side = threadIdx.x;
    int run = 0;
    for (int b = side * d.H * d.E; b < (side + 1) * d.H * d.E; ++b) {
      s_tbase[b] = run;
      run += (s_total[b] + SH_TILE_ROWS - 1) / SH_TILE_ROWS;
    }
    g.ntiles[side] = run;
  }
  __syncthreads();
  for (int b = threadIdx.x; b < nb; b += blockDim.x) {
    const int side = b / (d.H * d.E), h = (b / d.E) % d.H, e = b % d.E;
    int start = 0;
    for (int e2 = 0; e2 < e; ++e2) start += s_total[b - e + e2];
    const int cnt = s_total[b];
    ShTile* tp = g.tiles + (size_t)side * d.max_tiles + s_tbase[b];
    for (int rr = 0, i = 0; rr < cnt; rr += SH_TILE_ROWS, ++i) {
      ShTile tl;
      tl.h = h; tl.e = e; tl.row0 = start + rr; tl.nrows = min(SH_TILE_ROWS, cnt - rr);
      tp[i] = tl;
    }
  }
  if (threadIdx.x == 0) *g.done_counter = 0;            // ready for the next forward pass
}

}  // namespace shtc
