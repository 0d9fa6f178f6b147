// Output-expert projection with the gate-weighted sum kept on chip (the MoE output equation
// of Sec. 2.2):  y[t] = sum_h sum_{e in E_D^h(t)} s_D^h[t,e] * Ahat^h[t] W_O^{h,e}.
//
// One CTA owns 128 consecutive tokens and 128 output features.  For every head h the tokens'
// Ahat^h rows are one TMA tile (token order, no gather); for every expert e that at least one
// token of the tile selected, one UMMA chain computes Z = W_O^{h,e}[features, :] Ahat^h[tokens, :]^T
// (features on the TMEM lanes, tokens on the columns).  Each epilogue thread owns one feature
// and keeps y[token, feature] for all 128 tokens in registers:  acc[t] += g_e[t] * Z[feature, t],
// where g_e[t] is the destination gate of expert e for token t, or 0 if t did not select e.
// The sum over experts and heads therefore never leaves the SM, out is written exactly once
// (no atomics, no clearing, run-to-run deterministic).  The price is that unselected tokens
// ride along in the UMMA (E/k times the useful FLOP of this stage).
//
// Warp roles (320 threads): warp 0 = TMA producer, warp 1 = TMEM owner + UMMA issuer,
// warps 2..9 = epilogue (thread = one feature = TMEM lane, and one half of the tile's tokens;
// two warps share a lane quarter so that twice as many TMEM loads are in flight).
// TMEM: four 128-column buffers.
#pragma once
#include "sh_tc_prims.cuh"

namespace shtc {

struct TcOprojArgs {
  ShDims d;
  const int* idx;        // destination side: [N, H, k]
  const float* gate;     // destination side: [N, H, k]
  const int* blockcnt;   // [nblk, G] per-tile selection counts (bucket = (side*H + h)*E + e)
  float* out;            // [N, M]
  int a_stages;
  int* status;
};

template <int D>
struct OprojSmem {
  static constexpr int A_BYTES = 128 * D * 2;            // weights tile: 128 features x D
  static constexpr int B_BYTES = 128 * D * 2;            // Ahat tile: 128 tokens x D
  static int total(int a_stages, int H, int E, int k) {
    return a_stages * A_BYTES + 2 * B_BYTES + 128 * H * k * 8 + E * 128 * 4 + H * E * 4 + 512 + 1024;
  }
};

template <int D>
__global__ void __launch_bounds__(320)
sh_tc_oproj_kernel(const __grid_constant__ CUtensorMap mapAhat, const __grid_constant__ CUtensorMap mapWo, TcOprojArgs g) {
  using SM = OprojSmem<D>;
  constexpr int DB = D / 64;
  constexpr uint32_t BLK = 128 * 128;
  constexpr int MAX_A = 5;
  extern __shared__ unsigned char smem_raw[];
  const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* sgen = smem_raw + (sbase - smem_u32(smem_raw));
  const ShDims& d = g.d;
  const int AS = g.a_stages;
  const int HE = d.H * d.E;
  const uint32_t a_off = 0, b_off = AS * SM::A_BYTES, misc_off = b_off + 2 * SM::B_BYTES;
  int* s_idx = (int*)(sgen + misc_off);                       // [128, H, k]
  float* s_gt = (float*)(s_idx + 128 * d.H * d.k);            // [128, H, k]
  float* s_g = s_gt + 128 * d.H * d.k;                        // [E, 128] gates of the current head
  int* s_cnt = (int*)(s_g + d.E * 128);                       // [H*E]
  uint64_t* bars = (uint64_t*)(((uintptr_t)(s_cnt + HE) + 15) & ~(uintptr_t)15);
  uint64_t* a_full = bars;               // [MAX_A]
  uint64_t* a_empty = bars + MAX_A;      // [MAX_A]
  uint64_t* b_full = bars + 2 * MAX_A;   // [2]
  uint64_t* b_empty = b_full + 2;        // [2]
  uint64_t* d_full = b_empty + 2;        // [4]
  uint64_t* d_empty = d_full + 4;        // [4]
  uint32_t* tmem_slot = (uint32_t*)(d_empty + 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nfc = d.M / 128;
  const int tt = blockIdx.x / nfc, fc = blockIdx.x % nfc;
  const int row0 = tt * 128;
  const int nrows = min(128, d.N - row0);
  bool dead = false;

  if (threadIdx.x == 0) {
    for (int s = 0; s < MAX_A; ++s) { mbar_init(&a_full[s], 1); mbar_init(&a_empty[s], 1); }
    for (int s = 0; s < 2; ++s) { mbar_init(&b_full[s], 1); mbar_init(&b_empty[s], 1); }
    for (int s = 0; s < 4; ++s) { mbar_init(&d_full[s], 1); mbar_init(&d_empty[s], 256); }
    fence_barrier_init();
    tma_prefetch_desc(&mapAhat); tma_prefetch_desc(&mapWo);
  }
  if (warp == 1) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
  // destination-side counts of this tile, and its selections (contiguous in global memory)
  for (int i = threadIdx.x; i < HE; i += blockDim.x) s_cnt[i] = g.blockcnt[(size_t)tt * d.G + HE + i];
  {
    const int per_tok = d.H * d.k;
    const int total = nrows * per_tok;
    const int* gi = g.idx + (size_t)row0 * per_tok;
    const float* gg = g.gate + (size_t)row0 * per_tok;
    for (int i = threadIdx.x; i < 128 * per_tok; i += blockDim.x) {
      s_idx[i] = i < total ? gi[i] : 0;
      s_gt[i] = i < total ? gg[i] : 0.f;
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      int s = 0;
      uint32_t e_par = 1;                                   // parity of a_empty[s] for the current ring pass
      for (int h = 0; h < d.H; ++h) {
        const int bs = h & 1;
        if (!mbar_wait(&b_empty[bs], ((h >> 1) & 1) ^ 1, g.status, dead)) break;
        mbar_expect_tx(&b_full[bs], SM::B_BYTES);
#pragma unroll
        for (int c = 0; c < DB; ++c)
          tma_load_2d(sbase + b_off + bs * SM::B_BYTES + c * BLK, &mapAhat, &b_full[bs], h * D + c * 64, row0);
        for (int e = 0; e < d.E && !dead; ++e) {
          if (s_cnt[h * d.E + e] == 0) continue;
          if (!mbar_wait(&a_empty[s], e_par, g.status, dead)) break;
          mbar_expect_tx(&a_full[s], SM::A_BYTES);
#pragma unroll
          for (int c = 0; c < DB; ++c)
            tma_load_2d(sbase + a_off + s * SM::A_BYTES + c * BLK, &mapWo, &a_full[s], c * 64,
                        (h * d.E + e) * d.M + fc * 128);
          if (++s == AS) { s = 0; e_par ^= 1; }
        }
        if (dead) break;
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc_f16(128, 128, 0, 0, 0);
      const uint32_t a_lo0 = desc_lo_k(sbase + a_off), b_lo0 = desc_lo_k(sbase + b_off);
      int it = 0, s = 0;
      uint32_t a_par = 0;                                   // parity of a_full[s] for the current ring pass
      for (int h = 0; h < d.H && !dead; ++h) {
        const int bs = h & 1;
        if (!mbar_wait(&b_full[bs], (h >> 1) & 1, g.status, dead)) break;
        const uint32_t b_lo = b_lo0 + bs * (SM::B_BYTES >> 4);
        for (int e = 0; e < d.E; ++e) {
          if (s_cnt[h * d.E + e] == 0) continue;
          const int buf = it & 3;
          if (!mbar_wait(&a_full[s], a_par, g.status, dead)) break;
          if (!mbar_wait(&d_empty[buf], ((it >> 2) & 1) ^ 1, g.status, dead)) break;
          tc_fence_after();
          const uint32_t a_lo = a_lo0 + s * (SM::A_BYTES >> 4);
          const uint32_t td = tmem + buf * 128;
#pragma unroll
          for (int k = 0; k < D / 16; ++k) {
            const uint32_t koff = (k / 4) * (BLK >> 4) + 2 * (k % 4);
            umma_f16(td, desc_pack(a_lo + koff), desc_pack(b_lo + koff), idesc, k != 0);
          }
          umma_commit(&a_empty[s]);
          umma_commit(&d_full[buf]);
          ++it;
          if (++s == AS) { s = 0; a_par ^= 1; }
        }
        umma_commit(&b_empty[bs]);
      }
    }
  } else {
    // ---- epilogue: thread = output feature x token half; acc[t] = y[row0 + half*64 + t, feature] ----
    const int q = warp & 3;
    const int half = (warp - 2) >> 2;
    const int f = q * 32 + lane;
    const int et = threadIdx.x - 64;                      // 0..255; the first 128 build s_g (thread = token)
    const uint32_t lane_off = (uint32_t)(q * 32) << 16;
    float acc[64];
#pragma unroll
    for (int t = 0; t < 64; ++t) acc[t] = 0.f;
    int it = 0;
    bool ok = true;
    for (int h = 0; h < d.H && ok; ++h) {
      // gates of this head: s_g[e][t] = gate if token t selected e, else 0
      asm volatile("bar.sync 1, 256;" ::: "memory");      // everyone finished the previous head
      for (int i = et; i < d.E * 128; i += 256) s_g[i] = 0.f;
      asm volatile("bar.sync 1, 256;" ::: "memory");
      if (et < nrows)
        for (int j = 0; j < d.k; ++j) {
          const int o = (et * d.H + h) * d.k + j;
          s_g[s_idx[o] * 128 + et] = s_gt[o];
        }
      asm volatile("bar.sync 1, 256;" ::: "memory");
      for (int e = 0; e < d.E; ++e) {
        if (s_cnt[h * d.E + e] == 0) continue;
        const int buf = it & 3;
        if (!mbar_wait(&d_full[buf], (it >> 2) & 1, g.status, dead)) { ok = false; break; }
        tc_fence_after();
        const float4* ge = reinterpret_cast<const float4*>(s_g + e * 128 + half * 64);
        uint32_t v[64];
        tmem_ld32(tmem + lane_off + buf * 128 + half * 64, *reinterpret_cast<uint32_t(*)[32]>(&v[0]));
        tmem_ld32(tmem + lane_off + buf * 128 + half * 64 + 32, *reinterpret_cast<uint32_t(*)[32]>(&v[32]));
        tmem_ld_wait();
        tc_fence_before();
        mbar_arrive(&d_empty[buf]);
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const float4 gv = ge[i];
          acc[4 * i + 0] = fmaf(gv.x, __uint_as_float(v[4 * i + 0]), acc[4 * i + 0]);
          acc[4 * i + 1] = fmaf(gv.y, __uint_as_float(v[4 * i + 1]), acc[4 * i + 1]);
          acc[4 * i + 2] = fmaf(gv.z, __uint_as_float(v[4 * i + 2]), acc[4 * i + 2]);
          acc[4 * i + 3] = fmaf(gv.w, __uint_as_float(v[4 * i + 3]), acc[4 * i + 3]);
        }
        ++it;
      }
    }
    if (ok) {
      float* dst = g.out + (size_t)(row0 + half * 64) * d.M + fc * 128 + f;
#pragma unroll
      for (int t = 0; t < 64; ++t)
        if (half * 64 + t < nrows) dst[(size_t)t * d.M] = acc[t];
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

}  // namespace shtc
