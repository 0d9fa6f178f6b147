// Output-expert projection with the gate-weighted sum kept on chip (the MoE output equation
// of Sec. 2.2):  y[t] = sum_h sum_{e in E_D^h(t)} s_D^h[t,e] * Ahat^h[t] W_O^{h,e}.
//
// Work unit = 128 consecutive tokens x 128 output features; a persistent CTA (one per SM)
// walks work units blockIdx.x, blockIdx.x + gridDim.x, ...  For every head h the tokens'
// Ahat^h rows are one TMA tile (token order, no gather); for every expert e one UMMA chain
// computes Z = Ahat^h[tokens, :] W_O^{h,e}[:, features] (tokens on the TMEM lanes, features
// on the columns).  Each epilogue thread owns one token and 64 of the features and keeps
// y[token, feature] in registers:  acc[f] += g * Z[token, f], where g is the token's
// destination gate for expert e, or 0 if it did not select e - a per-thread scalar, so the
// epilogue is pure FFMA.  The sum over experts and heads therefore never leaves the SM and
// out is written exactly once (no atomics, no clearing, run-to-run deterministic).  The price
// is that unselected tokens ride along in the UMMA (E/k times the useful FLOP of this stage).
//
// Warp roles (384 threads): warps 0 and 11 = TMA producers (warp 0: token tiles and the first
// 64-column block of every weight tile, warp 11: the second block - one thread issues a TMA
// box only every ~150 ns), warp 1 = TMEM owner + UMMA issuer for the even pipeline items,
// warp 10 = UMMA issuer for the odd items, warps 2..9 = epilogue (thread =
// one token = TMEM lane, and one half of the 128 features; two warps share a lane quarter).
// One expert = one pipeline item: a weight-tile slot (ring of 4) and a 128-column TMEM buffer
// (ring of 4).  Both rings are deep on purpose: L2 answers a TMA load after ~0.9 us and the
// epilogue hands a TMEM buffer back ~1000 cycles after the UMMAs that filled it were issued,
// so with only two of either the tensor pipe idles most of the time.  The issuers alternate
// experts, so one thread's barrier round trips hide behind the other's UMMAs.  All rings run
// on across work units, so the producers and the issuers work ahead into the next unit while the epilogue
// stores the last one.
#pragma once
#include "sh_tc_prims.cuh"

namespace shtc {

struct TcOprojArgs {
  ShDims d;
  const int* idx;        // destination side: [N, H, k]
  const float* gate;     // destination side: [N, H, k]
  float* out;            // [N, M]
  int a_slots;           // weight-tile slots in the ring (power of two: 2 or 4)
  int nwork;             // nblk * (M / 128)
  int* status;
};

template <int D>
struct OprojSmem {
  static constexpr int A_BYTES = 128 * D * 2;            // one weight tile: 128 features x D
  static constexpr int B_BYTES = 128 * D * 2;            // Ahat tile: 128 tokens x D
  static int total(int a_slots, int H, int k) {
    return a_slots * A_BYTES + 2 * B_BYTES + 128 * H * k * 8 + 512 + 1024;
  }
};

template <int D>
__global__ void __launch_bounds__(384, 1)
sh_tc_oproj_kernel(const __grid_constant__ CUtensorMap mapAhat, const __grid_constant__ CUtensorMap mapWo, TcOprojArgs g) {
  using SM = OprojSmem<D>;
  constexpr int DB = D / 64;
  constexpr uint32_t BLK = 128 * 128;
  constexpr int MAX_A = 4;
  extern __shared__ unsigned char smem_raw[];
  const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* sgen = smem_raw + (sbase - smem_u32(smem_raw));
  const ShDims& d = g.d;
  const int AS = g.a_slots;                // power of two
  const int as_shift = AS == 4 ? 2 : 1;
  const uint32_t a_off = 0, b_off = AS * SM::A_BYTES, misc_off = b_off + 2 * SM::B_BYTES;
  int* s_idx = (int*)(sgen + misc_off);                       // [128, H, k] selections of the current tokens
  float* s_gt = (float*)(s_idx + 128 * d.H * d.k);            // [128, H, k]
  uint64_t* bars = (uint64_t*)(((uintptr_t)(s_gt + 128 * d.H * d.k) + 15) & ~(uintptr_t)15);
  uint64_t* a_full = bars;               // [MAX_A]
  uint64_t* a_empty = bars + MAX_A;      // [MAX_A]
  uint64_t* b_full = bars + 2 * MAX_A;   // [2]
  uint64_t* b_empty = b_full + 2;        // [2]
  uint64_t* d_full = b_empty + 2;        // [4]
  uint64_t* d_empty = d_full + 4;        // [4]
  uint64_t* sel_free = d_empty + 4;      // epilogue threads are done with the selections copy
  uint64_t* sel_ready = sel_free + 1;    // the selections copy of the current work unit is complete
  uint32_t* tmem_slot = (uint32_t*)(sel_ready + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nfc = d.M / 128;
  bool dead = false;

  if (threadIdx.x == 0) {
    for (int s = 0; s < MAX_A; ++s) { mbar_init(&a_full[s], DB); mbar_init(&a_empty[s], 1); }
    for (int s = 0; s < 2; ++s) { mbar_init(&b_full[s], 1); mbar_init(&b_empty[s], 2); }
    for (int s = 0; s < 4; ++s) { mbar_init(&d_full[s], 1); mbar_init(&d_empty[s], 256); }
    mbar_init(sel_free, 256); mbar_init(sel_ready, 256);
    fence_barrier_init();
    tma_prefetch_desc(&mapAhat); tma_prefetch_desc(&mapWo);
  }
  if (warp == 1) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp == 0 || warp == 11) {
    if (lane == 0 && (warp == 0 || DB == 2)) {
      const int c = warp == 0 ? 0 : 1;                      // the 64-column block this producer loads
      int gh = 0, ge = 0;                                   // running head / expert counters
      for (int w = blockIdx.x; w < g.nwork && !dead; w += gridDim.x) {
        const int row0 = (w / nfc) * 128, fc = w % nfc;
        for (int h = 0; h < d.H && !dead; ++h, ++gh) {
          if (warp == 0) {
            const int bs = gh & 1;
            if (!mbar_wait(&b_empty[bs], ((gh >> 1) & 1) ^ 1, g.status, dead)) break;
            mbar_expect_tx(&b_full[bs], SM::B_BYTES);
#pragma unroll
            for (int cc = 0; cc < DB; ++cc)
              tma_load_2d(sbase + b_off + bs * SM::B_BYTES + cc * BLK, &mapAhat, &b_full[bs], h * D + cc * 64, row0);
          }
          for (int e = 0; e < d.E; ++e, ++ge) {
            const int s = ge & (AS - 1);
            if (!mbar_wait(&a_empty[s], ((ge >> as_shift) & 1) ^ 1, g.status, dead)) break;
            mbar_expect_tx(&a_full[s], BLK);
            tma_load_2d(sbase + a_off + s * SM::A_BYTES + c * BLK, &mapWo, &a_full[s], c * 64,
                        (h * d.E + e) * d.M + fc * 128);
          }
        }
      }
    }
  } else if (warp == 1 || warp == 10) {
    if (lane == 0) {
      const int iss = warp == 1 ? 0 : 1;                    // this issuer takes the experts with ge % 2 == iss
      constexpr uint32_t idesc = make_idesc_f16(128, 128, 0, 0, 0);
      const uint32_t w_lo0 = desc_lo_k(sbase + a_off), t_lo0 = desc_lo_k(sbase + b_off);
      int gh = 0, ge = 0;
      for (int w = blockIdx.x; w < g.nwork && !dead; w += gridDim.x) {
        for (int h = 0; h < d.H && !dead; ++h, ++gh) {
          const int bs = gh & 1;
          if (!mbar_wait(&b_full[bs], (gh >> 1) & 1, g.status, dead)) break;
          const uint32_t t_lo = t_lo0 + bs * (SM::B_BYTES >> 4);
          for (int e = 0; e < d.E; ++e, ++ge) {
            if ((ge & 1) != iss) continue;
            const int s = ge & (AS - 1), buf = ge & 3;
            if (!mbar_wait(&a_full[s], (ge >> as_shift) & 1, g.status, dead)) break;
            if (!mbar_wait(&d_empty[buf], ((ge >> 2) & 1) ^ 1, g.status, dead)) break;
            tc_fence_after();
            const uint32_t w_lo = w_lo0 + s * (SM::A_BYTES >> 4);
#pragma unroll
            for (int k = 0; k < D / 16; ++k) {
              const uint32_t koff = (k / 4) * (BLK >> 4) + 2 * (k % 4);
              umma_f16(tmem + buf * 128, desc_pack(t_lo + koff), desc_pack(w_lo + koff), idesc, k != 0);
            }
            umma_commit(&a_empty[s]);                       // this slot can load its next tile
            umma_commit(&d_full[buf]);
          }
          umma_commit(&b_empty[bs]);
        }
      }
    }
  } else {
    // ---- epilogue: thread = token x feature half; acc[f] = y[row0 + token, fc*128 + half*64 + f] ----
    const int q = warp & 3;
    const int half = (warp - 2) >> 2;
    const int tok = q * 32 + lane;
    const int et = threadIdx.x - 64;                       // 0..255
    const uint32_t lane_off = (uint32_t)(q * 32) << 16;
    const int per_tok = d.H * d.k;
    int ge = 0;
    uint32_t wpar = 0;                                     // parity of this work unit for sel_free / sel_ready
    bool ok = true;
    for (int w = blockIdx.x; w < g.nwork && ok; w += gridDim.x, wpar ^= 1) {
      const int row0 = (w / nfc) * 128, fc = w % nfc;
      const int nrows = min(128, d.N - row0);
      // this tile's destination-side selections (contiguous in global memory) -> shared memory
      // (mbarriers with bounded waits rather than bar.sync, so that a thread that gave up cannot
      //  leave the others stuck)
      mbar_arrive(sel_free);                               // this thread is done with the previous copy
      if (!mbar_wait(sel_free, wpar, g.status, dead)) { ok = false; break; }
      {
        const int total = nrows * per_tok;
        const int* gi_ = g.idx + (size_t)row0 * per_tok;
        const float* gg = g.gate + (size_t)row0 * per_tok;
        for (int i = et; i < 128 * per_tok; i += 256) {
          s_idx[i] = i < total ? gi_[i] : -1;
          s_gt[i] = i < total ? gg[i] : 0.f;
        }
      }
      mbar_arrive(sel_ready);
      if (!mbar_wait(sel_ready, wpar, g.status, dead)) { ok = false; break; }
      float acc[64];
#pragma unroll
      for (int f = 0; f < 64; ++f) acc[f] = 0.f;
      for (int h = 0; h < d.H && ok; ++h) {
        const int sel = (tok * d.H + h) * d.k;               // this token's selections for head h
        for (int e = 0; e < d.E; ++e, ++ge) {
          const int buf = ge & 3;
          float gv = 0.f;                                    // gate of expert e for this token (0: not selected)
          for (int j = 0; j < d.k; ++j)
            if (s_idx[sel + j] == e) gv = s_gt[sel + j];
          if (!mbar_wait(&d_full[buf], (ge >> 2) & 1, g.status, dead)) { ok = false; break; }
          tc_fence_after();
          uint32_t v[64];
          const uint32_t ta = tmem + lane_off + buf * 128 + half * 64;
          tmem_ld32(ta, *reinterpret_cast<uint32_t(*)[32]>(&v[0]));
          tmem_ld32(ta + 32, *reinterpret_cast<uint32_t(*)[32]>(&v[32]));
          tmem_ld_wait();
          tc_fence_before();
          mbar_arrive(&d_empty[buf]);
#pragma unroll
          for (int f = 0; f < 64; ++f) acc[f] = fmaf(gv, __uint_as_float(v[f]), acc[f]);
        }
      }
      if (ok && tok < nrows) {
        float4* dst = reinterpret_cast<float4*>(g.out + (size_t)(row0 + tok) * d.M + fc * 128 + half * 64);
#pragma unroll
        for (int f = 0; f < 16; ++f) dst[f] = make_float4(acc[4 * f], acc[4 * f + 1], acc[4 * f + 2], acc[4 * f + 3]);
      }
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
