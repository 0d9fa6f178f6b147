// Output-expert projection with the gate-weighted sum kept on chip (the MoE output equation
// of Sec. 2.2):  y[t] = sum_h sum_{e in E_D^h(t)} s_D^h[t,e] * Ahat^h[t] W_O^{h,e}.
//
// Work unit = 128 consecutive tokens x 256 output features; a persistent CTA (one per SM)
// walks work units blockIdx.x, blockIdx.x + gridDim.x, ...  For every head h the tokens'
// Ahat^h rows are one TMA tile (token order, no gather); for every expert e one UMMA chain
// computes Z = Ahat^h[tokens, :] W_O^{h,e}[:, features] (tokens on the TMEM lanes, features
// on the columns).  Each epilogue thread owns one token and 128 of the features and keeps
// y[token, feature] in registers:  acc[f] += g * Z[token, f], where g is the token's
// destination gate for expert e, or 0 if it did not select e - a per-thread scalar, so the
// epilogue is pure FFMA.  The sum over experts and heads therefore never leaves the SM and
// out is written exactly once (no atomics, no clearing, run-to-run deterministic).  The price
// is that unselected tokens ride along in the UMMA (E/k times the useful FLOP of this stage).
//
// Why 256 features: the UMMA-issuing thread pays a fixed price per expert (barrier waits,
// fence, commits: ~400 cycles during which the tensor pipe drains, because tcgen05.mma issue
// is throttled to the pipe's own rate and queues almost nothing ahead), and every work unit
// re-reads the token tiles.  N = 256 doubles the tensor work behind each fixed price and
// halves the token-tile traffic; the accumulators (128 tokens x 256 features fp32) just fit
// the registers of 256 epilogue threads.
//
// Warp roles (320 threads): warp 0 = TMA producer, warp 1 = TMEM owner + UMMA issuer (a second
// issuing thread for the odd experts was tried: no gain), warps 2..9 = epilogue (thread = one token = TMEM lane, and one half of the 256 features;
// two warps share a lane quarter).  One expert = one 256-column TMEM buffer (ring of 2); its
// weights arrive as D/64 stages of 256 features x 64 columns (32 KB, one TMA box each) through
// a ring of 3 (or 2) stages that are released one by one: L2 answers a TMA load after ~0.9 us,
// so the bytes in flight set the fill rate and a stage handed back early is loading again.
// All rings run on across work units, so the producer and the issuer work ahead into the
// next unit while the epilogue stores the last one.
#pragma once
#include "sh_tc_prims.cuh"

namespace shtc {

struct TcOprojArgs {
  ShDims d;
  const int* idx;        // destination side: [N, H, k]
  const float* gate;     // destination side: [N, H, k]
  float* out;            // [N, M] fp32, or (out_f16) [N, M] fp16 at the same address
  int out_f16;           // 1: the result rows are rounded to fp16 once, on their way out
  int a_slots;           // 32 KB weight stages in the ring: 3 or 2
  int nwork;             // nblk * ceil(M / 256)
  int* status;
};

// Four consecutive features of one result row (element index elem of [N, M]): fp32, or rounded to fp16.
__device__ __forceinline__ void oproj_put4(float* out, size_t elem, float4 v, int out_f16) {
  if (out_f16) {
    const __half2 a = __floats2half2_rn(v.x, v.y), b = __floats2half2_rn(v.z, v.w);
    *reinterpret_cast<uint2*>(reinterpret_cast<__half*>(out) + elem) =
        make_uint2(*reinterpret_cast<const uint32_t*>(&a), *reinterpret_cast<const uint32_t*>(&b));
  } else {
    *reinterpret_cast<float4*>(out + elem) = v;
  }
}

template <int D>
struct OprojSmem {
  static constexpr int A_BYTES = 256 * 64 * 2;           // one weight stage: 256 features x 64 columns
  static constexpr int B_BYTES = 128 * D * 2;            // Ahat tile: 128 tokens x D
  static constexpr int STAGING = 8 * 32 * 32 * 4;        // per epilogue warp a 32 x 32 fp32 transpose tile
  static int total(int a_slots, int H, int k) {
    return a_slots * A_BYTES + 2 * B_BYTES + STAGING + 128 * H * k * 8 + 512 + 1024;
  }
};

template <int D>
__global__ void __launch_bounds__(320, 1)
sh_tc_oproj_kernel(const __grid_constant__ CUtensorMap mapAhat, const __grid_constant__ CUtensorMap mapWo, TcOprojArgs g) {
  using SM = OprojSmem<D>;
  constexpr int DB = D / 64;
  constexpr uint32_t TBLK = 128 * 128;                   // one 64-column block of the token tile
  extern __shared__ unsigned char smem_raw[];
  const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* sgen = smem_raw + (sbase - smem_u32(smem_raw));
  const ShDims& d = g.d;
  const int AS = g.a_slots;                              // 3 or 2
  const uint32_t a_off = 0, b_off = AS * SM::A_BYTES, stg_off = b_off + 2 * SM::B_BYTES, misc_off = stg_off + SM::STAGING;
  int* s_idx = (int*)(sgen + misc_off);                       // [128, H, k] selections of the current tokens
  float* s_gt = (float*)(s_idx + 128 * d.H * d.k);            // [128, H, k]
  uint64_t* bars = (uint64_t*)(((uintptr_t)(s_gt + 128 * d.H * d.k) + 15) & ~(uintptr_t)15);
  uint64_t* a_full = bars;               // [4]
  uint64_t* a_empty = bars + 4;          // [4]
  uint64_t* b_full = bars + 8;           // [2]
  uint64_t* b_empty = bars + 10;         // [2]
  uint64_t* d_full = bars + 12;          // [2]
  uint64_t* d_empty = bars + 14;         // [2]
  uint64_t* sel_free = bars + 16;        // epilogue threads are done with the selections copy
  uint64_t* sel_ready = bars + 17;       // the selections copy of the current work unit is complete
  uint32_t* tmem_slot = (uint32_t*)(bars + 18);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nfc = (d.M + 255) / 256;
  bool dead = false;

  if (threadIdx.x == 0) {
    for (int s = 0; s < 4; ++s) { mbar_init(&a_full[s], 1); mbar_init(&a_empty[s], 1); }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&b_full[s], 1); mbar_init(&b_empty[s], 1);
      mbar_init(&d_full[s], 1); mbar_init(&d_empty[s], 8);
    }
    mbar_init(sel_free, 256); mbar_init(sel_ready, 256);
    fence_barrier_init();
    tma_prefetch_desc(&mapAhat); tma_prefetch_desc(&mapWo);
  }
  if (warp == 1) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  pdl_trigger();                                         // programmatic dependent launch: the next kernel may become resident,
  if (threadIdx.x == 0) sh_stamp_resident(d.stamps, SH_K_O);
  pdl_wait();                                            // and this one starts consuming once the kernel before it has completed
  if (threadIdx.x == 0) sh_stamp_start(d.stamps, SH_K_O);

  if (warp == 0) {
    if (lane == 0) {
      int gh = 0, s = 0;                                    // running head counter, weight-ring stage
      uint32_t apar = 1;                                    // parity of a_empty[s] for the current ring pass
      for (int w = blockIdx.x; w < g.nwork && !dead; w += gridDim.x) {
        // (a 128-row tile of out is 128 consecutive tokens: with a cache in front of every sequence the
        //  chunk length is a multiple of 128, so a tile never straddles two sequences)
        const int row0 = sh_ctx_tok(d, (w / nfc) * 128), fc = w % nfc;
        for (int h = 0; h < d.H && !dead; ++h, ++gh) {
          const int bs = gh & 1;
          if (!mbar_wait(&b_empty[bs], ((gh >> 1) & 1) ^ 1, g.status, dead)) break;
          mbar_expect_tx(&b_full[bs], SM::B_BYTES);
#pragma unroll
          for (int c = 0; c < DB; ++c)
            tma_load_2d(sbase + b_off + bs * SM::B_BYTES + c * TBLK, &mapAhat, &b_full[bs], h * D + c * 64, row0);
          for (int e = 0; e < d.E && !dead; ++e) {
            // 256 feature rows of expert (h, e), one 64-column stage at a time; a box that runs past
            // the expert's rows (M not a multiple of 256) fetches rows whose columns are never stored
            for (int c = 0; c < DB; ++c) {
              if (!mbar_wait(&a_empty[s], apar, g.status, dead)) break;
              mbar_expect_tx(&a_full[s], SM::A_BYTES);
              tma_load_2d(sbase + a_off + s * SM::A_BYTES, &mapWo, &a_full[s], c * 64, (h * d.E + e) * d.M + fc * 256);
              if (++s == AS) { s = 0; apar ^= 1; }
            }
          }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc_f16(128, 256, 0, 0, 0);
      const uint32_t w_lo0 = desc_lo_k(sbase + a_off), t_lo0 = desc_lo_k(sbase + b_off);
      int gh = 0, ge = 0, s = 0;
      uint32_t apar = 0;                                    // parity of a_full[s] for the current ring pass
      for (int w = blockIdx.x; w < g.nwork && !dead; w += gridDim.x) {
        for (int h = 0; h < d.H && !dead; ++h, ++gh) {
          const int bs = gh & 1;
          if (!mbar_wait(&b_full[bs], (gh >> 1) & 1, g.status, dead)) break;
          const uint32_t t_lo = t_lo0 + bs * (SM::B_BYTES >> 4);
          for (int e = 0; e < d.E && !dead; ++e, ++ge) {
            const int buf = ge & 1;
            if (!mbar_wait(&d_empty[buf], ((ge >> 1) & 1) ^ 1, g.status, dead)) break;
            for (int c = 0; c < DB; ++c) {
              if (!mbar_wait(&a_full[s], apar, g.status, dead)) break;
              tc_fence_after();
              const uint32_t w_lo = w_lo0 + s * (SM::A_BYTES >> 4), tc_lo = t_lo + c * (TBLK >> 4);
#pragma unroll
              for (int k = 0; k < 4; ++k)
                umma_f16(tmem + buf * 256, desc_pack(tc_lo + 2 * k), desc_pack(w_lo + 2 * k), idesc, (c | k) != 0);
              umma_commit(&a_empty[s]);                     // this stage can load its next box
              if (++s == AS) { s = 0; apar ^= 1; }
            }
            if (dead) break;
            umma_commit(&d_full[buf]);
          }
          umma_commit(&b_empty[bs]);
        }
      }
    }
  } else {
    // ---- epilogue: thread = token x feature half; acc[f] = y[row0 + token, fc*256 + half*128 + f] ----
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
      const int row0 = (w / nfc) * 128, fc = w % nfc;      // rows of out
      const int nrows = min(128, sh_out_rows(d) - row0);
      const int tok0 = sh_ctx_tok(d, row0);                // their tokens (consecutive)
      // this tile's destination-side selections (contiguous in global memory) -> shared memory
      // (mbarriers with bounded waits rather than bar.sync, so that a thread that gave up cannot
      //  leave the others stuck)
      mbar_arrive(sel_free);                               // this thread is done with the previous copy
      if (!mbar_wait(sel_free, wpar, g.status, dead)) { ok = false; break; }
      {
        const int total = nrows * per_tok;
        const int* gi_ = g.idx + (size_t)tok0 * per_tok;
        const float* gg = g.gate + (size_t)tok0 * per_tok;
        for (int i = et; i < 128 * per_tok; i += 256) {
          s_idx[i] = i < total ? gi_[i] : -1;
          s_gt[i] = i < total ? gg[i] : 0.f;
        }
      }
      mbar_arrive(sel_ready);
      if (!mbar_wait(sel_ready, wpar, g.status, dead)) { ok = false; break; }
      float2 acc2[64];                                     // packed fp32 pairs: one FFMA2 per two features
#pragma unroll
      for (int f = 0; f < 64; ++f) acc2[f] = make_float2(0.f, 0.f);
      for (int h = 0; h < d.H && ok; ++h) {
        const int sel = (tok * d.H + h) * d.k;               // this token's selections for head h
        for (int e = 0; e < d.E; ++e, ++ge) {
          const int buf = ge & 1;
          float gv = 0.f;                                    // gate of expert e for this token (0: not selected)
          for (int j = 0; j < d.k; ++j)
            if (s_idx[sel + j] == e) gv = s_gt[sel + j];
          if (!mbar_wait(&d_full[buf], (ge >> 1) & 1, g.status, dead)) { ok = false; break; }
          tc_fence_after();
          const uint32_t ta = tmem + lane_off + buf * 256 + half * 128;
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            uint32_t v[32];
            tmem_ld32(ta + c * 32, v);
            tmem_ld_wait();
            if (c == 3) {                                    // everything is in registers: hand the buffer back
              tc_fence_before();
              __syncwarp();                                  // one arrival per warp: 256 arrivals on one barrier
              if (lane == 0) mbar_arrive(&d_empty[buf]);     // word would serialise in the LSU
            }
            const float2 g2 = make_float2(gv, gv);
#pragma unroll
            for (int f = 0; f < 16; ++f)
              acc2[c * 16 + f] = __ffma2_rn(g2, make_float2(__uint_as_float(v[2 * f]), __uint_as_float(v[2 * f + 1])), acc2[c * 16 + f]);
          }
        }
      }
      // store: the accumulators are token-per-lane; a 32 x 32 transpose through shared memory per
      // warp turns them into 128-byte row segments (a lane-per-row store is ~8 times slower)
      const int col0 = fc * 256 + half * 128;
      if (ok && col0 < d.M) {
        float* stg = reinterpret_cast<float*>(sgen + stg_off) + (warp - 2) * 1024;
        const size_t obase = (size_t)(row0 + q * 32) * d.M + col0;
        const int rows_here = min(32, nrows - q * 32);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          __syncwarp();
#pragma unroll
          for (int ch = 0; ch < 8; ++ch)                     // 16-byte chunk ch of row `lane` sits at chunk ch ^ (lane & 7)
            *reinterpret_cast<float4*>(stg + lane * 32 + ((ch ^ (lane & 7)) << 2)) =
                make_float4(acc2[c * 16 + 2 * ch].x, acc2[c * 16 + 2 * ch].y, acc2[c * 16 + 2 * ch + 1].x, acc2[c * 16 + 2 * ch + 1].y);
          __syncwarp();
          // 8 lanes cover one row's 128 bytes, a warp instruction four rows
#pragma unroll
          for (int r4 = 0; r4 < 32; r4 += 4) {
            const int r = r4 + (lane >> 3), ch = lane & 7;
            if (r < rows_here)
              oproj_put4(g.out, obase + (size_t)r * d.M + c * 32 + 4 * ch, *reinterpret_cast<const float4*>(stg + r * 32 + ((ch ^ (r & 7)) << 2)), g.out_f16);
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0) sh_stamp_end(d.stamps, SH_K_O);
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

}  // namespace shtc
