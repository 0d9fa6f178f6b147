// Causal softmax attention, one matrix per head (Eq. 1 with the autoregressive mask), on
// tcgen05: S = Q K^T and O += P V on the tensor pipe with accumulators in TMEM, K/V tiles
// staged by TMA, online softmax in base 2 on the CUDA cores (Q carries log2(e)/sqrt(D)).
//
// One CTA per (batch, head, 128-query tile); key/value tiles of 128 up to the diagonal.
// Warp roles (192 threads): warp 0 = TMA producer, warp 1 = TMEM owner + UMMA issuer,
// warps 2..5 = softmax (thread = query row = TMEM lane).
// TMEM columns: S double-buffered at 0 and 128, O accumulator at 256.
// The running maximum is only raised when a row's new maximum exceeds it by more than 8
// (in log2 units); O is then rescaled in TMEM.  P and l use the same (possibly stale)
// maximum, so the final O / l is exact up to rounding.
#pragma once
#include "sh_tc_prims.cuh"

namespace shtc {

struct TcAttnArgs {
  ShDims d;
  __half* ahat;          // [B*T, H, D]
  int* status;
  int balanced;          // two-tile kernel: pair query tile p with tile ntile-1-p (grid fits the GPU in one wave)
};

template <int D>
struct AttnSmem {
  static constexpr int Q_BYTES = 128 * D * 2;
  static constexpr int KV_BYTES = 128 * D * 2;
  static constexpr int P_BYTES = 128 * 128 * 2;
  static constexpr int Q_OFF = 0;
  static constexpr int K_OFF = Q_OFF + Q_BYTES;            // 2 stages
  static constexpr int V_OFF = K_OFF + 2 * KV_BYTES;       // 2 stages
  static constexpr int P_OFF = V_OFF + 2 * KV_BYTES;
  static constexpr int BAR_OFF = P_OFF + P_BYTES;
  static constexpr int TOTAL = BAR_OFF + 256 + 1024;
};

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
        "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
        "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

template <int D>
__global__ void __launch_bounds__(192)
sh_tc_attention_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
                       const __grid_constant__ CUtensorMap mapV, TcAttnArgs g) {
  using SM = AttnSmem<D>;
  constexpr int DB = D / 64;                 // 64-element column blocks of a Q/K/V tile
  constexpr uint32_t BLK = 128 * 128;        // bytes of one 128-row x 64-element block
  extern __shared__ unsigned char smem_raw[];
  const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* sgen = smem_raw + (sbase - smem_u32(smem_raw));
  uint64_t* bars = (uint64_t*)(sgen + SM::BAR_OFF);
  uint64_t* q_full = bars;
  uint64_t* k_full = bars + 1;    // [2]
  uint64_t* k_empty = bars + 3;   // [2]
  uint64_t* v_full = bars + 5;    // [2]
  uint64_t* v_empty = bars + 7;   // [2]
  uint64_t* s_full = bars + 9;    // [2]
  uint64_t* s_empty = bars + 11;  // [2]
  uint64_t* p_full = bars + 13;
  uint64_t* pv_done = bars + 14;
  uint32_t* tmem_slot = (uint32_t*)(bars + 15);

  const ShDims& d = g.d;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nq = (d.T + 127) / 128;
  const int BH = d.B * d.H;
  const int qt = nq - 1 - (int)(blockIdx.x / BH);        // heaviest query tiles first
  const int bh = blockIdx.x % BH;
  const int q0 = qt * 128;
  const int ntiles = qt + 1;
  bool dead = false;

  if (threadIdx.x == 0) {
    mbar_init(q_full, 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(&k_full[i], 1); mbar_init(&k_empty[i], 1);
      mbar_init(&v_full[i], 1); mbar_init(&v_empty[i], 1);
      mbar_init(&s_full[i], 1); mbar_init(&s_empty[i], 128);
    }
    mbar_init(p_full, 128);
    mbar_init(pv_done, 1);
    fence_barrier_init();
    tma_prefetch_desc(&mapQ); tma_prefetch_desc(&mapK); tma_prefetch_desc(&mapV);
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t tmem_o = tmem + 256;

  if (warp == 0) {
    if (lane == 0) {
      mbar_expect_tx(q_full, SM::Q_BYTES);
#pragma unroll
      for (int c = 0; c < DB; ++c) tma_load_3d(sbase + SM::Q_OFF + c * BLK, &mapQ, q_full, c * 64, q0, bh);
      for (int j = 0; j < ntiles; ++j) {
        const int s = j & 1;
        if (!mbar_wait(&k_empty[s], ((j >> 1) & 1) ^ 1, g.status, dead)) break;
        mbar_expect_tx(&k_full[s], SM::KV_BYTES);
#pragma unroll
        for (int c = 0; c < DB; ++c)
          tma_load_3d(sbase + SM::K_OFF + s * SM::KV_BYTES + c * BLK, &mapK, &k_full[s], c * 64, j * 128, bh);
        if (!mbar_wait(&v_empty[s], ((j >> 1) & 1) ^ 1, g.status, dead)) break;
        mbar_expect_tx(&v_full[s], SM::KV_BYTES);
#pragma unroll
        for (int c = 0; c < DB; ++c)
          tma_load_3d(sbase + SM::V_OFF + s * SM::KV_BYTES + c * BLK, &mapV, &v_full[s], c * 64, j * 128, bh);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc_s = make_idesc_f16(128, 128, 0, 0, 0);
      constexpr uint32_t idesc_pv = make_idesc_f16(128, D, 0, 0, 1);
      const uint32_t q_lo = desc_lo_k(sbase + SM::Q_OFF), k_lo0 = desc_lo_k(sbase + SM::K_OFF);
      const uint32_t p_lo = desc_lo_k(sbase + SM::P_OFF), v_lo0 = desc_lo_mn(sbase + SM::V_OFF, BLK);
      auto issue_s = [&](int j) {
        const int s = j & 1;
        const uint32_t k_lo = k_lo0 + s * (SM::KV_BYTES >> 4);
#pragma unroll
        for (int k = 0; k < D / 16; ++k) {
          const uint32_t koff = (k / 4) * (BLK >> 4) + 2 * (k % 4);
          umma_f16(tmem + s * 128, desc_pack(q_lo + koff), desc_pack(k_lo + koff), idesc_s, k != 0);
        }
        umma_commit(&k_empty[s]);
        umma_commit(&s_full[s]);
      };
      bool ok = mbar_wait(q_full, 0, g.status, dead) && mbar_wait(&k_full[0], 0, g.status, dead);
      if (ok) {
        tc_fence_after();
        issue_s(0);
      }
      for (int j = 0; ok && j < ntiles; ++j) {
        if (j + 1 < ntiles) {
          const int s1 = (j + 1) & 1;
          if (!mbar_wait(&k_full[s1], ((j + 1) >> 1) & 1, g.status, dead)) break;
          if (!mbar_wait(&s_empty[s1], (((j + 1) >> 1) & 1) ^ 1, g.status, dead)) break;
          tc_fence_after();
          issue_s(j + 1);
        }
        const int s = j & 1;
        if (!mbar_wait(&v_full[s], (j >> 1) & 1, g.status, dead)) break;
        if (!mbar_wait(p_full, j & 1, g.status, dead)) break;
        tc_fence_after();
        const uint32_t v_lo = v_lo0 + s * (SM::KV_BYTES >> 4);
#pragma unroll
        for (int k = 0; k < 8; ++k) {                       // 128 keys in steps of 16
          const uint32_t koff = (k / 4) * (BLK >> 4) + 2 * (k % 4);
          umma_f16(tmem_o, desc_pack(p_lo + koff), desc_pack(v_lo + k * (2048 >> 4)), idesc_pv, (j | k) != 0);
        }
        umma_commit(&v_empty[s]);
        umma_commit(pv_done);
      }
    }
  } else {
    // ---- softmax: thread = query row -----------------------------------------------------------
    const int q = warp & 3;
    const int r = q * 32 + lane;
    const uint32_t lane_off = (uint32_t)(q * 32) << 16;
    float m = -INFINITY, l = 0.f;
    const uint32_t prow = sbase + SM::P_OFF + r * 128;
    const uint32_t sw = (uint32_t)(r & 7);
    bool ok = true;
    for (int j = 0; j < ntiles; ++j) {
      const int b = j & 1;
      if (!mbar_wait(&s_full[b], (j >> 1) & 1, g.status, dead)) { ok = false; break; }
      tc_fence_after();
      uint32_t sv[128];
#pragma unroll
      for (int c = 0; c < 4; ++c) tmem_ld32(tmem + lane_off + b * 128 + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&sv[c * 32]));
      tmem_ld_wait();
      tc_fence_before();
      mbar_arrive(&s_empty[b]);
      float mx = -INFINITY;
      if (j == ntiles - 1) {                                 // diagonal tile: key c visible iff c <= r
#pragma unroll
        for (int c = 0; c < 128; ++c) {
          float v = (c <= r) ? __uint_as_float(sv[c]) : -INFINITY;
          sv[c] = __float_as_uint(v);
          mx = fmaxf(mx, v);
        }
      } else {
#pragma unroll
        for (int c = 0; c < 128; ++c) mx = fmaxf(mx, __uint_as_float(sv[c]));
      }
      float alpha = 1.f;
      bool raise = false;
      if (mx > m + 8.f) {
        alpha = fast_exp2(m - mx);                           // first tile: exp2(-inf) = 0
        m = mx;
        raise = j > 0;
      }
      float sum = 0.f;
      uint32_t pk[64];
#pragma unroll
      for (int c = 0; c < 64; ++c) {
        const float p0 = fast_exp2(__uint_as_float(sv[2 * c]) - m);
        const float p1 = fast_exp2(__uint_as_float(sv[2 * c + 1]) - m);
        sum += p0 + p1;
        __half2 h = __floats2half2_rn(p0, p1);
        pk[c] = *reinterpret_cast<uint32_t*>(&h);
      }
      l = l * alpha + sum;
      if (j > 0) {
        if (!mbar_wait(pv_done, (j - 1) & 1, g.status, dead)) { ok = false; break; }
        tc_fence_after();
        if (__any_sync(0xffffffffu, raise)) {                // rescale this warp's 32 rows of O
#pragma unroll
          for (int c = 0; c < D / 32; ++c) {
            uint32_t ov[32];
            tmem_ld32(tmem_o + lane_off + c * 32, ov);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 32; ++i) ov[i] = __float_as_uint(__uint_as_float(ov[i]) * alpha);
            tmem_st32(tmem_o + lane_off + c * 32, ov);
          }
          tmem_st_wait();
        }
      }
      // P tile, K-major, 128-byte swizzle: two blocks of 64 keys; 16-byte chunk ch of row r
      // sits at chunk position ch ^ (r & 7)
#pragma unroll
      for (int ch = 0; ch < 16; ++ch) {
        const uint32_t addr = prow + (ch >> 3) * BLK + (((uint32_t)(ch & 7) ^ sw) << 4);
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(pk[4 * ch]), "r"(pk[4 * ch + 1]),
                     "r"(pk[4 * ch + 2]), "r"(pk[4 * ch + 3]) : "memory");
      }
      fence_proxy_async_smem();
      tc_fence_before();
      mbar_arrive(p_full);
    }
    if (ok && mbar_wait(pv_done, (ntiles - 1) & 1, g.status, dead)) {
      tc_fence_after();
      const int t = q0 + r;
      const float inv = 1.f / l;
      const int bb = bh / d.H, hh = bh % d.H;
      __half* dst = g.ahat + (((size_t)bb * d.T + t) * d.H + hh) * D;
#pragma unroll
      for (int c = 0; c < D / 32; ++c) {
        uint32_t ov[32];
        tmem_ld32(tmem_o + lane_off + c * 32, ov);
        tmem_ld_wait();
        if (t < d.T) {
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            uint32_t w[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              __half2 h = __floats2half2_rn(__uint_as_float(ov[8 * i + 2 * u]) * inv, __uint_as_float(ov[8 * i + 2 * u + 1]) * inv);
              w[u] = *reinterpret_cast<uint32_t*>(&h);
            }
            *reinterpret_cast<uint4*>(dst + c * 32 + 8 * i) = make_uint4(w[0], w[1], w[2], w[3]);
          }
        }
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
