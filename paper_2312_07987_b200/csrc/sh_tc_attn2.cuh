// Causal softmax attention (Eq. 1 with the autoregressive mask), two 128-query tiles per CTA,
// with the probabilities P kept in tensor memory.
//
// Per query tile: S = Q K^T lands in 128 TMEM columns (fp32); the tile's softmax warps read
// their rows, and write P = exp2(S - m) back as packed fp16 into the first 64 of the SAME
// columns (tcgen05.st); the product O += P V then takes its A operand from tensor memory
// (tcgen05.mma with [a_tmem]).  The next S of the tile is issued right behind that product:
// the tensor pipe executes in issue order, so it overwrites P only after the product has read
// it, and no barrier is needed between the two.  Compared with P staged in shared memory
// (the earlier version of this kernel) this drops 16 shared-memory stores and a proxy fence per thread and step,
// the UMMA's shared-memory reads of P, and above all the single P buffer the two tiles had to
// take turns on; the two tiles now interleave freely: while one tile's softmax runs, the pipe
// works for the other.
//
// CTA = (batch, head, two query tiles); key/value tiles of 128 up to the diagonal of each
// query tile.  Warp roles (320 threads): warp 0 = TMA producer, warp 1 = TMEM owner + UMMA
// issuer, warps 2..5 / 6..9 = softmax of query tile 0 / 1 (thread = query row = TMEM lane).
// TMEM columns: S0 / P0 at 0, S1 / P1 at 128, O0 at 256, O1 at 384.  Running maximum and
// rescale: raise only by more than 8 in log2 units; O rescaled in TMEM when that happens.
#pragma once
#include "sh_tc_prims.cuh"

namespace shtc {

struct TcAttnArgs {
  ShDims d;
  __half* ahat;          // [B*T, H, D]
  int* status;
  int balanced;          // pair query tile p with tile ntile-1-p (causal mask, grid fits the GPU in one wave)
  const __half* bias;    // [B, H, T - Tc, T] added to the scores (Transformer-XL position and content-bias terms, log2 units), or nullptr
};

// Adds 64 or 128 consecutive bias values (fp16, 16-byte aligned run of this query row) to the scores in sv.
template <int N>
__device__ __forceinline__ void add_score_bias(uint32_t* sv, const __half* run) {
#pragma unroll
  for (int i = 0; i < N / 8; ++i) {
    const uint4 b4 = __ldg(reinterpret_cast<const uint4*>(run) + i);
    const __half2* h2 = reinterpret_cast<const __half2*>(&b4);
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const float2 f = __half22float2(h2[u]);
      sv[8 * i + 2 * u] = __float_as_uint(__uint_as_float(sv[8 * i + 2 * u]) + f.x);
      sv[8 * i + 2 * u + 1] = __float_as_uint(__uint_as_float(sv[8 * i + 2 * u + 1]) + f.y);
    }
  }
}

template <int D>
struct Attn2Smem {
  static constexpr int T_BYTES = 128 * D * 2;            // one 128-row tile of Q, K or V
  static constexpr int Q_OFF = 0;                          // 2 tiles
  static constexpr int K_OFF = Q_OFF + 2 * T_BYTES;        // 2 stages
  static constexpr int V_OFF = K_OFF + 2 * T_BYTES;        // 2 stages
  static constexpr int BAR_OFF = V_OFF + 2 * T_BYTES;
  static constexpr int TOTAL = BAR_OFF + 256 + 1024;
};

template <int D>
__global__ void __launch_bounds__(320, 1)
sh_tc_attention2_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
                        const __grid_constant__ CUtensorMap mapV, TcAttnArgs g) {
  using SM = Attn2Smem<D>;
  constexpr int DB = D / 64;
  constexpr uint32_t BLK = 128 * 128;
  extern __shared__ unsigned char smem_raw[];
  const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* sgen = smem_raw + (sbase - smem_u32(smem_raw));
  uint64_t* bars = (uint64_t*)(sgen + SM::BAR_OFF);
  uint64_t* q_full = bars;
  uint64_t* k_full = bars + 1;    // [2]
  uint64_t* k_empty = bars + 3;   // [2]
  uint64_t* v_full = bars + 5;    // [2]
  uint64_t* v_empty = bars + 7;   // [2]
  uint64_t* s_full = bars + 9;    // [2] per query tile: S of the step is in TMEM
  uint64_t* p_full = bars + 11;   // [2] per query tile: P of the step is in TMEM (one arrival per softmax warp)
  uint64_t* pv_done = bars + 13;  // [2] per query tile: the step's P V product has completed
  uint32_t* tmem_slot = (uint32_t*)(bars + 15);

  const ShDims& d = g.d;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int BH = d.B * d.H;
  const int bh = blockIdx.x % BH;
  // The two 128-query tiles of this CTA.  Saturated grid: adjacent tiles, heaviest pairs first (the
  // most steps in which both tiles share a K/V stage).  Grid that fits the GPU in one wave
  // (g.balanced): tile p with tile ntile-1-p, so that under the causal mask every CTA has the same
  // number of tile-steps and the kernel ends when the average CTA ends, not the heaviest.
  // (with a Transformer-XL cache of d.Tc tokens - a multiple of 128 - in front of the sequence, the
  //  query tiles start behind it; the key tiles start at 0 as ever)
  const int ntile = (d.T + 127) / 128, t_first = d.Tc / 128;
  const int nq = (ntile - t_first + 1) / 2;
  const int pr = (int)(blockIdx.x / BH);
  int ta, tb;
  if (g.balanced) { ta = t_first + pr; tb = ntile - 1 - pr; }
  else { ta = t_first + 2 * (nq - 1 - pr); tb = ta + 1; }
  const bool has_b = tb < ntile && tb != ta;
  const int qrow[2] = {ta * 128, tb * 128};
  // key tiles each query tile attends to: up to its diagonal tile, or (d.causal == 0) all of them
  const int nkt = ntile;
  const int n0 = d.causal ? ta + 1 : nkt;                // steps of query tile 0
  const int n1 = has_b ? (d.causal ? tb + 1 : nkt) : 0;  // steps of query tile 1 (0: no such tile)
  const int nsteps = n1 > n0 ? n1 : n0;
  bool dead = false;

  if (threadIdx.x == 0) {
    mbar_init(q_full, 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(&k_full[i], 1); mbar_init(&k_empty[i], 1);
      mbar_init(&v_full[i], 1); mbar_init(&v_empty[i], 1);
      mbar_init(&s_full[i], 1); mbar_init(&p_full[i], 4);
      mbar_init(&pv_done[i], 1);
    }
    fence_barrier_init();
    tma_prefetch_desc(&mapQ); tma_prefetch_desc(&mapK); tma_prefetch_desc(&mapV);
  }
  if (warp == 1) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  if (threadIdx.x == 0) sh_stamp_resident(d.stamps, SH_K_ATTN);
  pdl_wait();                                            // programmatic dependent launch: consume once the kernel before this one has completed;
  pdl_trigger();                                         // only then may the next kernel become resident: what it does ahead of ITS wait (the
                                                         // output projection reads the selections there) sees every earlier kernel of the pass complete
  if (threadIdx.x == 0) sh_stamp_start(d.stamps, SH_K_ATTN);

  if (warp == 0) {
    if (lane == 0) {
      mbar_expect_tx(q_full, (n1 > 0 ? 2 : 1) * SM::T_BYTES);
      for (int t = 0; t < (n1 > 0 ? 2 : 1); ++t)
#pragma unroll
        for (int c = 0; c < DB; ++c)
          tma_load_3d(sbase + SM::Q_OFF + t * SM::T_BYTES + c * BLK, &mapQ, q_full, c * 64, qrow[t], bh);
      for (int j = 0; j < nsteps; ++j) {
        const int s = j & 1;
        if (!mbar_wait(&k_empty[s], ((j >> 1) & 1) ^ 1, g.status, dead)) break;
        mbar_expect_tx(&k_full[s], SM::T_BYTES);
#pragma unroll
        for (int c = 0; c < DB; ++c)
          tma_load_3d(sbase + SM::K_OFF + s * SM::T_BYTES + c * BLK, &mapK, &k_full[s], c * 64, j * 128, bh);
        if (!mbar_wait(&v_empty[s], ((j >> 1) & 1) ^ 1, g.status, dead)) break;
        mbar_expect_tx(&v_full[s], SM::T_BYTES);
#pragma unroll
        for (int c = 0; c < DB; ++c)
          tma_load_3d(sbase + SM::V_OFF + s * SM::T_BYTES + c * BLK, &mapV, &v_full[s], c * 64, j * 128, bh);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc_s = make_idesc_f16(128, 128, 0, 0, 0);
      constexpr uint32_t idesc_pv = make_idesc_f16(128, D, 0, 0, 1);
      const uint32_t q_lo0 = desc_lo_k(sbase + SM::Q_OFF), k_lo0 = desc_lo_k(sbase + SM::K_OFF);
      const uint32_t v_lo0 = desc_lo_mn(sbase + SM::V_OFF, BLK);
      const int nt[2] = {n0, n1};
      auto issue_s = [&](int t, int j) {                     // S_t = Q_t K_j^T
        const uint32_t q_lo = q_lo0 + t * (SM::T_BYTES >> 4), k_lo = k_lo0 + (j & 1) * (SM::T_BYTES >> 4);
#pragma unroll
        for (int k = 0; k < D / 16; ++k) {
          const uint32_t koff = (k / 4) * (BLK >> 4) + 2 * (k % 4);
          umma_f16(tmem + t * 128, desc_pack(q_lo + koff), desc_pack(k_lo + koff), idesc_s, k != 0);
        }
        umma_commit(&s_full[t]);
      };
      bool ok = mbar_wait(q_full, 0, g.status, dead) && mbar_wait(&k_full[0], 0, g.status, dead);
      if (ok) {
        tc_fence_after();
        issue_s(0, 0);
        if (n1 > 0) issue_s(1, 0);
        umma_commit(&k_empty[0]);
      }
      for (int j = 0; ok && j < nsteps; ++j) {
        const int s = j & 1;
        const bool more = j + 1 < nsteps;
        if (more && !mbar_wait(&k_full[(j + 1) & 1], ((j + 1) >> 1) & 1, g.status, dead)) break;
        if (!mbar_wait(&v_full[s], (j >> 1) & 1, g.status, dead)) break;
        const uint32_t v_lo = v_lo0 + s * (SM::T_BYTES >> 4);
        for (int t = 0; t < 2 && ok; ++t) {
          if (j >= nt[t]) continue;
          if (!mbar_wait(&p_full[t], j & 1, g.status, dead)) { ok = false; break; }
          tc_fence_after();
#pragma unroll
          for (int k = 0; k < 8; ++k)                       // 128 keys in steps of 16: A = P_t from tensor memory
            umma_f16_tmem_a(tmem + 256 + t * 128, tmem + t * 128 + 8 * k, desc_pack(v_lo + k * (2048 >> 4)), idesc_pv, (j | k) != 0);
          umma_commit(&pv_done[t]);
          // the tile's next S goes right behind: executed in issue order, it overwrites P_t only
          // after the product above has read it
          if (j + 1 < nt[t]) issue_s(t, j + 1);
        }
        if (!ok) break;
        umma_commit(&v_empty[s]);
        if (more) umma_commit(&k_empty[(j + 1) & 1]);
      }
    }
  } else {
    // ---- softmax: warps 2..5 own query tile 0, warps 6..9 query tile 1; thread = query row ------
    const int t = (warp - 2) >> 2;
    const int n = t == 0 ? n0 : n1;
    const int q = warp & 3;
    const int r = q * 32 + lane;
    const uint32_t lane_off = (uint32_t)(q * 32) << 16;
    const uint32_t tmem_s = tmem + t * 128, tmem_o = tmem + 256 + t * 128;
    float m = -INFINITY, l = 0.f;
    bool ok = true;
    for (int j = 0; j < n; ++j) {
      if (!mbar_wait(&s_full[t], j & 1, g.status, dead)) { ok = false; break; }
      tc_fence_after();
      uint32_t sv[128];
#pragma unroll
      for (int c = 0; c < 4; ++c) tmem_ld32(tmem_s + lane_off + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&sv[c * 32]));
      tmem_ld_wait();
      if (g.bias && qrow[t] + r < d.T)
        add_score_bias<128>(sv, g.bias + ((size_t)bh * (d.T - d.Tc) + (qrow[t] - d.Tc + r)) * d.T + j * 128);
      if (j == n - 1) {
        // last tile: the diagonal one (key c visible iff c <= r), or without the causal mask the
        // tile that holds the end of the sequence (keys past it were zero-filled by the loads)
        const int cmax = d.causal ? r : d.T - 1 - j * 128;
#pragma unroll
        for (int c = 0; c < 128; ++c)
          if (c > cmax) sv[c] = 0xff800000u;                 // -inf
      }
      float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};   // four independent chains
#pragma unroll
      for (int c = 0; c < 128; c += 4) {
        mx4[0] = fmaxf(mx4[0], __uint_as_float(sv[c]));
        mx4[1] = fmaxf(mx4[1], __uint_as_float(sv[c + 1]));
        mx4[2] = fmaxf(mx4[2], __uint_as_float(sv[c + 2]));
        mx4[3] = fmaxf(mx4[3], __uint_as_float(sv[c + 3]));
      }
      const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
      float alpha = 1.f;
      bool raise = false;
      if (mx > m + 8.f) {
        alpha = fast_exp2(m - mx);                           // first tile: exp2(-inf) = 0
        m = mx;
        raise = j > 0;
      }
      float2 sum2[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
      const float2 negm = make_float2(-m, -m);
      uint32_t pk[64];
#pragma unroll
      for (int c = 0; c < 64; ++c) {
        const float2 x = __fadd2_rn(make_float2(__uint_as_float(sv[2 * c]), __uint_as_float(sv[2 * c + 1])), negm);
        float2 pr;
        pr.x = fast_exp2(x.x);
        pr.y = fast_exp2(x.y);
        sum2[c & 1] = __fadd2_rn(sum2[c & 1], pr);
        __half2 h = __floats2half2_rn(pr.x, pr.y);
        pk[c] = *reinterpret_cast<uint32_t*>(&h);
      }
      l = l * alpha + ((sum2[0].x + sum2[0].y) + (sum2[1].x + sum2[1].y));
      if (j > 0 && __any_sync(0xffffffffu, raise)) {         // rescale this warp's 32 rows of O
        // (S of this step was issued behind the previous P V product, so that product has completed)
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
          uint32_t ov[32];
          tmem_ld32(tmem_o + lane_off + c * 32, ov);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 32; ++i) ov[i] = __float_as_uint(__uint_as_float(ov[i]) * alpha);
          tmem_st32(tmem_o + lane_off + c * 32, ov);
        }
      }
      // P (packed fp16 pairs) over the first 64 columns of this row's S
      tmem_st32(tmem_s + lane_off, *reinterpret_cast<uint32_t(*)[32]>(&pk[0]));
      tmem_st32(tmem_s + lane_off + 32, *reinterpret_cast<uint32_t(*)[32]>(&pk[32]));
      tmem_st_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&p_full[t]);
    }
    if (ok && n > 0 && mbar_wait(&pv_done[t], (n - 1) & 1, g.status, dead)) {
      tc_fence_after();
      const int tq = qrow[t] + r;
      const float inv = 1.f / l;
      const int bb = bh / d.H, hh = bh % d.H;
      __half* dst = g.ahat + (((size_t)bb * d.T + tq) * d.H + hh) * D;
#pragma unroll
      for (int c = 0; c < D / 32; ++c) {
        uint32_t ov[32];
        tmem_ld32(tmem_o + lane_off + c * 32, ov);
        tmem_ld_wait();
        if (tq < d.T) {
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
  if (threadIdx.x == 0) sh_stamp_end(d.stamps, SH_K_ATTN);
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

}  // namespace shtc
