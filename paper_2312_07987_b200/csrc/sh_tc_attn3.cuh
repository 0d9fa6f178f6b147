// Causal softmax attention (Eq. 1 with the autoregressive mask), two 128-query tiles per CTA, the
// 128 keys of a step handled as TWO independently pipelined halves of 64.
//
// Per query tile and key half x: S_x = Q K_x^T lands in 64 TMEM columns (fp32); the tile's softmax
// warps read their rows and write P_x = exp2(S_x - m) back as packed fp16 over the first 32 of the
// SAME columns; the product O += P_x V_x takes its A operand from tensor memory; the half's next S
// (next step) is issued right behind that product - the tensor pipe executes in issue order, so it
// overwrites P_x only after the product has read it.
//
// Why halves: with one 128-key S per tile and step (sh_tc_attention2_kernel) the loop of a tile is a
// chain - S ready -> softmax (~2000 cycles) -> P ready -> P V and the next S -> S ready.  With halves
// the softmax of half b runs while the pipe does P_a V_a and the next S_a, and vice versa: the same
// 256 TMEM columns per tile (S_a 64 + S_b 64 + O 128), the same K / V stages of 128 keys, twice as
// many (half as long) hand-overs.  Measured: the chain of a SHORT sequence gets shorter (T = 512:
// 13.4 -> 11.5 us), but S_x is eight UMMAs of N = 64 - 32 cycles of tensor time each against the ~60
// cycles one thread needs to issue one - so at T = 4096 the issuing thread bounds the loop (72 -> 97 us).
// The layer therefore uses this kernel up to 1024 keys per query tile and the whole-S kernel beyond.
//
// The running maximum is only raised when a row's new maximum exceeds it by more than 8 (log2
// units); O is then rescaled in TMEM.  A product of the OTHER half may still be accumulating into O
// at that moment (it is issued when its P arrives, which can be after this half's S completed), so a
// warp that rescales first waits for the last product issued for its tile (pv_done counts them).
//
// CTA = (batch, head, two query tiles); warp roles (320 threads): warp 0 = TMA producer, warp 1 =
// TMEM owner + UMMA issuer, warps 2..5 / 6..9 = softmax of query tile 0 / 1 (thread = query row).
// TMEM columns: tile t: S_a at t*128, S_b at t*128 + 64, O at 256 + t*128.
#pragma once
#include "sh_tc_attn2.cuh"

namespace shtc {

template <int D>
struct Attn3Smem {
  static constexpr int T_BYTES = 128 * D * 2;            // one 128-row tile of Q, K or V
  static constexpr int Q_OFF = 0;                          // 2 tiles
  static constexpr int K_OFF = Q_OFF + 2 * T_BYTES;        // 2 stages
  static constexpr int V_OFF = K_OFF + 2 * T_BYTES;        // 2 stages
  static constexpr int BAR_OFF = V_OFF + 2 * T_BYTES;
  static constexpr int TOTAL = BAR_OFF + 256 + 1024;
};

template <int D>
__global__ void __launch_bounds__(320, 1)
sh_tc_attention3_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
                        const __grid_constant__ CUtensorMap mapV, TcAttnArgs g) {
  using SM = Attn3Smem<D>;
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
  uint64_t* s_full = bars + 9;    // [2 tiles][2 halves]: S_x of the step is in TMEM
  uint64_t* p_full = bars + 13;   // [2][2]: P_x of the step is in TMEM (one arrival per softmax warp)
  uint64_t* pv_done = bars + 17;  // [2] per query tile: one more P V product has completed (two per step)
  uint32_t* tmem_slot = (uint32_t*)(bars + 19);
  uint64_t* o_done = bars + 20;   // [2] per query tile: its last product has completed (one phase per launch)

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
      mbar_init(&pv_done[i], 1);
      mbar_init(&o_done[i], 1);
    }
    for (int i = 0; i < 4; ++i) { mbar_init(&s_full[i], 1); mbar_init(&p_full[i], 4); }
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
      constexpr uint32_t idesc_s = make_idesc_f16(128, 64, 0, 0, 0);
      constexpr uint32_t idesc_pv = make_idesc_f16(128, D, 0, 0, 1);
      const uint32_t q_lo0 = desc_lo_k(sbase + SM::Q_OFF), k_lo0 = desc_lo_k(sbase + SM::K_OFF);
      const uint32_t v_lo0 = desc_lo_mn(sbase + SM::V_OFF, BLK);
      const int nt[2] = {n0, n1};
      // S_x of tile t for step j: Q_t times the keys 64x .. 64x+63 of stage j & 1 (rows 64.. of a K-major
      // 128-byte-swizzled tile start 8 row groups = 8192 bytes into each 64-column block)
      auto issue_s = [&](int t, int x, int j) {
        const uint32_t q_lo = q_lo0 + t * (SM::T_BYTES >> 4), k_lo = k_lo0 + (j & 1) * (SM::T_BYTES >> 4) + x * (8192 >> 4);
#pragma unroll
        for (int k = 0; k < D / 16; ++k) {
          const uint32_t koff = (k / 4) * (BLK >> 4) + 2 * (k % 4);
          umma_f16(tmem + t * 128 + x * 64, desc_pack(q_lo + koff), desc_pack(k_lo + koff), idesc_s, k != 0);
        }
        umma_commit(&s_full[t * 2 + x]);
      };
      bool ok = mbar_wait(q_full, 0, g.status, dead) && mbar_wait(&k_full[0], 0, g.status, dead);
      if (ok) {
        tc_fence_after();
        issue_s(0, 0, 0);
        if (n1 > 0) issue_s(1, 0, 0);
        issue_s(0, 1, 0);
        if (n1 > 0) issue_s(1, 1, 0);
        umma_commit(&k_empty[0]);
      }
      for (int j = 0; ok && j < nsteps; ++j) {
        const int s = j & 1;
        const bool more = j + 1 < nsteps;
        if (more && !mbar_wait(&k_full[(j + 1) & 1], ((j + 1) >> 1) & 1, g.status, dead)) break;
        if (!mbar_wait(&v_full[s], (j >> 1) & 1, g.status, dead)) break;
        const uint32_t v_lo = v_lo0 + s * (SM::T_BYTES >> 4);
        for (int x = 0; x < 2 && ok; ++x) {
          for (int t = 0; t < 2 && ok; ++t) {
            if (j >= nt[t]) continue;
            if (!mbar_wait(&p_full[t * 2 + x], j & 1, g.status, dead)) { ok = false; break; }
            tc_fence_after();
#pragma unroll
            for (int k = 0; k < 4; ++k)                     // the half's 64 keys in steps of 16: A = P_x from tensor memory
              umma_f16_tmem_a(tmem + 256 + t * 128, tmem + t * 128 + x * 64 + 8 * k, desc_pack(v_lo + (4 * x + k) * (2048 >> 4)), idesc_pv,
                              (j | x | k) != 0);
            umma_commit(&pv_done[t]);
            if (x == 1 && j == nt[t] - 1) umma_commit(&o_done[t]);   // the tile's O is final when this completes
            // the half's next S goes right behind: executed in issue order, it overwrites P_x only after
            // the product above has read it
            if (j + 1 < nt[t]) issue_s(t, x, j + 1);
          }
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
    const uint32_t tmem_o = tmem + 256 + t * 128;
    float m = -INFINITY, l = 0.f;
    bool ok = true;
    int npv = 0;                                           // products issued for this tile before the half being processed
    for (int j = 0; j < n && ok; ++j) {
#pragma unroll
      for (int x = 0; x < 2; ++x, ++npv) {
        const uint32_t tmem_s = tmem + t * 128 + x * 64;
        if (!mbar_wait(&s_full[t * 2 + x], j & 1, g.status, dead)) { ok = false; break; }
        tc_fence_after();
        uint32_t sv[64];
        tmem_ld32(tmem_s + lane_off, *reinterpret_cast<uint32_t(*)[32]>(&sv[0]));
        tmem_ld32(tmem_s + lane_off + 32, *reinterpret_cast<uint32_t(*)[32]>(&sv[32]));
        tmem_ld_wait();
        if (g.bias && qrow[t] + r < d.T)
          add_score_bias<64>(sv, g.bias + ((size_t)bh * (d.T - d.Tc) + (qrow[t] - d.Tc + r)) * d.T + j * 128 + 64 * x);
        if (j == n - 1) {
          // last tile: the diagonal one (key c visible iff c <= r), or without the causal mask the
          // tile that holds the end of the sequence (keys past it were zero-filled by the loads)
          const int cmax = (d.causal ? r : d.T - 1 - j * 128) - 64 * x;
#pragma unroll
          for (int c = 0; c < 64; ++c)
            if (c > cmax) sv[c] = 0xff800000u;               // -inf
        }
        float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};   // four independent chains
#pragma unroll
        for (int c = 0; c < 64; c += 4) {
          mx4[0] = fmaxf(mx4[0], __uint_as_float(sv[c]));
          mx4[1] = fmaxf(mx4[1], __uint_as_float(sv[c + 1]));
          mx4[2] = fmaxf(mx4[2], __uint_as_float(sv[c + 2]));
          mx4[3] = fmaxf(mx4[3], __uint_as_float(sv[c + 3]));
        }
        const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
        float alpha = 1.f;
        bool raise = false;
        if (mx > m + 8.f) {
          alpha = fast_exp2(m - mx);                         // first half: exp2(-inf) = 0
          m = mx;
          raise = npv > 0;
        }
        float2 sum2[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
        const float2 negm = make_float2(-m, -m);
        uint32_t pk[32];
#pragma unroll
        for (int c = 0; c < 32; ++c) {
          const float2 xx = __fadd2_rn(make_float2(__uint_as_float(sv[2 * c]), __uint_as_float(sv[2 * c + 1])), negm);
          float2 pr2;
          pr2.x = fast_exp2(xx.x);
          pr2.y = fast_exp2(xx.y);
          sum2[c & 1] = __fadd2_rn(sum2[c & 1], pr2);
          __half2 h = __floats2half2_rn(pr2.x, pr2.y);
          pk[c] = *reinterpret_cast<uint32_t*>(&h);
        }
        l = l * alpha + ((sum2[0].x + sum2[0].y) + (sum2[1].x + sum2[1].y));
        if (npv > 0 && __any_sync(0xffffffffu, raise)) {     // rescale this warp's 32 rows of O
          // every product issued for this tile so far must have left O alone: the other half's may have
          // been issued after this half's S completed.  pv_done has had npv arrivals when they are done.
          if (!mbar_wait(&pv_done[t], (npv - 1) & 1, g.status, dead)) { ok = false; break; }
          tc_fence_after();
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
        // P_x (packed fp16 pairs) over the first 32 columns of this row's S_x
        tmem_st32(tmem_s + lane_off, pk);
        tmem_st_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&p_full[t * 2 + x]);
      }
    }
    // The tile's last product.  (Not a parity wait on pv_done: after its last arrival on p_full a warp
    // can be late - the tail below is cold code - and find BOTH of the last two products complete; a
    // parity wait for the first of them would then wait for a phase that never comes.  Seen as a 1 s
    // time-out once in ~500 passes at T = 512 with 160 (batch, head) pairs.)
    if (ok && n > 0 && mbar_wait(&o_done[t], 0, g.status, dead)) {
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
