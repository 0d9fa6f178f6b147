// CUDA-core (FFMA) kernels: the whole fp32 configuration runs on these; the gate, top-k and
// bucket-sort kernels also serve the bf16 configuration.
#pragma once
#include "sh_internal.cuh"

// ---------------------------------------------------------------------------------------
// Weight repack: out[b*obs + c*ors + r*oes] = in[b*rows*cols + r*cols + c]  (a batched
// transpose with free output strides), with type conversion.
// ---------------------------------------------------------------------------------------
template <typename TI, typename TO>
__global__ void sh_repack_kernel(const TI* __restrict__ in, TO* __restrict__ out, int batch, int rows,
                                 int cols, long obs, long ors, long oes) {
  long total = (long)batch * rows * cols;
  for (long i = blockIdx.x * (long)blockDim.x + threadIdx.x; i < total; i += (long)gridDim.x * blockDim.x) {
    int r = (int)(i % rows);
    long t = i / rows;
    int c = (int)(t % cols);
    int b = (int)(t / cols);
    float v = sh_to_float<TI>(in[((long)b * rows + r) * cols + c]);
    out[b * obs + c * ors + r * oes] = sh_from_float<TO>(v);
  }
}

// ---------------------------------------------------------------------------------------
// Gate: z = x W (+ b) per (side, head), sigmoid, top-k with lower-index-wins, per-block
// histogram of the selections (Sec. 2.2: s = sigmoid(x W_S), E = arg top-k).
// One warp per token; lane e owns expert e's logit during selection.
// Wg is [G, M] (one row per gate column g = (side*H + h)*E + e).
// ---------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256)
sh_gate_topk_kernel(const T* __restrict__ x, const T* __restrict__ Wg, const float* __restrict__ gbias,
                    int* __restrict__ idx, float* __restrict__ gate, int* __restrict__ blockcnt, ShDims d) {
  extern __shared__ int s_hist[];            // [G]
  const int nb = d.G;
  for (int i = threadIdx.x; i < nb; i += blockDim.x) s_hist[i] = 0;
  __syncthreads();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
  const int tok0 = blockIdx.x * SH_TILE_ROWS;
  for (int tt = warp; tt < SH_TILE_ROWS; tt += nwarps) {
    const int t = tok0 + tt;
    if (t >= d.N) break;
    const T* xr = x + (size_t)t * d.M;
    for (int grp = 0; grp < d.sides * d.H; ++grp) {
      float z = 0.f;                         // lane e keeps logit e
      for (int e0 = 0; e0 < d.E; e0 += 4) {
        float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
        const T* w0 = Wg + (size_t)(grp * d.E + e0) * d.M;
        const bool h1 = e0 + 1 < d.E, h2 = e0 + 2 < d.E, h3 = e0 + 3 < d.E;
        for (int m = lane; m < d.M; m += 32) {
          float xv = sh_to_float<T>(xr[m]);
          a0 = fmaf(xv, sh_to_float<T>(w0[m]), a0);
          if (h1) a1 = fmaf(xv, sh_to_float<T>(w0[d.M + m]), a1);
          if (h2) a2 = fmaf(xv, sh_to_float<T>(w0[2 * (size_t)d.M + m]), a2);
          if (h3) a3 = fmaf(xv, sh_to_float<T>(w0[3 * (size_t)d.M + m]), a3);
        }
#pragma unroll
        for (int s = 16; s > 0; s >>= 1) {
          a0 += __shfl_xor_sync(0xffffffffu, a0, s);
          a1 += __shfl_xor_sync(0xffffffffu, a1, s);
          a2 += __shfl_xor_sync(0xffffffffu, a2, s);
          a3 += __shfl_xor_sync(0xffffffffu, a3, s);
        }
        if (lane == e0) z = a0;
        if (lane == e0 + 1) z = a1;
        if (lane == e0 + 2) z = a2;
        if (lane == e0 + 3) z = a3;
      }
      if (lane < d.E) z += gbias[grp * d.E + lane];
      int rank = 0;
      for (int e = 0; e < d.E; ++e) {
        float ze = __shfl_sync(0xffffffffu, z, e);
        rank += (ze > z || (ze == z && e < lane)) ? 1 : 0;
      }
      if (lane < d.E && rank < d.k) {
        const int side = grp / d.H, h = grp % d.H;
        size_t o = (((size_t)side * d.N + t) * d.H + h) * d.k + rank;
        idx[o] = lane;
        gate[o] = 1.f / (1.f + expf(-z));
        atomicAdd(&s_hist[grp * d.E + lane], 1);
      }
    }
  }
  __syncthreads();
  for (int i = threadIdx.x; i < nb; i += blockDim.x) blockcnt[(size_t)blockIdx.x * nb + i] = s_hist[i];
}

// ---------------------------------------------------------------------------------------
// Bucket sort (one launch).  Block b owns tokens [b*128, b*128+128).  From the per-block
// selection histograms every block derives, per bucket (side, head, expert): the number of
// selections in earlier blocks and the bucket total; from the totals the per-head exclusive
// scan over experts.  It then places its own tokens, in ascending order, behind those of the
// earlier blocks (a stable counting sort: within a bucket tokens stay ascending).  Block 0
// also writes the offsets array and the row-tile table of the grouped GEMMs (tiles of
// d.tile_rows_src rows on the source side, 128 on the destination side).
// Dynamic shared memory: 128*H*k*2*8 bytes (the block's idx and gate values, both sides)
// + (6*G + 8) * 4 bytes.
// ---------------------------------------------------------------------------------------
// The block's part of the sort, for `nthreads` = 128 * GS threads numbered tid; `sync` is a barrier
// over exactly those threads.  have_sel: the block's idx / gate values are already in the
// shared-memory arrays (the fused gate kernel put them there), otherwise they are copied from idx /
// gate.  blockcnt must be complete for ALL blocks.
template <class Sync>
static __device__ __forceinline__ void sh_sort_block(const int* __restrict__ idx, const float* __restrict__ gate, const int* __restrict__ blockcnt,
                                                     int* __restrict__ offsets, int* __restrict__ lists, float* __restrict__ lgate,
                                                     ShTile* __restrict__ tiles, int* __restrict__ ntiles, const ShDims& d,
                                                     int* s_sort, int tid, int nthreads, int blk, bool have_sel, Sync sync) {
  const int nb = d.G;
  const int per_tok = d.H * d.k;
  int* s_pre = s_sort;                 // [nb] selections of this bucket in earlier blocks
  int* s_tot = s_pre + nb;             // [nb] bucket totals
  int* s_off = s_tot + nb;             // [nb] start of the bucket inside its (side, head) list
  int* s_tbase = s_off + nb;           // [nb] first tile of the bucket (block 0 only)
  int* s_wcnt = s_tbase + nb;          // [nb][4] per-warp counts of this block's tokens
  int* s_idx = s_wcnt + 4 * nb;        // [2][128*per_tok]
  float* s_gt = (float*)(s_idx + 2 * 128 * per_tok);
  const int lane = tid & 31;
  const int tl = tid & 127, gs = tid >> 7, GS = nthreads >> 7;
  const int twarp = tl >> 5;           // warp index among the 4 warps of a slice
  const int tok0 = blk * SH_TILE_ROWS;
  const int nrows = min(SH_TILE_ROWS, d.N - tok0);
  for (int i = tid; i < 2 * nb; i += nthreads) s_pre[i] = 0;   // s_pre and s_tot
  for (int i = tid; i < 4 * nb; i += nthreads) s_wcnt[i] = 0;  // (k = 1: only the buckets a warp meets are written)
  // bucket b = tid % nb; the thread sums the blocks part, part + parts, ... in registers.  These
  // loads do not depend on the selections copy below, so both are in flight together.
  int my_b = -1, my_tot = 0, my_pre = 0;
  {
    const int parts = max(1, nthreads / nb);
    if (nb <= nthreads) {
      if (tid / nb < parts) {
        my_b = tid % nb;
        const int part = tid / nb;
#pragma unroll 8
        for (int bk = part; bk < d.nblk; bk += parts) {
          const int c = blockcnt[(size_t)bk * nb + my_b];
          my_tot += c;
          my_pre += bk < blk ? c : 0;
        }
      }
    }
  }
  for (int side = 0; side < (have_sel ? 0 : d.sides); ++side) {  // this block's selections
    const size_t base = ((size_t)side * d.N + tok0) * per_tok;
    for (int i = tid; i < nrows * per_tok; i += nthreads) {
      s_idx[side * 128 * per_tok + i] = idx[base + i];
      s_gt[side * 128 * per_tok + i] = gate[base + i];
    }
  }
  sync();
  if (my_b >= 0) {
    if (my_tot) atomicAdd(&s_tot[my_b], my_tot);
    if (my_pre) atomicAdd(&s_pre[my_b], my_pre);
  } else if (nb > nthreads) {                              // more buckets than threads: plain loop
    for (int b = tid; b < nb; b += nthreads) {
      int tot = 0, pre = 0;
      for (int bk = 0; bk < d.nblk; ++bk) {
        const int c = blockcnt[(size_t)bk * nb + b];
        tot += c;
        pre += bk < blk ? c : 0;
      }
      s_tot[b] = tot;
      s_pre[b] = pre;
    }
  }
  sync();
  for (int g = tid; g < d.sides * d.H; g += nthreads) {
    int run = 0;
    for (int e = 0; e < d.E; ++e) {
      s_off[g * d.E + e] = run;
      run += s_tot[g * d.E + e];
    }
  }
  // One entry per (token, group) (k = 1: also the (head, expert pair) buckets of the pair-tiled value
  // projection, which can be many): the lanes of a warp that share a bucket find each other with
  // match.any instead of one ballot per bucket.
  const bool one_sel = d.k == 1;
  for (int grp = gs; one_sel && grp < d.sides * d.H; grp += GS) {
    const int side = grp / d.H, h = grp % d.H;
    int ev = tl < nrows ? s_idx[side * 128 * per_tok + tl * d.H + h] : -1;
    if (ev >= 0 && !SH_INDEX_OK(ev, d.E, d.status, SH_SITE_SORT_EXPERT)) ev = -1;
    const unsigned m = __match_any_sync(0xffffffffu, ev >= 0 ? ev : 0x10000 + lane);
    if (ev >= 0 && lane == __ffs(m) - 1) s_wcnt[(grp * d.E + ev) * 4 + twarp] = __popc(m);
  }
  for (int grp = gs; !one_sel && grp < d.sides * d.H; grp += GS) {            // per-warp counts of this block's tokens
    const int side = grp / d.H, h = grp % d.H;
    unsigned mask = 0;
    if (tl < nrows)
      for (int j = 0; j < d.k; ++j) {
        const int ev = s_idx[side * 128 * per_tok + (tl * d.H + h) * d.k + j];
        if (SH_INDEX_OK(ev, d.E, d.status, SH_SITE_SORT_EXPERT)) mask |= 1u << ev;
      }
    for (int e = 0; e < d.E; ++e) {
      const unsigned bal = __ballot_sync(0xffffffffu, (mask >> e) & 1u);
      if (lane == 0) s_wcnt[(grp * d.E + e) * 4 + twarp] = __popc(bal);
    }
  }
  sync();
  {
    const int t = tok0 + tl;
    for (int grp = gs; one_sel && grp < d.sides * d.H; grp += GS) {
      const int side = grp / d.H, h = grp % d.H;
      const int sel = side * 128 * per_tok + tl * d.H + h;
      int ev = tl < nrows ? s_idx[sel] : -1;
      if ((unsigned)ev >= (unsigned)d.E) ev = -1;
      const unsigned m = __match_any_sync(0xffffffffu, ev >= 0 ? ev : 0x10000 + lane);
      if (ev >= 0) {
        const int b = grp * d.E + ev;
        int pos = __popc(m & ((1u << lane) - 1u));
        for (int w = 0; w < twarp; ++w) pos += s_wcnt[b * 4 + w];
        const size_t dst = (size_t)grp * d.N + s_off[b] + s_pre[b] + pos;
        if (SH_INDEX_OK(s_off[b] + s_pre[b] + pos, (long long)d.N, d.status, SH_SITE_SORT_SLOT)) {
          lists[dst] = t;
          lgate[dst] = s_gt[sel];
        }
      }
    }
    for (int grp = gs; !one_sel && grp < d.sides * d.H; grp += GS) {
      const int side = grp / d.H, h = grp % d.H;
      const int sel = side * 128 * per_tok + (tl * d.H + h) * d.k;
      unsigned mask = 0;
      if (tl < nrows)
        for (int j = 0; j < d.k; ++j) {
          const int ev = s_idx[sel + j];
          if (SH_INDEX_OK(ev, d.E, d.status, SH_SITE_SORT_EXPERT)) mask |= 1u << ev;
        }
      for (int e = 0; e < d.E; ++e) {
        const bool mine = (mask >> e) & 1u;
        const unsigned bal = __ballot_sync(0xffffffffu, mine);
        if (mine) {
          const int b = grp * d.E + e;
          int pos = __popc(bal & ((1u << lane) - 1u));
          for (int w = 0; w < twarp; ++w) pos += s_wcnt[b * 4 + w];
          float gv = 0.f;
          for (int j = 0; j < d.k; ++j)
            if (s_idx[sel + j] == e) gv = s_gt[sel + j];
          const size_t dst = (size_t)grp * d.N * d.k + s_off[b] + s_pre[b] + pos;
          if (SH_INDEX_OK(s_off[b] + s_pre[b] + pos, (long long)d.N * d.k, d.status, SH_SITE_SORT_SLOT)) {
            lists[dst] = t;
            lgate[dst] = gv;
          }
        }
      }
    }
  }
  if (blk != 0) return;
  for (int g = tid; g < d.sides * d.H; g += nthreads) {
    for (int e = 0; e < d.E; ++e) offsets[g * (d.E + 1) + e] = s_off[g * d.E + e];
    offsets[g * (d.E + 1) + d.E] = s_off[g * d.E + d.E - 1] + s_tot[g * d.E + d.E - 1];
  }
  // Tile table of a side.  Kernel of its own (the larger problems): the full tiles of all buckets first,
  // then the partial ones (one per bucket at most), so that a persistent kernel whose CTAs take tiles
  // t, t + grid, t + 2 grid, ... gets an even share of both kinds (bucket by bucket, full and partial
  // tiles alternate with a period that can divide the grid size).  Fused into the gate kernel (small
  // problems, where this block's tail is on the layer's critical path and every cold instruction line
  // costs an L2 round trip): bucket by bucket, by one thread per side.
  int* s_pbase = s_wcnt;                 // [nb] index of the bucket's partial tile (the per-warp counts are done with)
  if (!have_sel) {
    sync();
    if (tid < 32 * d.sides) {            // one warp per side: prefix sums over its buckets, 32 at a time
      const int side = tid >> 5;
      const int tr = side == 0 ? d.tile_rows_src : SH_TILE_ROWS;    // 128 or 256
      const int sh = 31 - __clz(tr);
      const int b_lo = side * d.H * d.E, b_hi = b_lo + d.H * d.E;
      int run = 0;
      for (int pass = 0; pass < 2; ++pass)                          // full tiles, then partial ones
        for (int b0 = b_lo; b0 < b_hi; b0 += 32) {
          const int b = b0 + lane;
          const int v = b < b_hi ? (pass == 0 ? s_tot[b] >> sh : (int)((s_tot[b] & (tr - 1)) != 0)) : 0;
          int inc = v;
#pragma unroll
          for (int o = 1; o < 32; o <<= 1) {
            const int u = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += u;
          }
          if (b < b_hi) (pass == 0 ? s_tbase : s_pbase)[b] = run + inc - v;
          run += __shfl_sync(0xffffffffu, inc, 31);
        }
      if (lane == 0) ntiles[side] = run;
    }
  } else if (tid < d.sides) {
    const int side = tid;
    const int tr = side == 0 ? d.tile_rows_src : SH_TILE_ROWS;
    const int sh = 31 - __clz(tr);
    int run = 0;
    for (int b = side * d.H * d.E; b < (side + 1) * d.H * d.E; ++b) {
      s_tbase[b] = run;
      run += (s_tot[b] + tr - 1) >> sh;
    }
    ntiles[side] = run;
  }
  sync();
  for (int i = tid; i < d.sides * d.H * d.E * 32; i += nthreads) {   // 32 threads share a bucket's tiles
    const int b = i >> 5;
    const int side = b / (d.H * d.E), h = (b / d.E) % d.H, e = b % d.E;
    const int cnt = s_tot[b];
    ShTile* tp = tiles + (size_t)side * d.max_tiles;
    const int tr = side == 0 ? d.tile_rows_src : SH_TILE_ROWS;
    for (int ti = i & 31; ti * tr < cnt; ti += 32) {
      ShTile tl2;
      tl2.h = h; tl2.e = e; tl2.row0 = s_off[b] + ti * tr;
      tl2.nrows = min(tr, cnt - ti * tr);
      tp[(have_sel || tl2.nrows == tr) ? s_tbase[b] + ti : s_pbase[b]] = tl2;
    }
  }
}

// Threads: 128 * GS, thread = (token tid % 128, group slice tid / 128); slice gs handles the
// (side, head) groups gs, gs + GS, ...
static __global__ void __launch_bounds__(1024)
sh_sort_kernel(const int* __restrict__ idx, const float* __restrict__ gate, const int* __restrict__ blockcnt,
               int* __restrict__ offsets, int* __restrict__ lists, float* __restrict__ lgate,
               ShTile* __restrict__ tiles, int* __restrict__ ntiles, ShDims d) {
  extern __shared__ int s_sort[];
  // programmatic dependent launch (no-ops in an ordinary launch): let the next kernel in the
  // stream become resident, then wait for the gate kernel's selections to be complete and visible
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (threadIdx.x == 0) sh_stamp_resident(d.stamps, SH_K_SORT);
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (threadIdx.x == 0) sh_stamp_start(d.stamps, SH_K_SORT);
  sh_sort_block(idx, gate, blockcnt, offsets, lists, lgate, tiles, ntiles, d, s_sort, (int)threadIdx.x, (int)blockDim.x, (int)blockIdx.x,
                false, [] { __syncthreads(); });
  if (d.stamps) {
    __syncthreads();
    if (threadIdx.x == 0) sh_stamp_end(d.stamps, SH_K_SORT);
  }
}

static inline int sh_sort_threads(const ShDims& d) {
  // at most 512 threads (16 K registers), so that a block fits beside a 320-thread GEMM CTA on an SM
  int gs = d.sides * d.H;
  if (gs > 4) gs = 4;
  // (the histogram prefix is shared out over all threads - bucket by bucket, block range by block range -
  //  and is a chain of L2 round trips: with many buckets or blocks, more threads than token slices pay)
  if ((long)d.G * d.nblk > 2048 && gs < 4) gs = 4;
  return 128 * gs;
}

static inline size_t sh_sort_smem_bytes(const ShDims& d) {
  return (size_t)(8 * d.G + 8) * 4 + (size_t)2 * 128 * d.H * d.k * 8;
}

// ---------------------------------------------------------------------------------------
// CUDA-core GEMM, 128 x 64 x 16 tiles, 256 threads, 8 x 4 outputs per thread.
//   acc[r, n] = sum_k A[row(r), a_col0 + k] * Bt[b_row0 + n, k]
// A rows are addressed through an optional row list (token ids); Bt is "K-major": one row
// of K contiguous values per output column.  The epilogue decides where acc goes.
// ---------------------------------------------------------------------------------------
enum { SH_EPI_QKV = 0, SH_EPI_V = 1, SH_EPI_O = 2, SH_EPI_PLAIN = 3 };

struct ShGemmArgs {
  const void* A; long lda;          // A [*, lda]
  const void* Bt; long ldb;         // Bt [*, ldb]
  int K;                            // reduction length
  int ncols;                        // output columns (per group)
  int nrows;                        // dense: number of rows; grouped: unused
  const int* lists;                 // grouped: lists[side] base ([H, N*k]) or nullptr
  const float* lgate;               // grouped: gates aligned with lists
  const ShTile* tiles;              // grouped: row-tile table
  const int* ntiles;                // grouped: number of valid tiles (device)
  long b_group_stride;              // grouped: elements of Bt per (h*E + e)
  int a_head_stride;                // grouped O: column offset of head h inside an A row
  void* out0; void* out1; void* out2;
  float qscale;
  float vscale;                     // grouped V-type epilogue: extra factor on the gate-scaled result (0 = none)
  const float2* rope;               // QKV epilogue: (cos, sin) table [D/2, T] of the rotary embedding, or nullptr
  ShDims d;
};

template <typename TA, typename TB, typename TC, int EPI>
__global__ void __launch_bounds__(256)
sh_simt_gemm_kernel(ShGemmArgs g) {
  constexpr int BM = 128, BN = 64, BK = 16;
  __shared__ float sA[BK][BM + 4];
  __shared__ float sB[BK][BN + 4];
  __shared__ int s_row[BM];
  __shared__ float s_gate[BM];
  const int tid = threadIdx.x;
  const ShDims& d = g.d;
  int h = 0, e = 0, row0, nrows;
  constexpr bool grouped = (EPI == SH_EPI_V || EPI == SH_EPI_O);
  if (grouped) {
    if ((int)blockIdx.x >= *g.ntiles) return;
    ShTile tl = g.tiles[blockIdx.x];
    h = tl.h; e = tl.e; row0 = tl.row0; nrows = tl.nrows;
  } else {
    row0 = blockIdx.x * BM;
    nrows = min(BM, g.nrows - row0);
  }
  const int col0 = blockIdx.y * BN;
  if (tid < BM) {
    int r = -1; float gt = 0.f;
    if (tid < nrows) {
      if (grouped) {
        size_t li = (size_t)h * d.N * d.k + row0 + tid;
        r = g.lists[li]; gt = g.lgate[li];
      } else {
        r = row0 + tid;
      }
    }
    s_row[tid] = r; s_gate[tid] = gt;
  }
  __syncthreads();
  const TA* A = (const TA*)g.A + (EPI == SH_EPI_O ? (long)h * g.a_head_stride : 0);
  const TB* Bt = (const TB*)g.Bt + (grouped ? (long)(h * d.E + e) * g.b_group_stride : 0);
  float acc[8][4];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
  const int tr = tid / 16, tc = tid % 16;   // 16 x 16 thread grid: rows tr*8.., cols tc*4..
  for (int k0 = 0; k0 < g.K; k0 += BK) {
    // A tile: 128 rows x 16 k: thread loads row = tid/2, 8 consecutive k
    {
      const int r = tid >> 1, kk = (tid & 1) * 8;
      const int gr = s_row[r];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        float v = 0.f;
        if (gr >= 0 && k0 + kk + i < g.K) v = sh_to_float<TA>(A[(long)gr * g.lda + k0 + kk + i]);
        sA[kk + i][r] = v;
      }
    }
    {
      const int n = tid >> 2, kk = (tid & 3) * 4;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        float v = 0.f;
        if (col0 + n < g.ncols && k0 + kk + i < g.K) v = sh_to_float<TB>(Bt[(long)(col0 + n) * g.ldb + k0 + kk + i]);
        sB[kk + i][n] = v;
      }
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      float a[8], b[4];
#pragma unroll
      for (int i = 0; i < 8; ++i) a[i] = sA[kk][tr * 8 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = sB[kk][tc * 4 + j];
#pragma unroll
      for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int lr = tr * 8 + i;
    const int gr = s_row[lr];
    if (gr < 0) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = col0 + tc * 4 + j;
      if (n >= g.ncols) continue;
      float v = acc[i][j];
      if (EPI == SH_EPI_QKV) {
        // column n -> (which, head, dd); row gr -> (b, t); target layout [B, H, T, D]
        const int HD = d.H * d.D;
        const int which = n / HD, hh = (n % HD) / d.D, dd = n % d.D;
        const int b = gr / d.T, t = gr % d.T;
        if (g.rope && which < 2) {
          // rotary embedding: the pair (dd even, dd + 1) sits in acc[i][j even], acc[i][j + 1]
          const float2 cs = g.rope[(size_t)(dd >> 1) * d.T + t];
          const float a0 = acc[i][j & ~1], a1 = acc[i][j | 1];
          v = (j & 1) ? a0 * cs.y + a1 * cs.x : a0 * cs.x - a1 * cs.y;
        }
        TC* dst = (TC*)(which == 0 ? g.out0 : which == 1 ? g.out1 : g.out2);
        dst[(((size_t)b * d.H + hh) * d.T + t) * d.D + dd] = sh_from_float<TC>(which == 0 ? v * g.qscale : v);
      } else if (EPI == SH_EPI_V) {
        const int b = gr / d.T, t = gr % d.T;
        atomicAdd((TC*)g.out0 + (((size_t)b * d.H + h) * d.T + t) * d.D + n, sh_from_float<TC>(s_gate[lr] * v * (g.vscale != 0.f ? g.vscale : 1.f)));
      } else if (EPI == SH_EPI_O) {
        const int orow = sh_out_row(d, gr);                // (cache tokens have no output row)
        if (orow >= 0) atomicAdd((float*)g.out0 + (size_t)orow * d.M + n, s_gate[lr] * v);
      } else {
        ((float*)g.out0)[(size_t)gr * g.ncols + n] = v;
      }
    }
  }
}

// ---------------------------------------------------------------------------------------
// CUDA-core attention (Eq. 1, with the autoregressive mask unless d.causal == 0): one warp per query row,
// keys in chunks of 32 (lane = key), online softmax in base 2 (Q carries log2(e)/sqrt(D)).
// Q, K, V [B, H, T, D]; Ahat [B*T, H, D].
// ---------------------------------------------------------------------------------------
// Optional relative-position term of Transformer-XL (fp32 configuration, sh_set_xl_positions):
//   score[t, s] = ((q_t + u) . k_s + (q_t + v) . r_{t-s}) / sqrt(D),   r_dist = xl.R[h, dist, :]
// Q is stored pre-multiplied by c = log2(e)/sqrt(D), so the kernel keeps q + c*u and q + c*v.
struct ShXlPos {
  const float* R;        // [H, T, D] projected embeddings of the distances 0..T-1, or nullptr: plain q.k scores
  const float* u;        // [H, D] content bias
  const float* v;        // [H, D] position bias
  float qscale;          // c
};

template <typename TM>
__global__ void __launch_bounds__(128)
sh_simt_attention_kernel(const TM* __restrict__ Q, const TM* __restrict__ K, const TM* __restrict__ V,
                         TM* __restrict__ Ahat, ShDims d, ShXlPos xl) {
  __shared__ float s_q[4][256];
  __shared__ float s_qv[4][256];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long qi = (long)blockIdx.x * 4 + warp;          // index over (b, h, t)
  const long total = (long)d.B * d.H * d.T;
  if (qi >= total) return;
  const int t = (int)(qi % d.T);
  if (t < d.Tc) return;                                 // a cache token: it is a key, not a query
  const long bh = qi / d.T;
  const TM* q = Q + qi * d.D;
  const TM* Kb = K + bh * d.T * d.D;
  const TM* Vb = V + bh * d.T * d.D;
  const int hq = (int)(bh % d.H);
  const float* Rh = xl.R ? xl.R + (size_t)hq * d.T * d.D : nullptr;
  for (int i = lane; i < d.D; i += 32) {
    const float qv = sh_to_float<TM>(q[i]);
    s_q[warp][i] = Rh ? qv + xl.qscale * xl.u[hq * d.D + i] : qv;
    s_qv[warp][i] = Rh ? qv + xl.qscale * xl.v[hq * d.D + i] : 0.f;
  }
  __syncwarp();
  float o[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};   // lane owns d = lane + 32*i (d_head up to 256)
  float m = -INFINITY, l = 0.f;
  const int last = d.causal ? t : d.T - 1;              // last visible key
  for (int s0 = 0; s0 <= last; s0 += 32) {
    const int s = s0 + lane;
    float sc = -INFINITY;
    if (s <= last) {
      const TM* kr = Kb + (long)s * d.D;
      float a = 0.f;
      for (int i = 0; i < d.D; ++i) a = fmaf(s_q[warp][i], sh_to_float<TM>(kr[i]), a);
      if (Rh) {                                         // position term: the embedding of the distance t - s (keys behind the query only)
        const float* rr = Rh + (long)max(t - s, 0) * d.D;
        float p2 = 0.f;
        for (int i = 0; i < d.D; ++i) p2 = fmaf(s_qv[warp][i], rr[i], p2);
        a += p2;
      }
      sc = a;
    }
    float cm = sc;
#pragma unroll
    for (int x = 16; x > 0; x >>= 1) cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, x));
    const float mn = fmaxf(m, cm);
    const float alpha = exp2f(m - mn);                  // m = -inf first time -> 0
    const float p = (s <= last) ? exp2f(sc - mn) : 0.f;
    float ps = p;
#pragma unroll
    for (int x = 16; x > 0; x >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, x);
    l = l * alpha + ps;
    m = mn;
#pragma unroll
    for (int i = 0; i < 8; ++i) o[i] *= alpha;
    const int cnt = min(32, last - s0 + 1);
    for (int j = 0; j < cnt; ++j) {
      const float pj = __shfl_sync(0xffffffffu, p, j);
      const TM* vr = Vb + (long)(s0 + j) * d.D;
#pragma unroll
      for (int i = 0; i < 8; ++i)
        if (lane + 32 * i < d.D) o[i] = fmaf(pj, sh_to_float<TM>(vr[lane + 32 * i]), o[i]);
    }
  }
  const int b = (int)(bh / d.H), h = (int)(bh % d.H);
  TM* dst = Ahat + (((long)b * d.T + t) * d.H + h) * d.D;
  const float inv = 1.f / l;
#pragma unroll
  for (int i = 0; i < 8; ++i)
    if (lane + 32 * i < d.D) dst[lane + 32 * i] = sh_from_float<TM>(o[i] * inv);
}

// ---------------------------------------------------------------------------------------
// Transformer-XL relative positions, one-time set-up: the sinusoidal embedding of the distances
// 0..T-1 (row dist = [sin(dist w_0) .. sin(dist w_{M/2-1}), cos(dist w_0) .. cos(dist w_{M/2-1})],
// w_i = 10000^(-2i/M), angles in double precision), and its projection R[h, dist, :] = emb[dist] Wr^h.
// ---------------------------------------------------------------------------------------
static __global__ void sh_xl_embedding_kernel(float* emb, int T, int M) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= T * (M / 2)) return;
  const int dist = i / (M / 2), f = i % (M / 2);
  const double w = pow(10000.0, -2.0 * (double)f / (double)M);
  double s, c;
  sincos((double)dist * w, &s, &c);
  emb[(size_t)dist * M + f] = (float)s;
  emb[(size_t)dist * M + M / 2 + f] = (float)c;
}

// R[h, dist, dd] = sum_m emb[dist, m] * Wr[h, m, dd]   (Wr row-major [H, M, Dt]; columns dd >= Dt of the padded D are zero)
static __global__ void sh_xl_project_kernel(const float* __restrict__ emb, const float* __restrict__ Wr, float* __restrict__ R,
                                            int H, int T, int M, int D, int Dt) {
  const long i = (long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (long)H * T * D) return;
  const int dd = (int)(i % D), dist = (int)((i / D) % T), h = (int)(i / ((long)D * T));
  double acc = 0.0;
  if (dd < Dt)
    for (int m = 0; m < M; ++m) acc += (double)emb[(size_t)dist * M + m] * (double)Wr[((size_t)h * M + m) * Dt + dd];
  R[i] = (float)acc;
}

// Tensor-core path: R16[h, dist, :] = fp16(R[h, dist, :]) and vr[h, dist] = c * v^h . R[h, dist, :]
// (one thread per element of R; the dot product by the thread of element dd == 0).
static __global__ void sh_xl_tables16_kernel(const float* __restrict__ R, const float* __restrict__ v, __half* __restrict__ R16,
                                             float* __restrict__ vr, int H, int T, int D, float c) {
  const long i = (long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (long)H * T * D) return;
  R16[i] = __float2half_rn(R[i]);
  if (i % D == 0) {
    const int h = (int)(i / ((long)D * T));
    double acc = 0.0;
    for (int dd = 0; dd < D; ++dd) acc += (double)v[h * D + dd] * (double)R[i + dd];
    vr[i / D] = c * (float)acc;
  }
}

// Per-key content bias of the Transformer-XL score: uk[b, h, s] = c * u^h . K[b, h, s, :]  (K fp16 [B, H, T, D],
// D a multiple of 64); eight lanes per key, 16-byte loads (a warp reads four keys' rows at a time).
static __global__ void __launch_bounds__(256)
sh_xl_uk_kernel(const __half* __restrict__ K, const float* __restrict__ u, float* __restrict__ uk, int H, int T, int D, long nkeys, float c) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const long key = ((long)blockIdx.x * blockDim.x + threadIdx.x) >> 3;
  const int sub = threadIdx.x & 7;
  float acc = 0.f;
  if (key < nkeys) {
    const int h = (int)((key / T) % H);
    const uint4* kr = reinterpret_cast<const uint4*>(K + key * D);
    const float* uh = u + h * D;
    for (int i = sub; i < D / 8; i += 8) {                 // 16-byte chunk i of the row: 8 values
      const uint4 v = __ldg(kr + i);
      const __half2* hv = reinterpret_cast<const __half2*>(&v);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const float2 f = __half22float2(hv[q]);
        acc = fmaf(uh[8 * i + 2 * q], f.x, acc);
        acc = fmaf(uh[8 * i + 2 * q + 1], f.y, acc);
      }
    }
  }
#pragma unroll
  for (int x = 4; x > 0; x >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, x);
  if (sub == 0 && key < nkeys) uk[key] = c * acc;
}
