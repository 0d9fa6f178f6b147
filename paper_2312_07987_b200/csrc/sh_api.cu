// Host side of libswitchhead: argument validation, workspace layout, weight repacking and
// the launch sequence of the forward pass.  Every entry point is documented in
// include/switchhead.h.
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>

#include "sh_internal.cuh"
#include "sh_simt.cuh"
#include "sh_backward.cuh"

static thread_local char g_err[512] = "";

void sh_set_error(const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
}

#define SH_CUDA_CHECK(expr)                                                          \
  do {                                                                               \
    cudaError_t _e = (expr);                                                         \
    if (_e != cudaSuccess) {                                                         \
      sh_set_error("%s failed: %s", #expr, cudaGetErrorString(_e));                  \
      return SH_ERR_CUDA;                                                            \
    }                                                                                \
  } while (0)

static size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

static size_t elem_bytes_in(int dtype) { return dtype == SH_F32 ? 4 : 2; }
static size_t elem_bytes_mid(int dtype) { return dtype == SH_F32 ? 4 : 2; }

static void layout_workspace(sh_layer* L) {
  const ShDims& d = L->d;
  const size_t in = elem_bytes_in(L->dtype), mid = elem_bytes_mid(L->dtype);
  size_t off = 0;
  // every sub-buffer is followed by a guard of SH_GUARD_BYTES that sh_set_weights fills with a
  // pattern and sh_check_guards verifies: a kernel that writes past the end of its buffer shows there
  L->n_guards = 0;
  auto take = [&](size_t bytes) {
    size_t o = off;
    const size_t end = align_up(off + bytes, 256);
    if (L->n_guards < SH_MAX_GUARDS) L->guard_off[L->n_guards++] = end;
    off = align_up(end + SH_GUARD_BYTES, 1024);
    return o;
  };
  ShWorkspace& o = L->o;
  const size_t HD = (size_t)d.H * d.D;
  const size_t nproj = L->dense ? 3 : 2;
  o.status = take(256);
  o.wqk = take(nproj * HD * d.M * in);
  o.wgate = take((size_t)d.G * d.M * in);
  o.gbias = take((size_t)d.G * 4);
  o.wv = take(L->dense ? 16 : HD * d.E * d.M * in);
  o.wo = take(HD * d.E * d.M * mid);
  o.q = take((size_t)d.N * HD * mid);
  o.k = take((size_t)d.N * HD * mid);
  o.v = take((size_t)d.N * HD * mid);
  o.ahat = take((size_t)d.N * HD * mid);
  const size_t slots = (size_t)2 * d.N * d.H * d.k;
  o.idx = take(slots * 4);
  o.gate = take(slots * 4);
  // (a layer whose value projection is tiled by expert pairs sorts H * E(E-1)/2 buckets in a forward pass)
  const bool vp = sh_v_pairs_ok(L);
  const size_t hist = vp && 2 * d.H * sh_pair_count(d.E) > d.G ? (size_t)2 * d.H * sh_pair_count(d.E) : (size_t)d.G;
  o.blockcnt = take((size_t)d.nblk * hist * 4);
  o.blockoff = take((size_t)d.nblk * hist * 4);
  o.offsets = take(((size_t)2 * d.H * (d.E + 1) + (vp ? (size_t)2 * d.H * (sh_pair_count(d.E) + 1) : 0)) * 4);
  o.lists = take(slots * 4);
  o.lgate = take(slots * 4);
  o.tiles = take((size_t)2 * d.max_tiles * sizeof(ShTile));
  o.ntiles = take(256);
  o.rope = take((size_t)d.T * (d.D / 2) * 8);     // (cos, sin) per feature pair and position
  // 16-bit storage: fp32 sums of the value rows of the first SH_EARLY_ROWS tokens of every sequence,
  // and how many of a row's k contributions have arrived (both zero between passes)
  const bool early = L->dtype == SH_BF16 && !L->dense;
  o.vearly = take(early ? (size_t)d.B * HD * SH_EARLY_ROWS * 4 : 16);
  o.vearly_cnt = take(early ? (size_t)d.B * d.H * SH_EARLY_ROWS * 4 : 16);
  // fp32 configuration: Transformer-XL relative positions (sh_set_xl_positions): the embedding of the
  // distances [T, M], its projection R [H, T, D] and the two bias vectors [2, H, D]
  // (bf16 storage: only for a layer with a cache, the setting the paper's XL models run in; besides the
  //  fp32 tables an fp16 copy of R, the per-distance bias v.r [H, T], the per-key bias u.k [B, H, T] and
  //  the score bias [B, H, Tq, T] fp16 that the attention kernel adds to its S tiles)
  const bool xlp = !L->dense && (L->dtype == SH_F32 || d.Tc > 0);
  const bool xlb = xlp && L->dtype == SH_BF16;
  o.xl_emb = take(xlp ? (size_t)d.T * d.M * 4 : 16);
  o.xl_r = take(xlp ? (size_t)d.H * d.T * d.D * 4 : 16);
  o.xl_uv = take(xlp ? (size_t)2 * d.H * d.D * 4 : 16);
  o.xl_r16 = take(xlb ? (size_t)d.H * d.T * d.D * 2 : 16);
  o.xl_vr = take(xlb ? (size_t)d.H * d.T * 4 : 16);
  o.xl_uk = take(xlb ? (size_t)d.B * d.H * d.T * 4 : 16);
  o.xl_bias = take(xlb ? (size_t)d.B * d.H * (d.T - d.Tc) * d.T * 2 : 16);
  // W_O once more with the experts innermost on the contraction axis: [H, M, D*E] (sparse output projection)
  o.wos = take(sh_o_sparse_ok(L) ? HD * d.E * d.M * mid : 16);
  o.gid = take(vp ? (size_t)2 * d.N * d.H * 4 : 16);  // (both sides: query experts are tiled by the destination side's pairs)
  // query / key experts (sh_create_moe_qk): [H, E, D, M] like the value experts
  o.wq_e = take(L->moe_q ? HD * d.E * d.M * in : 16);
  o.wk_e = take(L->moe_k ? HD * d.E * d.M * in : 16);      // pair number of every (token, head), source side
  // fp32 configuration: scratch of the backward pass (dQ, dK, dV, dAhat [N, H, D] and the gate gradients [2, N, H, k])
  o.bw = take(L->dtype == SH_F32 && !L->dense ? ((size_t)4 * d.N * HD + (size_t)2 * d.N * d.H * d.k) * 4 : 16);
  o.stamps = take(sizeof(ShStampBlock));
  o.total = off;
}

static sh_layer* create_common(int d_model, int n_heads, int d_head, int n_experts, int k, bool dense, int sides = 2) {
  g_err[0] = 0;
  if (d_model <= 0 || d_model % 64 != 0) { sh_set_error("d_model must be a positive multiple of 64 (got %d)", d_model); return nullptr; }
  if (n_heads < 1) { sh_set_error("n_heads must be >= 1 (got %d)", n_heads); return nullptr; }
  if (d_head < 1 || d_head > 256) { sh_set_error("d_head must be in 1..256 (got %d)", d_head); return nullptr; }
  if (n_experts < 1 || n_experts > 32) { sh_set_error("n_experts must be in 1..32 (got %d)", n_experts); return nullptr; }
  if (k < 1 || k > n_experts) { sh_set_error("k must be in 1..n_experts (got k=%d, n_experts=%d)", k, n_experts); return nullptr; }
  sh_layer* L = new (std::nothrow) sh_layer();
  if (!L) { sh_set_error("out of host memory"); return nullptr; }
  L->d.M = d_model; L->d.H = n_heads; L->d.Dt = d_head; L->d.E = n_experts; L->d.k = k;
  L->d.D = d_head <= 32 ? 32 : d_head <= 64 ? 64 : d_head <= 128 ? 128 : 256;   // sh_configure fixes it for the storage type
  L->d.sides = sides;
  L->d.causal = 1;
  L->d.Tc = 0;
  L->d.stamps = nullptr;
  L->d.status = nullptr;
  L->d.G = sides * n_heads * n_experts;
  L->dense = dense;
  return L;
}

extern "C" sh_layer* sh_create(int d_model, int n_heads, int d_head, int n_experts, int k) {
  return create_common(d_model, n_heads, d_head, n_experts, k, false);
}

extern "C" sh_layer* sh_create_shared(int d_model, int n_heads, int d_head, int n_experts, int k) {
  return create_common(d_model, n_heads, d_head, n_experts, k, false, 1);
}

extern "C" sh_layer* sh_create_moe_qk(int d_model, int n_heads, int d_head, int n_experts, int k, int moe_q, int moe_k,
                                      int shared_selection) {
  sh_layer* L = create_common(d_model, n_heads, d_head, n_experts, k, false, shared_selection ? 1 : 2);
  if (L) { L->moe_q = moe_q != 0; L->moe_k = moe_k != 0; }
  return L;
}

extern "C" sh_layer* sh_create_dense(int d_model, int n_heads, int d_head) {
  return create_common(d_model, n_heads, d_head, 1, 1, true);
}

static int configure_common(sh_layer* L, int dtype, int batch, int seq, int cache_len) {
  g_err[0] = 0;
  if (!L) { sh_set_error("layer is NULL"); return SH_ERR_INVALID_ARG; }
  if (dtype != SH_F32 && dtype != SH_BF16) { sh_set_error("dtype must be SH_F32 or SH_BF16 (got %d)", dtype); return SH_ERR_INVALID_ARG; }
  if (batch < 1 || seq < 1) { sh_set_error("batch and seq must be >= 1 (got %d, %d)", batch, seq); return SH_ERR_INVALID_ARG; }
  if (cache_len < 0) { sh_set_error("cache_len must be >= 0 (got %d)", cache_len); return SH_ERR_INVALID_ARG; }
  const ShDims& d0 = L->d;
  if (dtype == SH_BF16 && d0.M % 128 != 0) {
    sh_set_error("bf16 path needs d_model %% 128 == 0 (got d_model=%d)", d0.M);
    return SH_ERR_UNSUPPORTED;
  }
  if (dtype == SH_BF16 && d0.Dt > 128 && (L->dense || cache_len > 0)) {
    // (the tensor-core attention kernel keeps S and O of two query tiles in the 512 TMEM columns: d_head <= 128;
    //  above that a bf16 layer runs on the CUDA-core kernels - see sh_tc_prepare - which this build keeps to the plain layer)
    sh_set_error("bf16 storage with d_head above 128 (got %d): the plain layer without a cache only; the fp32 configuration takes every form", d0.Dt);
    return SH_ERR_UNSUPPORTED;
  }
  if (cache_len > 0 && L->dense) { sh_set_error("the dense comparator has no cache"); return SH_ERR_UNSUPPORTED; }
  if ((L->moe_q || L->moe_k) && dtype != SH_F32) {
    // on the tensor-core path an expert projection of keys or queries is the pair-tiled value kernel with
    // other weights: the shapes that kernel serves, and a dense half (if any) the CTA-pair GEMM can tile
    const bool ok = d0.k == 2 && d0.E >= 2 && d0.E <= 8 && d0.Dt > 64 && d0.Dt <= 128 &&
                    ((L->moe_q && L->moe_k) || (d0.H * 128) % 256 == 0);
    if (!ok) {
      sh_set_error("query / key experts with bf16 storage need k = 2, 2..8 experts, d_head in 65..128 and, when only one of the "
                   "two is an expert projection, an even number of heads (the fp32 configuration takes every shape)");
      return SH_ERR_UNSUPPORTED;
    }
  }
  if (cache_len > 0 && dtype == SH_BF16 && (cache_len % 128 != 0 || seq % 128 != 0)) {
    // the tensor-core attention and output kernels work on 128-token tiles that must not straddle the
    // boundary between cache and chunk, nor two sequences
    sh_set_error("bf16 path with a cache needs cache_len and seq to be multiples of 128 (got %d, %d)", cache_len, seq);
    return SH_ERR_UNSUPPORTED;
  }
  // d_head is stored padded with zero columns: to 64 or 128 on the tensor-core path, to 32, 64 or
  // 128 on the fp32 path (zero columns of W_Q, W_K, W_V and zero rows of W_O change no result)
  L->d.D = dtype == SH_BF16 ? (d0.Dt <= 64 ? 64 : d0.Dt <= 128 ? 128 : 256) : (d0.Dt <= 32 ? 32 : d0.Dt <= 64 ? 64 : d0.Dt <= 128 ? 128 : 256);
  const int T = cache_len + seq;                           // tokens of a sequence the layer sees: cache, then chunk
  const long long slots = (long long)batch * T * d0.H * d0.k;
  if (slots >= (1ll << 31) || (long long)batch * T * d0.M >= (1ll << 40)) {
    sh_set_error("problem too large: batch*(cache_len+seq)*n_heads*k = %lld must be below 2^31", slots);
    return SH_ERR_UNSUPPORTED;
  }
  L->dtype = dtype;
  L->d.B = batch; L->d.T = T; L->d.Tc = cache_len; L->d.N = batch * T;
  L->d.nblk = (L->d.N + SH_TILE_ROWS - 1) / SH_TILE_ROWS;
  L->d.max_tiles = (int)((slots + SH_TILE_ROWS - 1) / SH_TILE_ROWS) + d0.H * d0.E + d0.H * sh_pair_count(d0.E > 8 ? 2 : d0.E);
  L->d.tile_rows_src = SH_TILE_ROWS;
  // (k >= 3: the fp16 reductions of a value row arrive in a different order from run to run - two
  //  passes have been seen 1e-2 of the output RMS apart; with the first rows, which reach the output
  //  unaveraged, summed in fp32 they stay within 4e-3)
  L->d.early_rows = (dtype == SH_BF16 && (T >= SH_EARLY_MIN_SEQ || d0.k >= 3)) ? SH_EARLY_ROWS : 0;
  L->ws = nullptr; L->ws_bytes = 0; L->rope = false; L->xl_positions = false;
  L->d.status = nullptr;
  L->weights_set = false;
  sh_tc_release(L);
  layout_workspace(L);
  return SH_OK;
}

extern "C" int sh_configure(sh_layer* L, int dtype, int batch, int seq) { return configure_common(L, dtype, batch, seq, 0); }

extern "C" int sh_configure_xl(sh_layer* L, int dtype, int batch, int seq, int cache_len) {
  return configure_common(L, dtype, batch, seq, cache_len);
}

extern "C" size_t sh_workspace_bytes(const sh_layer* L) {
  if (!L || L->dtype < 0) return 0;
  return L->o.total;
}

extern "C" int sh_set_workspace(sh_layer* L, void* workspace, size_t bytes) {
  g_err[0] = 0;
  if (!L) { sh_set_error("layer is NULL"); return SH_ERR_INVALID_ARG; }
  if (L->dtype < 0) { sh_set_error("sh_configure has not been called"); return SH_ERR_NOT_CONFIGURED; }
  if (!workspace) { sh_set_error("workspace is NULL"); return SH_ERR_WORKSPACE; }
  if ((uintptr_t)workspace % 256 != 0) { sh_set_error("workspace must be 256-byte aligned"); return SH_ERR_WORKSPACE; }
  if (bytes < L->o.total) { sh_set_error("workspace too small: %zu bytes given, %zu needed", bytes, L->o.total); return SH_ERR_WORKSPACE; }
  L->ws = (char*)workspace; L->ws_bytes = bytes; L->weights_set = false; L->rope = false; L->xl_positions = false;
  L->d.status = (int*)(L->ws + L->o.status);
  sh_tc_release(L);
  return SH_OK;
}

template <typename TI, typename TO>
static void repack(const void* in, void* out, int batch, int rows, int cols, long obs, long ors, long oes,
                   cudaStream_t st) {
  long total = (long)batch * rows * cols;
  int blocks = (int)((total + 255) / 256);
  if (blocks > 65535 * 4) blocks = 65535 * 4;
  if (blocks < 1) blocks = 1;
  sh_repack_kernel<TI, TO><<<blocks, 256, 0, st>>>((const TI*)in, (TO*)out, batch, rows, cols, obs, ors, oes);
}

template <typename TI, typename TM>
static int set_weights_t(sh_layer* L, const void* Wq, const void* Wk, const void* Wv, const void* Wo,
                         const void* Ws, const void* Wd, const float* bias_s, const float* bias_d,
                         cudaStream_t st) {
  const ShDims& d = L->d;
  char* ws = L->ws;
  const long HD = (long)d.H * d.D;
  SH_CUDA_CHECK(cudaMemsetAsync(ws + L->o.status, 0, 256, st));
  SH_CUDA_CHECK(cudaMemsetAsync(ws + L->o.vearly, 0, L->o.xl_emb - L->o.vearly, st));   // early-row sums and counters
  for (int i = 0; i < L->n_guards; ++i) SH_CUDA_CHECK(cudaMemsetAsync(ws + L->guard_off[i], SH_GUARD_BYTE, SH_GUARD_BYTES, st));
  // Wq, Wk [H, M, Dt] -> Wqk[(which*H + h)*D + dd][m]   (rows dd >= Dt stay zero)
  TI* wqk = (TI*)(ws + L->o.wqk);
  if (d.D != d.Dt) {
    SH_CUDA_CHECK(cudaMemsetAsync(ws + L->o.wqk, 0, (size_t)(L->dense ? 3 : 2) * HD * d.M * sizeof(TI), st));
    SH_CUDA_CHECK(cudaMemsetAsync(ws + L->o.wo, 0, (size_t)HD * d.E * d.M * sizeof(TM), st));
    if (!L->dense) SH_CUDA_CHECK(cudaMemsetAsync(ws + L->o.wv, 0, (size_t)HD * d.E * d.M * sizeof(TI), st));
  }
  // (with query / key experts: Wq / Wk [H, E, M, Dt] -> [H, E, D, M], like the value experts)
  if (L->moe_q) {
    if (d.D != d.Dt) SH_CUDA_CHECK(cudaMemsetAsync(ws + L->o.wq_e, 0, (size_t)HD * d.E * d.M * sizeof(TI), st));
    repack<TI, TI>(Wq, ws + L->o.wq_e, d.H * d.E, d.M, d.Dt, (long)d.D * d.M, d.M, 1, st);
  } else {
    repack<TI, TI>(Wq, wqk, d.H, d.M, d.Dt, (long)d.D * d.M, d.M, 1, st);
  }
  if (L->moe_k) {
    if (d.D != d.Dt) SH_CUDA_CHECK(cudaMemsetAsync(ws + L->o.wk_e, 0, (size_t)HD * d.E * d.M * sizeof(TI), st));
    repack<TI, TI>(Wk, ws + L->o.wk_e, d.H * d.E, d.M, d.Dt, (long)d.D * d.M, d.M, 1, st);
  } else {
    repack<TI, TI>(Wk, wqk + HD * d.M, d.H, d.M, d.Dt, (long)d.D * d.M, d.M, 1, st);
  }
  if (L->dense) {
    // Wv [H, 1, M, D] joins the fused projection; Wo [H, 1, D, M] -> Wo_t[m][h*D + dd]
    repack<TI, TI>(Wv, wqk + 2 * HD * d.M, d.H, d.M, d.Dt, (long)d.D * d.M, d.M, 1, st);
    repack<TI, TM>(Wo, ws + L->o.wo, d.H, d.Dt, d.M, d.D, HD, 1, st);
  } else {
    // Ws, Wd [H, M, E] -> Wgate[(side*H + h)*E + e][m]
    TI* wg = (TI*)(ws + L->o.wgate);
    repack<TI, TI>(Ws, wg, d.H, d.M, d.E, (long)d.E * d.M, d.M, 1, st);
    if (d.sides == 2) repack<TI, TI>(Wd, wg + (long)d.H * d.E * d.M, d.H, d.M, d.E, (long)d.E * d.M, d.M, 1, st);
    float* gb = (float*)(ws + L->o.gbias);
    const size_t hb = (size_t)d.H * d.E * 4;
    if (bias_s) SH_CUDA_CHECK(cudaMemcpyAsync(gb, bias_s, hb, cudaMemcpyDeviceToDevice, st));
    else SH_CUDA_CHECK(cudaMemsetAsync(gb, 0, hb, st));
    if (d.sides == 2) {
      if (bias_d) SH_CUDA_CHECK(cudaMemcpyAsync(gb + d.H * d.E, bias_d, hb, cudaMemcpyDeviceToDevice, st));
      else SH_CUDA_CHECK(cudaMemsetAsync(gb + d.H * d.E, 0, hb, st));
    }
    // Wv [H, E, M, D] -> [H, E, D, M];  Wo [H, E, D, M] -> [H, E, M, D]
    repack<TI, TI>(Wv, ws + L->o.wv, d.H * d.E, d.M, d.Dt, (long)d.D * d.M, d.M, 1, st);
    repack<TI, TM>(Wo, ws + L->o.wo, d.H * d.E, d.Dt, d.M, (long)d.D * d.M, d.D, 1, st);
    if (sh_o_sparse_ok(L)) {
      // Wo [H, E, D, M] -> [H, M, D*E]: element (h, e, dd, m) at (h*M + m)*(D*E) + dd*E + e
      if (d.D != d.Dt) SH_CUDA_CHECK(cudaMemsetAsync(ws + L->o.wos, 0, (size_t)HD * d.E * d.M * sizeof(TM), st));
      for (int h = 0; h < d.H; ++h)
        repack<TI, TM>((const TI*)Wo + (size_t)h * d.E * d.Dt * d.M, (TM*)(ws + L->o.wos) + (size_t)h * d.M * d.D * d.E, d.E, d.Dt, d.M, 1, (long)d.D * d.E, d.E, st);
    }
  }
  SH_CUDA_CHECK(cudaGetLastError());
  return SH_OK;
}

extern "C" int sh_set_weights(sh_layer* L, const void* Wq, const void* Wk, const void* Wv, const void* Wo,
                              const void* Ws, const void* Wd, const float* bias_s, const float* bias_d,
                              void* stream) {
  g_err[0] = 0;
  if (!L) { sh_set_error("layer is NULL"); return SH_ERR_INVALID_ARG; }
  if (L->dtype < 0) { sh_set_error("sh_configure has not been called"); return SH_ERR_NOT_CONFIGURED; }
  if (!L->ws) { sh_set_error("sh_set_workspace has not been called"); return SH_ERR_WORKSPACE; }
  if (!Wq || !Wk || !Wv || !Wo) { sh_set_error("Wq, Wk, Wv and Wo must not be NULL"); return SH_ERR_INVALID_ARG; }
  if (!L->dense && (!Ws || (!Wd && L->d.sides == 2))) { sh_set_error("Ws and Wd must not be NULL for a SwitchHead layer"); return SH_ERR_INVALID_ARG; }
  if (!L->dense && L->d.sides == 1 && (Wd || bias_d)) { sh_set_error("a shared-selection layer has one gate: pass NULL for Wd and bias_d"); return SH_ERR_INVALID_ARG; }
  if (L->dense && (Ws || Wd || bias_s || bias_d)) { sh_set_error("a dense layer has no gates: pass NULL for Ws, Wd and the biases"); return SH_ERR_INVALID_ARG; }
  cudaStream_t st = (cudaStream_t)stream;
  int rc = (L->dtype == SH_F32)
               ? set_weights_t<float, float>(L, Wq, Wk, Wv, Wo, Ws, Wd, bias_s, bias_d, st)
               : set_weights_t<__nv_bfloat16, __half>(L, Wq, Wk, Wv, Wo, Ws, Wd, bias_s, bias_d, st);
  if (rc != SH_OK) return rc;
  if (L->dtype == SH_BF16) {
    rc = sh_tc_prepare(L);
    if (rc != SH_OK) return rc;
  }
  L->weights_set = true;
  return SH_OK;
}

static int check_ready(sh_layer* L) {
  if (!L) { sh_set_error("layer is NULL"); return SH_ERR_INVALID_ARG; }
  if (L->dtype < 0) { sh_set_error("sh_configure has not been called"); return SH_ERR_NOT_CONFIGURED; }
  if (!L->ws) { sh_set_error("sh_set_workspace has not been called"); return SH_ERR_WORKSPACE; }
  if (!L->weights_set) { sh_set_error("sh_set_weights has not been called"); return SH_ERR_NOT_CONFIGURED; }
  return SH_OK;
}

// gate + top-k + bucket sort (three launches)
template <typename TI>
static int launch_gate_sort(sh_layer* L, const void* x, cudaStream_t st) {
  const ShDims& d = L->d;
  char* ws = L->ws;
  const size_t hist = (size_t)d.G * 4;
  sh_gate_topk_kernel<TI><<<d.nblk, 256, hist, st>>>((const TI*)x, (const TI*)(ws + L->o.wgate),
      (const float*)(ws + L->o.gbias), (int*)(ws + L->o.idx), (float*)(ws + L->o.gate),
      (int*)(ws + L->o.blockcnt), d);
  const size_t ssm = sh_sort_smem_bytes(d);
  // (set on every call that needs it: the attribute belongs to the current device's copy of the function)
  if (ssm > 48 * 1024)
    SH_CUDA_CHECK(cudaFuncSetAttribute(sh_sort_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ssm));
  sh_sort_kernel<<<d.nblk, sh_sort_threads(d), ssm, st>>>((const int*)(ws + L->o.idx), (const float*)(ws + L->o.gate),
      (const int*)(ws + L->o.blockcnt), (int*)(ws + L->o.offsets), (int*)(ws + L->o.lists),
      (float*)(ws + L->o.lgate), (ShTile*)(ws + L->o.tiles), (int*)(ws + L->o.ntiles), d);
  L->launches += 2;
  SH_CUDA_CHECK(cudaGetLastError());
  return SH_OK;
}

template <typename TI, typename TM>
static int forward_simt(sh_layer* L, int stages, const void* x, void* out, cudaStream_t st) {
  const ShDims& d = L->d;
  char* ws = L->ws;
  const int HD = d.H * d.D;
  const float qscale = 1.4426950408889634f / sqrtf((float)d.Dt);
  const bool all = stages == SH_STAGE_ALL;
  if (all) sh_mark(L, 0, st);
  if (!L->dense && (stages & SH_STAGE_GATE)) {
    int rc = launch_gate_sort<TI>(L, x, st);
    if (rc != SH_OK) return rc;
  }
  if (all) sh_mark(L, 1, st);
  if (stages & SH_STAGE_QK) {
    ShGemmArgs g{};
    g.d = d;
    g.A = x; g.lda = d.M; g.ldb = d.M; g.K = d.M; g.nrows = d.N;
    g.rope = L->rope ? (const float2*)(ws + L->o.rope) : nullptr;
    if (!L->moe_q && !L->moe_k) {
      // Q, K (and V for the dense comparator)
      g.Bt = ws + L->o.wqk;
      g.ncols = (L->dense ? 3 : 2) * HD;
      g.out0 = ws + L->o.q; g.out1 = ws + L->o.k; g.out2 = ws + L->o.v; g.qscale = qscale;
      dim3 grid_qk(d.nblk, (g.ncols + 63) / 64);
      sh_simt_gemm_kernel<TI, TI, TM, SH_EPI_QKV><<<grid_qk, 256, 0, st>>>(g);
      L->launches += 1;
    } else {
      // query / key experts: whichever of the two is dense is one projection of HD columns; an expert
      // projection is the value experts' grouped GEMM with its own weights, side and output
      g.ncols = HD;
      dim3 grid_1(d.nblk, (HD + 63) / 64);
      if (!L->moe_q) {
        g.Bt = ws + L->o.wqk; g.out0 = ws + L->o.q; g.qscale = qscale;
        sh_simt_gemm_kernel<TI, TI, TM, SH_EPI_QKV><<<grid_1, 256, 0, st>>>(g);
        L->launches += 1;
      }
      if (!L->moe_k) {
        g.Bt = (const TI*)(ws + L->o.wqk) + (size_t)HD * d.M; g.out0 = ws + L->o.k; g.qscale = 1.f;
        sh_simt_gemm_kernel<TI, TI, TM, SH_EPI_QKV><<<grid_1, 256, 0, st>>>(g);
        L->launches += 1;
      }
      ShGemmArgs e{};
      e.d = d; e.A = x; e.lda = d.M; e.ldb = d.M; e.K = d.M; e.ncols = d.D; e.b_group_stride = (long)d.D * d.M;
      dim3 grid_e(d.max_tiles, (d.D + 63) / 64);
      if (L->moe_k) {                                      // source side, like the values
        SH_CUDA_CHECK(cudaMemsetAsync(ws + L->o.k, 0, (size_t)d.N * HD * sizeof(TM), st));
        e.Bt = ws + L->o.wk_e; e.out0 = ws + L->o.k; e.vscale = 0.f;
        e.lists = (const int*)(ws + L->o.lists); e.lgate = (const float*)(ws + L->o.lgate);
        e.tiles = (const ShTile*)(ws + L->o.tiles); e.ntiles = (const int*)(ws + L->o.ntiles);
        sh_simt_gemm_kernel<TI, TI, TM, SH_EPI_V><<<grid_e, 256, 0, st>>>(e);
        L->launches += 2;
      }
      if (L->moe_q) {                                      // destination side, like the output (stored scaled, as the dense queries are)
        SH_CUDA_CHECK(cudaMemsetAsync(ws + L->o.q, 0, (size_t)d.N * HD * sizeof(TM), st));
        const size_t side1 = d.sides == 2 ? (size_t)d.H * d.N * d.k : 0;
        e.Bt = ws + L->o.wq_e; e.out0 = ws + L->o.q; e.vscale = qscale;
        e.lists = (const int*)(ws + L->o.lists) + side1; e.lgate = (const float*)(ws + L->o.lgate) + side1;
        e.tiles = (const ShTile*)(ws + L->o.tiles) + (d.sides == 2 ? d.max_tiles : 0);
        e.ntiles = (const int*)(ws + L->o.ntiles) + (d.sides == 2 ? 1 : 0);
        sh_simt_gemm_kernel<TI, TI, TM, SH_EPI_V><<<grid_e, 256, 0, st>>>(e);
        L->launches += 2;
      }
    }
  }
  if (all) sh_mark(L, 2, st);
  if (!L->dense && (stages & SH_STAGE_V)) {
    SH_CUDA_CHECK(cudaMemsetAsync(ws + L->o.v, 0, (size_t)d.N * HD * sizeof(TM), st));
    ShGemmArgs v{};
    v.d = d; v.A = x; v.lda = d.M; v.Bt = ws + L->o.wv; v.ldb = d.M; v.K = d.M; v.ncols = d.D;
    v.lists = (const int*)(ws + L->o.lists); v.lgate = (const float*)(ws + L->o.lgate);
    v.tiles = (const ShTile*)(ws + L->o.tiles); v.ntiles = (const int*)(ws + L->o.ntiles);
    v.b_group_stride = (long)d.D * d.M; v.out0 = ws + L->o.v;
    dim3 grid_v(d.max_tiles, (d.D + 63) / 64);
    sh_simt_gemm_kernel<TI, TI, TM, SH_EPI_V><<<grid_v, 256, 0, st>>>(v);
    L->launches += 2;
  }
  if (all) sh_mark(L, 3, st);
  if (stages & SH_STAGE_ATTN) {
    const long nq = (long)d.B * d.H * d.T;
    ShXlPos xl{};
    if (L->xl_positions) {
      xl.R = (const float*)(ws + L->o.xl_r);
      xl.u = (const float*)(ws + L->o.xl_uv); xl.v = xl.u + (size_t)d.H * d.D;
      xl.qscale = qscale;
    }
    sh_simt_attention_kernel<TM><<<(unsigned)((nq + 3) / 4), 128, 0, st>>>((const TM*)(ws + L->o.q),
        (const TM*)(ws + L->o.k), (const TM*)(ws + L->o.v), (TM*)(ws + L->o.ahat), d, xl);
    L->launches += 1;
  }
  if (all) sh_mark(L, 4, st);
  if (!(stages & SH_STAGE_O)) {
  } else if (!L->dense) {
    SH_CUDA_CHECK(cudaMemsetAsync(out, 0, (size_t)sh_out_rows(d) * d.M * 4, st));
    ShGemmArgs o{};
    o.d = d; o.A = ws + L->o.ahat; o.lda = HD; o.a_head_stride = d.D; o.Bt = ws + L->o.wo; o.ldb = d.D;
    o.K = d.D; o.ncols = d.M;
    // destination-side lists and tiles (with a shared selection: the one side there is)
    const size_t side1 = d.sides == 2 ? (size_t)d.H * d.N * d.k : 0;
    o.lists = (const int*)(ws + L->o.lists) + side1; o.lgate = (const float*)(ws + L->o.lgate) + side1;
    o.tiles = (const ShTile*)(ws + L->o.tiles) + (d.sides == 2 ? d.max_tiles : 0);
    o.ntiles = (const int*)(ws + L->o.ntiles) + (d.sides == 2 ? 1 : 0);
    o.b_group_stride = (long)d.M * d.D; o.out0 = out;
    dim3 grid_o(d.max_tiles, (d.M + 63) / 64);
    sh_simt_gemm_kernel<TM, TM, float, SH_EPI_O><<<grid_o, 256, 0, st>>>(o);
    L->launches += 2;
  } else {
    ShGemmArgs o{};
    o.d = d; o.A = ws + L->o.ahat; o.lda = HD; o.Bt = ws + L->o.wo; o.ldb = HD; o.K = HD; o.ncols = d.M;
    o.nrows = d.N; o.out0 = out;
    dim3 grid_o(d.nblk, (d.M + 63) / 64);
    sh_simt_gemm_kernel<TM, TM, float, SH_EPI_PLAIN><<<grid_o, 256, 0, st>>>(o);
    L->launches += 1;
  }
  if (all) sh_mark(L, 5, st);
  SH_CUDA_CHECK(cudaGetLastError());
  return SH_OK;
}

int sh_simt_run_bf16(sh_layer* L, int stages, const void* x, void* out, cudaStream_t st) {
  return forward_simt<__nv_bfloat16, __half>(L, stages, x, out, st);
}

// (cos, sin)(t * base^(-2i/D)) for every feature pair i < D/2 and position t < T, computed in
// double precision, stored as float2 [D/2][T] (positions contiguous: the epilogue threads of a
// warp hold consecutive tokens and read one pair at a time).
static __global__ void sh_rope_table_kernel(float2* table, int T, int D, int Dt, double base) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  const int half = D / 2;
  if (idx >= T * half) return;
  const int t = idx / half, i = idx % half;
  // pairs past the given d_head are zero padding: identity
  const double ang = 2 * i < Dt ? (double)t * pow(base, -2.0 * (double)i / (double)Dt) : 0.0;
  double s, c;
  sincos(ang, &s, &c);
  table[(size_t)i * T + t] = make_float2((float)c, (float)s);
}

extern "C" int sh_set_causal(sh_layer* L, int causal) {
  g_err[0] = 0;
  if (!L) { sh_set_error("layer is NULL"); return SH_ERR_INVALID_ARG; }
  L->d.causal = causal ? 1 : 0;
  return SH_OK;
}

extern "C" int sh_set_output_f16(sh_layer* L, int enable) {
  g_err[0] = 0;
  if (!L) { sh_set_error("layer is NULL"); return SH_ERR_INVALID_ARG; }
  if (L->dtype < 0) { sh_set_error("sh_set_output_f16 needs a configured layer"); return SH_ERR_NOT_CONFIGURED; }
  if (enable && (L->dtype != SH_BF16 || L->dense)) {
    sh_set_error("fp16 output exists for the bf16 storage configuration of the SwitchHead layer only");
    return SH_ERR_UNSUPPORTED;
  }
  L->out_f16 = enable != 0;
  return SH_OK;
}

extern "C" int sh_set_xl_positions(sh_layer* L, const float* Wr, const float* u, const float* v, void* stream) {
  g_err[0] = 0;
  if (!L) { sh_set_error("layer is NULL"); return SH_ERR_INVALID_ARG; }
  if (L->dtype < 0 || !L->ws) { sh_set_error("sh_set_xl_positions needs a configured layer with its workspace"); return SH_ERR_NOT_CONFIGURED; }
  if (!Wr) { L->xl_positions = false; return SH_OK; }
  if (L->dense) { sh_set_error("the dense comparator has no relative positions"); return SH_ERR_UNSUPPORTED; }
  if (L->dtype == SH_BF16 && L->d.Tc == 0) {
    sh_set_error("bf16 storage: the relative-position term needs a layer configured with a cache (sh_configure_xl, cache_len >= 128)");
    return SH_ERR_UNSUPPORTED;
  }
  if (L->rope) { sh_set_error("rotary embeddings are switched on: one positional encoding at a time"); return SH_ERR_UNSUPPORTED; }
  const ShDims& d = L->d;
  if (d.M % 2) { sh_set_error("the sinusoidal embedding needs an even d_model"); return SH_ERR_UNSUPPORTED; }
  cudaStream_t st = (cudaStream_t)stream;
  float* emb = (float*)(L->ws + L->o.xl_emb);
  float* R = (float*)(L->ws + L->o.xl_r);
  float* uv = (float*)(L->ws + L->o.xl_uv);
  const int ne = d.T * (d.M / 2);
  sh_xl_embedding_kernel<<<(ne + 255) / 256, 256, 0, st>>>(emb, d.T, d.M);
  const long nr = (long)d.H * d.T * d.D;
  sh_xl_project_kernel<<<(unsigned)((nr + 255) / 256), 256, 0, st>>>(emb, Wr, R, d.H, d.T, d.M, d.D, d.Dt);
  // u, v [H, Dt] -> [H, D] (zero padding: the padded columns of K and R are zero anyway)
  SH_CUDA_CHECK(cudaMemsetAsync(uv, 0, (size_t)2 * d.H * d.D * 4, st));
  if (u) SH_CUDA_CHECK(cudaMemcpy2DAsync(uv, (size_t)d.D * 4, u, (size_t)d.Dt * 4, (size_t)d.Dt * 4, d.H, cudaMemcpyDeviceToDevice, st));
  if (v) SH_CUDA_CHECK(cudaMemcpy2DAsync(uv + (size_t)d.H * d.D, (size_t)d.D * 4, v, (size_t)d.Dt * 4, (size_t)d.Dt * 4, d.H, cudaMemcpyDeviceToDevice, st));
  if (L->dtype == SH_BF16) {
    // tensor-core path: R as fp16 (the B operand of the score-bias GEMM) and the per-distance term c * v . r
    const float qscale = 1.4426950408889634f / sqrtf((float)d.Dt);
    sh_xl_tables16_kernel<<<(unsigned)((nr + 255) / 256), 256, 0, st>>>(R, uv + (size_t)d.H * d.D, (__half*)(L->ws + L->o.xl_r16),
                                                                       (float*)(L->ws + L->o.xl_vr), d.H, d.T, d.D, qscale);
  }
  SH_CUDA_CHECK(cudaGetLastError());
  L->xl_positions = true;
  return SH_OK;
}

extern "C" int sh_set_rope(sh_layer* L, double base, void* stream) {
  g_err[0] = 0;
  if (!L) { sh_set_error("layer is NULL"); return SH_ERR_INVALID_ARG; }
  if (L->dtype < 0 || !L->ws) { sh_set_error("sh_set_rope needs a configured layer with its workspace"); return SH_ERR_NOT_CONFIGURED; }
  if (!(base >= 0.0) || base != base) { sh_set_error("rotary base must be positive (0 switches it off), got %g", base); return SH_ERR_INVALID_ARG; }
  if (base == 0.0) { L->rope = false; return SH_OK; }
  if (L->xl_positions) { sh_set_error("relative positions are switched on: one positional encoding at a time"); return SH_ERR_UNSUPPORTED; }
  if (L->d.Tc > 0) { sh_set_error("rotary embeddings are for the cache-less layer (the paper's RoPE models have no cache)"); return SH_ERR_UNSUPPORTED; }
  if (L->d.Dt % 2) { sh_set_error("rotary embedding needs an even d_head (got %d)", L->d.Dt); return SH_ERR_UNSUPPORTED; }
  if (L->moe_q || L->moe_k) { sh_set_error("rotary embeddings are applied in the dense Q/K projection's epilogue: not with query / key experts"); return SH_ERR_UNSUPPORTED; }
  const int n = L->d.T * (L->d.D / 2);
  sh_rope_table_kernel<<<(n + 255) / 256, 256, 0, (cudaStream_t)stream>>>((float2*)(L->ws + L->o.rope), L->d.T, L->d.D, L->d.Dt, base);
  SH_CUDA_CHECK(cudaGetLastError());
  L->rope = true;
  return SH_OK;
}

extern "C" int sh_forward(sh_layer* L, const void* x, void* out, void* stream) {
  g_err[0] = 0;
  int rc = check_ready(L);
  if (rc != SH_OK) return rc;
  if (!x || !out) { sh_set_error("x and out must not be NULL"); return SH_ERR_INVALID_ARG; }
  if ((uintptr_t)x % 16 != 0 || (uintptr_t)out % 16 != 0) { sh_set_error("x and out must be 16-byte aligned"); return SH_ERR_INVALID_ARG; }
  cudaStream_t st = (cudaStream_t)stream;
  L->launches = 0;
  L->fwd_x = x;
  if (L->dtype == SH_F32) return forward_simt<float, float>(L, SH_STAGE_ALL, x, out, st);
  return sh_tc_forward(L, x, out, st);
}

extern "C" int sh_backward(sh_layer* L, const void* x, const float* dout, float* dx, float* dWq, float* dWk, float* dWv,
                           float* dWo, float* dWs, float* dWd, void* stream) {
  g_err[0] = 0;
  int rc = check_ready(L);
  if (rc != SH_OK) return rc;
  if (L->dtype != SH_F32 || L->dense || L->d.sides != 2 || L->d.Tc > 0 || L->rope || L->xl_positions || L->moe_q || L->moe_k) {
    sh_set_error("sh_backward serves the fp32 configuration of the plain layer (two gates, dense Q/K, no cache, no positional term)");
    return SH_ERR_UNSUPPORTED;
  }
  if (!x || !dout || !dx || !dWq || !dWk || !dWv || !dWo || !dWs || !dWd) { sh_set_error("sh_backward: NULL argument"); return SH_ERR_INVALID_ARG; }
  if (L->fwd_x != x) { sh_set_error("sh_backward needs the intermediates of sh_forward on the same x: call sh_forward(layer, x, ...) first"); return SH_ERR_NOT_CONFIGURED; }
  const ShDims& d = L->d;
  char* ws = L->ws;
  cudaStream_t st = (cudaStream_t)stream;
  const size_t nhd = (size_t)d.N * d.H * d.D;
  ShBwArgs a{};
  a.d = d; a.x = (const float*)x; a.dy = dout;
  a.q = (const float*)(ws + L->o.q); a.k = (const float*)(ws + L->o.k); a.v = (const float*)(ws + L->o.v);
  a.ahat = (const float*)(ws + L->o.ahat);
  a.idx = (const int*)(ws + L->o.idx); a.gate = (const float*)(ws + L->o.gate);
  a.wqk = (const float*)(ws + L->o.wqk); a.wv = (const float*)(ws + L->o.wv); a.wo = (const float*)(ws + L->o.wo);
  a.wgate = (const float*)(ws + L->o.wgate);
  float* scratch = (float*)(ws + L->o.bw);
  a.dq = scratch; a.dk = scratch + nhd; a.dv = scratch + 2 * nhd; a.dahat = scratch + 3 * nhd; a.dgate = scratch + 4 * nhd;
  a.dx = dx; a.dWq = dWq; a.dWk = dWk; a.dWv = dWv; a.dWo = dWo; a.dWs = dWs; a.dWd = dWd;
  SH_CUDA_CHECK(cudaMemsetAsync(a.dk, 0, 2 * nhd * 4, st));                                   // dK, dV: summed by atomics
  SH_CUDA_CHECK(cudaMemsetAsync(dx, 0, (size_t)d.N * d.M * 4, st));
  SH_CUDA_CHECK(cudaMemsetAsync(dWq, 0, (size_t)d.H * d.M * d.Dt * 4, st));
  SH_CUDA_CHECK(cudaMemsetAsync(dWk, 0, (size_t)d.H * d.M * d.Dt * 4, st));
  SH_CUDA_CHECK(cudaMemsetAsync(dWv, 0, (size_t)d.H * d.E * d.M * d.Dt * 4, st));
  SH_CUDA_CHECK(cudaMemsetAsync(dWo, 0, (size_t)d.H * d.E * d.Dt * d.M * 4, st));
  SH_CUDA_CHECK(cudaMemsetAsync(dWs, 0, (size_t)d.H * d.M * d.E * 4, st));
  SH_CUDA_CHECK(cudaMemsetAsync(dWd, 0, (size_t)d.H * d.M * d.E * 4, st));
  sh_bw_o_kernel<<<d.N * d.H, 128, 0, st>>>(a);
  const long rows = (long)d.B * d.H * d.T;
  sh_bw_attn_kernel<<<(unsigned)((rows + 3) / 4), 128, 0, st>>>(a);
  sh_bw_v_kernel<<<d.N * d.H, 128, 0, st>>>(a);
  sh_bw_qk_kernel<<<d.N, 128, (size_t)2 * d.H * d.D * 4, st>>>(a);
  sh_bw_gate_kernel<<<d.N, 128, 0, st>>>(a);
  SH_CUDA_CHECK(cudaGetLastError());
  L->launches = 5;
  return SH_OK;
}

extern "C" int sh_forward_timed(sh_layer* L, const void* x, void* out, void* stream, float* stage_ms) {
  g_err[0] = 0;
  if (!stage_ms) { sh_set_error("stage_ms must not be NULL"); return SH_ERR_INVALID_ARG; }
  if (!L) { sh_set_error("layer is NULL"); return SH_ERR_INVALID_ARG; }
  cudaEvent_t ev[6];
  for (int i = 0; i < 6; ++i) SH_CUDA_CHECK(cudaEventCreate(&ev[i]));
  L->ev = ev;
  int rc = sh_forward(L, x, out, stream);
  L->ev = nullptr;
  if (rc == SH_OK) {
    cudaError_t e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e != cudaSuccess) { sh_set_error("stream synchronise failed: %s", cudaGetErrorString(e)); rc = SH_ERR_CUDA; }
  }
  if (rc == SH_OK) {
    for (int i = 0; i < 5; ++i) cudaEventElapsedTime(&stage_ms[i], ev[i], ev[i + 1]);
    cudaEventElapsedTime(&stage_ms[5], ev[0], ev[5]);
  }
  for (int i = 0; i < 6; ++i) cudaEventDestroy(ev[i]);
  return rc;
}

extern "C" int sh_forward_stamped(sh_layer* L, const void* x, void* out, void* stream, uint64_t* stamps) {
  g_err[0] = 0;
  if (!stamps) { sh_set_error("stamps must not be NULL"); return SH_ERR_INVALID_ARG; }
  int rc = check_ready(L);
  if (rc != SH_OK) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  ShStampBlock* blk = (ShStampBlock*)(L->ws + L->o.stamps);
  SH_CUDA_CHECK(cudaMemsetAsync(blk->resident, 0xFF, 2 * sizeof(blk->resident), st));   // resident and start: minima
  SH_CUDA_CHECK(cudaMemsetAsync(blk->end, 0, sizeof(blk->end), st));                    // end: a maximum
  L->d.stamps = (unsigned long long*)blk;
  rc = sh_forward(L, x, out, stream);
  L->d.stamps = nullptr;
  if (rc != SH_OK) return rc;
  SH_CUDA_CHECK(cudaMemcpyAsync(stamps, blk, sizeof(ShStampBlock), cudaMemcpyDeviceToHost, st));
  SH_CUDA_CHECK(cudaStreamSynchronize(st));
  return SH_OK;
}

struct ShGuardList { size_t off[SH_MAX_GUARDS]; int n; };

// One thread per guard word; counts the damaged ones in *bad.
static __global__ void sh_check_guards_kernel(const unsigned char* ws, ShGuardList gl, int* bad) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  constexpr int words = SH_GUARD_BYTES / 4;
  if (i >= gl.n * words) return;
  const unsigned int v = *(const unsigned int*)(ws + gl.off[i / words] + (size_t)(i % words) * 4);
  if (v != 0x01010101u * SH_GUARD_BYTE) atomicAdd(bad, 1);
}

extern "C" int sh_check_guards(sh_layer* L, void* stream) {
  g_err[0] = 0;
  int rc = check_ready(L);
  if (rc != SH_OK) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  int* bad = (int*)(L->ws + L->o.status) + SH_ST_GUARD_BAD;
  ShGuardList gl{};
  gl.n = L->n_guards;
  for (int i = 0; i < gl.n; ++i) gl.off[i] = L->guard_off[i];
  SH_CUDA_CHECK(cudaMemsetAsync(bad, 0, 4, st));
  const int n = gl.n * (SH_GUARD_BYTES / 4);
  sh_check_guards_kernel<<<(n + 255) / 256, 256, 0, st>>>((const unsigned char*)L->ws, gl, bad);
  int h = 0;
  SH_CUDA_CHECK(cudaMemcpyAsync(&h, bad, 4, cudaMemcpyDeviceToHost, st));
  SH_CUDA_CHECK(cudaStreamSynchronize(st));
  if (h != 0) { sh_set_error("%d guard words behind workspace sub-buffers were overwritten", h); return SH_ERR_BOUNDS; }
  return SH_OK;
}

extern "C" int sh_status_block(sh_layer* L, int32_t* words, void* stream) {
  g_err[0] = 0;
  if (!L || !words) { sh_set_error("NULL argument"); return SH_ERR_INVALID_ARG; }
  if (L->dtype < 0 || !L->ws) { sh_set_error("layer has no workspace yet"); return SH_ERR_NOT_CONFIGURED; }
  SH_CUDA_CHECK(cudaMemcpyAsync(words, L->ws + L->o.status, 16 * 4, cudaMemcpyDeviceToHost, (cudaStream_t)stream));
  SH_CUDA_CHECK(cudaStreamSynchronize((cudaStream_t)stream));
  return SH_OK;
}

extern "C" int sh_clear_status(sh_layer* L, void* stream) {
  g_err[0] = 0;
  if (!L) { sh_set_error("layer is NULL"); return SH_ERR_INVALID_ARG; }
  if (L->dtype < 0 || !L->ws) { sh_set_error("layer has no workspace yet"); return SH_ERR_NOT_CONFIGURED; }
  // the whole block: status word, diagnostics, and the tile and grid-barrier counters a kernel that
  // gave up may have left half-way
  SH_CUDA_CHECK(cudaMemsetAsync(L->ws + L->o.status, 0, 256, (cudaStream_t)stream));
  // (and the early-row value sums with their arrival counters, which the last arrival of a row clears;
  //  the guards between and behind the two are rewritten)
  SH_CUDA_CHECK(cudaMemsetAsync(L->ws + L->o.vearly, 0, L->o.xl_emb - L->o.vearly, (cudaStream_t)stream));
  for (int i = 0; i < L->n_guards; ++i)
    if (L->guard_off[i] >= L->o.vearly && L->guard_off[i] < L->o.xl_emb)
      SH_CUDA_CHECK(cudaMemsetAsync(L->ws + L->guard_off[i], SH_GUARD_BYTE, SH_GUARD_BYTES, (cudaStream_t)stream));
  return SH_OK;
}

extern "C" int sh_selftest(sh_layer* L, int which, uint64_t arg, void* stream) {
  g_err[0] = 0;
  if (!L) { sh_set_error("layer is NULL"); return SH_ERR_INVALID_ARG; }
  if (L->dtype < 0 || !L->ws) { sh_set_error("layer has no workspace yet"); return SH_ERR_NOT_CONFIGURED; }
  if (which != 0 && which != 1) { sh_set_error("unknown self-test %d", which); return SH_ERR_INVALID_ARG; }
  if (which == 0 && arg > 1000000000ull) { sh_set_error("wait limit above one second (got %llu ns)", (unsigned long long)arg); return SH_ERR_INVALID_ARG; }
  return sh_tc_selftest(L, which, arg, (cudaStream_t)stream);
}

extern "C" int sh_is_debug_build(void) {
#ifdef SH_DEBUG
  return 1;
#else
  return 0;
#endif
}

extern "C" int sh_gate_topk(sh_layer* L, const void* x, int32_t* idx, float* gate, int32_t* offsets,
                            int32_t* lists, void* stream) {
  g_err[0] = 0;
  int rc = check_ready(L);
  if (rc != SH_OK) return rc;
  if (L->dense) { sh_set_error("a dense layer has no gates"); return SH_ERR_UNSUPPORTED; }
  if (!x) { sh_set_error("x must not be NULL"); return SH_ERR_INVALID_ARG; }
  cudaStream_t st = (cudaStream_t)stream;
  L->launches = 0;
  rc = (L->dtype == SH_F32) ? launch_gate_sort<float>(L, x, st) : sh_tc_gate_sort(L, x, st);
  if (rc != SH_OK) return rc;
  const ShDims& d = L->d;
  // side s of the outputs <- side s of the workspace (with a shared selection both <- the one side)
  const size_t half = (size_t)d.N * d.H * d.k * 4, ohalf = (size_t)d.H * (d.E + 1) * 4;
  for (int side = 0; side < 2; ++side) {
    const size_t src = d.sides == 2 ? side : 0;
    if (idx) SH_CUDA_CHECK(cudaMemcpyAsync((char*)idx + side * half, L->ws + L->o.idx + src * half, half, cudaMemcpyDeviceToDevice, st));
    if (gate) SH_CUDA_CHECK(cudaMemcpyAsync((char*)gate + side * half, L->ws + L->o.gate + src * half, half, cudaMemcpyDeviceToDevice, st));
    if (offsets) SH_CUDA_CHECK(cudaMemcpyAsync((char*)offsets + side * ohalf, L->ws + L->o.offsets + src * ohalf, ohalf, cudaMemcpyDeviceToDevice, st));
    if (lists) SH_CUDA_CHECK(cudaMemcpyAsync((char*)lists + side * half, L->ws + L->o.lists + src * half, half, cudaMemcpyDeviceToDevice, st));
  }
  return SH_OK;
}

extern "C" int sh_debug_buffer(sh_layer* L, int which, void** dev_ptr, size_t* bytes) {
  g_err[0] = 0;
  if (!L || !dev_ptr || !bytes) { sh_set_error("NULL argument"); return SH_ERR_INVALID_ARG; }
  if (L->dtype < 0 || !L->ws) { sh_set_error("layer has no workspace yet"); return SH_ERR_NOT_CONFIGURED; }
  const ShDims& d = L->d;
  const size_t mid = elem_bytes_mid(L->dtype), act = (size_t)d.N * d.H * d.D * mid;
  const size_t slots = (size_t)2 * d.N * d.H * d.k * 4;
  size_t off, sz;
  switch (which) {
    case SH_BUF_Q: off = L->o.q; sz = act; break;
    case SH_BUF_K: off = L->o.k; sz = act; break;
    case SH_BUF_V: off = L->o.v; sz = act; break;
    case SH_BUF_AHAT: off = L->o.ahat; sz = act; break;
    case SH_BUF_IDX: off = L->o.idx; sz = slots; break;
    case SH_BUF_GATE: off = L->o.gate; sz = slots; break;
    case SH_BUF_OFFSETS: off = L->o.offsets; sz = (size_t)2 * d.H * (d.E + 1) * 4; break;
    case SH_BUF_LISTS: off = L->o.lists; sz = slots; break;
    default: sh_set_error("unknown buffer id %d", which); return SH_ERR_INVALID_ARG;
  }
  *dev_ptr = L->ws + off; *bytes = sz;
  return SH_OK;
}

extern "C" int sh_last_status(sh_layer* L, void* stream) {
  g_err[0] = 0;
  if (!L) { sh_set_error("layer is NULL"); return SH_ERR_INVALID_ARG; }
  if (L->dtype < 0 || !L->ws) { sh_set_error("layer has no workspace yet"); return SH_ERR_NOT_CONFIGURED; }
  int v = 0;
  SH_CUDA_CHECK(cudaMemcpyAsync(&v, L->ws + L->o.status, 4, cudaMemcpyDeviceToHost, (cudaStream_t)stream));
  SH_CUDA_CHECK(cudaStreamSynchronize((cudaStream_t)stream));
  return v;
}

extern "C" int sh_launch_count(const sh_layer* L) { return L ? L->launches : 0; }

extern "C" const char* sh_last_error(void) { return g_err; }

extern "C" void sh_destroy(sh_layer* L) {
  if (!L) return;
  sh_tc_release(L);
  delete L;
}
