// Internal declarations shared by the translation units of libswitchhead.
#pragma once
#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>
#include "../../include/switchhead.h"

#define SH_TILE_ROWS 128   // rows of one grouped-GEMM tile and tokens per gate/sort block

struct ShTile {            // one row tile of one (head, expert) group
  int h, e, row0, nrows;   // row0: position inside lists[side][h]; nrows <= SH_TILE_ROWS
};

struct ShDims {
  int M, H, D, E, k;       // D: d_head as stored (padded with zero columns to 32, 64 or 128)
  int Dt;                  // d_head as given (scale 1/sqrt(Dt), rotary angles)
  int B, T;
  int N;                   // B*T tokens
  int sides;               // 2: source and destination gates; 1: shared selection (one gate serves both)
  int G;                   // gate columns = sides*H*E
  int nblk;                // ceil(N / SH_TILE_ROWS)
  int max_tiles;           // upper bound on row tiles per side
  int tile_rows_src;       // rows per tile of the source-side (value expert) tile table: 128 or 256
  int Tc;                  // Transformer-XL context: the first Tc tokens of every sequence are the cache (keys and values
                           // only); queries, destination gates and out rows exist for the last T - Tc tokens.  0: no cache.
  int causal;              // 1: key s visible to query t iff s <= t (default); 0: every key of the sequence
  int early_rows;          // first tokens of every sequence whose value rows are summed in fp32 (SH_EARLY_ROWS or 0)
  unsigned long long* stamps;   // sh_forward_stamped: the pass's ShStampBlock in the workspace; nullptr otherwise
  int* status;             // the status block at the start of the workspace (nullptr: the allocation-free gate entry point)
};

// Unordered pairs {a < b} of E experts, numbered row by row: (0,1), (0,2), ..., (0,E-1), (1,2), ...
// (the value projection of a k = 2 layer is tiled by (head, pair): sh_tc_vpair_kernel).
__host__ __device__ __forceinline__ int sh_pair_count(int E) { return E * (E - 1) / 2; }
__host__ __device__ __forceinline__ int sh_pair_id(int a, int b, int E) { return a * (2 * E - a - 1) / 2 + (b - a - 1); }
__host__ __device__ __forceinline__ void sh_pair_decode(int id, int E, int& a, int& b) {
  a = 0;
  while (a < E - 2 && id >= E - 1 - a) { id -= E - 1 - a; ++a; }
  b = a + 1 + id;
}

// With a cache in front of every sequence (ShDims::Tc): the row of `out` that belongs to context token
// `tok` (-1 for a cache token), and the context token of an out row.
__host__ __device__ __forceinline__ int sh_out_row(const ShDims& d, int tok) {
  if (d.Tc == 0) return tok;
  const int b = tok / d.T, t = tok % d.T;
  return t < d.Tc ? -1 : b * (d.T - d.Tc) + t - d.Tc;
}
__host__ __device__ __forceinline__ int sh_ctx_tok(const ShDims& d, int row) {
  if (d.Tc == 0) return row;
  const int Tq = d.T - d.Tc;
  return (row / Tq) * d.T + d.Tc + row % Tq;
}
__host__ __device__ __forceinline__ int sh_out_rows(const ShDims& d) { return d.B * (d.T - d.Tc); }

// Per-kernel time stamps of one forward pass (sh_forward_stamped), %globaltimer nanoseconds:
// resident = first CTA of the kernel running, start = first CTA past its wait for the kernel before
// it, end = last CTA done.  Slot = kernel identifier below.
enum { SH_K_GATE = 0, SH_K_SORT = 1, SH_K_QK_A = 2, SH_K_QK_B = 3, SH_K_V = 4, SH_K_ATTN = 5, SH_K_O = 6, SH_K_COUNT = 7 };
struct ShStampBlock { unsigned long long resident[SH_K_COUNT], start[SH_K_COUNT], end[SH_K_COUNT]; };
#ifdef __CUDACC__
// (one thread per CTA calls these; no-ops in an ordinary pass, where the block pointer is null)
__device__ __forceinline__ unsigned long long sh_globaltimer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void sh_stamp_resident(unsigned long long* s, int k) { if (s) atomicMin(s + k, sh_globaltimer_ns()); }
__device__ __forceinline__ void sh_stamp_start(unsigned long long* s, int k) { if (s) atomicMin(s + SH_K_COUNT + k, sh_globaltimer_ns()); }
__device__ __forceinline__ void sh_stamp_end(unsigned long long* s, int k) { if (s) atomicMax(s + 2 * SH_K_COUNT + k, sh_globaltimer_ns()); }
#endif

// Workspace sub-buffers (byte offsets from the workspace base).
// Precision policy of the 16-bit path.  Under the causal mask the first tokens of a sequence attend
// to a handful of keys: their attention read-out is hardly averaged, their output rows are 10-15
// times larger than the RMS of the whole output (which is what the tolerance is measured against),
// and every fp16 rounding on their way - 2^-11 of a LARGE value - counts.  The first SH_EARLY_ROWS
// tokens of every sequence therefore take a more exact route where it is cheap to give them one:
// their value rows are summed in fp32 (scratch of [B, H, SH_EARLY_ROWS, D] floats) and rounded to
// fp16 once by whichever of the k contributions arrives last.  Later rows, averaged over many keys,
// keep the fast form (k fp16 vector reductions into V).  The ratio between the first rows and the RMS
// grows with the sequence length (measured max-abs error / RMS of the fast form alone: 8e-3 at 512
// tokens, 1.4-1.9e-2 at 2048, 1.8-2.4e-2 at 4096, against a tolerance of 2e-2), so the exact route is
// taken from SH_EARLY_MIN_SEQ tokens per sequence on.
#define SH_EARLY_ROWS 32
#define SH_EARLY_MIN_SEQ 1024

struct ShWorkspace {
  size_t status, wqk, wgate, gbias, wv, wo, q, k, v, ahat, idx, gate, blockcnt, blockoff,
         offsets, lists, lgate, tiles, ntiles, rope, vearly, vearly_cnt, xl_emb, xl_r, xl_uv, xl_r16, xl_vr, xl_uk, xl_bias, wos, gid, wq_e, wk_e, bw, stamps, total;
};

// Words of the 256-byte status block at the start of the workspace.
enum {
  SH_ST_STATUS = 0,       // 0, or the first SH_ERR_TIMEOUT / SH_ERR_BOUNDS a kernel recorded
  SH_ST_DIAG = 1,         // 1..6: where the first bounded wait gave up (block, thread, barrier address, parity, grid, block size)
  SH_ST_BOUNDS = 8,       // 8..11: the first failed index check of a debug build (site, value, limit, block)
  SH_ST_SCHED = 16,       // 16, 17: tile counter and finished-claimer counter of the dense Q/K projection
  SH_ST_GRIDBAR = 24,     // 24, 25: grid barrier of the fused gate + sort kernel
  SH_ST_SORTED = 26,      // one-grid front: 128-token blocks whose selections, list entries and tiles are in memory
  SH_ST_GUARD_BAD = 32    // damaged guard words counted by sh_check_guards
};

#define SH_GUARD_BYTES 256
#define SH_GUARD_BYTE 0xC5u
#define SH_MAX_GUARDS 40

struct sh_layer {
  ShDims d{};
  bool dense = false;
  bool moe_q = false, moe_k = false;   // query / key projections are experts too (destination / source side selection)
  bool out_f16 = false;                // sh_set_output_f16: sh_forward writes its result as fp16 (bf16 storage, tensor-core output projection)
  int dtype = -1;
  char* ws = nullptr;
  size_t ws_bytes = 0;
  ShWorkspace o{};
  bool weights_set = false;
  const void* fwd_x = nullptr;   // input of the last forward pass (sh_backward wants the same one)
  bool rope = false;       // rotary position embeddings on Q, K (table in the workspace)
  bool xl_positions = false;   // Transformer-XL relative-position term (fp32 configuration; tables in the workspace)
  int launches = 0;
  int sm_count = 0;
  void* tc = nullptr;      // tensor-core path state (tensor maps), owned by the layer
  cudaEvent_t* ev = nullptr;  // when set (sh_forward_timed): 6 events recorded at the stage boundaries
  size_t guard_off[SH_MAX_GUARDS] = {};   // byte offsets of the guards behind the workspace sub-buffers
  int n_guards = 0;
};

// Shapes the sparse output projection (sh_tc_oproj_sp_kernel) serves: with at most two selections out of
// every four neighbouring experts a token's gate-scaled rows are 2:4 sparse along an expert-innermost
// contraction axis.  The layer then keeps a second, expert-interleaved copy of W_O in the workspace.
inline bool sh_o_sparse_ok(const sh_layer* L) {
  const ShDims& d = L->d;
  return L->dtype == SH_BF16 && !L->dense && d.k <= 2 && (d.E == 4 || d.E == 8) && d.D == 128 && d.H <= 4;
}

// Shapes whose value projection is tiled by (head, pair of selected experts) instead of (head, expert):
// k = 2, so every (token, head) belongs to exactly one pair; few enough pairs for the sort's 32-bit masks.
inline bool sh_v_pairs_ok(const sh_layer* L) {
  const ShDims& d = L->d;
  return L->dtype == SH_BF16 && !L->dense && d.k == 2 && d.E >= 2 && d.E <= 8 && d.D == 128;
}

template <typename T> __device__ __forceinline__ float sh_to_float(T v);
template <> __device__ __forceinline__ float sh_to_float<float>(float v) { return v; }
template <> __device__ __forceinline__ float sh_to_float<__half>(__half v) { return __half2float(v); }
template <> __device__ __forceinline__ float sh_to_float<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T sh_from_float(float v);
template <> __device__ __forceinline__ float sh_from_float<float>(float v) { return v; }
template <> __device__ __forceinline__ __half sh_from_float<__half>(float v) { return __float2half_rn(v); }
template <> __device__ __forceinline__ __nv_bfloat16 sh_from_float<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

void sh_set_error(const char* fmt, ...);

// Index checks of the debug library (built with -DSH_DEBUG): a list entry, tile-table field or
// expert index read from memory is checked against its range before it is used as an address; a
// failed check records SH_ERR_BOUNDS with the site, the value and the limit in the status block and
// the caller skips the access.  The release library compiles them away.
enum { SH_SITE_V_LIST = 1, SH_SITE_V_TILE = 2, SH_SITE_V_TOKEN = 3, SH_SITE_SORT_EXPERT = 4, SH_SITE_SORT_SLOT = 5,
       SH_SITE_O_EXPERT = 6, SH_SITE_SELFTEST = 7 };
#ifdef __CUDACC__
__device__ __forceinline__ bool sh_index_record(long long v, long long limit, int* status, int site) {
  if (v >= 0 && v < limit) return true;
  if (status && atomicCAS(status, 0, SH_ERR_BOUNDS) == 0) {
    status[SH_ST_BOUNDS] = site; status[SH_ST_BOUNDS + 1] = (int)v; status[SH_ST_BOUNDS + 2] = (int)limit; status[SH_ST_BOUNDS + 3] = (int)blockIdx.x;
  }
  return false;
}
#ifdef SH_DEBUG
#define SH_INDEX_OK(v, limit, status, site) sh_index_record((long long)(v), (long long)(limit), (status), (site))
#else
#define SH_INDEX_OK(v, limit, status, site) true
#endif
#endif

// Stage boundary marker: boundary 0 = start, 1 = after gate+sort, 2 = after Q/K, 3 = after V,
// 4 = after attention, 5 = after the output projection.
static inline void sh_mark(sh_layer* L, int boundary, cudaStream_t st) {
  if (L->ev) cudaEventRecord(L->ev[boundary], st);
}

enum { SH_STAGE_GATE = 1, SH_STAGE_QK = 2, SH_STAGE_V = 4, SH_STAGE_ATTN = 8, SH_STAGE_O = 16, SH_STAGE_ALL = 31 };

// CUDA-core stages on bf16 storage with fp16 intermediates (same buffers and layouts as the
// tensor-core kernels): the on-device reference used while a tensor-core stage is brought up.
int sh_simt_run_bf16(sh_layer* L, int stages, const void* x, void* out, cudaStream_t st);

// Tensor-core (tcgen05) path of the bf16 configuration.
int sh_tc_prepare(sh_layer* L);                 // builds tensor maps after the weights are repacked
void sh_tc_release(sh_layer* L);
int sh_tc_forward(sh_layer* L, const void* x, void* out, cudaStream_t st);
int sh_tc_gate_sort(sh_layer* L, const void* x, cudaStream_t st);
int sh_tc_selftest(sh_layer* L, int which, unsigned long long arg, cudaStream_t st);
