// sh_noalloc_gate_topk: the gate + top-k + bucket-sort stage for callers that cannot allocate.
// Its scratch memory (per-block selection histograms, the gate values in list order and the
// row-tile table that the sort kernel emits) lives in file-scope __device__ arrays of fixed
// size instead of a caller-provided workspace.  Documented in include/switchhead.h.
#include <cstdio>

#include "sh_internal.cuh"
#include "sh_simt.cuh"

#define SH_NOALLOC_MAX_TOKENS 16384
#define SH_NOALLOC_MAX_GATE_COLS 256
#define SH_NOALLOC_MAX_SLOTS 262144     /* n_tokens * n_heads * k, per side */
#define SH_NOALLOC_MAX_DEVICES 64

namespace {

constexpr int kMaxBlocks = SH_NOALLOC_MAX_TOKENS / SH_TILE_ROWS;
constexpr int kMaxTiles = SH_NOALLOC_MAX_SLOTS / SH_TILE_ROWS + SH_NOALLOC_MAX_GATE_COLS;

// Every GPU that loads the library holds these arrays (about 2.3 MB) until the process exits.
static __device__ __align__(256) int g_blockcnt[kMaxBlocks * SH_NOALLOC_MAX_GATE_COLS];
static __device__ __align__(256) float g_lgate[2 * SH_NOALLOC_MAX_SLOTS];
static __device__ __align__(256) ShTile g_tiles[2 * kMaxTiles];
static __device__ __align__(256) int g_ntiles[64];
static __device__ __align__(256) float g_zero_bias[SH_NOALLOC_MAX_GATE_COLS];   // never written: stays zero

struct DeviceScratch {
  bool ready = false;
  int* blockcnt = nullptr;
  float* lgate = nullptr;
  ShTile* tiles = nullptr;
  int* ntiles = nullptr;
  float* zero_bias = nullptr;
};
DeviceScratch g_scratch[SH_NOALLOC_MAX_DEVICES];

// In host code the array names are host-side stand-ins, not device addresses: the addresses
// the kernels need come from cudaGetSymbolAddress, once per device, with that device current.
int setup_device(int dev, DeviceScratch** out) {
  if (dev < 0 || dev >= SH_NOALLOC_MAX_DEVICES) { sh_set_error("device ordinal %d is out of range", dev); return SH_ERR_UNSUPPORTED; }
  DeviceScratch& s = g_scratch[dev];
  if (!s.ready) {
    cudaError_t e;
    if ((e = cudaGetSymbolAddress((void**)&s.blockcnt, g_blockcnt)) != cudaSuccess ||
        (e = cudaGetSymbolAddress((void**)&s.lgate, g_lgate)) != cudaSuccess ||
        (e = cudaGetSymbolAddress((void**)&s.tiles, g_tiles)) != cudaSuccess ||
        (e = cudaGetSymbolAddress((void**)&s.ntiles, g_ntiles)) != cudaSuccess ||
        (e = cudaGetSymbolAddress((void**)&s.zero_bias, g_zero_bias)) != cudaSuccess) {
      sh_set_error("cudaGetSymbolAddress failed: %s", cudaGetErrorString(e));
      return SH_ERR_CUDA;
    }
    s.ready = true;
  }
  *out = &s;
  return SH_OK;
}

template <typename T>
int run(const ShDims& d, DeviceScratch* s, const void* x, const void* w_gate, const float* bias, int32_t* idx,
        float* gate, int32_t* offsets, int32_t* lists, cudaStream_t st) {
  const size_t ssm = sh_sort_smem_bytes(d);
  if (ssm > 48 * 1024) {
    sh_set_error("n_heads * k = %d needs %zu bytes of shared memory in the sort kernel; the limit of this entry point is 48 KB",
                 d.H * d.k, ssm);
    return SH_ERR_UNSUPPORTED;
  }
  // every block overwrites its whole histogram row, so the array needs no clearing
  sh_gate_topk_kernel<T><<<d.nblk, 256, (size_t)d.G * 4, st>>>((const T*)x, (const T*)w_gate, bias ? bias : s->zero_bias,
                                                              idx, gate, s->blockcnt, d);
  sh_sort_kernel<<<d.nblk, sh_sort_threads(d), ssm, st>>>(idx, gate, s->blockcnt, offsets, lists, s->lgate, s->tiles,
                                                        s->ntiles, d);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) { sh_set_error("kernel launch failed: %s", cudaGetErrorString(e)); return SH_ERR_CUDA; }
  return SH_OK;
}

}  // namespace

extern "C" int sh_noalloc_gate_topk(int dtype, int n_tokens, int d_model, int n_heads, int n_experts, int k,
                                    const void* x, const void* w_gate, const float* bias, int32_t* idx, float* gate,
                                    int32_t* offsets, int32_t* lists, void* stream) {
  sh_set_error("%s", "");
  if (dtype != SH_F32 && dtype != SH_BF16) { sh_set_error("dtype must be SH_F32 or SH_BF16 (got %d)", dtype); return SH_ERR_INVALID_ARG; }
  if (n_tokens < 1 || d_model < 1 || n_heads < 1 || n_experts < 1 || n_experts > 32 || k < 1 || k > n_experts) {
    sh_set_error("invalid dimensions: n_tokens=%d d_model=%d n_heads=%d n_experts=%d k=%d", n_tokens, d_model, n_heads, n_experts, k);
    return SH_ERR_INVALID_ARG;
  }
  if (!x || !w_gate || !idx || !gate || !offsets || !lists) { sh_set_error("x, w_gate, idx, gate, offsets and lists must not be NULL"); return SH_ERR_INVALID_ARG; }
  const long long G = 2ll * n_heads * n_experts, slots = (long long)n_tokens * n_heads * k;
  if (n_tokens > SH_NOALLOC_MAX_TOKENS || G > SH_NOALLOC_MAX_GATE_COLS || slots > SH_NOALLOC_MAX_SLOTS) {
    sh_set_error("sh_noalloc_gate_topk is limited to %d tokens, %d gate columns (2*n_heads*n_experts) and %d selections per side "
                 "(n_tokens*n_heads*k); got %d, %lld, %lld", SH_NOALLOC_MAX_TOKENS, SH_NOALLOC_MAX_GATE_COLS,
                 SH_NOALLOC_MAX_SLOTS, n_tokens, G, slots);
    return SH_ERR_UNSUPPORTED;
  }
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) { sh_set_error("cudaGetDevice failed: %s", cudaGetErrorString(e)); return SH_ERR_CUDA; }
  DeviceScratch* s = nullptr;
  int rc = setup_device(dev, &s);
  if (rc != SH_OK) return rc;
  ShDims d{};
  d.M = d_model; d.H = n_heads; d.D = 0; d.E = n_experts; d.k = k;
  d.B = 1; d.T = n_tokens; d.N = n_tokens; d.sides = 2; d.G = (int)G;
  d.nblk = (n_tokens + SH_TILE_ROWS - 1) / SH_TILE_ROWS;
  d.max_tiles = kMaxTiles;
  d.tile_rows_src = SH_TILE_ROWS;
  cudaStream_t st = (cudaStream_t)stream;
  return dtype == SH_F32 ? run<float>(d, s, x, w_gate, bias, idx, gate, offsets, lists, st)
                         : run<__nv_bfloat16>(d, s, x, w_gate, bias, idx, gate, offsets, lists, st);
}
