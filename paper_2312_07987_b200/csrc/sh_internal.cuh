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
  int causal;              // 1: key s visible to query t iff s <= t (default); 0: every key of the sequence
};

// Workspace sub-buffers (byte offsets from the workspace base).
struct ShWorkspace {
  size_t status, wqk, wgate, gbias, wv, wo, q, k, v, ahat, idx, gate, blockcnt, blockoff,
         offsets, lists, lgate, tiles, ntiles, rope, v32, total;
};

struct sh_layer {
  ShDims d{};
  bool dense = false;
  int dtype = -1;
  char* ws = nullptr;
  size_t ws_bytes = 0;
  ShWorkspace o{};
  bool weights_set = false;
  bool rope = false;       // rotary position embeddings on Q, K (table in the workspace)
  int launches = 0;
  int sm_count = 0;
  void* tc = nullptr;      // tensor-core path state (tensor maps), owned by the layer
  cudaEvent_t* ev = nullptr;  // when set (sh_forward_timed): 6 events recorded at the stage boundaries
};

template <typename T> __device__ __forceinline__ float sh_to_float(T v);
template <> __device__ __forceinline__ float sh_to_float<float>(float v) { return v; }
template <> __device__ __forceinline__ float sh_to_float<__half>(__half v) { return __half2float(v); }
template <> __device__ __forceinline__ float sh_to_float<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T sh_from_float(float v);
template <> __device__ __forceinline__ float sh_from_float<float>(float v) { return v; }
template <> __device__ __forceinline__ __half sh_from_float<__half>(float v) { return __float2half_rn(v); }
template <> __device__ __forceinline__ __nv_bfloat16 sh_from_float<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

void sh_set_error(const char* fmt, ...);

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
