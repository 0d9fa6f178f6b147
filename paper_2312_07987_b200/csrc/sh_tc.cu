// Tensor-core (tcgen05) path of the bf16 configuration: tensor maps and launch sequence.
#include <cstdlib>
#include <mutex>
#include <new>
#include <utility>

#include "sh_internal.cuh"
#include "sh_simt.cuh"
#include "sh_tc_gemm.cuh"
#include "sh_tc_pgemm.cuh"
#include "sh_tc_attn2.cuh"
#include "sh_tc_attn3.cuh"
#include "sh_tc_gate.cuh"
#include "sh_tc_oproj2.cuh"
#include "sh_tc_qkpair.cuh"
#include "sh_tc_xlbias.cuh"
#include "sh_tc_oproj_sp.cuh"
#include "sh_tc_vpair.cuh"
#include "sh_tc_front.cuh"

using namespace shtc;

#define SH_CUDA_CHECK(expr)                                                          \
  do {                                                                               \
    cudaError_t _e = (expr);                                                         \
    if (_e != cudaSuccess) {                                                         \
      sh_set_error("%s failed: %s", #expr, cudaGetErrorString(_e));                  \
      return SH_ERR_CUDA;                                                            \
    }                                                                                \
  } while (0)

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)p;
  }
  return fn;
}

// 2-D row-major tensor [outer, inner] of 16-bit elements, 128-byte swizzle, box = box_outer
// rows of box_inner (= 64) elements.
int sh_tc_encode_2d(CUtensorMap* map, int elem_kind, const void* base, uint64_t inner, uint64_t outer,
                    uint64_t outer_stride_bytes, uint32_t box_inner, uint32_t box_outer) {
  EncodeTiledFn enc = get_encode();
  if (!enc) { sh_set_error("cuTensorMapEncodeTiled is not available from the driver"); return SH_ERR_CUDA; }
  cuuint64_t dims[2] = {inner, outer};
  cuuint64_t strides[1] = {outer_stride_bytes};
  cuuint32_t box[2] = {box_inner, box_outer};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = enc(map, elem_kind == 0 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2,
                   const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                   CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) { sh_set_error("cuTensorMapEncodeTiled failed with CUresult %d", (int)r); return SH_ERR_CUDA; }
  return SH_OK;
}

// 3-D tensor [n2, n1, inner] of fp16 (Q, K, V as [B*H, T, D]); box = 128 rows of 64 elements of
// one (batch, head) slice, so rows past the end of a sequence read as zero.
static int encode_3d_f16(CUtensorMap* map, const void* base, uint64_t inner, uint64_t n1, uint64_t n2) {
  EncodeTiledFn enc = get_encode();
  if (!enc) { sh_set_error("cuTensorMapEncodeTiled is not available from the driver"); return SH_ERR_CUDA; }
  cuuint64_t dims[3] = {inner, n1, n2};
  cuuint64_t strides[2] = {inner * 2, inner * n1 * 2};
  cuuint32_t box[3] = {64, 128, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) { sh_set_error("cuTensorMapEncodeTiled (3-D) failed with CUresult %d", (int)r); return SH_ERR_CUDA; }
  return SH_OK;
}

// The same tensor in boxes of 32 rows of 32 elements with the 64-byte swizzle: the tiles one epilogue
// warp of the one-grid front stores.
static int encode_3d_f16_store32(CUtensorMap* map, const void* base, uint64_t inner, uint64_t n1, uint64_t n2) {
  EncodeTiledFn enc = get_encode();
  if (!enc) { sh_set_error("cuTensorMapEncodeTiled is not available from the driver"); return SH_ERR_CUDA; }
  cuuint64_t dims[3] = {inner, n1, n2};
  cuuint64_t strides[2] = {inner * 2, inner * n1 * 2};
  cuuint32_t box[3] = {32, 32, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) { sh_set_error("cuTensorMapEncodeTiled (3-D, store) failed with CUresult %d", (int)r); return SH_ERR_CUDA; }
  return SH_OK;
}

struct TcState {
  CUtensorMap map_q, map_k, map_v;
  CUtensorMap map_q_st, map_k_st;   // Q and K as the one-grid front's epilogue stores them
  CUtensorMap map_wqk, map_wqk128, map_wv, map_wq_e, map_wk_e, map_wo, map_wo256, map_wos, map_ahat, map_wgate;
  CUtensorMap map_q2d, map_r16;  // score-bias GEMM of the Transformer-XL position term: Q as [B*H*T, D], R16 as [H*T, D]
  CUtensorMap map_x;             // tensor map of the last x pointer seen (x_cached)
  CUtensorMap map_x64;           // the same tensor in 64-token boxes (gate tile of the one-grid front, 64 tokens per CTA)
  CUtensorMap map_wgate_half;    // gate weights in boxes of gate_gp / 2 rows (each CTA of a pair loads half)
  const void* x_cached = nullptr;
  int gate_gp;          // gate columns padded to a multiple of 16; 0 = CUDA-core gate kernel (more than 256 gate columns)
  int qk_bn;            // column tile of the dense projection: 256 (CTA pairs / persistent) when 2*H*D allows, else 128
  int o_pairs_max;      // clusters of the CTA-pair output projection the device holds at once (0: not asked yet, -1: none)
  int qk_pairs_max;     // the same for the dense Q/K projection
  int gate_coop;        // 1: the gate kernel can be launched cooperatively (fused sort), -1: it cannot
  int front = 0;        // one-grid front (sh_tc_front_kernel): 0 = not asked yet, 1 = usable, -1 = not
  int front_stages = 0, front_smem = 0, front_pairs = 0, front_sort_bytes = 0;
  // Launch-structure switches.  The release library fixes them here; a library built with SH_DEBUG
  // reads them from the environment once, in sh_tc_prepare, for A/B runs and for the tests that
  // drive the less-travelled launch paths.
  bool pdl = true;          // kernels of the caller's stream chained by programmatic dependent launch
  bool overlap = true;      // Q/K projection on a side stream beside gate + sort
  bool qk_two_grids = true; // ... as two grids around the gate kernel
  bool qk_pair = true;      // CTA-pair Q/K kernel (else single-CTA persistent)
  bool o_pair = true;       // CTA-pair output projection for k <= 3 (else single-CTA)
  bool v_pairs = true;      // value projection tiled by (head, expert pair) on CTA pairs where the shape allows (sh_v_pairs_ok)
  int v_pairs_max = 0;      // clusters of that kernel the device holds at once (0: not asked yet, -1: none)
  bool o_sparse = true;     // sparse-A CTA-pair output projection where the shape allows (sh_o_sparse_ok)
  bool persistent = true;   // persistent Q/K and value-expert GEMMs (else one CTA per tile)
  bool fused_sort = true;   // sort fused into the gate kernel when it needs at most half of the SMs
  bool one_grid_front = true;   // gate, selection, sort and the dense Q/K projection as one grid where the shape allows
  bool attn_balanced = true;
  int simt_mask = 0;        // SH_DEBUG only: stages forced onto the CUDA-core kernels
  cudaStream_t side = nullptr, side2 = nullptr;   // Q/K grids A and B
  cudaEvent_t ev_fork = nullptr, ev_join = nullptr, ev_join2 = nullptr;
};

constexpr int QK_STAGES = 4;

// Kernel launch, optionally with the programmatic-stream-serialization attribute: the kernel may
// then become resident while the kernel before it in the stream is still running, and decides
// itself (griddepcontrol.wait) when it needs that kernel's results.
template <typename... P, typename... A>
static int launch_k(bool pdl, void (*kern)(P...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, A&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = pdl ? 1 : 0;
  SH_CUDA_CHECK(cudaLaunchKernelEx(&cfg, kern, std::forward<A>(args)...));
  return SH_OK;
}

// The same for a kernel that runs as clusters of two CTAs (grid.x even).
template <typename... P, typename... A>
static int launch_k_pairs(bool pdl, void (*kern)(P...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, A&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = pdl ? 2 : 1;
  SH_CUDA_CHECK(cudaLaunchKernelEx(&cfg, kern, std::forward<A>(args)...));
  return SH_OK;
}

// How many two-CTA clusters of a kernel the device holds at once (0 on error).
template <typename K>
static int max_pairs(K kern, int block, size_t smem) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2); cfg.blockDim = dim3(block); cfg.dynamicSmemBytes = smem;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess) { cudaGetLastError(); return 0; }
  return n;
}

// Dynamic shared memory limit and carve-out of a kernel, set once per (kernel, device, size): the
// attributes belong to the device's copy of the function, so a process that drives several GPUs
// must set them on each.  Always the largest shared-memory carve-out: kernels of one forward pass
// share SMs (a sort block beside a GEMM CTA; the next kernel's CTAs arriving while this one
// drains), and an SM set up with a smaller carve-out has to run empty before it can be set up again.
struct SmemAttr { const void* fn; int dev; int bytes; };
static SmemAttr g_smem_attr[128];
static int g_smem_attr_n = 0;
static std::mutex g_smem_attr_mutex;     // layers may be driven from several host threads

template <typename K>
static int set_smem(K kernel, int bytes) {
  std::lock_guard<std::mutex> lock(g_smem_attr_mutex);
  int dev = 0;
  SH_CUDA_CHECK(cudaGetDevice(&dev));
  const void* fn = (const void*)kernel;
  SmemAttr* slot = nullptr;
  for (int i = 0; i < g_smem_attr_n; ++i)
    if (g_smem_attr[i].fn == fn && g_smem_attr[i].dev == dev) slot = &g_smem_attr[i];
  if (slot && slot->bytes >= bytes) return SH_OK;
  if (bytes > 48 * 1024 || !slot)
    SH_CUDA_CHECK(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes > 48 * 1024 ? bytes : 48 * 1024));
  if (!slot) {
    SH_CUDA_CHECK(cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared));
    if (g_smem_attr_n < 128) slot = &g_smem_attr[g_smem_attr_n++];
  }
  if (slot) { slot->fn = fn; slot->dev = dev; slot->bytes = bytes; }
  return SH_OK;
}

void sh_tc_release(sh_layer* L) {
  if (L && L->tc) {
    TcState* S = (TcState*)L->tc;
    if (S->ev_fork) cudaEventDestroy(S->ev_fork);
    if (S->ev_join) cudaEventDestroy(S->ev_join);
    if (S->side) cudaStreamDestroy(S->side);
    if (S->ev_join2) cudaEventDestroy(S->ev_join2);
    if (S->side2) cudaStreamDestroy(S->side2);
    delete S;
    L->tc = nullptr;
  }
}

int sh_tc_prepare(sh_layer* L) {
  sh_tc_release(L);
  TcState* S = new (std::nothrow) TcState();
  if (!S) { sh_set_error("out of host memory"); return SH_ERR_INVALID_ARG; }
  L->tc = S;
  const ShDims& d = L->d;
  char* ws = L->ws;
  const int HD = d.H * d.D;
  const int nproj = L->dense ? 3 : 2;
#ifdef SH_DEBUG
  // A/B switches of the debug library (read once, here)
  S->pdl = !getenv("SH_NO_PDL");
  S->overlap = !getenv("SH_NO_OVERLAP");
  S->qk_two_grids = !getenv("SH_QK_ONE_GRID");
  S->qk_pair = !getenv("SH_QK_SINGLE");
  S->o_pair = !getenv("SH_O_SINGLE");
  S->o_sparse = !getenv("SH_O_MASKED");
  S->v_pairs = !getenv("SH_V_BY_EXPERT");
  S->persistent = !getenv("SH_NO_PERSISTENT");
  S->fused_sort = !getenv("SH_SORT_SEPARATE");
  S->one_grid_front = !getenv("SH_NO_FRONT");
  S->attn_balanced = !getenv("SH_ATTN_ADJACENT");
  if (const char* env = getenv("SH_SIMT_STAGES")) S->simt_mask = atoi(env);   // bit mask gate=1, qk=2, v=4, attention=8, o=16
#endif
  // d_head above 128 (stored as 256: the paper's 132 and 168): S and O of two query tiles no longer fit the 512
  // tensor-memory columns and the expert kernels are built for 64 / 128 columns, so every stage of such a layer
  // runs on the CUDA-core kernels (bf16 weights and x, fp16 intermediates, fp32 sums) - correct, not fast
  if (d.D > 128) S->simt_mask = SH_STAGE_GATE | SH_STAGE_QK | SH_STAGE_V | SH_STAGE_ATTN | SH_STAGE_O;
  // 256-column tiles (CTA pairs, or the persistent single-CTA kernel) need the projection's width to
  // be a multiple of 256; other widths take the one-CTA-per-tile kernel with 128-column tiles
  S->qk_bn = (nproj * HD) % 256 == 0 ? 256 : 128;
  // The kernels of the caller's stream are chained by programmatic dependent launch (each becomes
  // resident while the one before it drains, and waits on the device for its results); the dense
  // Q/K projection, which needs nothing from the gate and sort kernels, is launched the ordinary way
  // on side streams so that it runs beside them.
  if (!L->dense && S->overlap) {
    SH_CUDA_CHECK(cudaStreamCreateWithFlags(&S->side, cudaStreamNonBlocking));
    SH_CUDA_CHECK(cudaEventCreateWithFlags(&S->ev_fork, cudaEventDisableTiming));
    SH_CUDA_CHECK(cudaEventCreateWithFlags(&S->ev_join, cudaEventDisableTiming));
    SH_CUDA_CHECK(cudaStreamCreateWithFlags(&S->side2, cudaStreamNonBlocking));
    SH_CUDA_CHECK(cudaEventCreateWithFlags(&S->ev_join2, cudaEventDisableTiming));
  }
  S->o_pairs_max = 0;
  S->qk_pairs_max = 0;
  S->gate_coop = 0;
  if (L->sm_count == 0) {
    int dev = 0;
    SH_CUDA_CHECK(cudaGetDevice(&dev));
    SH_CUDA_CHECK(cudaDeviceGetAttribute(&L->sm_count, cudaDevAttrMultiProcessorCount, dev));
  }
  // value experts: 256-row tiles halve the weight traffic, but only pay off while there are
  // enough of them to fill the SMs one and a half times
  const long long slots = (long long)d.N * d.H * d.k;
  const bool big = slots / 256 >= (3ll * L->sm_count) / 2;
  // (the CUDA-core stages of the debug library read 128-row tiles; with a shared selection its output
  //  projection reads the source side's table)
  const bool simt_tiles = (S->simt_mask & SH_STAGE_V) || (L->d.sides == 1 && (S->simt_mask & SH_STAGE_O));
  L->d.tile_rows_src = (L->dense || simt_tiles || !big) ? 128 : 256;
  int rc;
  if ((rc = sh_tc_encode_2d(&S->map_wqk, 0, ws + L->o.wqk, d.M, (uint64_t)nproj * HD, (uint64_t)d.M * 2, 64, S->qk_bn))) return rc;
  if ((rc = sh_tc_encode_2d(&S->map_wqk128, 0, ws + L->o.wqk, d.M, (uint64_t)nproj * HD, (uint64_t)d.M * 2, 64, 128))) return rc;
  if (!L->dense) {
    if ((rc = sh_tc_encode_2d(&S->map_wv, 0, ws + L->o.wv, d.M, (uint64_t)d.H * d.E * d.D, (uint64_t)d.M * 2, 64, d.D))) return rc;
    if (L->moe_q && (rc = sh_tc_encode_2d(&S->map_wq_e, 0, ws + L->o.wq_e, d.M, (uint64_t)d.H * d.E * d.D, (uint64_t)d.M * 2, 64, d.D))) return rc;
    if (L->moe_k && (rc = sh_tc_encode_2d(&S->map_wk_e, 0, ws + L->o.wk_e, d.M, (uint64_t)d.H * d.E * d.D, (uint64_t)d.M * 2, 64, d.D))) return rc;
    if ((rc = sh_tc_encode_2d(&S->map_wo, 1, ws + L->o.wo, d.D, (uint64_t)d.H * d.E * d.M, (uint64_t)d.D * 2, 64, 128))) return rc;
    if ((rc = sh_tc_encode_2d(&S->map_wo256, 1, ws + L->o.wo, d.D, (uint64_t)d.H * d.E * d.M, (uint64_t)d.D * 2, 64, 256))) return rc;
    if (sh_o_sparse_ok(L) && (rc = sh_tc_encode_2d(&S->map_wos, 1, ws + L->o.wos, (uint64_t)d.D * d.E, (uint64_t)d.H * d.M, (uint64_t)d.D * d.E * 2, 64, 128))) return rc;
  } else {
    if ((rc = sh_tc_encode_2d(&S->map_wo, 1, ws + L->o.wo, HD, d.M, (uint64_t)HD * 2, 64, 128))) return rc;
  }
  S->gate_gp = 0;
  if (!L->dense && (d.G + 15) / 16 * 16 <= 256) {
    S->gate_gp = (d.G + 15) / 16 * 16;
    if ((rc = sh_tc_encode_2d(&S->map_wgate, 0, ws + L->o.wgate, d.M, d.G, (uint64_t)d.M * 2, 64, S->gate_gp))) return rc;
    if ((rc = sh_tc_encode_2d(&S->map_wgate_half, 0, ws + L->o.wgate, d.M, d.G, (uint64_t)d.M * 2, 64, S->gate_gp / 2))) return rc;
  }
  if ((rc = encode_3d_f16(&S->map_q, ws + L->o.q, d.D, d.T, (uint64_t)d.B * d.H))) return rc;
  if ((rc = encode_3d_f16(&S->map_k, ws + L->o.k, d.D, d.T, (uint64_t)d.B * d.H))) return rc;
  if ((rc = encode_3d_f16(&S->map_v, ws + L->o.v, d.D, d.T, (uint64_t)d.B * d.H))) return rc;
  if ((rc = encode_3d_f16_store32(&S->map_q_st, ws + L->o.q, d.D, d.T, (uint64_t)d.B * d.H))) return rc;
  if ((rc = encode_3d_f16_store32(&S->map_k_st, ws + L->o.k, d.D, d.T, (uint64_t)d.B * d.H))) return rc;
  if ((rc = sh_tc_encode_2d(&S->map_ahat, 1, ws + L->o.ahat, HD, d.N, (uint64_t)HD * 2, 64, 128))) return rc;
  if (!L->dense && d.Tc > 0) {
    if ((rc = sh_tc_encode_2d(&S->map_q2d, 1, ws + L->o.q, d.D, (uint64_t)d.B * d.H * d.T, (uint64_t)d.D * 2, 64, 128))) return rc;
    if ((rc = sh_tc_encode_2d(&S->map_r16, 1, ws + L->o.xl_r16, d.D, (uint64_t)d.H * d.T, (uint64_t)d.D * 2, 64, 64))) return rc;
  }
  return SH_OK;
}

// The tensor map of x [N, M] (128-token x 64-column boxes); kept for the pointer last seen, since a
// caller usually passes the same one or two buffers pass after pass.
static int x_map(sh_layer* L, const void* x, const CUtensorMap** out) {
  TcState* S = (TcState*)L->tc;
  if (S->x_cached != x) {
    const ShDims& d = L->d;
    if (int rc = sh_tc_encode_2d(&S->map_x, 0, x, d.M, d.N, (uint64_t)d.M * 2, 64, 128)) return rc;
    if (int rc = sh_tc_encode_2d(&S->map_x64, 0, x, d.M, d.N, (uint64_t)d.M * 2, 64, 64)) return rc;
    S->x_cached = x;
  }
  *out = &S->map_x;
  return SH_OK;
}

// The gate kernel's x stream comes cold from HBM (~1.2 us per box round trip), so what bounds its
// main loop is the bytes in flight per CTA: 8 stages when they fit, else 4.
static int gate_smem_bytes(int Gp, int G, int stages) {   // G: histogram width (gate columns, or (head, pair) buckets if more)
  const int stage = 128 * 64 * 2 + ((Gp * 128 + 1023) & ~1023);
  const int pipe = stages * stage, stag = 128 * (Gp + 1) * 4;
  const int bar_off = ((pipe > stag ? pipe : stag) + 1023) & ~1023;
  return bar_off + 256 + 3 * G * 4 + 1024;
}

using VPS = VPairSmem<6>;
// Forward passes of a k = 2 layer tile the value projection by (head, pair of selected experts): the gate
// kernel then buckets the source side by pair, and sh_tc_vpair_kernel replaces the expert-tiled kernel.
static bool use_v_pairs(sh_layer* L) {
  TcState* S = (TcState*)L->tc;
  if (!S->v_pairs || !sh_v_pairs_ok(L) || !S->gate_gp || (S->simt_mask & (SH_STAGE_GATE | SH_STAGE_V))) return false;
  if (S->v_pairs_max == 0) {
    if (set_smem(sh_tc_vpair_kernel<6>, VPS::TOTAL) != SH_OK) S->v_pairs_max = -1;
    else {
      S->v_pairs_max = max_pairs(sh_tc_vpair_kernel<6>, 320, VPS::TOTAL);
      if (S->v_pairs_max <= 0) S->v_pairs_max = -1;
    }
  }
  return S->v_pairs_max > 0;
}

// Gate + top-k + bucket sort.  With zero_for_forward the gate kernel also clears the value buffer.
static int tc_gate_sort(sh_layer* L, const void* x, void* out, bool zero_for_forward, cudaStream_t st, bool sort_apart = false) {
  TcState* S = (TcState*)L->tc;
  const ShDims& d = L->d;
  char* ws = L->ws;
  int rc;
  if (!S->gate_gp || (S->simt_mask & SH_STAGE_GATE)) {
    // more than 256 gate columns (or the debug library's switch): the CUDA-core gate kernel
    if ((rc = sh_simt_run_bf16(L, SH_STAGE_GATE, x, nullptr, st))) return rc;
    if (zero_for_forward) {
      SH_CUDA_CHECK(cudaMemsetAsync(ws + L->o.v, 0, (size_t)d.N * d.H * d.D * 2, st));
      if (S->simt_mask & SH_STAGE_O) SH_CUDA_CHECK(cudaMemsetAsync(out, 0, (size_t)sh_out_rows(d) * d.M * 4, st));
      L->launches += 2;
    }
    return SH_OK;
  }
  const CUtensorMap* map_x;
  if ((rc = x_map(L, x, &map_x))) return rc;
  TcGateArgs g{};
  g.d = d; g.Gp = S->gate_gp; g.gbias = (const float*)(ws + L->o.gbias);
  g.idx = (int*)(ws + L->o.idx); g.gate = (float*)(ws + L->o.gate);
  g.blockcnt = (int*)(ws + L->o.blockcnt);
  const bool vp = zero_for_forward && use_v_pairs(L);
  // (query experts are tiled by the DESTINATION side's pairs: then both sides are bucketed by pair)
  g.vpairs = vp ? ((L->moe_q && d.sides == 2) ? 2 : 1) : 0;
  g.NP = sh_pair_count(d.E); g.GH = vp ? g.vpairs * d.H * g.NP : d.G; g.gid = (int*)(ws + L->o.gid);
  const int GHmax = g.GH > d.G ? g.GH : d.G;
  g.zero_v = (zero_for_forward && !vp) ? (void*)(ws + L->o.v) : nullptr;    // (the pair-tiled kernel stores every value row once)
  g.zero_out = (zero_for_forward && (S->simt_mask & SH_STAGE_O) && d.Tc == 0) ? (float*)out : nullptr;
  if (zero_for_forward && (S->simt_mask & SH_STAGE_O) && d.Tc > 0)          // (out has fewer rows than there are tokens)
    SH_CUDA_CHECK(cudaMemsetAsync(out, 0, (size_t)sh_out_rows(d) * d.M * 4, st));
  g.status = (int*)(ws + L->o.status);
  const bool deep = gate_smem_bytes(S->gate_gp, GHmax, 8) <= 200 * 1024;
  const int smem = gate_smem_bytes(S->gate_gp, GHmax, deep ? 8 : 4);
  if ((rc = deep ? set_smem(sh_tc_gate_kernel<8>, smem) : set_smem(sh_tc_gate_kernel<4>, smem))) return rc;
  // In a forward pass only the value experts read sorted lists (the output projection works from
  // idx / gate, token tile by token tile), so only the source side is sorted there -- unless the
  // debug library's CUDA-core output projection is selected.  The histogram stride stays G; the
  // sort's loops run over sides * H groups.
  ShDims ds = d;
  if (zero_for_forward && !(S->simt_mask & SH_STAGE_O)) ds.sides = 1;
  if (vp) { ds.sides = g.vpairs; ds.E = g.NP; ds.k = 1; ds.G = g.GH; ds.tile_rows_src = 256; }   // buckets (side, head, pair), one entry per (token, head)
  // Fused sort: when every CTA of the gate kernel can be resident at once (cooperative launch) and the
  // sort's scratch fits behind the logits tile in the idle operand ring, the gate kernel places the
  // tokens itself and there is no sort kernel.  Used when the gate kernel needs at most half of the SMs:
  // 114.8 -> 110.7 us per forward at 8192 tokens (64 CTAs), but 270.7 -> 273.3 at 16384 (128 CTAs that
  // must all find a free SM before any of them starts).
  {
    const int stage = 128 * 64 * 2 + ((S->gate_gp * 128 + 1023) & ~1023);
    const int pipe = (deep ? 8 : 4) * stage, stag = 128 * (S->gate_gp + 1) * 4;
    const int sort_bytes = (int)(sh_sort_smem_bytes(d) > sh_sort_smem_bytes(ds) ? sh_sort_smem_bytes(d) : sh_sort_smem_bytes(ds));
    g.fused = S->fused_sort && 2 * d.nblk <= L->sm_count && ((stag + 15) & ~15) + sort_bytes <= pipe;
    if (g.fused && S->gate_coop == 0) {
      int dev = 0, coop = 0, per_sm = 0;
      SH_CUDA_CHECK(cudaGetDevice(&dev));
      SH_CUDA_CHECK(cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev));
      if (deep) SH_CUDA_CHECK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, sh_tc_gate_kernel<8>, GATE_THREADS, smem));
      else SH_CUDA_CHECK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, sh_tc_gate_kernel<4>, GATE_THREADS, smem));
      S->gate_coop = (coop && per_sm >= 1) ? 1 : -1;
    }
    if (S->gate_coop < 0) g.fused = 0;
  }
  g.sort_sides = ds.sides; g.tile_rows_src = ds.tile_rows_src; g.max_tiles = d.max_tiles;
  g.offsets = (int*)(ws + L->o.offsets); g.lists = (int*)(ws + L->o.lists); g.lgate = (float*)(ws + L->o.lgate);
  g.tiles = (ShTile*)(ws + L->o.tiles); g.ntiles = (int*)(ws + L->o.ntiles);
  g.gridbar = (int*)(ws + L->o.status) + SH_ST_GRIDBAR;
  if (g.fused) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(d.nblk); cfg.blockDim = dim3(GATE_THREADS); cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    if (deep) SH_CUDA_CHECK(cudaLaunchKernelEx(&cfg, sh_tc_gate_kernel<8>, *map_x, S->map_wgate, g));
    else SH_CUDA_CHECK(cudaLaunchKernelEx(&cfg, sh_tc_gate_kernel<4>, *map_x, S->map_wgate, g));
    L->launches += 1;
    return SH_OK;
  }
  if (deep) sh_tc_gate_kernel<8><<<d.nblk, GATE_THREADS, smem, st>>>(*map_x, S->map_wgate, g);
  else sh_tc_gate_kernel<4><<<d.nblk, GATE_THREADS, smem, st>>>(*map_x, S->map_wgate, g);
  size_t ssm = sh_sort_smem_bytes(ds);
  // sort_apart: ask for enough shared memory that a sort block fits beside a gate CTA but not beside a
  // ~198 KB GEMM CTA: next to the Q/K projection's CTAs (whose waiting warps poll) a block takes
  // 11 us instead of 4.7
  if (sort_apart && ssm < 40 * 1024) ssm = 40 * 1024;
  if ((rc = set_smem(sh_sort_kernel, (int)ssm))) return rc;
  if ((rc = launch_k(S->pdl && !L->ev, sh_sort_kernel, dim3(d.nblk), dim3(sh_sort_threads(ds)), ssm, st,
                     (const int*)(ws + (vp ? L->o.gid : L->o.idx)), (const float*)(ws + L->o.gate), (const int*)(ws + L->o.blockcnt),
                     (int*)(ws + L->o.offsets), (int*)(ws + L->o.lists), (float*)(ws + L->o.lgate),
                     (ShTile*)(ws + L->o.tiles), (int*)(ws + L->o.ntiles), ds)))
    return rc;
  L->launches += 2;
  return SH_OK;
}

int sh_tc_gate_sort(sh_layer* L, const void* x, cudaStream_t st) {
  if (!L->tc) { sh_set_error("tensor-core state missing: call sh_set_weights first"); return SH_ERR_NOT_CONFIGURED; }
  return tc_gate_sort(L, x, nullptr, false, st);
}

template <int BN, int STAGES, int MODE, int MT>
static int launch_pgemm(const CUtensorMap& mapA, const CUtensorMap& mapB, const TcGemmArgs& g, unsigned grid, cudaStream_t st, bool pdl) {
  auto kern = sh_tc_pgemm_kernel<BN, STAGES, MODE, MT>;
  constexpr int smem = PGemmSmem<BN, STAGES, MT>::TOTAL;
  if (int rc = set_smem(kern, smem)) return rc;
  return launch_k(pdl, kern, dim3(grid), dim3(352), smem, st, mapA, mapB, g);
}

template <int BN, int STAGES, int MODE, int A_BF16, int B_BF16, int MT = 1>
static int launch_gemm(const CUtensorMap& mapA, const CUtensorMap& mapB, const TcGemmArgs& g, dim3 grid, cudaStream_t st, bool pdl = false) {
  auto kern = sh_tc_gemm_kernel<BN, STAGES, MODE, A_BF16, B_BF16, MT>;
  constexpr int smem = GemmSmem<BN, STAGES, MT>::TOTAL;
  if (int rc = set_smem(kern, smem)) return rc;
  return launch_k(pdl, kern, grid, dim3(192), smem, st, mapA, mapB, g);
}

// ---- one-grid front ------------------------------------------------------------------------------
// Whether sh_tc_front_kernel serves this layer's forward passes, decided once per prepared layer: the
// plain bf16 layer with dense Q/K whose projection width is a multiple of 256, at most two 128-token
// blocks per CTA pair the device holds, shared memory for the operand ring plus the selection's
// scratch, and a device that launches cooperatively and holds all of the grid's CTA pairs at once.
static bool front_plan(sh_layer* L) {
  TcState* S = (TcState*)L->tc;
  if (S->front != 0) return S->front > 0;
  S->front = -1;
  const ShDims& d = L->d;
  if (!S->one_grid_front || L->dense || L->moe_q || L->moe_k || S->simt_mask || !S->gate_gp || S->qk_bn != 256 ||
      !S->persistent || !S->qk_pair)
    return false;
  const bool vp = use_v_pairs(L);
  ShDims ds = d;
  ds.sides = 1;
  if (vp) { ds.sides = 1; ds.E = sh_pair_count(d.E); ds.k = 1; ds.G = d.H * ds.E; }
  const int GH = vp ? ds.G : d.G;
  S->front_sort_bytes = (int)(vp ? sh_sort_smem_bytes(ds) : sh_sort_smem_bytes(d));
  int dev = 0, coop = 0, optin = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess || !coop) {
    cudaGetLastError();
    return false;
  }
  // (five ring stages: six measured the same, and the sixth's 32 KB hold the epilogue's staging tiles and
  //  the selection's scratch)
  S->front_stages = 5;
  S->front_smem = FrontSmem<5>::total(S->gate_gp, GH, S->front_sort_bytes);
  if (S->front_smem > optin) return false;
  if (set_smem(sh_tc_front_kernel<5>, S->front_smem) != SH_OK) return false;
  int pairs = max_pairs(sh_tc_front_kernel<5>, FRONT_THREADS, S->front_smem);
  if (pairs > L->sm_count / 2) pairs = L->sm_count / 2;
  if (pairs <= 0 || d.nblk > 2 * pairs) return false;
  S->front_pairs = pairs;
  S->front = 1;
  return true;
}

// Launches the one-grid front on `st`.  A device that refuses the launch turns the plan off (the
// caller then takes the separate kernels).
static int tc_front(sh_layer* L, const void* x, cudaStream_t st) {
  TcState* S = (TcState*)L->tc;
  const ShDims& d = L->d;
  char* ws = L->ws;
  const int HD = d.H * d.D;
  int rc;
  const CUtensorMap* map_x;
  if ((rc = x_map(L, x, &map_x))) return rc;
  int* status = (int*)(ws + L->o.status);
  TcFrontArgs fa{};
  TcGemmArgs& q = fa.q;
  q.d = d; q.K = d.M; q.ncols = 2 * HD; q.nrows = d.N;
  q.out0 = ws + L->o.q; q.out1 = ws + L->o.k; q.out2 = ws + L->o.v;
  q.qscale = 1.4426950408889634f / sqrtf((float)d.Dt);
  q.b_row0 = 0;
  q.status = status; q.sched = status + SH_ST_SCHED; q.claimers = 0;
  q.rope = L->rope ? (const float2*)(ws + L->o.rope) : nullptr;
  q.stamp_id = SH_K_QK_A;
  TcGateArgs& g = fa.g;
  g.d = d; g.Gp = S->gate_gp; g.gbias = (const float*)(ws + L->o.gbias);
  g.idx = (int*)(ws + L->o.idx); g.gate = (float*)(ws + L->o.gate);
  g.blockcnt = (int*)(ws + L->o.blockcnt);
  const bool vp = use_v_pairs(L);
  g.vpairs = vp ? 1 : 0;
  g.NP = sh_pair_count(d.E); g.GH = vp ? d.H * g.NP : d.G; g.gid = (int*)(ws + L->o.gid);
  g.zero_v = vp ? nullptr : (void*)(ws + L->o.v);          // (the pair-tiled kernel stores every value row once)
  g.zero_out = nullptr;
  g.status = status;
  g.fused = 1;
  g.sort_sides = 1;                                        // only the value experts read sorted lists in a forward pass
  g.tile_rows_src = vp ? 256 : d.tile_rows_src;
  g.max_tiles = d.max_tiles;
  g.offsets = (int*)(ws + L->o.offsets); g.lists = (int*)(ws + L->o.lists); g.lgate = (float*)(ws + L->o.lgate);
  g.tiles = (ShTile*)(ws + L->o.tiles); g.ntiles = (int*)(ws + L->o.ntiles);
  g.gridbar = status + SH_ST_GRIDBAR;
  fa.R = d.nblk <= S->front_pairs ? 64 : 128;
  fa.gate_pairs = fa.R == 64 ? d.nblk : (d.nblk + 1) / 2;
  fa.sort_bytes = S->front_sort_bytes;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2u * (unsigned)S->front_pairs); cfg.blockDim = dim3(FRONT_THREADS);
  cfg.dynamicSmemBytes = (size_t)S->front_smem; cfg.stream = st;
  // A cooperative launch (the grid's CTAs meet at a barrier: all of them have to be resident, whatever
  // else runs on the device); the cluster shape is the kernel's own (__cluster_dims__) - given as a
  // launch attribute beside the cooperative one, every launch failed under the profiler on this driver.
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;
  attr[0].val.cooperative = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  const CUtensorMap& map_g = fa.R == 64 ? S->map_x64 : *map_x;
  fa.tma_epi = d.T % 32 == 0;
  cudaError_t e = cudaLaunchKernelEx(&cfg, sh_tc_front_kernel<5>, *map_x, map_g, S->map_wqk128, S->map_wgate_half, S->map_q_st, S->map_k_st, fa);
  if (e != cudaSuccess) {
    cudaGetLastError();
    S->front = -1;
    sh_set_error("cooperative launch of the one-grid front failed: %s", cudaGetErrorString(e));
    return SH_ERR_CUDA;
  }
  L->launches += 1;
  return SH_OK;
}

using QkPS = QkPairSmem<6>;

// Clusters of the CTA-pair Q/K kernel the device holds at once (looked up once per layer; -1: none).
static int qk_pairs_max(TcState* S) {
  if (S->qk_pairs_max == 0) {
    if (set_smem(sh_tc_qk_pair_kernel<6>, QkPS::TOTAL) != SH_OK) return S->qk_pairs_max = -1;
    S->qk_pairs_max = max_pairs(sh_tc_qk_pair_kernel<6>, 320, QkPS::TOTAL);
    if (S->qk_pairs_max <= 0) S->qk_pairs_max = -1;
  }
  return S->qk_pairs_max;
}

// The launches of one forward pass after grid A of a split Q/K projection is out (see sh_tc_forward).
static int tc_forward_rest(sh_layer* L, const void* x, void* out, cudaStream_t st, const CUtensorMap& map_x, bool overlap,
                           int qkA, int qkB, TcGemmArgs& qg, bool front);

int sh_tc_forward(sh_layer* L, const void* x, void* out, cudaStream_t st) {
  TcState* S = (TcState*)L->tc;
  if (!S) { sh_set_error("tensor-core state missing: call sh_set_weights first"); return SH_ERR_NOT_CONFIGURED; }
  const ShDims& d = L->d;
  char* ws = L->ws;
  const int HD = d.H * d.D;
  int rc;
  const int simt = S->simt_mask;
  int* status = (int*)(ws + L->o.status);

  sh_mark(L, 0, st);
  // stage-timed runs (sh_forward_timed) stay serial so that the stage boundaries mean something
  // one grid for gate, selection, sort and Q/K where the shape allows; otherwise (and on a device that
  // refuses the launch) the separate kernels below
  bool front = false;
  if (!L->ev && front_plan(L)) {
    rc = tc_front(L, x, st);
    if (rc == SH_OK) front = true;
    else if (S->front > 0) return rc;
  }
  const bool overlap = S->side && !L->ev && !(simt & SH_STAGE_QK) && !front;
  if (overlap) {
    SH_CUDA_CHECK(cudaEventRecord(S->ev_fork, st));
    SH_CUDA_CHECK(cudaStreamWaitEvent(S->side, S->ev_fork, 0));
  }
  const CUtensorMap* map_x;
  if ((rc = x_map(L, x, &map_x))) return rc;
  // Split Q/K projection.  A grid whose CTAs cannot all start at once (the gate kernel holds SMs)
  // keeps every kernel launched after it, in any stream, from starting: the sort kernel, launched to
  // become resident while the gate kernel runs, then starts 4-8 us after the gate kernel has ended.
  // And launched after gate and sort, the projection starts two launch latencies late when the host
  // is not running ahead (a single forward pass at the 262M-scale shape: ~102 us instead of ~107).
  // So the projection goes out as two grids of CTA pairs that claim tiles from one counter: grid A,
  // launched BEFORE the gate kernel, sized for the SMs the gate kernel does not need; grid B, launched
  // AFTER the sort kernel on a stream of its own, takes over the gate kernel's SMs when they come
  // free.  The sort blocks are kept off the SMs of grid A (see tc_gate_sort): without that, about one
  // process in six ran every pass 6-8 us slower (as every process does when grid B's stream is given
  // a higher priority than the caller's: grid B's CTAs placed ahead of the sort and value-expert
  // kernels' CTAs, and as happens with a five-stage grid B, whose CTAs fit beside the sort blocks and
  // slow them down); with it, ten processes in a row ran 109.8-111.9 us per pass against 111.7-114.7
  // with one grid, and 265 against 270.5 at 16384 tokens.
  int qkA = 0, qkB = 0;                                    // CTA pairs of the two grids
  TcGemmArgs qg{};
  if (L->moe_q || L->moe_k) {
    // expert projections of keys / queries run on the pair-tiled kernel (pair-bucketed lists), or - debug
    // library, SH_SIMT_STAGES - on the CUDA-core kernels together with gate and value stage (expert lists)
    const bool bad = (simt & SH_STAGE_QK) ? use_v_pairs(L)
                                          : (!use_v_pairs(L) || !S->persistent || !S->qk_pair || qk_pairs_max(S) <= 0);
    if (bad) {
      sh_set_error("query / key experts need the CTA-pair projection kernels on this device and in this build");
      return SH_ERR_UNSUPPORTED;
    }
  }
  // a layer with query (key) experts projects only its keys (queries) densely; with both, nothing
  const int qk_ncols = (L->moe_q || L->moe_k) ? HD : 2 * HD;
  if (!front && overlap && !L->dense && !(simt & SH_STAGE_GATE) && S->gate_gp && S->qk_bn == 256 && S->persistent && S->qk_pair &&
      S->qk_two_grids && qk_pairs_max(S) > 0 && !(L->moe_q && L->moe_k)) {
    const int ptiles = ((d.N + 255) / 256) * ((qk_ncols + 255) / 256);
    const int pairs = ptiles < S->qk_pairs_max ? ptiles : S->qk_pairs_max;
    // (one gate CTA per SM; running two per SM with half the stages, to leave grid A more SMs when
    //  there are more gate CTAs than half the SMs, made the gate kernel 2.4 us slower and the layer
    //  8-10 us slower at 16384 tokens)
    int gate_sms = d.nblk;
    if (gate_sms > L->sm_count - 8) gate_sms = L->sm_count - 8;
    qkA = (L->sm_count - gate_sms) / 2;
    if (qkA > pairs) qkA = pairs;
    qkB = pairs - qkA;
    qg.d = d; qg.K = d.M; qg.ncols = qk_ncols; qg.nrows = d.N;
    qg.out0 = ws + (L->moe_q ? L->o.k : L->o.q); qg.out1 = ws + L->o.k; qg.out2 = ws + L->o.v;
    qg.qscale = L->moe_q ? 1.f : 1.4426950408889634f / sqrtf((float)d.Dt);
    qg.b_row0 = L->moe_q ? HD : 0;
    qg.status = status; qg.sched = status + SH_ST_SCHED; qg.claimers = qkA + qkB;
    qg.rope = L->rope ? (const float2*)(ws + L->o.rope) : nullptr;
    qg.stamp_id = SH_K_QK_A;
    if ((rc = launch_k_pairs(false, sh_tc_qk_pair_kernel<6>, dim3(2 * qkA), dim3(320), QkPS::TOTAL, S->side, *map_x, S->map_wqk128, qg))) return rc;
    L->launches += 1;
  }
  rc = tc_forward_rest(L, x, out, st, *map_x, overlap, qkA, qkB, qg, front);
  if (rc != SH_OK && qkA > 0) {
    // Grid A is out and something after it could not be launched: the tile counter it shares with
    // grid B would keep this pass's claims, and the caller's stream would never join the side
    // streams.  Put both right, so that a later pass starts from a clean state.
    cudaMemsetAsync(status + SH_ST_SCHED, 0, 8, S->side);
    cudaEventRecord(S->ev_join, S->side);
    cudaStreamWaitEvent(st, S->ev_join, 0);
    cudaGetLastError();
  }
  return rc;
}

static int tc_forward_rest(sh_layer* L, const void* x, void* out, cudaStream_t st, const CUtensorMap& map_x, bool overlap,
                           int qkA, int qkB, TcGemmArgs& qg, bool front) {
  TcState* S = (TcState*)L->tc;
  const ShDims& d = L->d;
  char* ws = L->ws;
  const int HD = d.H * d.D;
  int rc;
  const int simt = S->simt_mask;
  int* status = (int*)(ws + L->o.status);
  const bool pdl = S->pdl && !L->ev;                       // stage-timed runs use ordinary launches
  if (!L->dense && !front) {
    if ((rc = tc_gate_sort(L, x, out, true, st, qkA > 0))) return rc;
  }
  sh_mark(L, 1, st);
  if (qkA > 0 && qkB > 0) {
    SH_CUDA_CHECK(cudaStreamWaitEvent(S->side2, S->ev_fork, 0));
    qg.stamp_id = SH_K_QK_B;
    if ((rc = launch_k_pairs(false, sh_tc_qk_pair_kernel<6>, dim3(2 * qkB), dim3(320), QkPS::TOTAL, S->side2, map_x, S->map_wqk128, qg))) return rc;
    SH_CUDA_CHECK(cudaEventRecord(S->ev_join2, S->side2));
    L->launches += 1;
  }
  // ---- Q, K (and V for the dense comparator) ------------------------------------------------
  if (qkA > 0 || front) {
    // (launched above: as two grids, or inside the one-grid front)
  } else if (simt & SH_STAGE_QK) {
    if ((rc = sh_simt_run_bf16(L, SH_STAGE_QK, x, out, st))) return rc;
  } else if (L->moe_q && L->moe_k) {
    // (queries and keys are both expert projections: they follow the value experts below)
  } else {
    cudaStream_t qst = overlap ? S->side : st;              // side stream when overlapping
    TcGemmArgs g{};
    g.d = d; g.K = d.M; g.ncols = L->dense ? 3 * HD : (L->moe_q || L->moe_k) ? HD : 2 * HD; g.nrows = d.N;
    g.out0 = ws + (L->moe_q ? L->o.k : L->o.q); g.out1 = ws + L->o.k; g.out2 = ws + L->o.v;
    g.qscale = L->moe_q ? 1.f : 1.4426950408889634f / sqrtf((float)d.Dt);
    g.b_row0 = L->moe_q ? HD : 0;
    g.status = status;
    g.sched = status + SH_ST_SCHED;
    g.rope = L->rope ? (const float2*)(ws + L->o.rope) : nullptr;
    g.stamp_id = SH_K_QK_A;
    dim3 grid(d.nblk, (g.ncols + S->qk_bn - 1) / S->qk_bn);
    if (S->qk_bn == 256) {
      if (S->persistent && S->qk_pair && qk_pairs_max(S) > 0) {
        // CTA pairs: 256 x 256 tiles, each CTA loads half of the weight rows
        const int ptiles = ((d.N + 255) / 256) * ((g.ncols + 255) / 256);
        const unsigned pgrid = 2u * (unsigned)(ptiles < S->qk_pairs_max ? ptiles : S->qk_pairs_max);
        rc = launch_k_pairs(pdl && !overlap, sh_tc_qk_pair_kernel<6>, dim3(pgrid), dim3(320), QkPS::TOTAL, qst, map_x, S->map_wqk128, g);
      } else if (S->persistent) {
        // a device that cannot hold such a cluster: single-CTA persistent kernel, 128 x 256 tiles
        const unsigned tiles = (unsigned)(d.nblk * ((g.ncols + 255) / 256));
        rc = launch_pgemm<256, 4, PG_QKV, 1>(map_x, S->map_wqk, g, tiles < (unsigned)L->sm_count ? tiles : (unsigned)L->sm_count, qst, pdl && !overlap);
      } else {
        rc = launch_gemm<256, 4, GEMM_QKV, 1, 1>(map_x, S->map_wqk, g, grid, qst);
      }
    } else {
      // projection width not a multiple of 256: one CTA per 128 x 128 tile
      rc = launch_gemm<128, QK_STAGES, GEMM_QKV, 1, 1>(map_x, S->map_wqk, g, grid, qst);
    }
    if (rc) return rc;
    L->launches += 1;
  }
  if (overlap) SH_CUDA_CHECK(cudaEventRecord(S->ev_join, S->side));
  sh_mark(L, 2, st);
  // ---- value experts ---------------------------------------------------------------------------
  if (!L->dense) {
    if (simt & SH_STAGE_V) {
      if ((rc = sh_simt_run_bf16(L, SH_STAGE_V, x, out, st))) return rc;
    } else if (use_v_pairs(L)) {
      TcVPairArgs g{};
      g.d = d; g.x = x; g.lists = (const int*)(ws + L->o.lists);
      g.tiles = (const ShTile*)(ws + L->o.tiles); g.ntiles = (const int*)(ws + L->o.ntiles);
      g.idx = (const int*)(ws + L->o.idx); g.gate = (const float*)(ws + L->o.gate);
      g.v = (__half*)(ws + L->o.v); g.status = status;
      const int bound = (d.N * d.H + 255) / 256 + d.H * sh_pair_count(d.E);       // tiles: at most this many
      const unsigned pgrid = 2u * (unsigned)(bound < S->v_pairs_max ? bound : S->v_pairs_max);
      g.scale = 0.f; g.stamp_id = SH_K_V;
      // (behind the one-grid front: wait for the sort's counter, not for the grid - see sh_tc_vpair_kernel)
      if (front && pdl) { g.ready = status + SH_ST_SORTED; g.ready_count = d.nblk; }
      if ((rc = launch_k_pairs(pdl, sh_tc_vpair_kernel<6>, dim3(pgrid), dim3(320), VPS::TOTAL, st, S->map_wv, g))) return rc;
      g.ready = nullptr;
      L->launches += 1;
      // key / query experts: the same kernel with the key (query) experts' weights, the source
      // (destination) side's pair tiles and gates, into the K (Q) buffer; queries carry the score scale
      if (L->moe_k && !(simt & SH_STAGE_QK)) {
        g.v = (__half*)(ws + L->o.k); g.stamp_id = -1;
        if ((rc = launch_k_pairs(pdl, sh_tc_vpair_kernel<6>, dim3(pgrid), dim3(320), VPS::TOTAL, st, S->map_wk_e, g))) return rc;
        L->launches += 1;
      }
      if (L->moe_q && !(simt & SH_STAGE_QK)) {
        const size_t s1 = d.sides == 2 ? 1 : 0;            // destination side (with a shared selection: the one side there is)
        g.lists = (const int*)(ws + L->o.lists) + s1 * (size_t)d.H * d.N;
        g.tiles = (const ShTile*)(ws + L->o.tiles) + s1 * (size_t)d.max_tiles;
        g.ntiles = (const int*)(ws + L->o.ntiles) + s1;
        g.idx = (const int*)(ws + L->o.idx) + s1 * (size_t)d.N * d.H * d.k; g.gate = (const float*)(ws + L->o.gate) + s1 * (size_t)d.N * d.H * d.k;
        g.v = (__half*)(ws + L->o.q); g.scale = 1.4426950408889634f / sqrtf((float)d.Dt); g.stamp_id = -1;
        if ((rc = launch_k_pairs(pdl, sh_tc_vpair_kernel<6>, dim3(pgrid), dim3(320), VPS::TOTAL, st, S->map_wq_e, g))) return rc;
        L->launches += 1;
      }
    } else {
      TcGemmArgs g{};
      g.d = d; g.K = d.M; g.ncols = d.D;
      g.A = x; g.lda = d.M;
      g.lists = (const int*)(ws + L->o.lists); g.lgate = (const float*)(ws + L->o.lgate);
      g.tiles = (const ShTile*)(ws + L->o.tiles); g.ntiles = (const int*)(ws + L->o.ntiles);
      g.b_rows_per_group = d.D; g.out0 = ws + L->o.v; g.status = status;
      g.stamp_id = SH_K_V;
      g.v_early = (float*)(ws + L->o.vearly); g.v_early_cnt = (int*)(ws + L->o.vearly_cnt);
      // 256-row tiles (two accumulators sharing the weight operand): at most half the 128-row bound plus one per group
      dim3 grid(d.tile_rows_src == 256 ? d.max_tiles / 2 + d.H * d.E : d.max_tiles, 1);
      if (d.tile_rows_src == 256) {
        if (d.D == 128) rc = S->persistent ? launch_pgemm<128, 4, PG_V, 2>(map_x, S->map_wv, g, grid.x < (unsigned)L->sm_count ? grid.x : (unsigned)L->sm_count, st, pdl)
                                           : launch_gemm<128, 4, GEMM_V, 1, 1, 2>(map_x, S->map_wv, g, grid, st, pdl);
        else rc = launch_gemm<64, 4, GEMM_V, 1, 1, 2>(map_x, S->map_wv, g, grid, st, pdl);
      } else {
        // (128-row tiles of a small workload: the persistent kernel too - one prologue per SM instead of one per tile)
        const unsigned pg = grid.x < (unsigned)L->sm_count ? grid.x : (unsigned)L->sm_count;
        if (d.D == 128) rc = S->persistent ? launch_pgemm<128, 4, PG_V, 1>(map_x, S->map_wv, g, pg, st, pdl) : launch_gemm<128, 4, GEMM_V, 1, 1>(map_x, S->map_wv, g, grid, st, pdl);
        else rc = S->persistent ? launch_pgemm<64, 4, PG_V, 1>(map_x, S->map_wv, g, pg, st, pdl) : launch_gemm<64, 4, GEMM_V, 1, 1>(map_x, S->map_wv, g, grid, st, pdl);
      }
      if (rc) return rc;
      L->launches += 1;
    }
  }
  if (overlap) SH_CUDA_CHECK(cudaStreamWaitEvent(st, S->ev_join, 0));
  if (qkA > 0 && qkB > 0) SH_CUDA_CHECK(cudaStreamWaitEvent(st, S->ev_join2, 0));
  sh_mark(L, 3, st);
  // ---- attention ---------------------------------------------------------------------------------
  if (simt & SH_STAGE_ATTN) {
    if ((rc = sh_simt_run_bf16(L, SH_STAGE_ATTN, x, out, st))) return rc;
  } else {
    TcAttnArgs a{};
    a.d = d; a.ahat = (__half*)(ws + L->o.ahat); a.status = status;
    if (L->xl_positions) {
      // Transformer-XL position term: the per-key content bias c u.k, then the score bias
      // [B, H, Tq, T] = Q R^T (skewed to key order) + c v.r + c u.k by a tensor-core GEMM; the attention
      // kernel adds it to its S tiles
      const float qscale = 1.4426950408889634f / sqrtf((float)d.Dt);
      const long nkeys = (long)d.B * d.H * d.T;
      if ((rc = launch_k(false, sh_xl_uk_kernel, dim3((unsigned)((nkeys * 8 + 255) / 256)), dim3(256), 0, st, (const __half*)(ws + L->o.k),
                         (const float*)(ws + L->o.xl_uv), (float*)(ws + L->o.xl_uk), d.H, d.T, d.D, nkeys, qscale)))
        return rc;
      TcXlBiasArgs bg{};
      bg.d = d; bg.vr = (const float*)(ws + L->o.xl_vr); bg.uk = (const float*)(ws + L->o.xl_uk);
      bg.bias = (__half*)(ws + L->o.xl_bias); bg.status = status;
      const unsigned bgrid = (unsigned)(d.B * d.H * ((d.T - d.Tc) / 128));
      if (d.D == 128) {
        if ((rc = set_smem(sh_tc_xlbias_kernel<128>, XlBiasSmem<128>::TOTAL))) return rc;
        if ((rc = launch_k(pdl, sh_tc_xlbias_kernel<128>, dim3(bgrid), dim3(320), XlBiasSmem<128>::TOTAL, st, S->map_q2d, S->map_r16, bg))) return rc;
      } else {
        if ((rc = set_smem(sh_tc_xlbias_kernel<64>, XlBiasSmem<64>::TOTAL))) return rc;
        if ((rc = launch_k(pdl, sh_tc_xlbias_kernel<64>, dim3(bgrid), dim3(320), XlBiasSmem<64>::TOTAL, st, S->map_q2d, S->map_r16, bg))) return rc;
      }
      L->launches += 2;
      a.bias = (const __half*)(ws + L->o.xl_bias);
    }
    const int nq = ((d.T + 127) / 128 - d.Tc / 128 + 1) / 2;    // pairs of 128-query tiles behind the cache
    const unsigned grid = (unsigned)(nq * d.B * d.H);
    a.balanced = d.causal && (int)grid <= L->sm_count && S->attn_balanced;
    // up to 1024 keys per query tile: the kernel that pipelines the 128 keys of a step as two halves (its
    // finer hand-overs shorten the few-step chain of a short sequence); beyond: the whole-S kernel
    // (with halves the issuing thread, eight N = 64 UMMAs per half, bounds a long loop)
    const bool halves = d.T <= 1024;
    if (d.D == 128) {
      auto kern = halves ? sh_tc_attention3_kernel<128> : sh_tc_attention2_kernel<128>;
      const int smem = halves ? Attn3Smem<128>::TOTAL : Attn2Smem<128>::TOTAL;
      if ((rc = set_smem(kern, smem))) return rc;
      if ((rc = launch_k(pdl, kern, dim3(grid), dim3(320), smem, st, S->map_q, S->map_k, S->map_v, a))) return rc;
    } else {
      auto kern = halves ? sh_tc_attention3_kernel<64> : sh_tc_attention2_kernel<64>;
      const int smem = halves ? Attn3Smem<64>::TOTAL : Attn2Smem<64>::TOTAL;
      if ((rc = set_smem(kern, smem))) return rc;
      if ((rc = launch_k(pdl, kern, dim3(grid), dim3(320), smem, st, S->map_q, S->map_k, S->map_v, a))) return rc;
    }
    L->launches += 1;
  }
  sh_mark(L, 4, st);
  // ---- output experts ----------------------------------------------------------------------------
  if (L->out_f16 && ((simt & SH_STAGE_O) || L->dense)) {
    sh_set_error("fp16 output is written by the tensor-core output-expert kernels only");
    return SH_ERR_UNSUPPORTED;
  }
  if (simt & SH_STAGE_O) {
    if ((rc = sh_simt_run_bf16(L, SH_STAGE_O, x, out, st))) return rc;
  } else if (!L->dense) {
    TcOprojArgs a{};
    a.d = d;
    const size_t side1 = d.sides == 2 ? (size_t)d.N * d.H * d.k : 0;   // shared selection: the one side there is
    a.idx = (const int*)(ws + L->o.idx) + side1; a.gate = (const float*)(ws + L->o.gate) + side1;
    a.out = (float*)out; a.out_f16 = L->out_f16 ? 1 : 0; a.status = status;
    // Up to four selections per (token, head) the CTA-pair kernels serve (their builder threads keep a
    // token's selections in registers).  With more, the single-CTA kernel, which reads the selections
    // from shared memory and multiplies by the gate after the UMMA; a device that cannot hold a two-CTA
    // cluster of the pair kernel's size uses it too.
    bool pair = S->o_pair && d.k <= OPAIR_KMAX;
    const bool sparse = pair && S->o_sparse && sh_o_sparse_ok(L);
    if (sparse) {
      constexpr int psm = OprojSpSmem<128>::TOTAL;
      if (d.E == 4) { if ((rc = set_smem(sh_tc_oproj_sp_kernel<128, 1>, psm))) return rc; }
      else if ((rc = set_smem(sh_tc_oproj_sp_kernel<128, 2>, psm))) return rc;
      if (S->o_pairs_max == 0) {
        S->o_pairs_max = d.E == 4 ? max_pairs(sh_tc_oproj_sp_kernel<128, 1>, 480, psm) : max_pairs(sh_tc_oproj_sp_kernel<128, 2>, 480, psm);
        if (S->o_pairs_max <= 0) S->o_pairs_max = -1;
      }
      if (S->o_pairs_max < 0) pair = false;
    } else if (pair) {
      const int psm = d.D == 128 ? OprojPairSmem<128>::TOTAL : OprojPairSmem<64>::TOTAL;
      if (d.D == 128) { if ((rc = set_smem(sh_tc_oproj_pair_kernel<128>, psm))) return rc; }
      else if ((rc = set_smem(sh_tc_oproj_pair_kernel<64>, psm))) return rc;
      if (S->o_pairs_max == 0) {
        S->o_pairs_max = d.D == 128 ? max_pairs(sh_tc_oproj_pair_kernel<128>, 480, psm) : max_pairs(sh_tc_oproj_pair_kernel<64>, 480, psm);
        if (S->o_pairs_max <= 0) S->o_pairs_max = -1;
      }
      if (S->o_pairs_max < 0) pair = false;
    }
    if (pair && sparse) {
      // 256 tokens x 256 features per unit, the selection as 2:4 sparsity of the gate-scaled A operand
      constexpr int psm = OprojSpSmem<128>::TOTAL;
      a.nwork = ((sh_out_rows(d) + 255) / 256) * ((d.M + 255) / 256);
      const unsigned pgrid = 2u * (unsigned)(a.nwork < S->o_pairs_max ? a.nwork : S->o_pairs_max);
      const __half* ahat = (const __half*)(ws + L->o.ahat);
      if (d.E == 4) rc = launch_k_pairs(pdl, sh_tc_oproj_sp_kernel<128, 1>, dim3(pgrid), dim3(480), psm, st, S->map_wos, a, ahat);
      else rc = launch_k_pairs(pdl, sh_tc_oproj_sp_kernel<128, 2>, dim3(pgrid), dim3(480), psm, st, S->map_wos, a, ahat);
      if (rc) return rc;
    } else if (pair) {
      // 256 tokens x 256 features per unit, gates folded into the A operand
      const int psm = d.D == 128 ? OprojPairSmem<128>::TOTAL : OprojPairSmem<64>::TOTAL;
      a.nwork = ((sh_out_rows(d) + 255) / 256) * ((d.M + 255) / 256);
      const unsigned pgrid = 2u * (unsigned)(a.nwork < S->o_pairs_max ? a.nwork : S->o_pairs_max);
      const __half* ahat = (const __half*)(ws + L->o.ahat);
      if (d.D == 128) rc = launch_k_pairs(pdl, sh_tc_oproj_pair_kernel<128>, dim3(pgrid), dim3(480), psm, st, S->map_wo, a, ahat);
      else rc = launch_k_pairs(pdl, sh_tc_oproj_pair_kernel<64>, dim3(pgrid), dim3(480), psm, st, S->map_wo, a, ahat);
      if (rc) return rc;
    } else {
      a.nwork = ((sh_out_rows(d) + 127) / 128) * ((d.M + 255) / 256);
      const unsigned grid = (unsigned)(a.nwork < L->sm_count ? a.nwork : L->sm_count);
      int as = 3, smem = 0;
      for (; as >= 2; --as) {
        smem = d.D == 128 ? OprojSmem<128>::total(as, d.H, d.k) : OprojSmem<64>::total(as, d.H, d.k);
        if (smem <= 227 * 1024) break;
      }
      if (as < 2) { sh_set_error("output projection: n_heads*k = %d does not fit in shared memory", d.H * d.k); return SH_ERR_UNSUPPORTED; }
      a.a_slots = as;
      if (d.D == 128) {
        if ((rc = set_smem(sh_tc_oproj_kernel<128>, smem))) return rc;
        if ((rc = launch_k(pdl, sh_tc_oproj_kernel<128>, dim3(grid), dim3(320), smem, st, S->map_ahat, S->map_wo256, a))) return rc;
      } else {
        if ((rc = set_smem(sh_tc_oproj_kernel<64>, smem))) return rc;
        if ((rc = launch_k(pdl, sh_tc_oproj_kernel<64>, dim3(grid), dim3(320), smem, st, S->map_ahat, S->map_wo256, a))) return rc;
      }
    }
    L->launches += 1;
  } else {
    // dense comparator: out = Ahat W_O on the CTA-pair GEMM (256 x 256 tiles) when the device holds such
    // clusters and d_model allows, else one CTA per 128 x 128 tile
    TcGemmArgs g{};
    g.d = d; g.K = HD; g.ncols = d.M; g.nrows = d.N; g.out0 = out; g.status = status;
    g.stamp_id = SH_K_O;
    if (S->persistent && S->qk_pair && d.M % 256 == 0 && HD % 64 == 0 && qk_pairs_max(S) > 0) {
      g.sched = status + SH_ST_SCHED;                        // (the Q/K projection's claims of this pass are over: its last claimer put the counters back)
      if ((rc = set_smem(sh_tc_qk_pair_kernel<6, 1>, QkPS::TOTAL))) return rc;
      const int ptiles = ((d.N + 255) / 256) * (d.M / 256);
      const unsigned pgrid = 2u * (unsigned)(ptiles < S->qk_pairs_max ? ptiles : S->qk_pairs_max);
      if ((rc = launch_k_pairs(pdl, sh_tc_qk_pair_kernel<6, 1>, dim3(pgrid), dim3(320), QkPS::TOTAL, st, S->map_ahat, S->map_wo, g))) return rc;
    } else {
      dim3 grid(d.nblk, (d.M + 127) / 128);
      if ((rc = launch_gemm<128, 4, GEMM_PLAIN, 0, 0>(S->map_ahat, S->map_wo, g, grid, st))) return rc;
    }
    L->launches += 1;
  }
  sh_mark(L, 5, st);
  SH_CUDA_CHECK(cudaGetLastError());
  return SH_OK;
}

// ---- self-tests of the safety net (no memory access can go wrong in either) ---------------------------
// which = 0: one thread waits on an mbarrier nobody arrives on, with the given limit, through the
// same bounded wait every kernel uses; it gives up, records SH_ERR_TIMEOUT and where, and returns.
// which = 1 (debug library): one thread runs the index check on `arg` against the limit 10.
static __global__ void sh_selftest_kernel(int* status, int which, unsigned long long arg) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) { mbar_init(&bar, 1); fence_barrier_init(); }
  __syncthreads();
  if (threadIdx.x != 0) return;
  if (which == 0) {
    bool dead = false;
    mbar_wait_limit(&bar, 0, status, dead, arg);
  } else {
    (void)SH_INDEX_OK((long long)arg, 10, status, SH_SITE_SELFTEST);
  }
}

int sh_tc_selftest(sh_layer* L, int which, unsigned long long arg, cudaStream_t st) {
#ifndef SH_DEBUG
  if (which == 1) { sh_set_error("index checks exist only in the debug library (built with -DSH_DEBUG)"); return SH_ERR_UNSUPPORTED; }
#endif
  sh_selftest_kernel<<<1, 32, 0, st>>>((int*)(L->ws + L->o.status), which, arg);
  SH_CUDA_CHECK(cudaGetLastError());
  return SH_OK;
}
