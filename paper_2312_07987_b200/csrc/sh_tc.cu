// Tensor-core path of the bf16 configuration (interim: routes to the CUDA-core stages).
#include "sh_internal.cuh"

int sh_tc_prepare(sh_layer* L) { (void)L; return SH_OK; }
void sh_tc_release(sh_layer* L) { (void)L; }
int sh_tc_forward(sh_layer* L, const void* x, void* out, cudaStream_t st) {
  return sh_simt_run_bf16(L, SH_STAGE_ALL, x, out, st);
}
int sh_tc_gate_sort(sh_layer* L, const void* x, cudaStream_t st) {
  return sh_simt_run_bf16(L, SH_STAGE_GATE, x, nullptr, st);
}
