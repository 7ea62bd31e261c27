#include "tc_kernels.cuh"

struct TcState { int sm_count; };

TcState* tc_create(int sm_count) { return new TcState{sm_count}; }
void tc_destroy(TcState* s) { delete s; }
int tc_gemm(TcState*, const GemmArgs&, int*, cudaStream_t) { return 1; }
int tc_attn_fwd(TcState*, const CcaDims&, const bf16*, const bf16*, const bf16*, bf16*, float*, float*, int*, cudaStream_t) {
  return 1;
}
