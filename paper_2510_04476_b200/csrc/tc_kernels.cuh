// Tensor-core (tcgen05 / TMEM / TMA) kernels of the CCA library: host-side interface.
// Each tc_* launcher returns 0 if it enqueued the work, 1 if the case is outside its coverage
// (the caller then uses the SIMT kernel), or -cudaError on a CUDA failure.
#pragma once
#include "common.cuh"

struct TcState;

TcState* tc_create(int sm_count);
void tc_destroy(TcState* s);
int tc_gemm(TcState* s, const GemmArgs& g, int* d_status, cudaStream_t st);
// Same contraction on CTA pairs (256 x 256 tiles); covers large K-major-A cases only.
int tc_gemm_pair(TcState* s, const GemmArgs& g, int* d_status, cudaStream_t st);
// t_first > 0 (a multiple of 256): only the query rows [t_first, d.S) of every sequence; keys and values [0, d.S).
int tc_attn_fwd(TcState* s, const CcaDims& d, const bf16* q, const bf16* k, const bf16* v, bf16* o, float* o32,
                float* lse, const float* temp, int* d_status, cudaStream_t st, int t_first = 0);
// Head size 256 (one query tile per CTA, score buffers alternate over key tiles).
int tc_attn_fwd256(TcState* s, const CcaDims& d, const bf16* q, const bf16* k, const bf16* v, bf16* o, float* o32, float* lse,
                   const float* temp, int* d_status, cudaStream_t st);
// Attention adjoint (dq, dk, dv in fp32) from q, k, v, d_o, the forward's lse and delta = rowsum(dO o O).
int tc_attn_bwd(TcState* s, const CcaDims& d, const bf16* q, const bf16* k, const bf16* v, const bf16* d_o,
                const float* lse, const float* delta, float* dq, float* dk, float* dv, int* d_status, cudaStream_t st);
// The same adjoint as one kernel (head size 64): every (query, key) pair once; dq is zeroed, then summed by reductions.
int tc_attn_bwd_fused(TcState* s, const CcaDims& d, const bf16* q, const bf16* k, const bf16* v, const bf16* d_o,
                      const float* lse, const float* delta, float* dq, float* dk, float* dv, int* d_status, cudaStream_t st);
// Adjoint of conv2: dy1 [T, L] fp32 <- d_hat (dqh, dkh); d_w1 accumulates the conv2 weight gradient.
int tc_transform_bwd(TcState* s, const CcaDims& d, const float* qk0, const bf16* w0, const bf16* w1, const float* dqh,
                     const float* dkh, float* dy1, float* d_w1, int* d_status, cudaStream_t st);
// The same stage with TMA-fed operands (tc_transform2.cu): needs a bf16 copy of qk0 (the fused down-projection writes
// it) and the composed conv1 * conv2 weights wc that tc_transform2_compose forms from w0, w1 (tc_transform2_weight_bytes).
size_t tc_transform2_weight_bytes(const CcaDims& d);
bool tc_transform2_covers(const CcaDims& d);
int tc_transform2_compose(const CcaDims& d, const bf16* w0, const bf16* w1, bf16* wc, cudaStream_t st);
int tc_transform2_fwd(TcState* s, const CcaDims& d, const float* qk0, const bf16* qk0b, const bf16* wc, const float* temp,
                      const float2* rope, bf16* q, bf16* k, float* rnorm, int* d_status, cudaStream_t st, int t_first = 0);
int tc_transform_fwd(TcState* s, const CcaDims& d, const float* qk0, const bf16* w0, const bf16* w1,
                     const float* temp, const float2* rope, bf16* q, bf16* k, float* rnorm, int* d_status,
                     cudaStream_t st, int t_first = 0);   // t_first > 0 (multiple of 128): only tokens [t_first, d.S)
