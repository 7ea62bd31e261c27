// Shared declarations of the CCA library's translation units (host launchers + small helpers).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

typedef __nv_bfloat16 bf16;

#define CCA_DEVINL __device__ __forceinline__

// ---- problem description shared by the latent-transform and attention launchers ----
struct CcaDims {
  int B, S, E;
  int hq, hk, dh, g;
  int Lq, Lk, L;
  int k_seq, k_ch;
  int causal;
  unsigned flags;
  float rope_base;
};

// Strided operand of a GEMM: element (r, c) lives at p[r * rs + c * cs]; one stride is 1.
struct GemmOperand {
  const bf16* p;
  long long rs, cs;
};

// C[M,N] = sum_k A(m,k) * B(n,k), fp32 accumulate.
//   a_row_off / seq_len: row m of A is taken from row m + a_row_off of the same sequence (rows
//   are grouped in sequences of seq_len); rows whose source falls outside the sequence count as
//   zero.  This is how the value-shift reads x_{t-1}.
//   out_bf16 / out_f32: exactly one is non-null; ldc is the row stride of C in elements.
//   split_L > 0 selects the fused down-projection output instead (Eq. 7 and Eq. 10 in one contraction with the
//   rows of W_qk, W_v1, W_v2 stacked): columns [0, split_L) go to out_f32 (row stride ldc), the next split_Lk/2
//   columns to out_bf16 (row stride split_Lk) in the same row, the last split_Lk/2 columns to out_bf16 one row
//   later in the same sequence if split_shift (value-shift: v2 of token t is W_v2 x_{t-1}; row 0 gets zeros).
struct GemmArgs {
  GemmOperand A, B;
  int M, N, K;
  int a_row_off, seq_len;
  bf16* out_bf16;
  float* out_f32;
  long long ldc;
  int split_L, split_Lk, split_shift;
  int row0;          // fused output only: position inside its sequence of row 0 of A (a chunk of a longer sequence)
  bf16* out_lat_bf16;   // fused output only, optional: a bf16 copy of columns [0, split_L) (row stride split_L)
  int accumulate;       // out_f32 only: add the product to what the output holds (atomic adds) instead of overwriting
};

cudaError_t launch_gemm_simt(const GemmArgs& g, cudaStream_t st);

// ---- latent transforms (Eq. 8-11 without the attention) ----
cudaError_t launch_rope_table(float2* tab, int S, int dh, float base, cudaStream_t st);
cudaError_t launch_transform_fwd(const CcaDims& d, const float* qk0, const bf16* w0, const bf16* w1,
                                 const float* temp, const float2* rope_tab, bf16* q, bf16* k, float* rnorm,
                                 cudaStream_t st);
// rnorm[token, head] = sqrt(d_h) [* exp(temp)] / |pre-norm latent|, written by the forward.
// dq/dk (fp32, gradients w.r.t. the attention inputs) are replaced in place by the gradients
// w.r.t. the pre-norm latents; d_temp accumulates (must be zeroed by the caller).
cudaError_t launch_transform_bwd_norm(const CcaDims& d, const bf16* q, const bf16* k, const float* rnorm,
                                      const float* temp, const float2* rope_tab, float* dq, float* dk,
                                      float* d_temp, cudaStream_t st);
// dlat[T, ld_dlat] columns [0, L) <- gradient w.r.t. qk0 (bf16); d_w0 accumulates.
cudaError_t launch_transform_bwd_conv(const CcaDims& d, const float* qk0, const bf16* w0, const bf16* w1,
                                      const float* dqh, const float* dkh, bf16* dlat, long long ld_dlat,
                                      float* d_w0, cudaStream_t st);
// Same result as launch_transform_bwd_conv when dy1 [T, L] (fp32) already holds the conv2 adjoint of d_hat.
cudaError_t launch_conv1_adjoint(const CcaDims& d, const float* dy1, const float* dqh, const float* dkh, const float* qk0,
                                 const bf16* w0, bf16* dlat, long long ld_dlat, float* d_w0, cudaStream_t st);
// d_w1 accumulates.
cudaError_t launch_transform_bwd_w1(const CcaDims& d, const float* qk0, const bf16* w0, const float* dqh,
                                    const float* dkh, float* d_w1, cudaStream_t st);
// dlat columns [L, L+Lk) <- dv with the second half moved one token earlier (value-shift adjoint).
cudaError_t launch_pack_dv(const CcaDims& d, const float* dv, bf16* dlat, long long ld_dlat, cudaStream_t st);

// Same stages without the fused kernels, for head sizes those do not cover: conv1 output at the taps conv2 reads
// (y1s[t, c * k_ch + r], bf16; y2 [T, L] fp32 directly when conv2 is off), then -- after the caller's per-head
// contractions have filled y2 -- q-k-mean, norm, temperature and RoPE.
cudaError_t launch_conv1_taps(const CcaDims& d, const float* qk0, const bf16* w0, bf16* y1s, float* y2, cudaStream_t st);
cudaError_t launch_finalize(const CcaDims& d, const float* qk0, const float* y2, const float* temp, const float2* rope,
                            bf16* q, bf16* k, float* rnorm, cudaStream_t st);

// ---- element-wise pieces of the backward at head sizes without fused adjoint kernels (bwd_unfused.cu) ----
// P (bf16) and dS / sqrt(d_h) (bf16) of one chunk of `rows` query rows starting at m0 of one (sequence, query head) from
// its scores s and dP (fp32, row stride ld, keys [0, n_keys)); lse, delta: that head's rows.  Columns >= n_keys get 0.
cudaError_t launch_pds(const float* s, const float* dp, long long ld, const float* lse, const float* delta, int m0, int rows,
                       int n_keys, int S, int causal, int dh, bf16* p_out, bf16* ds_out, cudaStream_t st);
cudaError_t launch_cast_dhat(const CcaDims& d, const float* dqh, const float* dkh, bf16* out_bf16, float* out_f32, cudaStream_t st);
// dy1 [T, L] from dy1s [T, L * k_ch] (gradient of the conv1 output stored at the k_ch positions conv2 reads).
cudaError_t launch_taps_adjoint(const CcaDims& d, const float* dy1s, float* dy1, cudaStream_t st);

// ---- MLA baseline (Eq. 6): attention operands from the up-projected parts (mla.cu) ----
cudaError_t launch_mla_assemble(long long tokens, int S, int nh, int dn, int dr, const bf16* qn, const bf16* qr, const bf16* kn,
                                const bf16* kr, const float2* rope, bf16* q, bf16* k, cudaStream_t st);

// ---- attention (Eq. 11, softmax line), plain SIMT ----
// o32: optional fp32 copy of o (kept for the backward's delta = rowsum(dO * O)); may be null.
cudaError_t launch_attn_fwd_simt(const CcaDims& d, const bf16* q, const bf16* k, const bf16* v, bf16* o,
                                 float* o32, float* lse, cudaStream_t st);
// delta[b,i,t] = sum_c dO[t,i,c] * O[t,i,c] from the fp32 copy of o.
cudaError_t launch_attn_delta(const CcaDims& d, const float* o32, const bf16* d_o, float* delta, cudaStream_t st);
// dq, dk, dv from a delta that launch_attn_delta has filled.
cudaError_t launch_attn_bwd_simt(const CcaDims& d, const bf16* q, const bf16* k, const bf16* v, const float* o32,
                                 const bf16* d_o, const float* lse, float* delta, float* dq, float* dk,
                                 float* dv, cudaStream_t st);
