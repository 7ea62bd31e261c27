// Decode step against the latent KV cache: host-side launcher interface.
#pragma once
#include "common.cuh"

struct DecodeWeights {
  const bf16 *w_qk, *w_v1, *w_v2, *w_o, *conv0_w, *conv1_w;
  const float* temp;
};

struct DecodeState {
  bf16* k_cache;      // [B, S_max, Lk]
  bf16* v_cache;      // [B, S_max, Lk]
  float* qk0_hist;    // [B, k_seq + k_ch - 2, L]
  bf16* x_prev;       // [B, E]
  const int* pos;     // [B]
  long long S_max;
};

// Key chunk per CTA and number of chunks for sequences of up to max_len tokens.
void decode_plan(const CcaDims& d, int max_len, int sm_count, int* chunk, int* splits);
size_t decode_workspace_bytes(const CcaDims& d, int max_len, int sm_count);
// 0 = enqueued, 1 = shape not covered, < 0 = minus a cudaError_t.  *launches is advanced by the kernels enqueued.
// The two events (may be null) are recorded around the attention kernel.
int launch_decode_step(const CcaDims& d, const DecodeWeights& w, const bf16* x, bf16* out, const DecodeState& s,
                       int max_len, void* workspace, int sm_count, int* status, long long* launches, cudaEvent_t ev_attn_begin,
                       cudaEvent_t ev_attn_end, cudaStream_t st);
