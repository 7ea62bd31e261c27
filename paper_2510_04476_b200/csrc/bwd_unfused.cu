// Element-wise pieces of the backward for head sizes the fused adjoint kernels do not cover (d_h = 256).  There the
// attention adjoint and the conv2 adjoint run as plain contractions on the library's GEMM kernels over query chunks
// and heads (the host side is in cca_api.cu), with these kernels in between:
//
//   pds_kernel            P = 2^(S c - lse) (masked), dS = P o (dP - delta) / sqrt(d_h) from the score and dP chunks -> bf16
//   cast_dhat_kernel      pre-norm latent gradient (fp32 dq | dk) -> one [T, L] tensor, bf16 (operand) and / or fp32
//   taps_adjoint_kernel   dy1[t, c] = sum_r dy1s[t + (k_ch-1) - r, c k_ch + r]: adjoint of "conv1 output stored at the
//                         k_ch positions conv2 reads"
#include "common.cuh"

namespace {

constexpr float U_LOG2E = 1.4426950408889634f;

// One thread = 4 consecutive keys of one query row of the chunk.
__global__ void __launch_bounds__(256) pds_kernel(const float* __restrict__ s, const float* __restrict__ dp, long long ld,
                                                  const float* __restrict__ lse, const float* __restrict__ delta, int m0,
                                                  int rows, int n_keys, int S, int causal, float c_scale, float ds_scale,
                                                  bf16* __restrict__ p_out, bf16* __restrict__ ds_out) {
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const int quads = (int)(ld / 4);
  const int r = (int)(idx / quads), c4 = (int)(idx % quads) * 4;
  if (r >= rows) return;
  const int tq = m0 + r;
  const bool row_ok = tq < S;
  const float l2 = row_ok ? lse[tq] * U_LOG2E : 0.f, dl = row_ok ? delta[tq] : 0.f;
  const float4 sv = *reinterpret_cast<const float4*>(s + (long long)r * ld + c4);
  const float4 dv = *reinterpret_cast<const float4*>(dp + (long long)r * ld + c4);
  const float se[4] = {sv.x, sv.y, sv.z, sv.w}, de[4] = {dv.x, dv.y, dv.z, dv.w};
  float pv[4], gv[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int key = c4 + i;
    const bool vis = row_ok && key < n_keys && key < S && (!causal || key <= tq);
    const float pr = vis ? exp2f(fmaf(se[i], c_scale, -l2)) : 0.f;
    pv[i] = pr;
    gv[i] = vis ? pr * (de[i] - dl) * ds_scale : 0.f;     // columns past the chunk's keys hold stale scratch
  }
  __nv_bfloat162 a = __floats2bfloat162_rn(pv[0], pv[1]), b = __floats2bfloat162_rn(pv[2], pv[3]);
  uint2 w;
  w.x = *reinterpret_cast<uint32_t*>(&a);
  w.y = *reinterpret_cast<uint32_t*>(&b);
  *reinterpret_cast<uint2*>(p_out + (long long)r * ld + c4) = w;
  a = __floats2bfloat162_rn(gv[0], gv[1]);
  b = __floats2bfloat162_rn(gv[2], gv[3]);
  w.x = *reinterpret_cast<uint32_t*>(&a);
  w.y = *reinterpret_cast<uint32_t*>(&b);
  *reinterpret_cast<uint2*>(ds_out + (long long)r * ld + c4) = w;
}

__global__ void __launch_bounds__(256) cast_dhat_kernel(CcaDims d, const float* __restrict__ dqh, const float* __restrict__ dkh,
                                                        bf16* __restrict__ out, float* __restrict__ out32) {
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;      // one per 4 channels
  const int quads = d.L / 4;
  const long long row = idx / quads;
  const int c = (int)(idx % quads) * 4;
  if (row >= (long long)d.B * d.S) return;
  const float4 v = c < d.Lq ? *reinterpret_cast<const float4*>(dqh + row * d.Lq + c)
                            : *reinterpret_cast<const float4*>(dkh + row * d.Lk + (c - d.Lq));
  __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b = __floats2bfloat162_rn(v.z, v.w);
  uint2 w;
  w.x = *reinterpret_cast<uint32_t*>(&a);
  w.y = *reinterpret_cast<uint32_t*>(&b);
  if (out) *reinterpret_cast<uint2*>(out + row * d.L + c) = w;
  if (out32) *reinterpret_cast<float4*>(out32 + row * d.L + c) = v;
}

__global__ void __launch_bounds__(256) taps_adjoint_kernel(CcaDims d, const float* __restrict__ dy1s, float* __restrict__ dy1) {
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;      // one per (token, channel)
  const long long row = idx / d.L;
  const int c = (int)(idx % d.L);
  if (row >= (long long)d.B * d.S) return;
  const int t = (int)(row % d.S);
  const int kc = d.k_ch;
  float acc = 0.f;
  for (int r = 0; r < kc; ++r) {
    const int tt = t + (kc - 1) - r;               // the token whose conv2 window holds y1[t] at position r
    if (tt < d.S) acc += dy1s[(row + (tt - t)) * ((long long)d.L * kc) + (long long)c * kc + r];
  }
  dy1[row * d.L + c] = acc;
}

}  // namespace

cudaError_t launch_pds(const float* s, const float* dp, long long ld, const float* lse, const float* delta, int m0, int rows,
                       int n_keys, int S, int causal, int dh, bf16* p_out, bf16* ds_out, cudaStream_t st) {
  const long long n = (long long)rows * (ld / 4);
  pds_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(s, dp, ld, lse, delta, m0, rows, n_keys, S, causal,
                                                          rsqrtf((float)dh) * U_LOG2E, rsqrtf((float)dh), p_out, ds_out);
  return cudaGetLastError();
}

cudaError_t launch_cast_dhat(const CcaDims& d, const float* dqh, const float* dkh, bf16* out, float* out32, cudaStream_t st) {
  const long long n = (long long)d.B * d.S * (d.L / 4);
  cast_dhat_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(d, dqh, dkh, out, out32);
  return cudaGetLastError();
}

cudaError_t launch_taps_adjoint(const CcaDims& d, const float* dy1s, float* dy1, cudaStream_t st) {
  const long long n = (long long)d.B * d.S * d.L;
  taps_adjoint_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(d, dy1s, dy1);
  return cudaGetLastError();
}
