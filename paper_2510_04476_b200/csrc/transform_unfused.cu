// Latent transforms of Eq. 8, 9 and 11 for head sizes the fused kernel does not cover (d_h = 256): the same
// arithmetic in three steps with the channel convolution as ordinary contractions.
//   conv1_taps_kernel   y1 = conv1_seq(qk0) (Eq. 8) written, for every token, at the k_ch positions conv2 reads:
//                       y1s[t, c * k_ch + r] = y1[t - (k_ch - 1) + r, c] (bf16), so that conv2 of head h becomes
//                       y2[:, h] = y1s[:, h d_h k_ch : (h+1) d_h k_ch] W_h^T with W_h = conv1_w rows of the head,
//                       a [d_h, d_h k_ch] K-major matrix exactly as the parameter is stored
//   (the caller runs one tensor-core GEMM per head)
//   finalize_kernel     q-k-mean (Eq. 9), L2 norm * sqrt(d_h) [* exp(temp)], RoPE (Eq. 11): one warp per (token, head)
#include "common.cuh"

namespace {

enum : unsigned { F_CONV1 = 1, F_CONV2 = 2, F_QK_MEAN = 4, F_QK_NORM = 16, F_ROPE = 32 };

CCA_DEVINL uint32_t pack2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// thread = (token, 4 channels)
__global__ void __launch_bounds__(256) conv1_taps_kernel(CcaDims d, const float* __restrict__ qk0, const bf16* __restrict__ w0,
                                                         bf16* __restrict__ y1s, float* __restrict__ y2) {
  // blockIdx.x = token (of all sequences), blockIdx.y * 256 + thread = channel quad: no per-thread division
  const int quad = blockIdx.y * 256 + threadIdx.x;
  if (quad >= d.L / 4) return;
  const long long tok = blockIdx.x;
  const int ch = quad * 4;
  const int t = (int)(blockIdx.x % (unsigned)d.S);
  const int ks = (d.flags & F_CONV1) ? d.k_seq : 1;
  const int kc = (d.flags & F_CONV2) ? d.k_ch : 1;
  const int span = ks + kc - 1;                      // raw tokens t - span + 1 .. t
  float4 raw[7];
#pragma unroll
  for (int i = 0; i < 7; ++i) {
    raw[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    const int back = span - 1 - i;                   // raw[i] = token t - back
    if (i < span && t - back >= 0) raw[i] = *reinterpret_cast<const float4*>(qk0 + (tok - back) * d.L + ch);
  }
  float wt[4][4];
#pragma unroll
  for (int c = 0; c < 4; ++c)
#pragma unroll
    for (int j = 0; j < 4; ++j)
      wt[c][j] = (j < ks) ? ((d.flags & F_CONV1) ? __bfloat162float(w0[(size_t)(ch + c) * d.k_seq + j]) : 1.f) : 0.f;
  // the thread's 4 channels x kc taps are contiguous in y1s: element (c, r) at (ch + c) * kc + r
  float yv[4][4];
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    // y1 at token t - (kc - 1) + r: taps j = 0..ks-1 read raw tokens t - (kc-1) + r - (ks-1) + j = raw[r + j]
    float y[4] = {0.f, 0.f, 0.f, 0.f};
    if (r < kc && t - (kc - 1) + r >= 0) {
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        if (j < ks) {
          const float4 v = raw[r + j];
          y[0] = fmaf(wt[0][j], v.x, y[0]);
          y[1] = fmaf(wt[1][j], v.y, y[1]);
          y[2] = fmaf(wt[2][j], v.z, y[2]);
          y[3] = fmaf(wt[3][j], v.w, y[3]);
        }
      }
    }
#pragma unroll
    for (int c = 0; c < 4; ++c) yv[c][r] = y[c];
  }
  if (!(d.flags & F_CONV2)) {
    *reinterpret_cast<float4*>(y2 + tok * d.L + ch) = make_float4(yv[0][0], yv[1][0], yv[2][0], yv[3][0]);
    return;
  }
  bf16* dst = y1s + (tok * d.L + ch) * kc;          // 8 kc bytes, 8-byte aligned
  if (kc == 2) {
    uint4 w;
    w.x = pack2(yv[0][0], yv[0][1]); w.y = pack2(yv[1][0], yv[1][1]);
    w.z = pack2(yv[2][0], yv[2][1]); w.w = pack2(yv[3][0], yv[3][1]);
    *reinterpret_cast<uint4*>(dst) = w;
  } else if (kc == 4) {
#pragma unroll
    for (int c = 0; c < 4; ++c)
      reinterpret_cast<uint2*>(dst)[c] = make_uint2(pack2(yv[c][0], yv[c][1]), pack2(yv[c][2], yv[c][3]));
  } else if (kc == 1) {
    *reinterpret_cast<uint2*>(dst) = make_uint2(pack2(yv[0][0], yv[1][0]), pack2(yv[2][0], yv[3][0]));
  } else {                                           // kc == 3: 12 elements
    const float f[12] = {yv[0][0], yv[0][1], yv[0][2], yv[1][0], yv[1][1], yv[1][2],
                         yv[2][0], yv[2][1], yv[2][2], yv[3][0], yv[3][1], yv[3][2]};
#pragma unroll
    for (int i = 0; i < 3; ++i)
      reinterpret_cast<uint2*>(dst)[i] = make_uint2(pack2(f[4 * i], f[4 * i + 1]), pack2(f[4 * i + 2], f[4 * i + 3]));
  }
}

// one warp per (token, head); lane l owns channels l + 32 u, so the rotation partner c + d_h/2 is in the same lane
template <int DH>
__global__ void __launch_bounds__(256) finalize_kernel(CcaDims d, const float* __restrict__ qk0, const float* __restrict__ y2,
                                                       const float* __restrict__ temp, const float2* __restrict__ rope,
                                                       bf16* __restrict__ q, bf16* __restrict__ k, float* __restrict__ rnorm) {
  constexpr int U = DH / 32;
  const int lane = threadIdx.x & 31;
  const int heads = d.hq + d.hk;
  const long long tok = blockIdx.x;                  // token of all sequences; the block's 8 warps walk its heads
  const int t = (int)(blockIdx.x % (unsigned)d.S);
  for (int h = threadIdx.x >> 5; h < heads; h += 8) {
  const bool is_q = h < d.hq;
  const int hj = is_q ? h / d.g : h - d.hq;
  const float* lat = qk0 + tok * d.L;
  float v[U];
  float ss = 0.f;
#pragma unroll
  for (int u = 0; u < U; ++u) {
    const int c = lane + 32 * u;
    float x = y2[tok * d.L + h * DH + c];
    if (d.flags & F_QK_MEAN) {
      if (is_q) {
        x += 0.5f * (lat[h * DH + c] + lat[d.Lq + hj * DH + c]);
      } else {
        float sq = 0.f;
        for (int i = 0; i < d.g; ++i) sq += lat[(hj * d.g + i) * DH + c];
        x += 0.5f * lat[h * DH + c] + 0.5f * sq / (float)d.g;
      }
    }
    v[u] = x;
    ss = fmaf(x, x, ss);
  }
  float sc = 1.f;
  if (d.flags & F_QK_NORM) {
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, s);
    sc = sqrtf((float)DH) * rsqrtf(ss);
    if (!is_q) sc *= __expf(temp[hj]);
  }
  if (lane == 0) rnorm[tok * heads + h] = sc;
  bf16* dst = is_q ? q + tok * d.Lq + h * DH : k + tok * d.Lk + hj * DH;
#pragma unroll
  for (int u = 0; u < U / 2; ++u) {
    const int c = lane + 32 * u;                     // pair (c, c + DH/2)
    float a = v[u] * sc, b = v[u + U / 2] * sc;
    if (d.flags & F_ROPE) {
      const float2 cs = rope[(size_t)t * (DH / 2) + c];
      const float a2 = a * cs.x - b * cs.y;
      b = b * cs.x + a * cs.y;
      a = a2;
    }
    dst[c] = __float2bfloat16(a);
    dst[c + DH / 2] = __float2bfloat16(b);
  }
  }
}

}  // namespace

cudaError_t launch_conv1_taps(const CcaDims& d, const float* qk0, const bf16* w0, bf16* y1s, float* y2, cudaStream_t st) {
  dim3 grid((unsigned)((long long)d.B * d.S), (unsigned)((d.L / 4 + 255) / 256));
  conv1_taps_kernel<<<grid, 256, 0, st>>>(d, qk0, w0, y1s, y2);
  return cudaGetLastError();
}

cudaError_t launch_finalize(const CcaDims& d, const float* qk0, const float* y2, const float* temp, const float2* rope,
                            bf16* q, bf16* k, float* rnorm, cudaStream_t st) {
  const unsigned grid = (unsigned)((long long)d.B * d.S);
  switch (d.dh) {
    case 64: finalize_kernel<64><<<grid, 256, 0, st>>>(d, qk0, y2, temp, rope, q, k, rnorm); break;
    case 128: finalize_kernel<128><<<grid, 256, 0, st>>>(d, qk0, y2, temp, rope, q, k, rnorm); break;
    case 256: finalize_kernel<256><<<grid, 256, 0, st>>>(d, qk0, y2, temp, rope, q, k, rnorm); break;
    default: return cudaErrorInvalidValue;
  }
  return cudaGetLastError();
}
