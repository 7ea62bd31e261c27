// Plain SIMT softmax attention in the latent (Eq. 11, third line) with grouped kv heads, forward and
// backward.  64x64 tiles, 256 threads as 16x16, fp32 FMA.  These kernels are the always-available
// implementation and the on-device cross-check of the tensor-core kernels.
#include "common.cuh"

namespace {

constexpr int BT = 64;            // tile rows (queries) and columns (keys)
constexpr float LOG2E = 1.4426950408889634f;
constexpr float LN2 = 0.6931471805599453f;

template <int DH>
struct AL {
  static constexpr int LD = DH + 1;
  static constexpr int NC = DH / 16;     // output columns per thread
  static constexpr int PLD = BT + 1;
};

// Load a [BT][DH] tile of a [B,S,H,DH] tensor (rows = tokens t0.., head hh) as fp32; rows >= S are zero.
template <int DH>
CCA_DEVINL void load_rows(const bf16* __restrict__ src, int ld, int S, long long seq_base, int t0, int hh,
                          float* dst, float mul) {
  for (int f = threadIdx.x; f < BT * DH / 8; f += 256) {
    int r = f / (DH / 8), c8 = (f - r * (DH / 8)) * 8;
    int t = t0 + r;
    float* drow = dst + r * AL<DH>::LD + c8;
    if (t < S) {
      uint4 v = *reinterpret_cast<const uint4*>(src + (seq_base + t) * ld + hh * DH + c8);
      const bf16* e = reinterpret_cast<const bf16*>(&v);
#pragma unroll
      for (int i = 0; i < 8; ++i) drow[i] = __bfloat162float(e[i]) * mul;
    } else {
#pragma unroll
      for (int i = 0; i < 8; ++i) drow[i] = 0.f;
    }
  }
}

// s[a][c] = sum_d X[ty*4+a][d] * Y[tx*4+c][d]
template <int DH>
CCA_DEVINL void tile_dot(const float* X, const float* Y, int ty, int tx, float (&s)[4][4]) {
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int c = 0; c < 4; ++c) s[a][c] = 0.f;
  for (int dd = 0; dd < DH; ++dd) {
    float x[4], y[4];
#pragma unroll
    for (int a = 0; a < 4; ++a) x[a] = X[(ty * 4 + a) * AL<DH>::LD + dd];
#pragma unroll
    for (int c = 0; c < 4; ++c) y[c] = Y[(tx * 4 + c) * AL<DH>::LD + dd];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
      for (int c = 0; c < 4; ++c) s[a][c] = fmaf(x[a], y[c], s[a][c]);
  }
}

CCA_DEVINL float half_warp_max(float v) {
#pragma unroll
  for (int off = 8; off > 0; off >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, off));
  return v;
}
CCA_DEVINL float half_warp_sum(float v) {
#pragma unroll
  for (int off = 8; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
  return v;
}

// ------------------------------------------------------------------------------------------
template <int DH>
__global__ void __launch_bounds__(256) attn_fwd_kernel(CcaDims d, const bf16* __restrict__ q,
                                                       const bf16* __restrict__ k, const bf16* __restrict__ v,
                                                       bf16* __restrict__ o, float* __restrict__ o32,
                                                       float* __restrict__ lse) {
  extern __shared__ __align__(16) float smf[];
  constexpr int LD = AL<DH>::LD, NC = AL<DH>::NC, PLD = AL<DH>::PLD;
  float* Qs = smf;
  float* Ks = Qs + BT * LD;
  float* Vs = Ks + BT * LD;
  float* Ps = Vs + BT * LD;
  const int m0 = blockIdx.x * BT, hi = blockIdx.y, b = blockIdx.z, hj = hi / d.g;
  const int ty = threadIdx.x / 16, tx = threadIdx.x % 16;
  const long long seq_base = (long long)b * d.S;
  const float sc = rsqrtf((float)DH) * LOG2E;
  load_rows<DH>(q, d.Lq, d.S, seq_base, m0, hi, Qs, sc);
  float m_i[4], l_i[4], acc[4][NC];
#pragma unroll
  for (int a = 0; a < 4; ++a) {
    m_i[a] = -INFINITY;
    l_i[a] = 0.f;
#pragma unroll
    for (int c = 0; c < NC; ++c) acc[a][c] = 0.f;
  }
  const int n_end = d.causal ? min(d.S, m0 + BT) : d.S;
  for (int n0 = 0; n0 < n_end; n0 += BT) {
    __syncthreads();
    load_rows<DH>(k, d.Lk, d.S, seq_base, n0, hj, Ks, 1.f);
    load_rows<DH>(v, d.Lk, d.S, seq_base, n0, hj, Vs, 1.f);
    __syncthreads();
    float s[4][4];
    tile_dot<DH>(Qs, Ks, ty, tx, s);
#pragma unroll
    for (int a = 0; a < 4; ++a) {
      int tq = m0 + ty * 4 + a;
      float mx = -INFINITY;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        int tk = n0 + tx * 4 + c;
        if (tk >= d.S || (d.causal && tk > tq)) s[a][c] = -INFINITY;
        mx = fmaxf(mx, s[a][c]);
      }
      mx = half_warp_max(mx);
      float m_new = fmaxf(m_i[a], mx);
      float m_use = (m_new == -INFINITY) ? 0.f : m_new;
      float alpha = exp2f(m_i[a] - m_use);
      float rs = 0.f;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        float p = exp2f(s[a][c] - m_use);
        rs += p;
        Ps[(ty * 4 + a) * PLD + tx * 4 + c] = p;
      }
      rs = half_warp_sum(rs);
      l_i[a] = l_i[a] * alpha + rs;
      m_i[a] = m_new;
#pragma unroll
      for (int c = 0; c < NC; ++c) acc[a][c] *= alpha;
    }
    __syncthreads();
    for (int kk = 0; kk < BT; ++kk) {
      float p[4], vv[NC];
#pragma unroll
      for (int a = 0; a < 4; ++a) p[a] = Ps[(ty * 4 + a) * PLD + kk];
#pragma unroll
      for (int c = 0; c < NC; ++c) vv[c] = Vs[kk * LD + tx + 16 * c];
#pragma unroll
      for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int c = 0; c < NC; ++c) acc[a][c] = fmaf(p[a], vv[c], acc[a][c]);
    }
  }
#pragma unroll
  for (int a = 0; a < 4; ++a) {
    int tq = m0 + ty * 4 + a;
    if (tq >= d.S) continue;
    float inv = 1.f / l_i[a];
#pragma unroll
    for (int c = 0; c < NC; ++c) {
      long long idx = (seq_base + tq) * d.Lq + hi * DH + tx + 16 * c;
      o[idx] = __float2bfloat16(acc[a][c] * inv);
      if (o32) o32[idx] = acc[a][c] * inv;
    }
    if (tx == 0) lse[((long long)b * d.hq + hi) * d.S + tq] = (m_i[a] + log2f(l_i[a])) * LN2;
  }
}

// delta[b,i,t] = sum_c dO[t,i,c] * O[t,i,c].  O is the fp32 copy kept by the forward: delta is subtracted from
// dP = dO V^T inside the softmax adjoint, and rounding O to bf16 there would cost the dominant keys several
// digits.  A group of d_h/8 lanes owns one (token, head): 8 channels per lane, 128-bit loads.
template <int DH>
__global__ void __launch_bounds__(256) attn_delta_kernel(CcaDims d, const float* __restrict__ o,
                                                         const bf16* __restrict__ d_o, float* __restrict__ delta) {
  constexpr int TPR = DH / 8;                       // lanes per row
  const long long gt = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const long long w = gt / TPR;
  const int sub = (int)(gt % TPR);
  const long long total = (long long)d.B * d.S * d.hq;
  float s = 0.f;
  const bool act = w < total;
  int hi = 0;
  long long row = 0;
  if (act) {
    hi = (int)(w % d.hq);
    row = w / d.hq;
    const float4* po = reinterpret_cast<const float4*>(o + row * d.Lq + hi * DH + sub * 8);
    const uint4 dv = *reinterpret_cast<const uint4*>(d_o + row * d.Lq + hi * DH + sub * 8);
    const float4 a = po[0], c = po[1];
    const __nv_bfloat162* db = reinterpret_cast<const __nv_bfloat162*>(&dv);
    const float2 d0 = __bfloat1622float2(db[0]), d1 = __bfloat1622float2(db[1]), d2 = __bfloat1622float2(db[2]),
                 d3 = __bfloat1622float2(db[3]);
    s = a.x * d0.x + a.y * d0.y + a.z * d1.x + a.w * d1.y + c.x * d2.x + c.y * d2.y + c.z * d3.x + c.w * d3.y;
  }
#pragma unroll
  for (int off = TPR / 2; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
  if (act && sub == 0) {
    const int b = (int)(row / d.S), t = (int)(row % d.S);
    delta[((long long)b * d.hq + hi) * d.S + t] = s;
  }
}

// Recompute P and dS for the 4x4 sub-tile of (query tile m0, key tile n0); write them to smem.
template <int DH>
CCA_DEVINL void p_and_ds(const CcaDims& d, const float* Qs, const float* Ks, const float* dOs, const float* Vs,
                         const float* __restrict__ lse_row, const float* __restrict__ delta_row, int m0, int n0,
                         int ty, int tx, float* Ps, float* dSs) {
  constexpr int PLD = AL<DH>::PLD;
  float s[4][4], dp[4][4];
  tile_dot<DH>(Qs, Ks, ty, tx, s);       // Qs pre-scaled by log2(e)/sqrt(d_h)
  tile_dot<DH>(dOs, Vs, ty, tx, dp);
#pragma unroll
  for (int a = 0; a < 4; ++a) {
    int tq = m0 + ty * 4 + a;
    float l2 = 0.f, dl = 0.f;
    if (tq < d.S) {
      l2 = lse_row[tq] * LOG2E;
      dl = delta_row[tq];
    }
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      int tk = n0 + tx * 4 + c;
      bool ok = tq < d.S && tk < d.S && !(d.causal && tk > tq);
      float p = ok ? exp2f(s[a][c] - l2) : 0.f;
      Ps[(ty * 4 + a) * PLD + tx * 4 + c] = p;
      dSs[(ty * 4 + a) * PLD + tx * 4 + c] = p * (dp[a][c] - dl);
    }
  }
}

// dK, dV of one key tile: loops over the g query heads of the kv head and over the query tiles.
template <int DH>
__global__ void __launch_bounds__(256) attn_bwd_dkdv_kernel(CcaDims d, const bf16* __restrict__ q,
                                                            const bf16* __restrict__ k, const bf16* __restrict__ v,
                                                            const bf16* __restrict__ d_o,
                                                            const float* __restrict__ lse,
                                                            const float* __restrict__ delta, float* __restrict__ dk,
                                                            float* __restrict__ dv) {
  extern __shared__ __align__(16) float smf[];
  constexpr int LD = AL<DH>::LD, NC = AL<DH>::NC, PLD = AL<DH>::PLD;
  float* Ks = smf;
  float* Vs = Ks + BT * LD;
  float* Qs = Vs + BT * LD;
  float* dOs = Qs + BT * LD;
  float* Ps = dOs + BT * LD;
  float* dSs = Ps + BT * PLD;
  const int n0 = blockIdx.x * BT, hj = blockIdx.y, b = blockIdx.z;
  const int ty = threadIdx.x / 16, tx = threadIdx.x % 16;
  const long long seq_base = (long long)b * d.S;
  const float scale = rsqrtf((float)DH);
  load_rows<DH>(k, d.Lk, d.S, seq_base, n0, hj, Ks, 1.f);
  load_rows<DH>(v, d.Lk, d.S, seq_base, n0, hj, Vs, 1.f);
  float dk_acc[4][NC], dv_acc[4][NC];
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int c = 0; c < NC; ++c) dk_acc[a][c] = dv_acc[a][c] = 0.f;
  for (int gi = 0; gi < d.g; ++gi) {
    const int hi = hj * d.g + gi;
    const float* lse_row = lse + ((long long)b * d.hq + hi) * d.S;
    const float* delta_row = delta + ((long long)b * d.hq + hi) * d.S;
    for (int m0 = d.causal ? n0 : 0; m0 < d.S; m0 += BT) {
      __syncthreads();
      load_rows<DH>(q, d.Lq, d.S, seq_base, m0, hi, Qs, scale * LOG2E);
      load_rows<DH>(d_o, d.Lq, d.S, seq_base, m0, hi, dOs, 1.f);
      __syncthreads();
      p_and_ds<DH>(d, Qs, Ks, dOs, Vs, lse_row, delta_row, m0, n0, ty, tx, Ps, dSs);
      __syncthreads();
      for (int r = 0; r < BT; ++r) {
        float p[4], ds[4], dov[NC], qv[NC];
#pragma unroll
        for (int a = 0; a < 4; ++a) {
          p[a] = Ps[r * PLD + ty * 4 + a];
          ds[a] = dSs[r * PLD + ty * 4 + a];
        }
#pragma unroll
        for (int c = 0; c < NC; ++c) {
          dov[c] = dOs[r * LD + tx + 16 * c];
          qv[c] = Qs[r * LD + tx + 16 * c];
        }
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
          for (int c = 0; c < NC; ++c) {
            dv_acc[a][c] = fmaf(p[a], dov[c], dv_acc[a][c]);
            dk_acc[a][c] = fmaf(ds[a], qv[c], dk_acc[a][c]);
          }
      }
    }
  }
  // Qs carried scale*log2e; dK = dS^T Q * scale  =>  divide the log2e back out.
  const float fix = 1.f / LOG2E;
#pragma unroll
  for (int a = 0; a < 4; ++a) {
    int tk = n0 + ty * 4 + a;
    if (tk >= d.S) continue;
#pragma unroll
    for (int c = 0; c < NC; ++c) {
      long long idx = (seq_base + tk) * d.Lk + hj * DH + tx + 16 * c;
      dk[idx] = dk_acc[a][c] * fix;
      dv[idx] = dv_acc[a][c];
    }
  }
}

// dQ of one query tile.
template <int DH>
__global__ void __launch_bounds__(256) attn_bwd_dq_kernel(CcaDims d, const bf16* __restrict__ q,
                                                          const bf16* __restrict__ k, const bf16* __restrict__ v,
                                                          const bf16* __restrict__ d_o, const float* __restrict__ lse,
                                                          const float* __restrict__ delta, float* __restrict__ dq) {
  extern __shared__ __align__(16) float smf[];
  constexpr int LD = AL<DH>::LD, NC = AL<DH>::NC, PLD = AL<DH>::PLD;
  float* Ks = smf;
  float* Vs = Ks + BT * LD;
  float* Qs = Vs + BT * LD;
  float* dOs = Qs + BT * LD;
  float* Ps = dOs + BT * LD;
  float* dSs = Ps + BT * PLD;
  const int m0 = blockIdx.x * BT, hi = blockIdx.y, b = blockIdx.z, hj = hi / d.g;
  const int ty = threadIdx.x / 16, tx = threadIdx.x % 16;
  const long long seq_base = (long long)b * d.S;
  const float scale = rsqrtf((float)DH);
  const float* lse_row = lse + ((long long)b * d.hq + hi) * d.S;
  const float* delta_row = delta + ((long long)b * d.hq + hi) * d.S;
  load_rows<DH>(q, d.Lq, d.S, seq_base, m0, hi, Qs, scale * LOG2E);
  load_rows<DH>(d_o, d.Lq, d.S, seq_base, m0, hi, dOs, 1.f);
  float acc[4][NC];
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int c = 0; c < NC; ++c) acc[a][c] = 0.f;
  const int n_end = d.causal ? min(d.S, m0 + BT) : d.S;
  for (int n0 = 0; n0 < n_end; n0 += BT) {
    __syncthreads();
    load_rows<DH>(k, d.Lk, d.S, seq_base, n0, hj, Ks, 1.f);
    load_rows<DH>(v, d.Lk, d.S, seq_base, n0, hj, Vs, 1.f);
    __syncthreads();
    p_and_ds<DH>(d, Qs, Ks, dOs, Vs, lse_row, delta_row, m0, n0, ty, tx, Ps, dSs);
    __syncthreads();
    for (int kk = 0; kk < BT; ++kk) {
      float ds[4], kv[NC];
#pragma unroll
      for (int a = 0; a < 4; ++a) ds[a] = dSs[(ty * 4 + a) * PLD + kk];
#pragma unroll
      for (int c = 0; c < NC; ++c) kv[c] = Ks[kk * LD + tx + 16 * c];
#pragma unroll
      for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int c = 0; c < NC; ++c) acc[a][c] = fmaf(ds[a], kv[c], acc[a][c]);
    }
  }
#pragma unroll
  for (int a = 0; a < 4; ++a) {
    int tq = m0 + ty * 4 + a;
    if (tq >= d.S) continue;
#pragma unroll
    for (int c = 0; c < NC; ++c) dq[(seq_base + tq) * d.Lq + hi * DH + tx + 16 * c] = acc[a][c] * scale;
  }
}

template <typename K>
cudaError_t set_smem(K kern, size_t bytes) {
  return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
}

}  // namespace

#define DISPATCH_DH(dh, ...)                                    \
  switch (dh) {                                                 \
    case 32: { constexpr int DH = 32; __VA_ARGS__; break; }     \
    case 64: { constexpr int DH = 64; __VA_ARGS__; break; }     \
    case 128: { constexpr int DH = 128; __VA_ARGS__; break; }   \
    default: return cudaErrorInvalidValue;                      \
  }

cudaError_t launch_attn_fwd_simt(const CcaDims& d, const bf16* q, const bf16* k, const bf16* v, bf16* o, float* o32,
                                 float* lse, cudaStream_t st) {
  dim3 grid((d.S + BT - 1) / BT, d.hq, d.B);
  if (d.dh == 256) {                       // forward only exists at this head size
    constexpr int DH = 256;
    size_t sm = (size_t)(3 * BT * AL<DH>::LD + BT * AL<DH>::PLD) * sizeof(float);
    cudaError_t e = set_smem(attn_fwd_kernel<DH>, sm);
    if (e != cudaSuccess) return e;
    attn_fwd_kernel<DH><<<grid, 256, sm, st>>>(d, q, k, v, o, o32, lse);
    return cudaGetLastError();
  }
  DISPATCH_DH(d.dh, {
    size_t sm = (size_t)(3 * BT * AL<DH>::LD + BT * AL<DH>::PLD) * sizeof(float);
    cudaError_t e = set_smem(attn_fwd_kernel<DH>, sm);
    if (e != cudaSuccess) return e;
    attn_fwd_kernel<DH><<<grid, 256, sm, st>>>(d, q, k, v, o, o32, lse);
  });
  return cudaGetLastError();
}

cudaError_t launch_attn_delta(const CcaDims& d, const float* o32, const bf16* d_o, float* delta, cudaStream_t st) {
  const long long rows = (long long)d.B * d.S * d.hq;
  if (d.dh == 256) {
    const long long threads = rows * (256 / 8);
    attn_delta_kernel<256><<<(unsigned)((threads + 255) / 256), 256, 0, st>>>(d, o32, d_o, delta);
    return cudaGetLastError();
  }
  DISPATCH_DH(d.dh, {
    const long long threads = rows * (DH / 8);
    attn_delta_kernel<DH><<<(unsigned)((threads + 255) / 256), 256, 0, st>>>(d, o32, d_o, delta);
  });
  return cudaGetLastError();
}

cudaError_t launch_attn_bwd_simt(const CcaDims& d, const bf16* q, const bf16* k, const bf16* v, const float* o32,
                                 const bf16* d_o, const float* lse, float* delta, float* dq, float* dk, float* dv,
                                 cudaStream_t st) {
  (void)o32;
  cudaError_t e;
  DISPATCH_DH(d.dh, {
    size_t sm = (size_t)(4 * BT * AL<DH>::LD + 2 * BT * AL<DH>::PLD) * sizeof(float);
    e = set_smem(attn_bwd_dkdv_kernel<DH>, sm);
    if (e != cudaSuccess) return e;
    e = set_smem(attn_bwd_dq_kernel<DH>, sm);
    if (e != cudaSuccess) return e;
    dim3 gkv((d.S + BT - 1) / BT, d.hk, d.B);
    attn_bwd_dkdv_kernel<DH><<<gkv, 256, sm, st>>>(d, q, k, v, d_o, lse, delta, dk, dv);
    dim3 gq((d.S + BT - 1) / BT, d.hq, d.B);
    attn_bwd_dq_kernel<DH><<<gq, 256, sm, st>>>(d, q, k, v, d_o, lse, delta, dq);
  });
  return cudaGetLastError();
}
