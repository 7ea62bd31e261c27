// Latent transforms on q and k between the down-projection and the attention (Eq. 8, 9, 11):
// conv1_seq, conv2_seq+ch, q-k-mean, L2 norm * sqrt(d_h) (* exp(temp) for keys), RoPE;
// and their adjoints.  One thread block works on (a run of 32-token tiles, one head, one sequence).
// Thread layout: 256 threads = (256/DH) token groups x DH channels; a thread owns one channel of
// TT/(256/DH) consecutive tokens of the tile.
#include "common.cuh"

namespace {

constexpr int TT = 32;             // tokens per tile
constexpr int TILES_PER_BLOCK = 4; // tiles a block walks through with one load of the conv2 weights
constexpr int MAXK = 4;            // largest conv kernel size

enum : unsigned { F_CONV1 = 1, F_CONV2 = 2, F_QK_MEAN = 4, F_V_SHIFT = 8, F_QK_NORM = 16, F_ROPE = 32 };

template <int DH>
struct Lay {
  static constexpr int NG = 256 / DH;        // token groups
  static constexpr int TPT = TT / NG;        // tokens per thread
  static constexpr int WLD = DH + 2;         // bf16 row stride of the staged conv2 weights
  static constexpr int YLD = DH + 1;         // fp32 row stride of token-major tiles
  static constexpr int YROWS = TT + 2 * (MAXK - 1);
};

CCA_DEVINL float ldbf(const bf16* p) { return __bfloat162float(*p); }

// conv1_seq output (or the raw latent if the stage is off) of channel `ch` at token t of sequence b.
CCA_DEVINL float y1_at(const CcaDims& d, const float* qk0, const bf16* w0, int b, int t, int ch) {
  if (t < 0 || t >= d.S) return 0.f;
  const float* col = qk0 + (long long)b * d.S * d.L + ch;
  if (!(d.flags & F_CONV1)) return col[(long long)t * d.L];
  float acc = 0.f;
  for (int j = 0; j < d.k_seq; ++j) {
    int ts = t - (d.k_seq - 1) + j;
    if (ts >= 0) acc = fmaf(ldbf(w0 + ch * d.k_seq + j), col[(long long)ts * d.L], acc);
  }
  return acc;
}

// Stage the conv2 weights of head h as ws[(i*k_ch + j)][o]  (forward) or ws[(o*k_ch + j)][i] (adjoint).
template <int DH, bool kAdjoint>
CCA_DEVINL void stage_w1(const CcaDims& d, const bf16* w1, int h, bf16* ws) {
  const int per_o = DH * d.k_ch;
  const bf16* src = w1 + (long long)h * DH * per_o;
  for (int f = threadIdx.x; f < DH * per_o; f += 256) {
    int o = f / per_o, rem = f - o * per_o;       // rem = i*k_ch + j
    if (!kAdjoint) ws[rem * Lay<DH>::WLD + o] = src[f];
    else {
      int i = rem / d.k_ch, j = rem - i * d.k_ch;
      ws[(o * d.k_ch + j) * Lay<DH>::WLD + i] = src[f];
    }
  }
}

// y1s[r][c], r in [0, rows): conv1 output of head h's channels at token t_first + r.
template <int DH>
CCA_DEVINL void fill_y1(const CcaDims& d, const float* qk0, const bf16* w0, int b, int h, int t_first, int rows,
                        float* y1s) {
  for (int f = threadIdx.x; f < rows * DH; f += 256) {
    int r = f / DH, c = f - r * DH;
    y1s[r * Lay<DH>::YLD + c] = y1_at(d, qk0, w0, b, t_first + r, h * DH + c);
  }
}

// Pre-norm latent (conv2 output + q-k-mean term) of channel o for this thread's tokens.
// y1s row r holds token t0 - (k_ch-1) + r.
template <int DH>
CCA_DEVINL void hat_tile(const CcaDims& d, const float* qk0, const bf16* ws, const float* y1s, int b, int h, int t0,
                         float (&acc)[Lay<DH>::TPT]) {
  constexpr int TPT = Lay<DH>::TPT;
  const int o = threadIdx.x % DH, tg = threadIdx.x / DH;
  const int kc = (d.flags & F_CONV2) ? d.k_ch : 1;
#pragma unroll
  for (int n = 0; n < TPT; ++n) acc[n] = 0.f;
  if (d.flags & F_CONV2) {
    for (int i = 0; i < DH; ++i) {
      for (int j = 0; j < kc; ++j) {
        float w = __bfloat162float(ws[(i * kc + j) * Lay<DH>::WLD + o]);
        const float* yp = y1s + (tg * TPT + j) * Lay<DH>::YLD + i;
#pragma unroll
        for (int n = 0; n < TPT; ++n) acc[n] = fmaf(w, yp[n * Lay<DH>::YLD], acc[n]);
      }
    }
  } else {
#pragma unroll
    for (int n = 0; n < TPT; ++n) acc[n] = y1s[(tg * TPT + n + (d.k_ch - 1)) * Lay<DH>::YLD + o];
  }
  if (d.flags & F_QK_MEAN) {
    const float* base = qk0 + (long long)b * d.S * d.L;
#pragma unroll
    for (int n = 0; n < TPT; ++n) {
      int t = t0 + tg * TPT + n;
      if (t >= d.S) continue;
      const float* row = base + (long long)t * d.L;
      if (h < d.hq) {
        acc[n] += 0.5f * (row[h * DH + o] + row[d.Lq + (h / d.g) * DH + o]);
      } else {
        int jk = h - d.hq;
        float sq = 0.f;
        for (int i = 0; i < d.g; ++i) sq += row[(jk * d.g + i) * DH + o];
        acc[n] += 0.5f * row[d.Lq + jk * DH + o] + (0.5f / d.g) * sq;
      }
    }
  }
}

// Sum over the DH channels of each of this thread's tokens (all threads of the group get the result).
template <int DH>
CCA_DEVINL void reduce_channels(float (&v)[Lay<DH>::TPT], float* red /*[NG][DH/32][TPT]*/) {
  constexpr int TPT = Lay<DH>::TPT, NW = DH / 32;
  const int o = threadIdx.x % DH, tg = threadIdx.x / DH, wi = o / 32;
#pragma unroll
  for (int n = 0; n < TPT; ++n) {
    float s = v[n];
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
    v[n] = s;
  }
  if (NW > 1) {
    __syncthreads();
    if ((o & 31) == 0)
#pragma unroll
      for (int n = 0; n < TPT; ++n) red[(tg * NW + wi) * TPT + n] = v[n];
    __syncthreads();
#pragma unroll
    for (int n = 0; n < TPT; ++n) {
      float s = 0.f;
#pragma unroll
      for (int w = 0; w < NW; ++w) s += red[(tg * NW + w) * TPT + n];
      v[n] = s;
    }
  }
}

template <int DH>
constexpr size_t smem_bytes() {
  return (size_t)DH * MAXK * Lay<DH>::WLD * sizeof(bf16) + (size_t)Lay<DH>::YROWS * Lay<DH>::YLD * sizeof(float) +
         (size_t)(TT + 2 * (MAXK - 1)) * Lay<DH>::YLD * sizeof(float) + 256 * sizeof(float);
}

template <int DH>
struct Smem {
  bf16* ws;
  float* y1s;
  float* outs;
  float* red;
  __device__ explicit Smem(unsigned char* base) {
    ws = reinterpret_cast<bf16*>(base);
    y1s = reinterpret_cast<float*>(base + (size_t)DH * MAXK * Lay<DH>::WLD * sizeof(bf16));
    outs = y1s + Lay<DH>::YROWS * Lay<DH>::YLD;
    red = outs + (TT + 2 * (MAXK - 1)) * Lay<DH>::YLD;
  }
};

// ------------------------------------------------------------------------------------------
// forward
// ------------------------------------------------------------------------------------------
template <int DH>
__global__ void __launch_bounds__(256) transform_fwd_kernel(CcaDims d, const float* __restrict__ qk0,
                                                            const bf16* __restrict__ w0, const bf16* __restrict__ w1,
                                                            const float* __restrict__ temp,
                                                            const float2* __restrict__ rope_tab, bf16* __restrict__ q,
                                                            bf16* __restrict__ k, float* __restrict__ rnorm) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  Smem<DH> sm(smem_raw);
  constexpr int TPT = Lay<DH>::TPT, YLD = Lay<DH>::YLD;
  const int h = blockIdx.y, b = blockIdx.z;
  const int o = threadIdx.x % DH, tg = threadIdx.x / DH;
  if (d.flags & F_CONV2) stage_w1<DH, false>(d, w1, h, sm.ws);
  const float scale = (d.flags & F_QK_NORM) ? sqrtf((float)DH) * (h >= d.hq ? __expf(temp[h - d.hq]) : 1.f) : 1.f;
  for (int tile = 0; tile < TILES_PER_BLOCK; ++tile) {
    const int t0 = (blockIdx.x * TILES_PER_BLOCK + tile) * TT;
    if (t0 >= d.S) break;
    __syncthreads();
    fill_y1<DH>(d, qk0, w0, b, h, t0 - (d.k_ch - 1), TT + d.k_ch - 1, sm.y1s);
    __syncthreads();
    float acc[TPT];
    hat_tile<DH>(d, qk0, sm.ws, sm.y1s, b, h, t0, acc);
    if (d.flags & F_QK_NORM) {
      float ss[TPT];
#pragma unroll
      for (int n = 0; n < TPT; ++n) ss[n] = acc[n] * acc[n];
      reduce_channels<DH>(ss, sm.red);
#pragma unroll
      for (int n = 0; n < TPT; ++n) {
        const float sc = scale * rsqrtf(ss[n]);
        acc[n] *= sc;
        const int t = t0 + tg * TPT + n;
        if (o == 0 && t < d.S) rnorm[((long long)b * d.S + t) * (d.hq + d.hk) + h] = sc;
      }
    }
#pragma unroll
    for (int n = 0; n < TPT; ++n) sm.outs[(tg * TPT + n) * YLD + o] = acc[n];
    __syncthreads();
#pragma unroll
    for (int n = 0; n < TPT; ++n) {
      int tl = tg * TPT + n, t = t0 + tl;
      if (t >= d.S) continue;
      float val = acc[n];
      if (d.flags & F_ROPE) {
        constexpr int HALF = DH / 2;
        int c = o < HALF ? o : o - HALF;
        float2 cs = rope_tab[(long long)t * HALF + c];
        float other = sm.outs[tl * YLD + (o < HALF ? o + HALF : o - HALF)];
        val = o < HALF ? acc[n] * cs.x - other * cs.y : acc[n] * cs.x + other * cs.y;
      }
      long long row = (long long)b * d.S + t;
      if (h < d.hq) q[row * d.Lq + h * DH + o] = __float2bfloat16(val);
      else k[row * d.Lk + (h - d.hq) * DH + o] = __float2bfloat16(val);
    }
  }
}

// ------------------------------------------------------------------------------------------
// backward, part 1: RoPE adjoint, norm adjoint, d_temp.  In place on dq / dk (fp32).
// A group of d_h/8 lanes owns one (token, head); lane l of the group owns channels [4l, 4l+4) and their
// rotation partners [4l + d_h/2, ...), so every access is a 64- or 128-bit vector.
//   x = pre-norm latent, y = r x with r = sqrt(d_h)[beta]/|x| (kept by the forward), q = RoPE(y):
//   dy = RoPE^T(dq);  dx = r (dy - y (y . dy) / |y|^2),  |y|^2 = d_h [beta^2];  d_temp = sum y . dy.
// y is taken from the stored bf16 q / k (rotated back), r in fp32: the 1/|x| amplification is exact,
// the projection direction carries the bf16 rounding of q.
// ------------------------------------------------------------------------------------------
constexpr int BWD_NORM_TOK = 16;
template <int DH>
__global__ void __launch_bounds__(256) transform_bwd_norm_kernel(CcaDims d, const bf16* __restrict__ q,
                                                                 const bf16* __restrict__ k,
                                                                 const float* __restrict__ rnorm,
                                                                 const float* __restrict__ temp,
                                                                 const float2* __restrict__ rope_tab, float* dq,
                                                                 float* dk, float* d_temp) {
  constexpr int HALF = DH / 2, TPR = HALF / 4;     // lanes per row
  const int H = d.hq + d.hk;
  // a block walks BWD_NORM_TOK consecutive tokens; work item = (token, head, lane of the row), 32-bit arithmetic
  __shared__ float temp_acc[64];
  for (int i = threadIdx.x; i < d.hk && i < 64; i += blockDim.x) temp_acc[i] = 0.f;
  __syncthreads();
  const long long row0 = (long long)blockIdx.x * BWD_NORM_TOK;
  const long long n_rows = (long long)d.B * d.S;
  const int rows_here = (int)min((long long)BWD_NORM_TOK, n_rows - row0);
  const unsigned per_row = (unsigned)H * TPR, items = (unsigned)rows_here * per_row;
  const int t_first = (int)(row0 % d.S);
  for (unsigned it0 = 0; it0 < items; it0 += blockDim.x) {
  const unsigned item = it0 + threadIdx.x;
  const bool act = item < items;
  const unsigned ic = act ? item : 0u;
  const unsigned rl = ic / per_row, rem_i = ic - rl * per_row;
  const int h = (int)(rem_i / TPR);
  const int sub = (int)(rem_i % TPR);
  const long long row = row0 + rl;
  int t = t_first + (int)rl;
  if (t >= d.S) t -= d.S * (t / d.S);
  const bool is_q = h < d.hq;
  const int hj = is_q ? h : h - d.hq;
  float* g = (is_q ? dq + row * d.Lq : dk + row * d.Lk) + hj * DH + sub * 4;
  const bf16* y = (is_q ? q + row * d.Lq : k + row * d.Lk) + hj * DH + sub * 4;
  float ga[4], gb[4], ya[4], yb[4];
  {
    const float4 va = *reinterpret_cast<const float4*>(g), vb = *reinterpret_cast<const float4*>(g + HALF);
    ga[0] = va.x; ga[1] = va.y; ga[2] = va.z; ga[3] = va.w;
    gb[0] = vb.x; gb[1] = vb.y; gb[2] = vb.z; gb[3] = vb.w;
    const uint2 ua = *reinterpret_cast<const uint2*>(y), ub = *reinterpret_cast<const uint2*>(y + HALF);
    const __nv_bfloat162* pa = reinterpret_cast<const __nv_bfloat162*>(&ua);
    const __nv_bfloat162* pb = reinterpret_cast<const __nv_bfloat162*>(&ub);
    const float2 a0 = __bfloat1622float2(pa[0]), a1 = __bfloat1622float2(pa[1]);
    const float2 b0 = __bfloat1622float2(pb[0]), b1 = __bfloat1622float2(pb[1]);
    ya[0] = a0.x; ya[1] = a0.y; ya[2] = a1.x; ya[3] = a1.y;
    yb[0] = b0.x; yb[1] = b0.y; yb[2] = b1.x; yb[3] = b1.y;
  }
  if (d.flags & F_ROPE) {
    const float4* tab = reinterpret_cast<const float4*>(rope_tab + (long long)t * HALF + sub * 4);
    const float4 c01 = tab[0], c23 = tab[1];
    const float cs[4] = {c01.x, c01.z, c23.x, c23.z}, sn[4] = {c01.y, c01.w, c23.y, c23.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      // rotation by the negated angle
      const float a0 = ga[i] * cs[i] + gb[i] * sn[i], b0 = gb[i] * cs[i] - ga[i] * sn[i];
      ga[i] = a0; gb[i] = b0;
      const float a1 = ya[i] * cs[i] + yb[i] * sn[i], b1 = yb[i] * cs[i] - ya[i] * sn[i];
      ya[i] = a1; yb[i] = b1;
    }
  }
  if (d.flags & F_QK_NORM) {
    float dot = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) dot = fmaf(ya[i], ga[i], fmaf(yb[i], gb[i], dot));
#pragma unroll
    for (int off = TPR / 2; off > 0; off >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, off);
    const float beta = is_q ? 1.f : __expf(temp[hj]);
    const float r = rnorm[row * H + h];
    const float proj = dot / ((float)DH * beta * beta);
    if (act && !is_q && sub == 0) atomicAdd(&temp_acc[hj & 63], dot);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      ga[i] = r * (ga[i] - ya[i] * proj);
      gb[i] = r * (gb[i] - yb[i] * proj);
    }
  }
  if (act) {
    *reinterpret_cast<float4*>(g) = make_float4(ga[0], ga[1], ga[2], ga[3]);
    *reinterpret_cast<float4*>(g + HALF) = make_float4(gb[0], gb[1], gb[2], gb[3]);
  }
  }
  if (d.flags & F_QK_NORM) {
    __syncthreads();
    for (int i = threadIdx.x; i < d.hk && i < 64; i += blockDim.x) atomicAdd(d_temp + i, temp_acc[i]);
  }
}

// ------------------------------------------------------------------------------------------
// backward, part 2: q-k-mean adjoint, conv2 adjoint, conv1 adjoint -> gradient of the packed
// latent qk0 (bf16), and the gradient of the depth-wise taps.
// ------------------------------------------------------------------------------------------
CCA_DEVINL float dhat_at(const CcaDims& d, const float* dqh, const float* dkh, int b, int t, int h, int o) {
  if (t < 0 || t >= d.S) return 0.f;
  long long row = (long long)b * d.S + t;
  return h < d.hq ? dqh[row * d.Lq + h * d.dh + o] : dkh[row * d.Lk + (h - d.hq) * d.dh + o];
}

template <int DH>
__global__ void __launch_bounds__(256) transform_bwd_conv_kernel(CcaDims d, const float* __restrict__ qk0,
                                                                 const bf16* __restrict__ w0,
                                                                 const bf16* __restrict__ w1,
                                                                 const float* __restrict__ dqh,
                                                                 const float* __restrict__ dkh, bf16* __restrict__ dlat,
                                                                 long long ld_dlat, float* d_w0) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  Smem<DH> sm(smem_raw);
  constexpr int TPT = Lay<DH>::TPT, YLD = Lay<DH>::YLD, NG = Lay<DH>::NG;
  const int h = blockIdx.y, b = blockIdx.z;
  const int i = threadIdx.x % DH, tg = threadIdx.x / DH;   // this thread's channel (input side of conv2)
  const int ch = h * DH + i;
  const int kc = (d.flags & F_CONV2) ? d.k_ch : 1;
  const int ks = (d.flags & F_CONV1) ? d.k_seq : 1;
  if (d.flags & F_CONV2) stage_w1<DH, true>(d, w1, h, sm.ws);
  float w0r[MAXK];
  for (int j = 0; j < MAXK; ++j) w0r[j] = (j < d.k_seq) ? ldbf(w0 + ch * d.k_seq + j) : 0.f;
  float dw0[MAXK] = {0.f, 0.f, 0.f, 0.f};
  float* dy2s = sm.y1s;    // [TT + (kc-1) + (ks-1)][YLD]: dy2 at tokens t0 + r
  float* dy1s = sm.outs;   // [TT + (ks-1)][YLD]:          dy1 at tokens t0 + r
  for (int tile = 0; tile < TILES_PER_BLOCK; ++tile) {
    const int t0 = (blockIdx.x * TILES_PER_BLOCK + tile) * TT;
    if (t0 >= d.S) break;
    __syncthreads();
    const int rows2 = TT + (kc - 1) + (ks - 1), rows1 = TT + (ks - 1);
    for (int f = threadIdx.x; f < rows2 * DH; f += 256) {
      int r = f / DH, c = f - r * DH;
      dy2s[r * YLD + c] = dhat_at(d, dqh, dkh, b, t0 + r, h, c);
    }
    __syncthreads();
    // conv2 adjoint: dy1[t'][i] = sum_{o,j} w1[o][i][j] dy2[t' + (kc-1) - j][o]
    for (int r = tg; r < rows1; r += NG) {
      float a = 0.f;
      if (d.flags & F_CONV2) {
        for (int o = 0; o < DH; ++o)
          for (int j = 0; j < kc; ++j)
            a = fmaf(__bfloat162float(sm.ws[(o * kc + j) * Lay<DH>::WLD + i]), dy2s[(r + (kc - 1) - j) * YLD + o], a);
      } else {
        a = dy2s[r * YLD + i];
      }
      dy1s[r * YLD + i] = (t0 + r < d.S) ? a : 0.f;
    }
    __syncthreads();
    // conv1 adjoint + q-k-mean adjoint for this thread's tokens
#pragma unroll
    for (int n = 0; n < TPT; ++n) {
      int tl = tg * TPT + n, t = t0 + tl;
      if (t >= d.S) continue;
      float gq;
      if (d.flags & F_CONV1) {
        gq = 0.f;
        for (int j = 0; j < ks; ++j) gq = fmaf(w0r[j], dy1s[(tl + (ks - 1) - j) * YLD + i], gq);
        // taps' gradient: dw0[j] += dy1[t] * qk0[t - (ks-1) + j]
        float dy1_t = dy1s[tl * YLD + i];
        for (int j = 0; j < ks; ++j) {
          int ts = t - (ks - 1) + j;
          if (ts >= 0) dw0[j] = fmaf(dy1_t, qk0[((long long)b * d.S + ts) * d.L + ch], dw0[j]);
        }
      } else {
        gq = dy1s[tl * YLD + i];
      }
      if (d.flags & F_QK_MEAN) {
        if (h < d.hq) {
          gq += 0.5f * (dhat_at(d, dqh, dkh, b, t, h, i) + dhat_at(d, dqh, dkh, b, t, d.hq + h / d.g, i) / d.g);
        } else {
          int jk = h - d.hq;
          float s = dhat_at(d, dqh, dkh, b, t, h, i);
          for (int m = 0; m < d.g; ++m) s += dhat_at(d, dqh, dkh, b, t, jk * d.g + m, i);
          gq += 0.5f * s;
        }
      }
      dlat[((long long)b * d.S + t) * ld_dlat + ch] = __float2bfloat16(gq);
    }
  }
  if (d.flags & F_CONV1)
    for (int j = 0; j < d.k_seq; ++j) atomicAdd(d_w0 + ch * d.k_seq + j, dw0[j]);
}

// ------------------------------------------------------------------------------------------
// backward, part 3: gradient of the conv2 weights,
//   d_w1[h,o,i,j] = sum_{b,t} dy2[t,h,o] * y1[t-(k_ch-1)+j, h, i].
// Block = (token chunk, head, sequence); thread tile RO x RI outputs of the d_h x d_h block per tap.
// ------------------------------------------------------------------------------------------
template <int DH>
__global__ void __launch_bounds__(256) transform_bwd_w1_kernel(CcaDims d, const float* __restrict__ qk0,
                                                               const bf16* __restrict__ w0,
                                                               const float* __restrict__ dqh,
                                                               const float* __restrict__ dkh, float* d_w1,
                                                               int chunk_tokens) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  Smem<DH> sm(smem_raw);
  constexpr int YLD = Lay<DH>::YLD;
  constexpr int R = DH / 16;                // 16 x 16 threads, R x R outputs each
  const int h = blockIdx.y, b = blockIdx.z;
  const int to = threadIdx.x / 16, ti = threadIdx.x % 16;
  float* dy2s = sm.outs;   // [TT][YLD]
  float* y1s = sm.y1s;     // [TT + k_ch - 1][YLD], row r = token t0 - (k_ch-1) + r
  const int c_begin = blockIdx.x * chunk_tokens, c_end = min(d.S, c_begin + chunk_tokens);
  for (int j = 0; j < d.k_ch; ++j) {
    float acc[R][R];
#pragma unroll
    for (int a = 0; a < R; ++a)
#pragma unroll
      for (int c = 0; c < R; ++c) acc[a][c] = 0.f;
    for (int t0 = c_begin; t0 < c_end; t0 += TT) {
      __syncthreads();
      for (int f = threadIdx.x; f < TT * DH; f += 256) {
        int r = f / DH, c = f - r * DH;
        dy2s[r * YLD + c] = (t0 + r < c_end) ? dhat_at(d, dqh, dkh, b, t0 + r, h, c) : 0.f;
      }
      fill_y1<DH>(d, qk0, w0, b, h, t0 - (d.k_ch - 1), TT + d.k_ch - 1, y1s);
      __syncthreads();
      for (int r = 0; r < TT; ++r) {
        float dv[R], yv[R];
#pragma unroll
        for (int a = 0; a < R; ++a) dv[a] = dy2s[r * YLD + to + 16 * a];
#pragma unroll
        for (int c = 0; c < R; ++c) yv[c] = y1s[(r + j) * YLD + ti + 16 * c];
#pragma unroll
        for (int a = 0; a < R; ++a)
#pragma unroll
          for (int c = 0; c < R; ++c) acc[a][c] = fmaf(dv[a], yv[c], acc[a][c]);
      }
    }
#pragma unroll
    for (int a = 0; a < R; ++a)
#pragma unroll
      for (int c = 0; c < R; ++c) {
        int o = to + 16 * a, i = ti + 16 * c;
        atomicAdd(d_w1 + ((long long)(h * DH + o) * DH + i) * d.k_ch + j, acc[a][c]);
      }
  }
}

// conv1 adjoint + q-k-mean adjoint + gradient of the depth-wise taps, given dy1 = gradient w.r.t. conv1's output:
//   d_qk0[t][c]  = sum_j w0[c][j] dy1[t + (ks-1) - j][c]  +  (direct q-k-mean terms of d_hat)
//   d_w0[c][j]  += sum_t dy1[t][c] qk0[t - (ks-1) + j][c]
// One thread per channel (coalesced over channels), walking CONV1_TOK consecutive tokens with sliding windows.
constexpr int CONV1_TOK = 16;
template <int KS>
__global__ void __launch_bounds__(128) conv1_adjoint_kernel(CcaDims d, const float* __restrict__ dy1,
                                                            const float* __restrict__ dqh, const float* __restrict__ dkh,
                                                            const float* __restrict__ qk0, const bf16* __restrict__ w0,
                                                            bf16* __restrict__ dlat, long long ld, float* d_w0) {
  const int c = blockIdx.x * 128 + threadIdx.x;
  if (c >= d.L) return;
  const int b = blockIdx.z;
  const int t_begin = blockIdx.y * CONV1_TOK, t_end = min(d.S, t_begin + CONV1_TOK);
  const bool conv1 = (d.flags & F_CONV1) != 0;         // off: KS = 1 with unit weight
  float w[KS], dw[KS], win[KS], qwin[KS];
#pragma unroll
  for (int j = 0; j < KS; ++j) {
    w[j] = conv1 ? ldbf(w0 + c * KS + j) : 1.f;
    dw[j] = 0.f;
  }
  // every address is a pointer that advances by a row per token: no multiplications or divisions in the loop
  const long long row0 = (long long)b * d.S + t_begin;
  const float* pdy = dy1 + row0 * d.L + c;              // dy1 of token t_begin
  const float* pq0 = qk0 + row0 * d.L + c;              // qk0 of token t_begin
  bf16* pout = dlat + row0 * ld + c;
  // win[m] = dy1[t + m], qwin[m] = qk0[t - (KS-1) + m]
#pragma unroll
  for (int m = 0; m < KS; ++m) {
    win[m] = t_begin + m < d.S ? pdy[(long long)m * d.L] : 0.f;
    qwin[m] = t_begin - (KS - 1) + m >= 0 ? pq0[(long long)(m - (KS - 1)) * d.L] : 0.f;
  }
  // q-k-mean adjoint: a q channel takes half of its own d_hat and 1/(2g) of its kv head's; a k channel half of its
  // own and half of the sum over its g query heads
  const bool is_q = c < d.Lq;
  const int cj = is_q ? c : c - d.Lq, hh = cj / d.dh, o = cj - hh * d.dh;
  const bool mean = (d.flags & F_QK_MEAN) != 0;
  const float* pa = is_q ? dqh + row0 * d.Lq + c : dkh + row0 * d.Lk + cj;                       // own d_hat
  const float* pb = is_q ? dkh + row0 * d.Lk + (hh / d.g) * d.dh + o : dqh + row0 * d.Lq + (hh * d.g) * d.dh + o;
  const int sa = is_q ? d.Lq : d.Lk, sb = is_q ? d.Lk : d.Lq;                                   // row strides
  const int n_b = is_q ? 1 : d.g;
  const float scale_b = is_q ? 0.5f / (float)d.g : 0.5f;
  const int sL = d.L;
  constexpr int U = 4;                               // tokens per batch: all loads of a batch are issued together
  for (int tb = t_begin; tb < t_end; tb += U) {
    float ndy[U], nq[U], dir[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int t = tb + u;
      ndy[u] = t + KS < d.S ? pdy[(u + KS) * sL] : 0.f;
      nq[u] = t + 1 < d.S ? pq0[(u + 1) * sL] : 0.f;
      dir[u] = 0.f;
      if (mean && t < t_end) {
        float sbv = pb[u * sb];
        for (int m = 1; m < n_b; ++m) sbv += pb[u * sb + m * d.dh];
        dir[u] = 0.5f * pa[u * sa] + scale_b * sbv;
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int t = tb + u;
      if (t < t_end) {
        float gq = dir[u];
#pragma unroll
        for (int j = 0; j < KS; ++j) gq = fmaf(w[j], win[KS - 1 - j], gq);
#pragma unroll
        for (int j = 0; j < KS; ++j) dw[j] = fmaf(win[0], qwin[j], dw[j]);
        pout[(long long)u * ld] = __float2bfloat16(gq);
#pragma unroll
        for (int m = 0; m < KS - 1; ++m) {
          win[m] = win[m + 1];
          qwin[m] = qwin[m + 1];
        }
        win[KS - 1] = ndy[u];
        qwin[KS - 1] = nq[u];
      }
    }
    pdy += U * sL;
    pq0 += U * sL;
    pout += (long long)U * ld;
    pa += U * sa;
    pb += U * sb;
  }
  if (conv1)
#pragma unroll
    for (int j = 0; j < KS; ++j) atomicAdd(d_w0 + c * KS + j, dw[j]);
}

__global__ void rope_table_kernel(float2* tab, int S, int half, double log2_base) {
  long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (long long)S * half) return;
  int t = (int)(idx / half), c = (int)(idx % half);
  double theta = exp2(-(double)c / (double)half * log2_base);   // base^(-2c/d_h)
  double s, co;
  sincos((double)t * theta, &s, &co);
  tab[idx] = make_float2((float)co, (float)s);
}

// One thread per 4 consecutive value channels; a block covers PACK_ROWS tokens.
constexpr int PACK_ROWS = 8;
__global__ void __launch_bounds__(256) pack_dv_kernel(CcaDims d, const float* __restrict__ dv, bf16* __restrict__ dlat,
                                                      long long ld) {
  const int quads = d.Lk / 4;
  const long long row0 = (long long)blockIdx.x * PACK_ROWS, n_rows = (long long)d.B * d.S;
  const int rows_here = (int)min((long long)PACK_ROWS, n_rows - row0);
  const int t_first = (int)(row0 % d.S);
  for (int i = threadIdx.x; i < rows_here * quads; i += 256) {
    const int rl = i / quads, c = (i - rl * quads) * 4;
    const long long row = row0 + rl;
    int t = t_first + rl;
    if (t >= d.S) t -= d.S * (t / d.S);
    float4 v;
    if (c < d.Lk / 2 || !(d.flags & F_V_SHIFT)) v = *reinterpret_cast<const float4*>(dv + row * d.Lk + c);
    else v = (t + 1 < d.S) ? *reinterpret_cast<const float4*>(dv + (row + 1) * d.Lk + c) : make_float4(0.f, 0.f, 0.f, 0.f);
    __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
    uint2 pk;
    pk.x = *reinterpret_cast<uint32_t*>(&lo);
    pk.y = *reinterpret_cast<uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(dlat + row * ld + d.L + c) = pk;
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

cudaError_t launch_rope_table(float2* tab, int S, int dh, float base, cudaStream_t st) {
  long long n = (long long)S * (dh / 2);
  rope_table_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(tab, S, dh / 2, log2((double)base));
  return cudaGetLastError();
}

static dim3 tile_grid(const CcaDims& d) {
  return dim3((d.S + TT * TILES_PER_BLOCK - 1) / (TT * TILES_PER_BLOCK), d.hq + d.hk, d.B);
}

cudaError_t launch_transform_fwd(const CcaDims& d, const float* qk0, const bf16* w0, const bf16* w1, const float* temp,
                                 const float2* rope_tab, bf16* q, bf16* k, float* rnorm, cudaStream_t st) {
  DISPATCH_DH(d.dh, {
    cudaError_t e = set_smem(transform_fwd_kernel<DH>, smem_bytes<DH>());
    if (e != cudaSuccess) return e;
    transform_fwd_kernel<DH><<<tile_grid(d), 256, smem_bytes<DH>(), st>>>(d, qk0, w0, w1, temp, rope_tab, q, k, rnorm);
  });
  return cudaGetLastError();
}

cudaError_t launch_transform_bwd_norm(const CcaDims& d, const bf16* q, const bf16* k, const float* rnorm,
                                      const float* temp, const float2* rope_tab, float* dq, float* dk, float* d_temp,
                                      cudaStream_t st) {
  if (!(d.flags & (F_QK_NORM | F_ROPE))) return cudaSuccess;
  const long long blocks = ((long long)d.B * d.S + BWD_NORM_TOK - 1) / BWD_NORM_TOK;
  if (d.dh == 256) {
    transform_bwd_norm_kernel<256><<<(unsigned)blocks, 256, 0, st>>>(d, q, k, rnorm, temp, rope_tab, dq, dk, d_temp);
    return cudaGetLastError();
  }
  DISPATCH_DH(d.dh, {
    transform_bwd_norm_kernel<DH><<<(unsigned)blocks, 256, 0, st>>>(d, q, k, rnorm, temp, rope_tab, dq, dk, d_temp);
  });
  return cudaGetLastError();
}

cudaError_t launch_transform_bwd_conv(const CcaDims& d, const float* qk0, const bf16* w0, const bf16* w1,
                                      const float* dqh, const float* dkh, bf16* dlat, long long ld_dlat, float* d_w0,
                                      cudaStream_t st) {
  DISPATCH_DH(d.dh, {
    cudaError_t e = set_smem(transform_bwd_conv_kernel<DH>, smem_bytes<DH>());
    if (e != cudaSuccess) return e;
    transform_bwd_conv_kernel<DH><<<tile_grid(d), 256, smem_bytes<DH>(), st>>>(d, qk0, w0, w1, dqh, dkh, dlat, ld_dlat,
                                                                              d_w0);
  });
  return cudaGetLastError();
}

cudaError_t launch_transform_bwd_w1(const CcaDims& d, const float* qk0, const bf16* w0, const float* dqh,
                                    const float* dkh, float* d_w1, cudaStream_t st) {
  if (!(d.flags & F_CONV2)) return cudaSuccess;
  const int chunk = 512;
  dim3 grid((d.S + chunk - 1) / chunk, d.hq + d.hk, d.B);
  DISPATCH_DH(d.dh, {
    cudaError_t e = set_smem(transform_bwd_w1_kernel<DH>, smem_bytes<DH>());
    if (e != cudaSuccess) return e;
    transform_bwd_w1_kernel<DH><<<grid, 256, smem_bytes<DH>(), st>>>(d, qk0, w0, dqh, dkh, d_w1, chunk);
  });
  return cudaGetLastError();
}

cudaError_t launch_pack_dv(const CcaDims& d, const float* dv, bf16* dlat, long long ld_dlat, cudaStream_t st) {
  const long long blocks = ((long long)d.B * d.S + PACK_ROWS - 1) / PACK_ROWS;
  pack_dv_kernel<<<(unsigned)blocks, 256, 0, st>>>(d, dv, dlat, ld_dlat);
  return cudaGetLastError();
}

cudaError_t launch_conv1_adjoint(const CcaDims& d, const float* dy1, const float* dqh, const float* dkh, const float* qk0,
                                 const bf16* w0, bf16* dlat, long long ld_dlat, float* d_w0, cudaStream_t st) {
  dim3 grid((d.L + 127) / 128, (d.S + CONV1_TOK - 1) / CONV1_TOK, d.B);
  const int ks = (d.flags & F_CONV1) ? d.k_seq : 1;
  if (ks == 1) conv1_adjoint_kernel<1><<<grid, 128, 0, st>>>(d, dy1, dqh, dkh, qk0, w0, dlat, ld_dlat, d_w0);
  else if (ks == 2) conv1_adjoint_kernel<2><<<grid, 128, 0, st>>>(d, dy1, dqh, dkh, qk0, w0, dlat, ld_dlat, d_w0);
  else if (ks == 3) conv1_adjoint_kernel<3><<<grid, 128, 0, st>>>(d, dy1, dqh, dkh, qk0, w0, dlat, ld_dlat, d_w0);
  else conv1_adjoint_kernel<4><<<grid, 128, 0, st>>>(d, dy1, dqh, dkh, qk0, w0, dlat, ld_dlat, d_w0);
  return cudaGetLastError();
}
