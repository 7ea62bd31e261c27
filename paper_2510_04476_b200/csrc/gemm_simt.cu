// Plain SIMT GEMM (fp32 FMA, bf16 operands): the always-available contraction of the library.
// C[M,N] = sum_k A(m,k) B(n,k).  Either operand may be contiguous along k or along its row index.
// 128x128x16 tiles, 256 threads, 8x8 outputs per thread.
#include "common.cuh"

namespace {

constexpr int BM = 128, BN = 128, BK = 16, PADM = 4;

// Loads one 128(rows) x 16(k) tile of a strided operand into smem as [k][row] fp32.
// row_off / seq_len implement the sequence-local row shift (see GemmArgs).
template <bool kShift>
CCA_DEVINL void load_tile(const GemmOperand& op, int rows_total, int K, int row0, int k0,
                          float (*dst)[BM + PADM], int tid, int row_off, int seq_len) {
  if (op.cs == 1) {
    // contiguous along k: thread -> (row = tid/2, 8 consecutive k)
    int r = tid >> 1, kk = (tid & 1) * 8;
    int row = row0 + r;
    bool row_ok = row < rows_total;
    long long src_row = row;
    if (kShift && row_ok) {
      int t = row % seq_len + row_off;
      row_ok = (t >= 0) && (t < seq_len);
      src_row = (long long)row + row_off;
    }
    const bf16* p = op.p + src_row * op.rs + (k0 + kk);
    if (row_ok && k0 + kk + 8 <= K && ((reinterpret_cast<uintptr_t>(p) & 15) == 0)) {
      uint4 v = *reinterpret_cast<const uint4*>(p);
      const bf16* e = reinterpret_cast<const bf16*>(&v);
#pragma unroll
      for (int i = 0; i < 8; ++i) dst[kk + i][r] = __bfloat162float(e[i]);
    } else {
#pragma unroll
      for (int i = 0; i < 8; ++i)
        dst[kk + i][r] = (row_ok && k0 + kk + i < K) ? __bfloat162float(p[i]) : 0.f;
    }
  } else {
    // contiguous along the row index: thread -> (k = tid/16, 8 consecutive rows)
    int kk = tid >> 4, r = (tid & 15) * 8;
    int k = k0 + kk;
    const bf16* p = op.p + (long long)k * op.cs + (long long)(row0 + r) * op.rs;
    if (!kShift && k < K && row0 + r + 8 <= rows_total && op.rs == 1 &&
        ((reinterpret_cast<uintptr_t>(p) & 15) == 0)) {
      uint4 v = *reinterpret_cast<const uint4*>(p);
      const bf16* e = reinterpret_cast<const bf16*>(&v);
#pragma unroll
      for (int i = 0; i < 8; ++i) dst[kk][r + i] = __bfloat162float(e[i]);
    } else {
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        int row = row0 + r + i;
        bool ok = (k < K) && (row < rows_total);
        long long src_row = row;
        if (kShift && ok) {
          int t = row % seq_len + row_off;
          ok = (t >= 0) && (t < seq_len);
          src_row = (long long)row + row_off;
        }
        dst[kk][r + i] = ok ? __bfloat162float(op.p[(long long)k * op.cs + src_row * op.rs]) : 0.f;
      }
    }
  }
}

template <bool kShift>
__global__ void __launch_bounds__(256) gemm_simt_kernel(GemmArgs g) {
  __shared__ float As[BK][BM + PADM];
  __shared__ float Bs[BK][BN + PADM];
  const int tid = threadIdx.x;
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  const int ty = tid >> 4, tx = tid & 15;
  float acc[8][8];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;

  for (int k0 = 0; k0 < g.K; k0 += BK) {
    load_tile<kShift>(g.A, g.M, g.K, m0, k0, As, tid, g.a_row_off, g.seq_len);
    load_tile<false>(g.B, g.N, g.K, n0, k0, Bs, tid, 0, 1);
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      float a[8], b[8];
      *reinterpret_cast<float4*>(&a[0]) = *reinterpret_cast<const float4*>(&As[kk][ty * 4]);
      *reinterpret_cast<float4*>(&a[4]) = *reinterpret_cast<const float4*>(&As[kk][64 + ty * 4]);
      *reinterpret_cast<float4*>(&b[0]) = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4]);
      *reinterpret_cast<float4*>(&b[4]) = *reinterpret_cast<const float4*>(&Bs[kk][64 + tx * 4]);
#pragma unroll
      for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    int m = m0 + (i < 4 ? ty * 4 + i : 64 + ty * 4 + (i - 4));
    if (m >= g.M) continue;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      int n = n0 + (j < 4 ? tx * 4 + j : 64 + tx * 4 + (j - 4));
      if (n >= g.N) continue;
      long long idx = (long long)m * g.ldc + n;
      if (g.out_bf16) g.out_bf16[idx] = __float2bfloat16(acc[i][j]);
      else if (g.accumulate) atomicAdd(g.out_f32 + idx, acc[i][j]);
      else g.out_f32[idx] = acc[i][j];
    }
  }
}

}  // namespace

cudaError_t launch_gemm_simt(const GemmArgs& g, cudaStream_t st) {
  if (g.M <= 0 || g.N <= 0) return cudaSuccess;
  dim3 grid((g.N + BN - 1) / BN, (g.M + BM - 1) / BM);
  if (g.a_row_off != 0) gemm_simt_kernel<true><<<grid, 256, 0, st>>>(g);
  else gemm_simt_kernel<false><<<grid, 256, 0, st>>>(g);
  return cudaGetLastError();
}
