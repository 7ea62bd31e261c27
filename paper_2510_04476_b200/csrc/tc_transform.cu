// Tensor-core kernels, part 3: the latent transforms of Eq. 8, 9 and 11 on q and k, forward.
// One CTA = (128 tokens, one head, one sequence).
//   1. all threads: conv1_seq (depth-wise, fp32) of the head's channels from the fp32 latent qk0, written as
//      bf16 into k_ch row-shifted copies A_j[rho] = y1[t0 + rho - (k_ch-1) + j] in the 128-byte-swizzled
//      K-major layout the tensor core reads; the head's conv2 weights as B_j[o][i] = w1[o][i][j] likewise;
//   2. one thread: y2 = sum_j A_j B_j^T as tcgen05.mma into TMEM (128 tokens x d_h, K = d_h * k_ch);
//   3. threads 0..127, one token each (= one TMEM lane): q-k-mean, L2 norm * sqrt(d_h) (* exp(temp)),
//      RoPE, bf16 store.  The norm and the rotation pairs are local to the thread.
#include "tc_kernels.cuh"
#include "tc_ptx.cuh"
#include "tc_state.cuh"

using namespace tc;

namespace {

constexpr int TR_THREADS = 256;
enum : unsigned { F_CONV1 = 1, F_CONV2 = 2, F_QK_MEAN = 4, F_QK_NORM = 16, F_ROPE = 32 };

// byte offset of element (row, col) inside a K-major operand tile [128][DH] stored as DH/64 boxes of
// [128 rows][64 bf16] with the 128-byte swizzle (16-byte chunk index XOR row mod 8)
TC_DEVINL uint32_t sw_off(int row, int col) {
  return (uint32_t)((col >> 6) * 16384 + row * 128 + ((((col & 63) >> 3) ^ (row & 7)) << 4) + (col & 7) * 2);
}

template <int DH, int KC>
struct TrSmem {
  static constexpr int TILE = 128 * DH * 2;      // bytes of one A tile
  static constexpr int BT = DH * DH * 2;         // bytes of one B tile ([DH rows][DH])
  static constexpr int A_OFF = 0;
  static constexpr int B_OFF = KC * TILE;
  static constexpr int BAR_OFF = B_OFF + KC * (DH == 128 ? BT : 16384);
  static constexpr int TOTAL = BAR_OFF + 64 + 1024;
};

template <int DH, int KC>
__global__ void __launch_bounds__(TR_THREADS, 1)
tc_transform_fwd_kernel(CcaDims d, const float* __restrict__ qk0, const bf16* __restrict__ w0,
                        const bf16* __restrict__ w1, const float* __restrict__ temp,
                        const float2* __restrict__ rope_tab, bf16* __restrict__ q, bf16* __restrict__ k, int* status) {
  using SM = TrSmem<DH, KC>;
  constexpr int BTILE = (DH == 128 ? SM::BT : 16384);     // B tile stride (a 64-row tile still spans a 16 KB box)
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
  uint64_t* mma_bar = reinterpret_cast<uint64_t*>(smem + SM::BAR_OFF);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(mma_bar + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int t0 = blockIdx.x * 128, h = blockIdx.y, b = blockIdx.z;
  const long long seq_base = (long long)b * d.S;

  if (threadIdx.x == 0) {
    mbar_init(mma_bar, 1);
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, DH);
    tmem_relinquish();
  }

  // ---- stage B_j[o][i] = w1[h*DH + o][i][j] ------------------------------------------------
  {
    const bf16* wsrc = w1 + (size_t)h * DH * DH * KC;
    for (int f = threadIdx.x; f < DH * (DH / 8); f += TR_THREADS) {
      const int o = f / (DH / 8), i0 = (f % (DH / 8)) * 8;
      __align__(16) bf16 buf[8 * KC];
      const uint4* src = reinterpret_cast<const uint4*>(wsrc + ((size_t)o * DH + i0) * KC);
#pragma unroll
      for (int v = 0; v < KC; ++v) reinterpret_cast<uint4*>(buf)[v] = src[v];
#pragma unroll
      for (int j = 0; j < KC; ++j) {
        __align__(16) bf16 outv[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) outv[e] = buf[e * KC + j];
        *reinterpret_cast<uint4*>(smem + SM::B_OFF + j * BTILE + sw_off(o, i0)) = *reinterpret_cast<uint4*>(outv);
      }
    }
  }
  // ---- stage A_j: conv1 of the head's channels, rows r = 0 .. 127 + KC-1, token tau = t0 - (KC-1) + r ----
  {
    constexpr int CG = DH / 4;                 // channel quads per row
    constexpr int RG = TR_THREADS / CG;        // row groups
    constexpr int ROWS = 128 + KC - 1;
    constexpr int RPT = (ROWS + RG - 1) / RG;
    const int cq = (threadIdx.x % CG) * 4, rg = threadIdx.x / CG;
    const int ch = h * DH + cq;
    const int ks = (d.flags & F_CONV1) ? d.k_seq : 1;
    // 4-slot window ending at the current token: slot 3 = current, slot 2 = previous, ...; tap j of the
    // k_seq taps sits in slot 4 - k_seq + j, unused leading slots carry weight 0.
    float wt[4][4];                            // [channel][slot]
#pragma unroll
    for (int c = 0; c < 4; ++c)
#pragma unroll
      for (int sl = 0; sl < 4; ++sl) {
        const int j = sl - (4 - ks);
        wt[c][sl] = (j < 0) ? 0.f : ((d.flags & F_CONV1) ? __bfloat162float(w0[(ch + c) * d.k_seq + j]) : 1.f);
      }
    const float* col = qk0 + seq_base * d.L + ch;
    auto load = [&](int tau) -> float4 {
      if (tau < 0 || tau >= d.S) return make_float4(0.f, 0.f, 0.f, 0.f);
      return *reinterpret_cast<const float4*>(col + (long long)tau * d.L);
    };
    const int r_begin = rg * RPT, r_end = min(ROWS, r_begin + RPT);
    float4 win[4];
    const int tau0 = t0 - (KC - 1) + r_begin;
#pragma unroll
    for (int sl = 0; sl < 3; ++sl) win[sl] = (sl >= 4 - ks) ? load(tau0 - 3 + sl) : make_float4(0.f, 0.f, 0.f, 0.f);
    for (int r = r_begin; r < r_end; ++r) {
      const int tau = t0 - (KC - 1) + r;
      win[3] = load(tau);
      float y[4] = {0.f, 0.f, 0.f, 0.f};
      if (tau >= 0) {
#pragma unroll
        for (int sl = 0; sl < 4; ++sl) {
          y[0] = fmaf(wt[0][sl], win[sl].x, y[0]);
          y[1] = fmaf(wt[1][sl], win[sl].y, y[1]);
          y[2] = fmaf(wt[2][sl], win[sl].z, y[2]);
          y[3] = fmaf(wt[3][sl], win[sl].w, y[3]);
        }
      }
      uint2 packed;
      packed.x = pack_bf16(y[0], y[1]);
      packed.y = pack_bf16(y[2], y[3]);
#pragma unroll
      for (int j = 0; j < KC; ++j) {
        const int rho = r - j;
        if (rho >= 0 && rho < 128) *reinterpret_cast<uint2*>(smem + SM::A_OFF + j * SM::TILE + sw_off(rho, cq)) = packed;
      }
#pragma unroll
      for (int j = 0; j < 3; ++j) win[j] = win[j + 1];
    }
  }
  fence_proxy_async();          // generic-proxy smem writes -> visible to the tensor core
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (threadIdx.x == 32) {      // lane 0 of warp 1 issues the MMAs
    const uint32_t idesc = idesc_bf16(DH, 0, 0);
    const uint32_t a_addr = smem_u32(smem + SM::A_OFF), b_addr = smem_u32(smem + SM::B_OFF);
#pragma unroll
    for (int j = 0; j < KC; ++j)
#pragma unroll
      for (int kk = 0; kk < DH / 16; ++kk) {
        const uint32_t off = (kk >> 2) * 16384 + (kk & 3) * 32;
        mma_ss(tmem_base, smem_desc_sw128(a_addr + j * SM::TILE + off, 16, 1024),
               smem_desc_sw128(b_addr + j * BTILE + off, 16, 1024), idesc, (j | kk) != 0);
      }
    mma_commit(mma_bar);
  }

  if (warp < 4) {
    const int rho = threadIdx.x, t = t0 + rho;
    const bool valid = t < d.S;
    const bool is_q = h < d.hq;
    const int hj = is_q ? h / d.g : h - d.hq;
    const float* row = qk0 + (seq_base + (valid ? t : 0)) * d.L;
    if (!mbar_wait(mma_bar, 0, abort_flag)) {
      *abort_flag = 1;
      atomicCAS(status, 0, ST_TIMEOUT_EPI);
    } else {
      tc_fence_after();
      float v[DH];
#pragma unroll
      for (int c = 0; c < DH / 32; ++c) {
        uint32_t r[32];
        tmem_ld32(tmem_base + ((uint32_t)(warp * 32) << 16) + c * 32, r);
        tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 32; ++i) v[c * 32 + i] = __uint_as_float(r[i]);
      }
      if (valid) {
        if (d.flags & F_QK_MEAN) {
          const float4* own = reinterpret_cast<const float4*>(row + h * DH);
          if (is_q) {
            const float4* kk4 = reinterpret_cast<const float4*>(row + d.Lq + hj * DH);
#pragma unroll
            for (int c = 0; c < DH / 4; ++c) {
              const float4 a = own[c], bb = kk4[c];
              v[4 * c + 0] += 0.5f * (a.x + bb.x);
              v[4 * c + 1] += 0.5f * (a.y + bb.y);
              v[4 * c + 2] += 0.5f * (a.z + bb.z);
              v[4 * c + 3] += 0.5f * (a.w + bb.w);
            }
          } else {
            const float hg = 0.5f / (float)d.g;
#pragma unroll
            for (int c = 0; c < DH / 4; ++c) {
              const float4 a = own[c];
              v[4 * c + 0] += 0.5f * a.x;
              v[4 * c + 1] += 0.5f * a.y;
              v[4 * c + 2] += 0.5f * a.z;
              v[4 * c + 3] += 0.5f * a.w;
            }
            for (int m = 0; m < d.g; ++m) {
              const float4* q4 = reinterpret_cast<const float4*>(row + (hj * d.g + m) * DH);
#pragma unroll
              for (int c = 0; c < DH / 4; ++c) {
                const float4 a = q4[c];
                v[4 * c + 0] = fmaf(hg, a.x, v[4 * c + 0]);
                v[4 * c + 1] = fmaf(hg, a.y, v[4 * c + 1]);
                v[4 * c + 2] = fmaf(hg, a.z, v[4 * c + 2]);
                v[4 * c + 3] = fmaf(hg, a.w, v[4 * c + 3]);
              }
            }
          }
        }
        if (d.flags & F_QK_NORM) {
          float ss = 0.f;
#pragma unroll
          for (int c = 0; c < DH; ++c) ss = fmaf(v[c], v[c], ss);
          const float sc = sqrtf((float)DH) * (is_q ? 1.f : __expf(temp[hj])) * rsqrtf(ss);
#pragma unroll
          for (int c = 0; c < DH; ++c) v[c] *= sc;
        }
        if (d.flags & F_ROPE) {
          const float4* tab = reinterpret_cast<const float4*>(rope_tab + (long long)t * (DH / 2));
#pragma unroll
          for (int c = 0; c < DH / 4; ++c) {
            const float4 cs = tab[c];                       // (cos, sin) of channels 2c and 2c+1
            const float a0 = v[2 * c], b0 = v[2 * c + DH / 2];
            const float a1 = v[2 * c + 1], b1 = v[2 * c + 1 + DH / 2];
            v[2 * c] = a0 * cs.x - b0 * cs.y;
            v[2 * c + DH / 2] = b0 * cs.x + a0 * cs.y;
            v[2 * c + 1] = a1 * cs.z - b1 * cs.w;
            v[2 * c + 1 + DH / 2] = b1 * cs.z + a1 * cs.w;
          }
        }
        bf16* dst = is_q ? q + (seq_base + t) * d.Lq + h * DH : k + (seq_base + t) * d.Lk + hj * DH;
#pragma unroll
        for (int c = 0; c < DH / 8; ++c) {
          uint4 w;
          w.x = pack_bf16(v[8 * c + 0], v[8 * c + 1]);
          w.y = pack_bf16(v[8 * c + 2], v[8 * c + 3]);
          w.z = pack_bf16(v[8 * c + 4], v[8 * c + 5]);
          w.w = pack_bf16(v[8 * c + 6], v[8 * c + 7]);
          reinterpret_cast<uint4*>(dst)[c] = w;
        }
      }
    }
  }
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    const long long c0 = clock64();
    while (clock64() - c0 < 2000000) {}
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, DH);
  }
}

template <int DH, int KC>
int launch_tr(const CcaDims& d, const float* qk0, const bf16* w0, const bf16* w1, const float* temp,
              const float2* rope, bf16* q, bf16* k, int* status, cudaStream_t st) {
  static bool attr_done = false;
  using SM = TrSmem<DH, KC>;
  if (!attr_done) {
    cudaError_t e = cudaFuncSetAttribute(tc_transform_fwd_kernel<DH, KC>, cudaFuncAttributeMaxDynamicSharedMemorySize, SM::TOTAL);
    if (e != cudaSuccess) return -(int)e;
    attr_done = true;
  }
  dim3 grid((d.S + 127) / 128, d.hq + d.hk, d.B);
  tc_transform_fwd_kernel<DH, KC><<<grid, TR_THREADS, SM::TOTAL, st>>>(d, qk0, w0, w1, temp, rope, q, k, status);
  cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? 0 : -(int)e;
}

}  // namespace

int tc_transform_fwd(TcState* s, const CcaDims& d, const float* qk0, const bf16* w0, const bf16* w1,
                     const float* temp, const float2* rope, bf16* q, bf16* k, int* d_status, cudaStream_t st) {
  if (!s) return 1;
  if (!(d.flags & F_CONV2)) return 1;                 // no contraction to run: the SIMT kernel is the right tool
  if (d.L % 4 || d.Lq % 8 || d.Lk % 8) return 1;
  if ((reinterpret_cast<uintptr_t>(w1) & 15) || (reinterpret_cast<uintptr_t>(qk0) & 15)) return 1;
  if (d.dh == 128) {
    if (d.k_ch == 1) return launch_tr<128, 1>(d, qk0, w0, w1, temp, rope, q, k, d_status, st);
    if (d.k_ch == 2) return launch_tr<128, 2>(d, qk0, w0, w1, temp, rope, q, k, d_status, st);
    return 1;
  }
  if (d.dh == 64) {
    if (d.k_ch == 1) return launch_tr<64, 1>(d, qk0, w0, w1, temp, rope, q, k, d_status, st);
    if (d.k_ch == 2) return launch_tr<64, 2>(d, qk0, w0, w1, temp, rope, q, k, d_status, st);
    if (d.k_ch == 3) return launch_tr<64, 3>(d, qk0, w0, w1, temp, rope, q, k, d_status, st);
    if (d.k_ch == 4) return launch_tr<64, 4>(d, qk0, w0, w1, temp, rope, q, k, d_status, st);
  }
  return 1;
}
