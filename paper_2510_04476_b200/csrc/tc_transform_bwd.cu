// Tensor-core kernels, part 5: adjoint of conv2_seq+ch (Eq. 8) of the latent transforms.
//
// Given d_hat = gradient w.r.t. the pre-norm latents (fp32, per head) and the fp32 latent qk0:
//     d_y1[t][i]     = sum_j sum_o d_hat[t + (k_ch-1) - j][o] * w1[o][i][j]        (gradient w.r.t. conv1's output)
//     d_w1[o][i][j] += sum_t d_hat[t][o] * y1[t - (k_ch-1) + j][i]                  (gradient of the conv2 weights)
// Work unit = (one head, one sequence, 128 consecutive tokens); a persistent CTA walks a contiguous range
// of units, head-major, like the forward kernel:
//
//   warps 4-11 producers: recompute y1 = conv1_seq(qk0) for the unit (fp32 -> bf16, k_ch row-shifted tiles
//              Y_j[rho] = y1[t0 + rho - (k_ch-1) + j]) and convert d_hat into the k_ch row-shifted tiles
//              G_j[rho] = d_hat[t0 + rho + (k_ch-1) - j], all in the 128-byte-swizzled layout; stage the head's
//              weights as W_j[o][i] = w1[o][i][j].  The first producer thread then issues
//                  d_y1 tile  = sum_j G_j W_j              (128 tokens x d_h, K = d_h * k_ch)
//                  D_j       += Y_j^T G_{k_ch-1}           (d_h x d_h per tap, K = the unit's 128 tokens)
//              with every operand read through the descriptor form that matches how it lies in shared memory.
//   warps 0-3  epilogue: d_y1 rows (thread = token) to global fp32; after the last unit of a head the weight
//              gradient accumulators (thread = input channel i) are added to d_w1 with atomics.
//
// For d_h = 64 two taps share one accumulator (M = 128 = two stacked taps x 64 channels).
#include "tc_kernels.cuh"
#include "tc_ptx.cuh"
#include "tc_state.cuh"

using namespace tc;

namespace {

constexpr int TB_PRODUCERS = 256;
constexpr int TB_THREADS = 128 + TB_PRODUCERS;
constexpr int TB_ALLOC_WARP = 4;
enum : unsigned { F_CONV1 = 1, F_CONV2 = 2 };

TC_DEVINL uint32_t sw_off(int row, int col, int box_bytes) {
  return (uint32_t)((col >> 6) * box_bytes + row * 128 + ((((col & 63) >> 3) ^ (row & 7)) << 4) + (col & 7) * 2);
}

template <int DH, int KC>
struct TbSmem {
  static constexpr int TILE = 128 * DH * 2;      // one [128 tokens][DH] operand tile
  static constexpr int BT = DH * DH * 2;         // one [DH][DH] weight tile
  static constexpr int Y_OFF = 0;
  static constexpr int G_OFF = KC * TILE;
  static constexpr int W_OFF = 2 * KC * TILE;
  static constexpr int BAR_OFF = W_OFF + KC * BT;
  static constexpr int STG_OFF = BAR_OFF + 128;      // four epilogue warps x 4 KB: row blocks on their way to memory
  static constexpr int TOTAL = STG_OFF + 4 * 4096 + 1024;
  static_assert(TOTAL <= 232448, "shared memory");
  static constexpr int NGRP = DH == 128 ? KC : (KC + 1) / 2;          // weight-gradient accumulators
  static constexpr int GRP_COLS = DH == 128 ? 128 : 64;
  static constexpr int DW_COL = 2 * DH;                               // after the two d_y1 buffers
  static constexpr int TMEM_COLS = (DW_COL + NGRP * GRP_COLS) <= 256 ? 256 : 512;
};

struct TbParams {
  CcaDims d;
  const float* qk0;
  const bf16* w0;
  const bf16* w1;
  const float* dqh;     // d_hat of the q heads [T, Lq]
  const float* dkh;     // d_hat of the kv heads [T, Lk]
  float* dy1;           // [T, L] gradient w.r.t. conv1's output
  float* d_w1;          // [L, d_h, k_ch], accumulated
  int* status;
  int n_tiles, units_per_head, total_units;
};

TC_DEVINL void fail(volatile int* abort_flag, int* status, int code) {
  *abort_flag = 1;
  atomicCAS(status, 0, code);
}

template <int DH, int KC>
__global__ void __launch_bounds__(TB_THREADS, 1) tc_transform_bwd_kernel(const TbParams p) {
  using SM = TbSmem<DH, KC>;
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = smem_align1024(smem_dyn);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + SM::BAR_OFF);
  uint64_t* a_full = bars;           // producers -> MMA   (256 arrivals)
  uint64_t* a_empty = bars + 1;      // MMA -> producers   (commit)
  uint64_t* acc_full = bars + 2;     // [2] MMA -> epilogue (commit)
  uint64_t* acc_empty = bars + 4;    // [2] epilogue -> MMA (128 arrivals)
  uint64_t* dw_free = bars + 6;      // epilogue -> MMA: weight-gradient accumulators flushed (128 arrivals)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 7);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const CcaDims& d = p.d;
  const int warp = threadIdx.x >> 5;

  const int u_begin = (int)((long long)p.total_units * blockIdx.x / gridDim.x);
  const int u_end = (int)((long long)p.total_units * (blockIdx.x + 1) / gridDim.x);

  if (threadIdx.x == 0) {
    mbar_init(a_full, TB_PRODUCERS);
    mbar_init(a_empty, 1);
    for (int s = 0; s < 2; ++s) {
      mbar_init(&acc_full[s], 1);
      mbar_init(&acc_empty[s], 128);
    }
    mbar_init(dw_free, 128);
    wait_ctl_init(abort_flag, p.status);
    fence_barrier_init();
  }
  if (warp == TB_ALLOC_WARP) {
    tmem_alloc(tmem_slot, SM::TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp >= 4) {
    // ------------------------------------------------------------------ producers
    const int pt = threadIdx.x - 128;
    constexpr int CG = DH / 4;                   // channel quads per row
    constexpr int RG = TB_PRODUCERS / CG;        // row groups
    constexpr int RPG = 128 / RG;                // tile rows per thread
    constexpr int NR = RPG + KC - 1;             // rows of y1 (and of d_hat) a thread handles
    const int cq = (pt % CG) * 4, rg = pt / CG;
    const int ks = (d.flags & F_CONV1) ? d.k_seq : 1;
    int staged_head = -1, flushes = 0;
    int it = 0;
    for (int u = u_begin; u < u_end; ++u, ++it) {
      const int h = u / p.units_per_head, rem = u % p.units_per_head;
      const int b = rem / p.n_tiles, t0 = (rem % p.n_tiles) * 128;
      const bool is_q = h < d.hq;
      const int ch = h * DH + cq;
      const float* col = p.qk0 + (long long)b * d.S * d.L + ch;
      const float* gcol = is_q ? p.dqh + (long long)b * d.S * d.Lq + ch
                               : p.dkh + (long long)b * d.S * d.Lk + (ch - d.Lq);
      const long long gld = is_q ? d.Lq : d.Lk;
      auto load = [&](int tau) -> float4 {
        if (tau < 0 || tau >= d.S) return make_float4(0.f, 0.f, 0.f, 0.f);
        return *reinterpret_cast<const float4*>(col + (long long)tau * d.L);
      };
      auto gload = [&](int tau) -> float4 {
        if (tau >= d.S) return make_float4(0.f, 0.f, 0.f, 0.f);
        return *reinterpret_cast<const float4*>(gcol + (long long)tau * gld);
      };
      // conv1 taps in a 4-slot window ending at the current token (see the forward kernel)
      float wt[4][4];
#pragma unroll
      for (int c = 0; c < 4; ++c)
#pragma unroll
        for (int sl = 0; sl < 4; ++sl) {
          const int j = sl - (4 - ks);
          wt[c][sl] = (j < 0) ? 0.f : ((d.flags & F_CONV1) ? __bfloat162float(p.w0[(ch + c) * d.k_seq + j]) : 1.f);
        }
      // rows: y1 at x in [rg*RPG - (KC-1), (rg+1)*RPG), d_hat at x in [rg*RPG, (rg+1)*RPG + KC-1)
      const int xy = rg * RPG - (KC - 1), xg = rg * RPG;
      float4 win[4];
#pragma unroll
      for (int sl = 0; sl < 3; ++sl) win[sl] = (sl >= 4 - ks) ? load(t0 + xy - 3 + sl) : make_float4(0.f, 0.f, 0.f, 0.f);
      bool waited = false;
      constexpr int CHN = 8;
#pragma unroll 1
      for (int r0 = 0; r0 < NR; r0 += CHN) {
        float4 raw[CHN], gr[CHN];
#pragma unroll
        for (int i = 0; i < CHN; ++i) {
          raw[i] = (r0 + i < NR) ? load(t0 + xy + r0 + i) : make_float4(0.f, 0.f, 0.f, 0.f);
          gr[i] = (r0 + i < NR) ? gload(t0 + xg + r0 + i) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
        if (!waited) {
          // the loads above are in flight while the previous unit's MMAs finish reading the operand tiles
          if (!mbar_wait(a_empty, (it & 1) ^ 1, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_TMA); goto done; }
          waited = true;
          if (h != staged_head) {
            // W_j[o][i] = w1[h*DH + o][i][j]
            const bf16* wsrc = p.w1 + (size_t)h * DH * DH * KC;
            for (int f = pt; f < DH * (DH / 8); f += TB_PRODUCERS) {
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
                *reinterpret_cast<uint4*>(smem + SM::W_OFF + j * SM::BT + sw_off(o, i0, DH * 128)) =
                    *reinterpret_cast<uint4*>(outv);
              }
            }
          }
        }
#pragma unroll
        for (int i = 0; i < CHN; ++i) {
          if (r0 + i < NR) {
            // y1 at x = xy + r0 + i
            const int x = xy + r0 + i, tau = t0 + x;
            win[3] = raw[i];
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
              const int rho = x + (KC - 1) - j;
              if (rho >= rg * RPG && rho < (rg + 1) * RPG)
                *reinterpret_cast<uint2*>(smem + SM::Y_OFF + j * SM::TILE + sw_off(rho, cq, 16384)) = packed;
            }
#pragma unroll
            for (int j = 0; j < 3; ++j) win[j] = win[j + 1];
            // d_hat at x = xg + r0 + i
            const int x2 = xg + r0 + i;
            uint2 gp;
            gp.x = pack_bf16(gr[i].x, gr[i].y);
            gp.y = pack_bf16(gr[i].z, gr[i].w);
#pragma unroll
            for (int j = 0; j < KC; ++j) {
              const int rho = x2 - (KC - 1) + j;
              if (rho >= rg * RPG && rho < (rg + 1) * RPG)
                *reinterpret_cast<uint2*>(smem + SM::G_OFF + j * SM::TILE + sw_off(rho, cq, 16384)) = gp;
            }
          }
        }
      }
      fence_proxy_async();          // generic-proxy smem writes -> visible to the tensor core
      mbar_arrive(a_full);
      const bool first_of_head = h != staged_head;
      if (pt == 0) {
        // ---------------------------------------------------------------- MMA issue (one thread)
        const int buf = it & 1;
        if (!mbar_wait(&acc_empty[buf], ((it >> 1) & 1) ^ 1, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
        if (!mbar_wait(a_full, it & 1, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
        if (first_of_head && staged_head >= 0) {
          // the accumulators of the previous head must have been read out
          if (!mbar_wait(dw_free, flushes & 1, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
        }
        tc_fence_after();
        const uint32_t y_addr = smem_u32(smem + SM::Y_OFF), g_addr = smem_u32(smem + SM::G_OFF),
                       w_addr = smem_u32(smem + SM::W_OFF);
        // d_y1 = sum_j G_j W_j : A = G_j (K-major, K = o), B = W_j stored [o][i] read with N = i contiguous
        {
          const uint32_t idesc = idesc_bf16(DH, 0, 1);
#pragma unroll
          for (int j = 0; j < KC; ++j)
#pragma unroll
            for (int kk = 0; kk < DH / 16; ++kk) {
              const uint32_t off_a = (kk >> 2) * 16384 + (kk & 3) * 32;
              mma_ss(tmem_base + buf * DH, smem_desc_sw128(g_addr + j * SM::TILE + off_a, 16, 1024),
                     smem_desc_sw128(w_addr + j * SM::BT + kk * 2048, DH * 128, 1024), idesc, (j | kk) != 0);
            }
        }
        // D += Y^T G_{KC-1}: A = Y tile(s) read with M = i contiguous, B = G read with N = o contiguous, K = tokens
        {
          const uint32_t idesc = idesc_bf16(DH, 1, 1);
          const uint32_t gl = g_addr + (KC - 1) * SM::TILE;
          const uint32_t acc = first_of_head ? 0u : 1u;
#pragma unroll
          for (int gp = 0; gp < SM::NGRP; ++gp) {
            // d_h = 128: one tap, two 64-channel chunks 16 KB apart; d_h = 64: two taps, their tiles TILE apart
            const int j0 = DH == 128 ? gp : 2 * gp;
            const uint32_t lbo = DH == 128 ? 16384u : (uint32_t)SM::TILE;   // an odd last tap pairs with the tile after it (ignored)
#pragma unroll
            for (int kk = 0; kk < 8; ++kk)
              mma_ss(tmem_base + SM::DW_COL + gp * SM::GRP_COLS,
                     smem_desc_sw128(y_addr + j0 * SM::TILE + kk * 2048, lbo, 1024),
                     smem_desc_sw128(gl + kk * 2048, 16384, 1024), idesc, acc | (uint32_t)(kk != 0));
          }
        }
        mma_commit(a_empty);
        mma_commit(&acc_full[buf]);
      }
      __syncwarp();
      if (first_of_head && staged_head >= 0) ++flushes;
      staged_head = h;
    }
  } else {
    // ------------------------------------------------------------------ epilogue
    const int rho = threadIdx.x;
    const uint32_t lane_sel = (uint32_t)(warp * 32) << 16;
    int it = 0;
    for (int u = u_begin; u < u_end; ++u, ++it) {
      const int h = u / p.units_per_head, rem = u % p.units_per_head;
      const int b = rem / p.n_tiles, t0 = (rem % p.n_tiles) * 128;
      const int buf = it & 1;
      const int t = t0 + rho;
      const bool last_of_head = (u + 1 == u_end) || ((u + 1) / p.units_per_head != h);
      if (!mbar_wait(&acc_full[buf], (it >> 1) & 1, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_EPI); goto done; }
      tc_fence_after();
      const uint32_t acc = tmem_base + lane_sel + buf * DH;
#pragma unroll 1
      for (int c = 0; c < DH / 32; ++c) {
        uint32_t r[32];
        tmem_ld32(acc + c * 32, r);
        tmem_ld_wait();
        // the warp's 32 tokens x 32 channels leave as whole 128-byte row segments, four rows per instruction
        warp_store_rows<128>(smem + SM::STG_OFF + warp * 4096, r,
                             reinterpret_cast<unsigned char*>(p.dy1 + ((long long)b * d.S + t0 + warp * 32) * d.L + h * DH + c * 32),
                             (long long)d.L * 4, d.S - (t0 + warp * 32));
      }
      if (last_of_head) {
        // accumulator rows: d_h = 128: lane = i of tap gp; d_h = 64: lanes 0-63 = tap 2gp, lanes 64-127 = tap 2gp+1
#pragma unroll 1
        for (int gp = 0; gp < SM::NGRP; ++gp) {
          const int j = DH == 128 ? gp : 2 * gp + (rho >> 6);
          const int i = DH == 128 ? rho : (rho & 63);
#pragma unroll 1
          for (int c = 0; c < SM::GRP_COLS / 32; ++c) {
            uint32_t r[32];
            tmem_ld32(tmem_base + lane_sel + SM::DW_COL + gp * SM::GRP_COLS + c * 32, r);
            tmem_ld_wait();
            if (j < KC) {
#pragma unroll
              for (int e = 0; e < 32; ++e) {
                const int o = c * 32 + e;
                atomicAdd(p.d_w1 + (((size_t)h * DH + o) * DH + i) * KC + j, __uint_as_float(r[e]));
              }
            }
          }
        }
        tc_fence_before();
        mbar_arrive(dw_free);
      }
      tc_fence_before();
      mbar_arrive(&acc_empty[buf]);
    }
  }
done:
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    const long long c0 = clock64();
    while (clock64() - c0 < 2000000) {}
    __syncthreads();
  }
  if (warp == TB_ALLOC_WARP) {
    tc_fence_after();
    tmem_dealloc(tmem_base, SM::TMEM_COLS);
  }
}

template <int DH, int KC>
int launch_tb(TcState* s, const TbParams& p0, cudaStream_t st) {
  static bool attr_done[TC_MAX_DEVICES] = {};
  using SM = TbSmem<DH, KC>;
  if (!attr_done[s->device]) {
    cudaError_t e = cudaFuncSetAttribute(tc_transform_bwd_kernel<DH, KC>, cudaFuncAttributeMaxDynamicSharedMemorySize, SM::TOTAL);
    if (e != cudaSuccess) return -(int)e;
    attr_done[s->device] = true;
  }
  const int grid = p0.total_units < s->sm_count ? p0.total_units : s->sm_count;
  tc_transform_bwd_kernel<DH, KC><<<grid, TB_THREADS, SM::TOTAL, st>>>(p0);
  cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? 0 : -(int)e;
}

}  // namespace

int tc_transform_bwd(TcState* s, const CcaDims& d, const float* qk0, const bf16* w0, const bf16* w1, const float* dqh,
                     const float* dkh, float* dy1, float* d_w1, int* d_status, cudaStream_t st) {
  if (!s || s->sm_count < 1) return 1;
  if (!(d.flags & F_CONV2)) return 1;
  if (d.L % 4 || d.Lq % 4 || d.Lk % 4) return 1;
  if ((reinterpret_cast<uintptr_t>(w1) & 15) || (reinterpret_cast<uintptr_t>(qk0) & 15) ||
      (reinterpret_cast<uintptr_t>(dqh) & 15) || (reinterpret_cast<uintptr_t>(dkh) & 15) ||
      (reinterpret_cast<uintptr_t>(dy1) & 15))
    return 1;
  TbParams p;
  p.d = d; p.qk0 = qk0; p.w0 = w0; p.w1 = w1; p.dqh = dqh; p.dkh = dkh; p.dy1 = dy1; p.d_w1 = d_w1; p.status = d_status;
  p.n_tiles = (d.S + 127) / 128;
  const long long uph = (long long)d.B * p.n_tiles, total = uph * (d.hq + d.hk);
  if (total > 0x7fffffffLL) return 1;
  p.units_per_head = (int)uph;
  p.total_units = (int)total;
  if (d.dh == 128) {
    if (d.k_ch == 1) return launch_tb<128, 1>(s, p, st);
    if (d.k_ch == 2) return launch_tb<128, 2>(s, p, st);
    return 1;
  }
  if (d.dh == 64) {
    if (d.k_ch == 1) return launch_tb<64, 1>(s, p, st);
    if (d.k_ch == 2) return launch_tb<64, 2>(s, p, st);
    if (d.k_ch == 3) return launch_tb<64, 3>(s, p, st);
    if (d.k_ch == 4) return launch_tb<64, 4>(s, p, st);
  }
  return 1;
}
