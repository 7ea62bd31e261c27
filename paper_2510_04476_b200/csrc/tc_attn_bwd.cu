// Tensor-core kernels, part 4: adjoint of the softmax attention of Eq. 11 (the paper prints no backward;
// this is the exact adjoint).  With P = softmax(Q K^T / sqrt(d_h)) recomputed from the saved log-sum-exp,
// dP = dO V^T, delta = rowsum(dO o O) and dS = P o (dP - delta):
//     dV = P^T dO,   dK = dS^T Q / sqrt(d_h),   dQ = dS K / sqrt(d_h),
// dK and dV summed over the g query heads that share a kv head.  Two kernels, no atomics:
//
//   tc_attn_bwd_dq_kernel   one CTA = 128 query rows of one (sequence, query head), loops over KV tiles.
//                           TMEM: S (two buffers), dP, dQ accumulator; thread = query row.
//   tc_attn_bwd_dkv_kernel  one CTA = 128 keys of one (sequence, kv head), loops over the g query heads and
//                           their query tiles.  It works on the transposed tiles S^T = K Q^T and
//                           dP^T = V dO^T (thread = key), so that P^T and dS^T are the TMEM A operands of
//                           dV += P^T dO and dK += dS^T Q and both accumulators stay in TMEM.  A query tile is
//                           handled as two 64-query sub-tiles in alternating TMEM buffers, so the MMAs of one
//                           overlap the exponentials of the other.
//
// Both: warps 0-15 compute (four column groups x four TMEM lane quarters), warp 16 TMA loads, warp 17 issues
// the MMAs (warp-uniform loop, one elected lane).  P and dS are bf16 MMA operands, everything else fp32.
#include <type_traits>
#include "tc_kernels.cuh"
#include "tc_ptx.cuh"
#include "tc_state.cuh"

using namespace tc;

namespace {

constexpr int BW_COMPUTE_WARPS = 16;       // four warps per scheduler: the per-element chains are latency-bound
constexpr int BW_TMA_WARP = BW_COMPUTE_WARPS, BW_MMA_WARP = BW_COMPUTE_WARPS + 1;
constexpr int BW_THREADS = 32 * (BW_COMPUTE_WARPS + 2);
constexpr float LOG2E_F = 1.4426950408889634f;

struct BwdParams {
  int B, S, hq, hk, g, Lq, Lk, causal;
  const float* lse;     // [B, hq, S] natural-log sum of exponentials from the forward
  const float* delta;   // [B, hq, S]
  float* dq;            // [B*S, Lq]
  float* dk;            // [B*S, Lk]
  float* dv;            // [B*S, Lk]
  int n_tiles;          // 128-row tiles per sequence
  int* status;
};

template <int DH>
struct BwdSmem {
  static constexpr int TILE = 128 * DH * 2;
  static constexpr int HALF_TILE = 64 * DH * 2;        // 64 queries of Q or dO
  static constexpr int STAGES = DH == 128 ? 4 : 6;     // ring of (Q, dO) half-tile pairs (shared memory is full at 128)
  static constexpr int FIX_OFF = 0;                    // K and V tiles, loaded once
  static constexpr int RING_OFF = 2 * TILE;
  static constexpr int BAR_OFF = RING_OFF + STAGES * 2 * HALF_TILE;
  static constexpr int STAT_OFF = BAR_OFF + 256;       // float [2 groups][2 buffers][2][128]
  // at least 120 KB so that two CTAs (each wanting all 512 TMEM columns) never share an SM
  static constexpr int TOTAL = (STAT_OFF + 4096 + 1024) > 122880 ? (STAT_OFF + 4096 + 1024) : 122880;
};

// dQ kernel: Q, dO, three K stages, two V stages
template <int DH>
struct DqSmem {
  static constexpr int TILE = 128 * DH * 2;
  static constexpr int K_STAGES = 3;
  static constexpr int BAR_OFF = (4 + K_STAGES) * TILE;
  static constexpr int TOTAL = (BAR_OFF + 256 + 1024) > 122880 ? (BAR_OFF + 256 + 1024) : 122880;
};

TC_DEVINL void fail(volatile int* abort_flag, int* status, int code) {
  *abort_flag = 1;
  atomicCAS(status, 0, code);
}

// 2^x for a pair: on the FMA pipe (clamped to the polynomial's range) or on the transcendental unit
template <bool POLY>
TC_DEVINL uint64_t exp2_pair(uint64_t x) {
  uint32_t a, b;
  unpack2u(x, a, b);
  if (POLY) return exp2_poly2(pack2f(fmaxf(__uint_as_float(a), -120.f), fmaxf(__uint_as_float(b), -120.f)));
  return pack2f(ex2f(__uint_as_float(a)), ex2f(__uint_as_float(b)));
}
TC_DEVINL uint32_t cvt_bf16x2(uint64_t v) {
  uint32_t a, b;
  unpack2u(v, a, b);
  return pack_bf16(__uint_as_float(a), __uint_as_float(b));
}

// descriptor low words (address >> 4 | leading offset << 16) and the common high word
TC_DEVINL uint32_t lo_kmajor(uint32_t addr) { return (addr >> 4) | (1u << 16); }
TC_DEVINL uint32_t lo_mnmajor(uint32_t addr) { return (addr >> 4) | ((16384u >> 4) << 16); }

// C[128 x 128] = A[128 x DH] B[128 x DH]^T, both operands K-major tiles in shared memory
template <int DH>
TC_DEVINL void mma_kk(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t hi) {
  const uint32_t idesc = idesc_bf16(128, 0, 0);
#pragma unroll
  for (int kk = 0; kk < DH / 16; ++kk) {
    const uint32_t off = (uint32_t)(((kk >> 2) * 16384 + (kk & 3) * 32) >> 4);
    mma_ss_w(d_tmem, a_lo + off, hi, b_lo + off, hi, idesc, kk != 0);
  }
}
// C[128 x DH] (+)= A[128 x 128] B, A = bf16 pairs in TMEM (32 keys in 16 columns at every 32nd column of a_tmem),
// B = a [128 rows][DH] tile in shared memory read along its rows (MN-major)
template <int DH>
TC_DEVINL void mma_tm(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t hi, uint32_t accumulate) {
  const uint32_t idesc = idesc_bf16(DH, 0, 1);
#pragma unroll
  for (int kk = 0; kk < 8; ++kk)
    mma_ts_w(d_tmem, a_tmem + (kk >> 1) * 32 + (kk & 1) * 8, b_lo + kk * (2048 >> 4), hi, idesc, (accumulate | kk) != 0);
}

template <int DH>
TC_DEVINL void tma_tile(unsigned char* dst, const CUtensorMap* map, int c0, int row, int b, uint64_t* bar) {
#pragma unroll
  for (int c = 0; c < DH / 64; ++c) tma_load_3d(dst + c * 16384, map, c0 + c * 64, row, b, bar);
}

// ------------------------------------------------------------------------------------------ dQ
template <int DH, int POLY>
__global__ void __launch_bounds__(BW_THREADS, 1)
tc_attn_bwd_dq_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                      const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmDO, BwdParams p) {
  using SM = DqSmem<DH>;
  constexpr int KS = SM::K_STAGES;
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = smem_align1024(smem_dyn);
  unsigned char* sQ = smem;
  unsigned char* sDO = sQ + SM::TILE;
  unsigned char* sK = sDO + SM::TILE;                 // [KS]: K_j lives from S(j) (issued a tile ahead) to dQ(j)
  unsigned char* sV = sK + KS * SM::TILE;             // [2]
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + SM::BAR_OFF);
  uint64_t* qdo_full = bars;          // Q and dO tiles loaded
  uint64_t* k_full = bars + 1;        // [KS]
  uint64_t* k_empty = bars + 4;       // [KS]
  uint64_t* v_full = bars + 7;        // [2]
  uint64_t* v_empty = bars + 9;       // [2]
  uint64_t* s_full = bars + 11;       // [2] MMA -> compute: S buffer ready
  uint64_t* dp_full = bars + 13;      // MMA -> compute: dP ready
  uint64_t* ds_full = bars + 14;      // compute -> MMA: dS written, dP consumed (all compute threads)
  uint64_t* dq_done = bars + 15;
  uint64_t* dp_free = bars + 16;      // compute -> MMA: dP of the tile is in registers (all compute threads)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 17);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // heavy (late) query tiles first
  const int per_tile = p.B * p.hq;
  const int tile = p.n_tiles - 1 - (int)(blockIdx.x / per_tile);
  const int rem = blockIdx.x % per_tile;
  const int b = rem / p.hq, hi = rem % p.hq, hj = hi / p.g;
  const int m0 = tile * 128;
  const int n_kv = p.causal ? tile + 1 : p.n_tiles;

  if (threadIdx.x == 0) {
    mbar_init(qdo_full, 1);
    for (int i = 0; i < KS; ++i) {
      mbar_init(&k_full[i], 1);
      mbar_init(&k_empty[i], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&v_full[i], 1);
      mbar_init(&v_empty[i], 1);
      mbar_init(&s_full[i], 1);
    }
    mbar_init(dp_full, 1);
    mbar_init(ds_full, 32 * BW_COMPUTE_WARPS);
    mbar_init(dq_done, 1);
    mbar_init(dp_free, 32 * BW_COMPUTE_WARPS);
    wait_ctl_init(abort_flag, p.status);
    fence_barrier_init();
    prefetch_tmap(&tmQ);
    prefetch_tmap(&tmK);
    prefetch_tmap(&tmV);
    prefetch_tmap(&tmDO);
  }
  if (warp == BW_MMA_WARP) {
    tmem_alloc(tmem_slot, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // TMEM columns: S0 [0,128) S1 [128,256) dP [256,384) dQ [384,384+DH)

  if (warp == BW_TMA_WARP) {
    if (lane == 0) {
      mbar_expect_tx(qdo_full, 2 * SM::TILE);
      tma_tile<DH>(sQ, &tmQ, hi * DH, m0, b, qdo_full);
      tma_tile<DH>(sDO, &tmDO, hi * DH, m0, b, qdo_full);
      for (int j = 0; j < n_kv; ++j) {
        const int st = j & 1, ks = j % KS;
        const uint32_t ph = (j >> 1) & 1, kph = (j / KS) & 1;
        if (!mbar_wait(&k_empty[ks], kph ^ 1, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_TMA); goto done; }
        mbar_expect_tx(&k_full[ks], SM::TILE);
        tma_tile<DH>(sK + ks * SM::TILE, &tmK, hj * DH, j * 128, b, &k_full[ks]);
        if (!mbar_wait(&v_empty[st], ph ^ 1, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_TMA); goto done; }
        mbar_expect_tx(&v_full[st], SM::TILE);
        tma_tile<DH>(sV + st * SM::TILE, &tmV, hj * DH, j * 128, b, &v_full[st]);
      }
    }
  } else if (warp == BW_MMA_WARP) {
    const bool leader = elect_one();
    const uint32_t hi_w = (uint32_t)(smem_desc_sw128(0, 0, 1024) >> 32);
    const uint32_t q_lo = lo_kmajor(smem_u32(sQ)), do_lo = lo_kmajor(smem_u32(sDO));
    const uint32_t k_lo = lo_kmajor(smem_u32(sK)), v_lo = lo_kmajor(smem_u32(sV)), k_mn = lo_mnmajor(smem_u32(sK));
    constexpr uint32_t TILE16 = SM::TILE >> 4;
    auto wait_all = [&](uint64_t* bar, uint32_t parity) -> bool {
      return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag));
    };
    if (!wait_all(qdo_full, 0)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
    if (!wait_all(&k_full[0], 0)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
    tc_fence_after();
    if (leader) {
      mma_kk<DH>(tmem_base, q_lo, k_lo, hi_w);                         // S(0) = Q K_0^T
      mma_commit(&s_full[0]);
    }
    if (!wait_all(&v_full[0], 0)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
    tc_fence_after();
    if (leader) {
      mma_kk<DH>(tmem_base + 256, do_lo, v_lo, hi_w);                  // dP(0) = dO V_0^T
      mma_commit(dp_full);
      mma_commit(&v_empty[0]);
    }
    for (int j = 0; j < n_kv; ++j) {
      const int st = j & 1, nx = (j + 1) & 1, kst = j % KS, knx = (j + 1) % KS;
      const uint32_t nph = ((j + 1) >> 1) & 1, knph = ((j + 1) / KS) & 1;
      if (j + 1 < n_kv) {
        // S(j+1) into the other buffer; the dQ MMA that read dS(j-1) from it was issued earlier (in order)
        if (!wait_all(&k_full[knx], knph)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
        tc_fence_after();
        if (leader) {
          mma_kk<DH>(tmem_base + nx * 128, q_lo, k_lo + knx * TILE16, hi_w);
          mma_commit(&s_full[nx]);
        }
      }
      if (j + 1 < n_kv) {
        // dP(j+1) as soon as the compute warps hold dP(j) in registers: their exponentials then overlap it
        if (!wait_all(dp_free, j & 1)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
        if (!wait_all(&v_full[nx], nph)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
        tc_fence_after();
        if (leader) {
          mma_kk<DH>(tmem_base + 256, do_lo, v_lo + nx * TILE16, hi_w);
          mma_commit(dp_full);
          mma_commit(&v_empty[nx]);
        }
      }
      if (!wait_all(ds_full, j & 1)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
      tc_fence_after();
      if (leader) {
        mma_tm<DH>(tmem_base + 384, tmem_base + st * 128, k_mn + kst * TILE16, hi_w, j != 0);   // dQ += dS(j) K_j
        mma_commit(&k_empty[kst]);
      }
    }
    if (leader) mma_commit(dq_done);
  } else {
    // ------------------------------------------------------------------ compute, thread = query row
    const int part = warp >> 2;                        // which 32 keys of each KV tile
    const int row = (warp & 3) * 32 + lane;
    const uint32_t lane_sel = (uint32_t)((warp & 3) * 32) << 16;
    const int tq = m0 + row;
    const float c_scale = rsqrtf((float)DH) * LOG2E_F;
    const long long stat_idx = ((long long)b * p.hq + hi) * p.S + tq;
    const float l2 = tq < p.S ? p.lse[stat_idx] * LOG2E_F : INFINITY;     // rows past the end: P = 0
    const float dl = tq < p.S ? p.delta[stat_idx] : 0.f;
    const uint64_t scale2 = pack2f(c_scale, c_scale), nl2 = pack2f(-l2, -l2), ndl2 = pack2f(-dl, -dl);
    for (int j = 0; j < n_kv; ++j) {
      const uint32_t s_t = tmem_base + lane_sel + (j & 1) * 128 + part * 32;
      const uint32_t dp_t = tmem_base + lane_sel + 256 + part * 32;
      if (!mbar_wait(&s_full[j & 1], (j >> 1) & 1, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_SOFTMAX); goto done; }
      if (!mbar_wait(dp_full, j & 1, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_SOFTMAX); goto done; }
      tc_fence_after();
      const int k0 = j * 128 + part * 32;
      const bool need_mask = (p.causal && j * 128 + 127 > m0) || (j * 128 + 128 > p.S);
      const int lim = p.causal ? min(tq, p.S - 1) : p.S - 1;
      uint32_t sv[32], dv[32];
      tmem_ld32(s_t, sv);
      tmem_ld32(dp_t, dv);
      tmem_ld_wait();
      tc_fence_before();
      mbar_arrive(dp_free);                            // the dP buffer may be overwritten
      // masking is a compile-time variant of the whole tile's arithmetic: a branch per pair would end the instruction
      // scheduler's window sixteen times per tile
      auto tile_math = [&](auto mask_c) {
      constexpr bool MASK = decltype(mask_c)::value;
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
        uint32_t pk[8];
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          const int e = hf * 16 + 2 * c;
          const uint64_t x = fma2(pack2u(sv[e], sv[e + 1]), scale2, nl2);
          uint64_t ex = (c & 3) < POLY ? exp2_pair<true>(x) : exp2_pair<false>(x);
          if (MASK) {
            uint32_t a, bb;
            unpack2u(ex, a, bb);
            if (k0 + e > lim) a = 0u;
            if (k0 + e + 1 > lim) bb = 0u;
            ex = pack2u(a, bb);
          }
          pk[c] = cvt_bf16x2(mul2(ex, add2(pack2u(dv[e], dv[e + 1]), ndl2)));
        }
        // dS (bf16 pairs) over columns this thread has read: keys 32 part + [0,32) -> columns 32 part + [0,16)
        tmem_st8(s_t + hf * 8, pk);
      }
      };
      if (need_mask) tile_math(std::true_type{}); else tile_math(std::false_type{});
      tmem_st_wait();
      tc_fence_before();
      mbar_arrive(ds_full);
    }
    if (!mbar_wait(dq_done, 0, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_EPI); goto done; }
    tc_fence_after();
    {
      const float scale = rsqrtf((float)DH);
#pragma unroll 1
      for (int c = 0; c < DH / 64; ++c) {
        uint32_t t[16];
        const int col = part * (DH / 4) + c * 16;
        tmem_ld16(tmem_base + lane_sel + 384 + col, t);
        tmem_ld_wait();
        if (tq < p.S) {
          float* dst = p.dq + ((long long)b * p.S + tq) * p.Lq + hi * DH + col;
#pragma unroll
          for (int i = 0; i < 4; ++i)
            reinterpret_cast<float4*>(dst)[i] =
                make_float4(__uint_as_float(t[4 * i]) * scale, __uint_as_float(t[4 * i + 1]) * scale,
                            __uint_as_float(t[4 * i + 2]) * scale, __uint_as_float(t[4 * i + 3]) * scale);
        }
      }
    }
  }
done:
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000) {}
    __syncthreads();
  }
  if (warp == BW_MMA_WARP) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

// ------------------------------------------------------------------------------------------ dK, dV
template <int DH, int POLY>
__global__ void __launch_bounds__(BW_THREADS, 1)
tc_attn_bwd_dkv_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                       const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmDO, BwdParams p) {
  using SM = BwdSmem<DH>;
  constexpr int NST = SM::STAGES;
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = smem_align1024(smem_dyn);
  unsigned char* sK = smem + SM::FIX_OFF;
  unsigned char* sV = sK + SM::TILE;
  unsigned char* sRing = smem + SM::RING_OFF;         // [NST] stages of (Q half-tile, dO half-tile): 64 queries each
  float* stat = reinterpret_cast<float*>(smem + SM::STAT_OFF);   // [2 buffers][lse2 | delta][128 queries]
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + SM::BAR_OFF);
  uint64_t* kv_full = bars;
  uint64_t* qdo_full = bars + 1;      // [NST]
  uint64_t* qdo_empty = bars + 1 + NST;   // [NST]
  uint64_t* sdp_full = bars + 1 + 2 * NST;   // [2] MMA -> compute: S^T and dP^T of a 64-query sub-tile ready
  uint64_t* pds_full = sdp_full + 2;  // [2] compute group -> MMA: P^T and dS^T written (256 arrivals)
  uint64_t* acc_done = pds_full + 2;
  uint64_t* stat_ready = acc_done + 1;   // [2] per compute group: column statistics of the tile are in shared memory
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(stat_ready + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // heavy (early) key tiles first
  const int per_tile = p.B * p.hk;
  const int tile = (int)(blockIdx.x / per_tile);
  const int rem = blockIdx.x % per_tile;
  const int b = rem / p.hk, hj = rem % p.hk;
  const int n0 = tile * 128;
  const int i0 = p.causal ? tile : 0;                  // first query tile that sees these keys
  const int n_q = p.n_tiles - i0;
  const int n_it = n_q * p.g;                          // iteration it = (gi, i): gi = it / n_q, i = i0 + it % n_q

  if (threadIdx.x == 0) {
    mbar_init(kv_full, 1);
    for (int i = 0; i < NST; ++i) {
      mbar_init(&qdo_full[i], 1);
      mbar_init(&qdo_empty[i], 1);
    }
    mbar_init(&sdp_full[0], 1);
    mbar_init(&sdp_full[1], 1);
    mbar_init(&pds_full[0], 256);
    mbar_init(&pds_full[1], 256);
    mbar_init(acc_done, 1);
    mbar_init(&stat_ready[0], 256);
    mbar_init(&stat_ready[1], 256);
    wait_ctl_init(abort_flag, p.status);
    fence_barrier_init();
    prefetch_tmap(&tmQ);
    prefetch_tmap(&tmK);
    prefetch_tmap(&tmV);
    prefetch_tmap(&tmDO);
  }
  if (warp == BW_MMA_WARP) {
    tmem_alloc(tmem_slot, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // TMEM columns: S^T two 64-query buffers [0,64) [64,128), dP^T likewise [128,192) [192,256),
  // dV [256,256+DH), dK [384,384+DH)

  if (warp == BW_TMA_WARP) {
    if (lane == 0) {
      mbar_expect_tx(kv_full, 2 * SM::TILE);
      tma_tile<DH>(sK, &tmK, hj * DH, n0, b, kv_full);
      tma_tile<DH>(sV, &tmV, hj * DH, n0, b, kv_full);
      for (int sub = 0; sub < 2 * n_it; ++sub) {
        const int it = sub >> 1, st = sub % NST;
        const uint32_t ph = (sub / NST) & 1;
        const int hi = hj * p.g + it / n_q, m0 = (i0 + it % n_q) * 128 + (sub & 1) * 64;
        if (!mbar_wait(&qdo_empty[st], ph ^ 1, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_TMA); goto done; }
        mbar_expect_tx(&qdo_full[st], 2 * SM::HALF_TILE);
        unsigned char* dst = sRing + st * 2 * SM::HALF_TILE;
#pragma unroll
        for (int c = 0; c < DH / 64; ++c) {
          tma_load_3d(dst + c * 8192, &tmQ, hi * DH + c * 64, m0, b, &qdo_full[st]);
          tma_load_3d(dst + SM::HALF_TILE + c * 8192, &tmDO, hi * DH + c * 64, m0, b, &qdo_full[st]);
        }
      }
    }
  } else if (warp == BW_MMA_WARP) {
    // Sub-tile = 64 queries; S^T / dP^T of sub-tile s live in TMEM buffer s & 1, so the MMAs of sub-tile s + 1
    // run while the compute warps work on sub-tile s.
    const bool leader = elect_one();
    const uint32_t hi_w = (uint32_t)(smem_desc_sw128(0, 0, 1024) >> 32);
    const uint32_t k_lo = lo_kmajor(smem_u32(sK)), v_lo = lo_kmajor(smem_u32(sV));
    const uint32_t ring16 = smem_u32(sRing) >> 4;
    constexpr uint32_t STAGE16 = (2 * SM::HALF_TILE) >> 4, HALF16 = SM::HALF_TILE >> 4;
    const int n_sub = 2 * n_it;
    auto wait_all = [&](uint64_t* bar, uint32_t parity) -> bool {
      return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag));
    };
    // half-tiles are [64 rows][DH] as DH/64 boxes of 8 KB
    auto issue_sdp = [&](int sub) {     // S^T = K Q^T and dP^T = V dO^T for 64 queries
      const int sb = sub & 1;
      const uint32_t idesc = idesc_bf16(64, 0, 0);
      const uint32_t qb = (ring16 + (sub % NST) * STAGE16) | (1u << 16), ob = qb + HALF16;
      if (leader) {
#pragma unroll
        for (int kk = 0; kk < DH / 16; ++kk) {
          const uint32_t offk = (uint32_t)(((kk >> 2) * 16384 + (kk & 3) * 32) >> 4);
          const uint32_t offq = (uint32_t)(((kk >> 2) * 8192 + (kk & 3) * 32) >> 4);
          mma_ss_w(tmem_base + sb * 64, k_lo + offk, hi_w, qb + offq, hi_w, idesc, kk != 0);
        }
#pragma unroll
        for (int kk = 0; kk < DH / 16; ++kk) {
          const uint32_t offk = (uint32_t)(((kk >> 2) * 16384 + (kk & 3) * 32) >> 4);
          const uint32_t offq = (uint32_t)(((kk >> 2) * 8192 + (kk & 3) * 32) >> 4);
          mma_ss_w(tmem_base + 128 + sb * 64, v_lo + offk, hi_w, ob + offq, hi_w, idesc, kk != 0);
        }
        mma_commit(&sdp_full[sb]);
      }
    };
    auto issue_dvdk = [&](int sub) {    // dV += P^T dO, dK += dS^T Q over the sub-tile's 64 queries
      const int sb = sub & 1, st = sub % NST;
      const uint32_t idesc = idesc_bf16(DH, 0, 1);
      // read along the rows (N = d_h contiguous): 64-channel chunks are one 8 KB box apart
      const uint32_t qb = (ring16 + st * STAGE16) | ((8192u >> 4) << 16), ob = qb + HALF16;
      if (leader) {
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)
          mma_ts_w(tmem_base + 256, tmem_base + sb * 64 + (kk >> 1) * 32 + (kk & 1) * 8, ob + kk * (2048 >> 4), hi_w, idesc,
                   (sub | kk) != 0);
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)
          mma_ts_w(tmem_base + 384, tmem_base + 128 + sb * 64 + (kk >> 1) * 32 + (kk & 1) * 8, qb + kk * (2048 >> 4), hi_w,
                   idesc, (sub | kk) != 0);
        mma_commit(&qdo_empty[st]);
      }
    };
    if (!wait_all(kv_full, 0)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
    for (int s0 = 0; s0 < 2 && s0 < n_sub; ++s0) {
      if (!wait_all(&qdo_full[s0 % NST], (s0 / NST) & 1)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
      tc_fence_after();
      issue_sdp(s0);
    }
    for (int sub = 0; sub < n_sub; ++sub) {
      // sub-tile sub belongs to compute group sub & 1
      if (!wait_all(&pds_full[sub & 1], (sub >> 1) & 1)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
      tc_fence_after();
      issue_dvdk(sub);
      if (sub + 2 < n_sub) {
        const int nx = sub + 2;
        if (!wait_all(&qdo_full[nx % NST], (nx / NST) & 1)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
        tc_fence_after();
        issue_sdp(nx);             // into the buffer whose P^T / dS^T the MMAs just issued are reading (in order)
      }
    }
    if (leader) mma_commit(acc_done);
  } else {
    // ------------------------------------------------------------------ compute, thread = key
    // Two groups of eight warps: group gsel works on the sub-tiles with (sub & 1) == gsel, i.e. on queries
    // [64 gsel, 64 gsel + 64) of every query tile, in TMEM buffer gsel.
    const int gsel = warp >> 3;
    const int part = (warp >> 2) & 1;                  // which 32 of the sub-tile's 64 queries
    const int row = (warp & 3) * 32 + lane;
    const int ct = threadIdx.x & 255;                  // index inside the group
    const uint32_t lane_sel = (uint32_t)((warp & 3) * 32) << 16;
    const int tk = n0 + row;
    const float c_scale = rsqrtf((float)DH) * LOG2E_F;
    float* gstat = stat + gsel * 512;                  // [2 buffers][lse2 | delta][128 queries] of this group
    // column statistics of a query tile, negated: thread ct < 128 fetches -lse * log2(e) of query ct, the others
    // -delta; queries past the end of the sequence get -inf, so their P is 0
    auto fetch_stat = [&](int it) -> float {
      const int hi = hj * p.g + it / n_q, m0 = (i0 + it % n_q) * 128;
      const int tq = m0 + (ct & 127);
      const long long idx = ((long long)b * p.hq + hi) * p.S + tq;
      if (ct < 128) return tq < p.S ? -p.lse[idx] * LOG2E_F : -INFINITY;
      return tq < p.S ? -p.delta[idx] : 0.f;
    };
    float next_stat = n_it > 0 ? fetch_stat(0) : 0.f;
    const uint64_t scale2 = pack2f(c_scale, c_scale);
    const uint32_t s_t = tmem_base + lane_sel + gsel * 64 + part * 32;
    const uint32_t dp_t = tmem_base + lane_sel + 128 + gsel * 64 + part * 32;
    const int qoff = gsel * 64 + part * 32;            // first query (within the tile) of this thread's columns
    for (int it = 0; it < n_it; ++it) {
      const int stb = it & 1;
      gstat[stb * 256 + ct] = next_stat;               // buffer stb was last read two tiles ago
      if (it + 1 < n_it) next_stat = fetch_stat(it + 1);
      mbar_arrive(&stat_ready[gsel]);
      if (!mbar_wait(&stat_ready[gsel], it & 1, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_SOFTMAX); goto done; }
      const int m0 = (i0 + it % n_q) * 128;
      const bool diag = p.causal && m0 == n0;
      if (!mbar_wait(&sdp_full[gsel], it & 1, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_SOFTMAX); goto done; }
      tc_fence_after();
      const ulonglong2* nlv = reinterpret_cast<const ulonglong2*>(gstat + stb * 256 + qoff);        // pairs of -lse2
      const ulonglong2* ndv = reinterpret_cast<const ulonglong2*>(gstat + stb * 256 + 128 + qoff);  // pairs of -delta
      auto tile_math = [&](auto diag_c) {
      constexpr bool DIAG = decltype(diag_c)::value;
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
        uint32_t sv[16], dv[16], pk[8], dk_[8];
        tmem_ld16(s_t + hf * 16, sv);
        tmem_ld16(dp_t + hf * 16, dv);
        tmem_ld_wait();
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const ulonglong2 nl = nlv[hf * 4 + c], nd = ndv[hf * 4 + c];
          uint64_t e0 = fma2(pack2u(sv[4 * c + 0], sv[4 * c + 1]), scale2, nl.x);
          uint64_t e1 = fma2(pack2u(sv[4 * c + 2], sv[4 * c + 3]), scale2, nl.y);
          e0 = (2 * c & 3) < POLY ? exp2_pair<true>(e0) : exp2_pair<false>(e0);
          e1 = ((2 * c + 1) & 3) < POLY ? exp2_pair<true>(e1) : exp2_pair<false>(e1);
          if (DIAG) {
            const int q0 = m0 + qoff + hf * 16 + 4 * c;      // query of the first of the four
            uint32_t a0, a1, a2, a3;
            unpack2u(e0, a0, a1);
            unpack2u(e1, a2, a3);
            if (tk > q0) a0 = 0u;
            if (tk > q0 + 1) a1 = 0u;
            if (tk > q0 + 2) a2 = 0u;
            if (tk > q0 + 3) a3 = 0u;
            e0 = pack2u(a0, a1);
            e1 = pack2u(a2, a3);
          }
          pk[2 * c] = cvt_bf16x2(e0);
          pk[2 * c + 1] = cvt_bf16x2(e1);
          dk_[2 * c] = cvt_bf16x2(mul2(e0, add2(pack2u(dv[4 * c + 0], dv[4 * c + 1]), nd.x)));
          dk_[2 * c + 1] = cvt_bf16x2(mul2(e1, add2(pack2u(dv[4 * c + 2], dv[4 * c + 3]), nd.y)));
        }
        tmem_st8(s_t + hf * 8, pk);                    // P^T over S^T columns this thread has read
        tmem_st8(dp_t + hf * 8, dk_);                  // dS^T over dP^T columns this thread has read
      }
      };
      if (diag) tile_math(std::true_type{}); else tile_math(std::false_type{});
      tmem_st_wait();
      tc_fence_before();
      mbar_arrive(&pds_full[gsel]);
    }
    if (!mbar_wait(acc_done, 0, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_EPI); goto done; }
    tc_fence_after();
    {
      const float scale = rsqrtf((float)DH);
#pragma unroll 1
      for (int c = 0; c < DH / 64; ++c) {
        uint32_t t[16], u[16];
        const int col = (gsel * 2 + part) * (DH / 4) + c * 16;
        tmem_ld16(tmem_base + lane_sel + 256 + col, t);
        tmem_ld16(tmem_base + lane_sel + 384 + col, u);
        tmem_ld_wait();
        if (tk < p.S) {
          const long long off = ((long long)b * p.S + tk) * p.Lk + hj * DH + col;
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            reinterpret_cast<float4*>(p.dv + off)[i] = make_float4(__uint_as_float(t[4 * i]), __uint_as_float(t[4 * i + 1]),
                                                                    __uint_as_float(t[4 * i + 2]), __uint_as_float(t[4 * i + 3]));
            reinterpret_cast<float4*>(p.dk + off)[i] =
                make_float4(__uint_as_float(u[4 * i]) * scale, __uint_as_float(u[4 * i + 1]) * scale,
                            __uint_as_float(u[4 * i + 2]) * scale, __uint_as_float(u[4 * i + 3]) * scale);
          }
        }
      }
    }
  }
done:
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000) {}
    __syncthreads();
  }
  if (warp == BW_MMA_WARP) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

template <int DH, int POLY>
int launch_bwd(TcState* s, const CcaDims& d, const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV,
               const CUtensorMap& tmDO, const CUtensorMap& tmQh, const CUtensorMap& tmDOh, const BwdParams& p,
               cudaStream_t st) {
  static bool attr_set[TC_MAX_DEVICES] = {};
  if (!attr_set[s->device]) {
    cudaError_t e = cudaFuncSetAttribute(tc_attn_bwd_dq_kernel<DH, POLY>, cudaFuncAttributeMaxDynamicSharedMemorySize, DqSmem<DH>::TOTAL);
    if (e != cudaSuccess) return -(int)e;
    e = cudaFuncSetAttribute(tc_attn_bwd_dkv_kernel<DH, POLY>, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdSmem<DH>::TOTAL);
    if (e != cudaSuccess) return -(int)e;
    attr_set[s->device] = true;
  }
  const long long g_kv = (long long)p.n_tiles * d.B * d.hk, g_q = (long long)p.n_tiles * d.B * d.hq;
  if (g_q > 0x7fffffffLL) return 1;
  tc_attn_bwd_dkv_kernel<DH, POLY><<<(unsigned)g_kv, BW_THREADS, BwdSmem<DH>::TOTAL, st>>>(tmQh, tmK, tmV, tmDOh, p);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return -(int)e;
  tc_attn_bwd_dq_kernel<DH, POLY><<<(unsigned)g_q, BW_THREADS, DqSmem<DH>::TOTAL, st>>>(tmQ, tmK, tmV, tmDO, p);
  e = cudaGetLastError();
  return e == cudaSuccess ? 0 : -(int)e;
}

}  // namespace

// delta must already hold rowsum(dO o O).  Returns 0 if both kernels were enqueued (2 launches).
int tc_attn_bwd(TcState* s, const CcaDims& d, const bf16* q, const bf16* k, const bf16* v, const bf16* d_o,
                const float* lse, const float* delta, float* dq, float* dk, float* dv, int* d_status, cudaStream_t st) {
  if (!s || !s->encode) return 1;
  if (d.dh != 64 && d.dh != 128) return 1;
  if (d.Lq % 8 || d.Lk % 8) return 1;
  if (d.dh == 64 && s->attn_bwd_fused) {
    // one kernel that visits every (query, key) pair once; dQ by vector reductions into memory
    const int r = tc_attn_bwd_fused(s, d, q, k, v, d_o, lse, delta, dq, dk, dv, d_status, st);
    if (r != 1) return r;
  }
  CUtensorMap tmQ, tmK, tmV, tmDO;
  const uint64_t S = (uint64_t)d.S, B = (uint64_t)d.B, Lq = (uint64_t)d.Lq, Lk = (uint64_t)d.Lk;
  if (!tc_make_map_3d(s, &tmQ, q, Lq, S, B, Lq, S * Lq, 64, 128)) return 1;
  if (!tc_make_map_3d(s, &tmDO, d_o, Lq, S, B, Lq, S * Lq, 64, 128)) return 1;
  CUtensorMap tmQh, tmDOh;       // 64-row boxes for the dK/dV kernel's half-tiles
  if (!tc_make_map_3d(s, &tmQh, q, Lq, S, B, Lq, S * Lq, 64, 64)) return 1;
  if (!tc_make_map_3d(s, &tmDOh, d_o, Lq, S, B, Lq, S * Lq, 64, 64)) return 1;
  if (!tc_make_map_3d(s, &tmK, k, Lk, S, B, Lk, S * Lk, 64, 128)) return 1;
  if (!tc_make_map_3d(s, &tmV, v, Lk, S, B, Lk, S * Lk, 64, 128)) return 1;
  BwdParams p;
  p.B = d.B; p.S = d.S; p.hq = d.hq; p.hk = d.hk; p.g = d.g; p.Lq = d.Lq; p.Lk = d.Lk; p.causal = d.causal;
  p.lse = lse; p.delta = delta; p.dq = dq; p.dk = dk; p.dv = dv;
  p.n_tiles = (d.S + 127) / 128;
  p.status = d_status;
  const int poly = s->attn_poly_bwd < 0 ? (d.dh == 128 ? 0 : 1) : s->attn_poly_bwd;
  if (d.dh == 128) {
    if (poly == 0) return launch_bwd<128, 0>(s, d, tmQ, tmK, tmV, tmDO, tmQh, tmDOh, p, st);
    if (poly == 2) return launch_bwd<128, 2>(s, d, tmQ, tmK, tmV, tmDO, tmQh, tmDOh, p, st);
    return launch_bwd<128, 1>(s, d, tmQ, tmK, tmV, tmDO, tmQh, tmDOh, p, st);
  }
  if (poly == 0) return launch_bwd<64, 0>(s, d, tmQ, tmK, tmV, tmDO, tmQh, tmDOh, p, st);
  if (poly == 2) return launch_bwd<64, 2>(s, d, tmQ, tmK, tmV, tmDO, tmQh, tmDOh, p, st);
  return launch_bwd<64, 1>(s, d, tmQ, tmK, tmV, tmDO, tmQh, tmDOh, p, st);
}
