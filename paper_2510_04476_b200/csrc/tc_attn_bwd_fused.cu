// Tensor-core kernels, part 4b: adjoint of the softmax attention of Eq. 11 in ONE kernel (head size 64).
//
// The two-kernel adjoint (tc_attn_bwd.cu) recomputes S and dP in each kernel: seven contractions and two
// exponentials per (query, key) pair where the adjoint itself has five and one.  At head size 64 a score costs only
// 256 tensor FLOPs per contraction, so the exponentials and the element-wise chain bound both kernels; here every
// pair is visited once.
//
// One CTA = 128 keys of one (sequence, kv head); it walks the g query heads of the group and, for each, the query
// tiles that see these keys (thread = key, transposed tiles S^T = K Q^T, dP^T = V dO^T as in the dK/dV kernel), so
// that dV += P^T dO and dK += dS^T Q accumulate in TMEM over the whole walk with P^T and dS^T as TMEM operands.
// Two groups of four compute warps; a group owns the 64-query sub-tile of its TMEM buffer and a thread all 64 scores
// of its key there (16 at a time, the next 16 and their column statistics in flight meanwhile).  A group's loop is a
// chain  scores ready -> arithmetic -> P^T, dS^T written -> the tensor core's dV / dK and next S^T / dP^T -> ...;  the
// two groups' chains interleave, and everything that is not on the chain (the dQ hand-over) runs while the tensor
// core works.
// The compute warps also leave dS^T as bf16 in shared memory ([key][query], 128-byte swizzle): read with the queries
// as the M dimension it is the A operand of   dQ_tile = dS K   (M = 128 queries, N = d_h, K = 128 keys; the resident
// K tile read along its rows is the B operand).  A query tile's dQ gets such a contribution from every key tile it
// sees, i.e. from different CTAs: the compute warps copy the finished tile from TMEM to a shared-memory stage and a
// lane of the TMA warp adds it into the zeroed fp32 dq with TMA reductions (cp.reduce.async.bulk.tensor, whole 128-byte
// lines; rows past the end of the sequence are clipped by the tensor map).  The sum order of dq therefore varies from
// run to run (fp32 rounding only).
//
// TMEM columns: S^T two 64-query buffers [0,128), dP^T likewise [128,256), dV [256,320), dK [320,384),
// dQ two buffers [384,448) [448,512).
#include <type_traits>
#include "tc_kernels.cuh"
#include "tc_ptx.cuh"
#include "tc_state.cuh"

using namespace tc;

namespace {

constexpr int FB_COMPUTE_WARPS = 8;
// warp 16: lane 0 issues the TMA loads, lane 1 the dQ reductions (two independent loops of one warp: a third service
// warp would cost every thread 16 registers); warp 17 issues the MMAs
constexpr int FB_TMA_WARP = FB_COMPUTE_WARPS, FB_MMA_WARP = FB_COMPUTE_WARPS + 1;
constexpr int FB_THREADS = 32 * (FB_COMPUTE_WARPS + 2);
constexpr float FB_LOG2E = 1.4426950408889634f;
constexpr int DH = 64;

struct FbParams {
  int B, S, hq, hk, g, Lq, Lk, causal;
  const float* lse;     // [B, hq, S] natural-log sum of exponentials from the forward
  const float* delta;   // [B, hq, S]
  float* dq;            // [B*S, Lq], zeroed before the launch
  float* dk;            // [B*S, Lk]
  float* dv;            // [B*S, Lk]
  int n_tiles;          // 128-row tiles per sequence
  int* status;
};

struct FbSmem {
  static constexpr int TILE = 128 * DH * 2;            // 16 KB: K, V
  static constexpr int HALF_TILE = 64 * DH * 2;        // 64 queries of Q or dO
  static constexpr int STAGES = 4;                     // ring of (Q, dO) half-tile pairs
  static constexpr int DS_TILE = 128 * 128 * 2;        // dS^T [128 keys][128 queries] bf16: two 64-query boxes
  static constexpr int DQ_STAGE = 128 * DH * 4;        // one dQ tile in fp32: two boxes of [128 queries][32 channels]
  static constexpr int FIX_OFF = 0;
  static constexpr int RING_OFF = 2 * TILE;
  static constexpr int DS_OFF = RING_OFF + STAGES * 2 * HALF_TILE;
  static constexpr int DQ_OFF = DS_OFF + 2 * DS_TILE;
  static constexpr int BAR_OFF = DQ_OFF + DQ_STAGE;
  static constexpr int STAT_OFF = BAR_OFF + 256;       // float [2 groups][2 buffers][2][128]
  static constexpr int TOTAL = STAT_OFF + 4096 + 1024;
};

TC_DEVINL void fail(volatile int* abort_flag, int* status, int code) {
  *abort_flag = 1;
  atomicCAS(status, 0, code);
}
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
TC_DEVINL uint32_t lo_kmajor(uint32_t addr) { return (addr >> 4) | (1u << 16); }
TC_DEVINL uint32_t lo_mnmajor(uint32_t addr) { return (addr >> 4) | ((16384u >> 4) << 16); }

template <int POLY>
__global__ void __launch_bounds__(FB_THREADS, 1)
tc_attn_bwd_fused_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                         const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmDO,
                         const __grid_constant__ CUtensorMap tmDQ, FbParams p) {
  using SM = FbSmem;
  constexpr int NST = SM::STAGES;
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = smem_align1024(smem_dyn);
  unsigned char* sK = smem + SM::FIX_OFF;
  unsigned char* sV = sK + SM::TILE;
  unsigned char* sRing = smem + SM::RING_OFF;         // [NST] stages of (Q half-tile, dO half-tile): 64 queries each
  unsigned char* sDS = smem + SM::DS_OFF;             // [2] dS^T of a query tile
  float* stat = reinterpret_cast<float*>(smem + SM::STAT_OFF);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + SM::BAR_OFF);
  uint64_t* kv_full = bars;
  uint64_t* qdo_full = bars + 1;              // [NST]
  uint64_t* qdo_empty = bars + 1 + NST;       // [NST]
  uint64_t* sdp_full = bars + 1 + 2 * NST;    // [2] MMA -> compute: S^T and dP^T of a 64-query sub-tile ready
  uint64_t* pds_full = sdp_full + 2;          // [2] compute group -> MMA: P^T, dS^T written (TMEM and shared memory)
  uint64_t* acc_done = pds_full + 2;
  uint64_t* stat_ready = acc_done + 1;        // [2] per compute group
  uint64_t* dq_full = stat_ready + 2;         // [2] MMA -> compute: dQ of a query tile ready in its TMEM buffer
  uint64_t* dq_empty = dq_full + 2;           // [2] compute -> MMA: that buffer has been added to memory (512 arrivals)
  uint64_t* ds_free = dq_empty + 2;           // [2] MMA -> compute: the dQ contraction has read the dS^T tile
  uint64_t* stg_full = ds_free + 2;           // compute -> reduce warp: a dQ tile is in the stage (512 arrivals)
  uint64_t* stg_free = stg_full + 1;          // reduce warp -> compute: the TMA reduction has read the stage
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(stg_free + 1);
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
    for (int i = 0; i < 2; ++i) {
      mbar_init(&sdp_full[i], 1);
      mbar_init(&pds_full[i], 128);
      mbar_init(&stat_ready[i], 128);
      mbar_init(&dq_full[i], 1);
      mbar_init(&dq_empty[i], 32 * FB_COMPUTE_WARPS);
      mbar_init(&ds_free[i], 1);
    }
    mbar_init(acc_done, 1);
    mbar_init(stg_full, 32 * FB_COMPUTE_WARPS);
    mbar_init(stg_free, 1);
    wait_ctl_init(abort_flag, p.status);
    fence_barrier_init();
    prefetch_tmap(&tmQ);
    prefetch_tmap(&tmK);
    prefetch_tmap(&tmV);
    prefetch_tmap(&tmDO);
    prefetch_tmap(&tmDQ);
  }
  if (warp == FB_MMA_WARP) {
    tmem_alloc(tmem_slot, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == FB_TMA_WARP) {
    if (lane == 0) {
      mbar_expect_tx(kv_full, 2 * SM::TILE);
      tma_load_3d(sK, &tmK, hj * DH, n0, b, kv_full);
      tma_load_3d(sV, &tmV, hj * DH, n0, b, kv_full);
      for (int sub = 0; sub < 2 * n_it; ++sub) {
        const int it = sub >> 1, st = sub % NST;
        const uint32_t ph = (sub / NST) & 1;
        const int hi = hj * p.g + it / n_q, m0 = (i0 + it % n_q) * 128 + (sub & 1) * 64;
        if (!mbar_wait(&qdo_empty[st], ph ^ 1, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_TMA); goto done; }
        mbar_expect_tx(&qdo_full[st], 2 * SM::HALF_TILE);
        unsigned char* dst = sRing + st * 2 * SM::HALF_TILE;
        tma_load_3d(dst, &tmQ, hi * DH, m0, b, &qdo_full[st]);
        tma_load_3d(dst + SM::HALF_TILE, &tmDO, hi * DH, m0, b, &qdo_full[st]);
      }
    } else if (lane == 1) {
      // ---------------------------------------------------------------- dQ reductions into memory
      unsigned char* stg = smem + SM::DQ_OFF;
      for (int it = 0; it < n_it; ++it) {
        if (!mbar_wait(stg_full, it & 1, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_CORR); goto done; }
        const int hi = hj * p.g + it / n_q, m0 = (i0 + it % n_q) * 128;
#pragma unroll
        for (int c = 0; c < DH / 32; ++c)
          asm volatile("cp.reduce.async.bulk.tensor.3d.global.shared::cta.add.tile.bulk_group [%0, {%1, %2, %3}], [%4];"
                       ::"l"(&tmDQ), "r"(hi * DH + c * 32), "r"(m0), "r"(b), "r"(smem_u32(stg + c * 16384))
                       : "memory");
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        mbar_arrive(stg_free);
      }
      asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    }
  } else if (warp == FB_MMA_WARP) {
    const bool leader = elect_one();
    const uint32_t hi_w = (uint32_t)(smem_desc_sw128(0, 0, 1024) >> 32);
    const uint32_t k_lo = lo_kmajor(smem_u32(sK)), v_lo = lo_kmajor(smem_u32(sV)), k_mn = lo_mnmajor(smem_u32(sK));
    const uint32_t ds_mn = lo_mnmajor(smem_u32(sDS));
    const uint32_t ring16 = smem_u32(sRing) >> 4;
    constexpr uint32_t STAGE16 = (2 * SM::HALF_TILE) >> 4, HALF16 = SM::HALF_TILE >> 4, DS16 = SM::DS_TILE >> 4;
    const int n_sub = 2 * n_it;
    auto wait_all = [&](uint64_t* bar, uint32_t parity) -> bool {
      return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag));
    };
    auto issue_sdp = [&](int sub) {     // S^T = K Q^T and dP^T = V dO^T for 64 queries
      const int sb = sub & 1;
      const uint32_t idesc = idesc_bf16(64, 0, 0);
      const uint32_t qb = (ring16 + (sub % NST) * STAGE16) | (1u << 16), ob = qb + HALF16;
      if (leader) {
#pragma unroll
        for (int kk = 0; kk < DH / 16; ++kk)
          mma_ss_w(tmem_base + sb * 64, k_lo + kk * 2, hi_w, qb + kk * 2, hi_w, idesc, kk != 0);
#pragma unroll
        for (int kk = 0; kk < DH / 16; ++kk)
          mma_ss_w(tmem_base + 128 + sb * 64, v_lo + kk * 2, hi_w, ob + kk * 2, hi_w, idesc, kk != 0);
        mma_commit(&sdp_full[sb]);
      }
    };
    auto issue_dvdk = [&](int sub) {    // dV += P^T dO, dK += dS^T Q over the sub-tile's 64 queries
      const int sb = sub & 1, st = sub % NST;
      const uint32_t idesc = idesc_bf16(DH, 0, 1);
      const uint32_t qb = (ring16 + st * STAGE16) | ((8192u >> 4) << 16), ob = qb + HALF16;
      if (leader) {
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)
          mma_ts_w(tmem_base + 256, tmem_base + sb * 64 + (kk >> 1) * 32 + (kk & 1) * 8, ob + kk * (2048 >> 4), hi_w, idesc,
                   (sub | kk) != 0);
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)
          mma_ts_w(tmem_base + 320, tmem_base + 128 + sb * 64 + (kk >> 1) * 32 + (kk & 1) * 8, qb + kk * (2048 >> 4), hi_w,
                   idesc, (sub | kk) != 0);
        mma_commit(&qdo_empty[st]);
      }
    };
    auto issue_dq = [&](int it) {       // dQ_tile = dS K: A = dS^T tile read with the queries as M, B = K tile rows
      const int buf = it & 1;
      const uint32_t idesc = idesc_bf16(DH, 1, 1);
      if (leader) {
#pragma unroll
        for (int kk = 0; kk < 8; ++kk)
          mma_ss_w(tmem_base + 384 + buf * 64, ds_mn + buf * DS16 + kk * (2048 >> 4), hi_w, k_mn + kk * (2048 >> 4), hi_w, idesc,
                   kk != 0);
        mma_commit(&dq_full[buf]);
        mma_commit(&ds_free[buf]);
      }
    };
    if (!wait_all(kv_full, 0)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
    for (int s0 = 0; s0 < 2 && s0 < n_sub; ++s0) {
      if (!wait_all(&qdo_full[s0 % NST], (s0 / NST) & 1)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
      tc_fence_after();
      issue_sdp(s0);
    }
    for (int sub = 0; sub < n_sub; ++sub) {
      if (!wait_all(&pds_full[sub & 1], (sub >> 1) & 1)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
      tc_fence_after();
      issue_dvdk(sub);
      if (sub + 2 < n_sub) {
        const int nx = sub + 2;
        if (!wait_all(&qdo_full[nx % NST], (nx / NST) & 1)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
        tc_fence_after();
        issue_sdp(nx);
      }
      if (sub & 1) {
        const int it = sub >> 1;
        if (!wait_all(&dq_empty[it & 1], ((it >> 1) & 1) ^ 1)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
        tc_fence_after();
        issue_dq(it);
      }
    }
    if (leader) mma_commit(acc_done);
  } else {
    // ------------------------------------------------------------------ compute, thread = key
    // Two groups of four warps; group gsel owns the sub-tile of queries [64 gsel, 64 gsel + 64) of every query tile (TMEM
    // buffer gsel) and a thread all 64 of its key's scores there, in quarters of 16 with the next quarter's TMEM loads
    // in flight during the arithmetic (few warps with many independent chains each, instead of many short ones).
    const int gsel = warp >> 2;
    const int row = (warp & 3) * 32 + lane;
    const int ct = threadIdx.x & 127;
    const uint32_t lane_sel = (uint32_t)((warp & 3) * 32) << 16;
    const int tk = n0 + row;
    const float c_scale = rsqrtf((float)DH) * FB_LOG2E;
    const float q_scale = rsqrtf((float)DH);
    float* gstat = stat + gsel * 512;                  // [2 buffers][-lse2 | -delta][128 queries]
    auto fetch_stat = [&](int it, float& nl, float& nd) {
      const int hi = hj * p.g + it / n_q, m0 = (i0 + it % n_q) * 128;
      const int tq = m0 + ct;
      const long long idx = ((long long)b * p.hq + hi) * p.S + tq;
      nl = tq < p.S ? -p.lse[idx] * FB_LOG2E : -INFINITY;
      nd = tq < p.S ? -p.delta[idx] : 0.f;
    };
    // hands the finished dQ of iteration `it` (its TMEM buffer) to the reduction lane: thread = query row, 32 channels,
    // written into the fp32 stage (rows of 128 bytes, 128-byte swizzle; box gsel = channels [32 gsel, 32 gsel + 32))
    unsigned char* stg_row = smem + SM::DQ_OFF + gsel * 16384 + row * 128;
    // The finished dQ of iteration `it` goes from its TMEM buffer to the fp32 stage: flush_load (wait for the contraction,
    // issue the load) and, after a tcgen05.wait::ld, flush_store (release the buffer, wait for the stage, write it, hand it
    // to the reduction lane).
    auto flush_load = [&](int it, uint32_t (&t)[32]) -> bool {
      const int buf = it & 1;
      if (!mbar_wait(&dq_full[buf], (it >> 1) & 1, abort_flag)) return false;
      tc_fence_after();
      tmem_ld32(tmem_base + lane_sel + 384 + buf * 64 + gsel * 32, t);
      return true;
    };
    auto flush_store = [&](int it, const uint32_t (&t)[32]) -> bool {
      tc_fence_before();
      mbar_arrive(&dq_empty[it & 1]);
      if (!mbar_wait(stg_free, (it & 1) ^ 1, abort_flag)) return false;     // the previous tile has left the stage
#pragma unroll
      for (int i = 0; i < 8; ++i)
        *reinterpret_cast<float4*>(stg_row + ((i ^ (row & 7)) << 4)) =
            make_float4(__uint_as_float(t[4 * i]) * q_scale, __uint_as_float(t[4 * i + 1]) * q_scale,
                        __uint_as_float(t[4 * i + 2]) * q_scale, __uint_as_float(t[4 * i + 3]) * q_scale);
      fence_proxy_async();
      mbar_arrive(stg_full);
      return true;
    };
    float next_nl = 0.f, next_nd = 0.f;
    if (n_it > 0) fetch_stat(0, next_nl, next_nd);
    const uint64_t scale2 = pack2f(c_scale, c_scale);
    const uint32_t s_t = tmem_base + lane_sel + gsel * 64;
    const uint32_t dp_t = tmem_base + lane_sel + 128 + gsel * 64;
    const int qoff = gsel * 64;                        // first query (within the tile) of this thread's columns
    unsigned char* ds_row = sDS + gsel * 16384 + row * 128;      // this thread's 128-byte row of dS^T, box gsel
    for (int it = 0; it < n_it; ++it) {
      const int stb = it & 1;
      gstat[stb * 256 + ct] = next_nl;
      gstat[stb * 256 + 128 + ct] = next_nd;
      if (it + 1 < n_it) fetch_stat(it + 1, next_nl, next_nd);
      mbar_arrive(&stat_ready[gsel]);
      if (!mbar_wait(&stat_ready[gsel], it & 1, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_SOFTMAX); goto done; }
      const int m0 = (i0 + it % n_q) * 128;
      const bool diag = p.causal && m0 == n0;
      // the dS^T tile of two iterations ago must have been read by its dQ contraction
      if (!mbar_wait(&ds_free[stb], ((it >> 1) & 1) ^ 1, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_SOFTMAX); goto done; }
      if (!mbar_wait(&sdp_full[gsel], it & 1, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_SOFTMAX); goto done; }
      tc_fence_after();
      const ulonglong2* nlv = reinterpret_cast<const ulonglong2*>(gstat + stb * 256 + qoff);
      const ulonglong2* ndv = reinterpret_cast<const ulonglong2*>(gstat + stb * 256 + 128 + qoff);
      unsigned char* dsb = ds_row + stb * SM::DS_TILE;
      // the whole tile's arithmetic in one basic block: the diagonal tile's masking is a compile-time variant, not a branch
      // per group of four scores (a branch there ends the scheduler's window)
      auto tile_math = [&](auto diag_c) {
      constexpr bool DIAG = decltype(diag_c)::value;
      uint32_t sv[2][16], dv[2][16];
      ulonglong2 nlq[2][4], ndq[2][4];                 // this quarter's and the next one's column statistics
      tmem_ld16(s_t, sv[0]);
      tmem_ld16(dp_t, dv[0]);
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        nlq[0][c] = nlv[c];
        ndq[0][c] = ndv[c];
      }
#pragma unroll
      for (int hf = 0; hf < 4; ++hf) {
        uint32_t pk[8], dk_[8];
        tmem_ld_wait();
        if (hf < 3) {
          tmem_ld16(s_t + (hf + 1) * 16, sv[(hf + 1) & 1]);
          tmem_ld16(dp_t + (hf + 1) * 16, dv[(hf + 1) & 1]);
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            nlq[(hf + 1) & 1][c] = nlv[(hf + 1) * 4 + c];
            ndq[(hf + 1) & 1][c] = ndv[(hf + 1) * 4 + c];
          }
        }
        const uint32_t(&sq)[16] = sv[hf & 1];
        const uint32_t(&dq_)[16] = dv[hf & 1];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const ulonglong2 nl = nlq[hf & 1][c], nd = ndq[hf & 1][c];
          uint64_t e0 = fma2(pack2u(sq[4 * c + 0], sq[4 * c + 1]), scale2, nl.x);
          uint64_t e1 = fma2(pack2u(sq[4 * c + 2], sq[4 * c + 3]), scale2, nl.y);
          e0 = (2 * c & 3) < POLY ? exp2_pair<true>(e0) : exp2_pair<false>(e0);
          e1 = ((2 * c + 1) & 3) < POLY ? exp2_pair<true>(e1) : exp2_pair<false>(e1);
          if (DIAG) {
            const int q0 = m0 + qoff + hf * 16 + 4 * c;
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
          dk_[2 * c] = cvt_bf16x2(mul2(e0, add2(pack2u(dq_[4 * c + 0], dq_[4 * c + 1]), nd.x)));
          dk_[2 * c + 1] = cvt_bf16x2(mul2(e1, add2(pack2u(dq_[4 * c + 2], dq_[4 * c + 3]), nd.y)));
        }
        // 16 queries = k-step hf of the dV / dK contractions: 8 columns at (hf >> 1) * 32 + (hf & 1) * 8, all of them
        // columns this thread has already read
        tmem_st8(s_t + (hf >> 1) * 32 + (hf & 1) * 8, pk);
        tmem_st8(dp_t + (hf >> 1) * 32 + (hf & 1) * 8, dk_);
        // the same dS^T values for the dQ contraction: 16-byte chunks 2 hf, 2 hf + 1 of the row (swizzled)
        *reinterpret_cast<uint4*>(dsb + (((2 * hf) ^ (row & 7)) << 4)) = make_uint4(dk_[0], dk_[1], dk_[2], dk_[3]);
        *reinterpret_cast<uint4*>(dsb + (((2 * hf + 1) ^ (row & 7)) << 4)) = make_uint4(dk_[4], dk_[5], dk_[6], dk_[7]);
      }
      };
      if (diag) tile_math(std::true_type{}); else tile_math(std::false_type{});
      tmem_st_wait();
      tc_fence_before();
      fence_proxy_async();                             // shared-memory writes -> visible to the tensor core
      mbar_arrive(&pds_full[gsel]);
      // the previous tile's dQ leaves while the tensor core works on this sub-tile's contractions
      if (it >= 1) {
        uint32_t t[32];
        bool ok = flush_load(it - 1, t);
        tmem_ld_wait();
        if (ok) ok = flush_store(it - 1, t);
        if (!ok) { fail(abort_flag, p.status, ST_TIMEOUT_SOFTMAX); goto done; }
      }
    }
    if (n_it > 0) {
      uint32_t t[32];
      bool ok = flush_load(n_it - 1, t);
      tmem_ld_wait();
      if (ok) ok = flush_store(n_it - 1, t);
      if (!ok) { fail(abort_flag, p.status, ST_TIMEOUT_EPI); goto done; }
    }
    if (!mbar_wait(acc_done, 0, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_EPI); goto done; }
    tc_fence_after();
    {
      uint32_t t[32], u[32];
      const int col = gsel * 32;
      tmem_ld32(tmem_base + lane_sel + 256 + col, t);
      tmem_ld32(tmem_base + lane_sel + 320 + col, u);
      tmem_ld_wait();
      if (tk < p.S) {
        const long long off = ((long long)b * p.S + tk) * p.Lk + hj * DH + col;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          reinterpret_cast<float4*>(p.dv + off)[i] = make_float4(__uint_as_float(t[4 * i]), __uint_as_float(t[4 * i + 1]),
                                                                  __uint_as_float(t[4 * i + 2]), __uint_as_float(t[4 * i + 3]));
          reinterpret_cast<float4*>(p.dk + off)[i] =
              make_float4(__uint_as_float(u[4 * i]) * q_scale, __uint_as_float(u[4 * i + 1]) * q_scale,
                          __uint_as_float(u[4 * i + 2]) * q_scale, __uint_as_float(u[4 * i + 3]) * q_scale);
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
  if (warp == FB_MMA_WARP) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

template <int POLY>
int launch_fused(TcState* s, const CcaDims& d, const CUtensorMap& tmQh, const CUtensorMap& tmK, const CUtensorMap& tmV,
                 const CUtensorMap& tmDOh, const CUtensorMap& tmDQ, const FbParams& p, cudaStream_t st) {
  static bool attr_set[TC_MAX_DEVICES] = {};
  if (!attr_set[s->device]) {
    cudaError_t e = cudaFuncSetAttribute(tc_attn_bwd_fused_kernel<POLY>, cudaFuncAttributeMaxDynamicSharedMemorySize, FbSmem::TOTAL);
    if (e != cudaSuccess) return -(int)e;
    attr_set[s->device] = true;
  }
  const long long g_kv = (long long)p.n_tiles * d.B * d.hk;
  if (g_kv > 0x7fffffffLL) return 1;
  cudaError_t e = cudaMemsetAsync(p.dq, 0, (size_t)d.B * d.S * d.Lq * sizeof(float), st);
  if (e != cudaSuccess) return -(int)e;
  tc_attn_bwd_fused_kernel<POLY><<<(unsigned)g_kv, FB_THREADS, FbSmem::TOTAL, st>>>(tmQh, tmK, tmV, tmDOh, tmDQ, p);
  e = cudaGetLastError();
  return e == cudaSuccess ? 0 : -(int)e;
}

}  // namespace

// Head size 64 only.  delta must already hold rowsum(dO o O).  Returns 0 if the work was enqueued (a memset of dq and one
// kernel), 1 if the case is not covered.
int tc_attn_bwd_fused(TcState* s, const CcaDims& d, const bf16* q, const bf16* k, const bf16* v, const bf16* d_o,
                      const float* lse, const float* delta, float* dq, float* dk, float* dv, int* d_status, cudaStream_t st) {
  if (!s || !s->encode) return 1;
  if (d.dh != 64) return 1;
  if (d.Lq % 8 || d.Lk % 8) return 1;
  if (reinterpret_cast<uintptr_t>(dq) & 15) return 1;
  CUtensorMap tmK, tmV, tmQh, tmDOh;
  const uint64_t S = (uint64_t)d.S, B = (uint64_t)d.B, Lq = (uint64_t)d.Lq, Lk = (uint64_t)d.Lk;
  if (!tc_make_map_3d(s, &tmQh, q, Lq, S, B, Lq, S * Lq, 64, 64)) return 1;
  if (!tc_make_map_3d(s, &tmDOh, d_o, Lq, S, B, Lq, S * Lq, 64, 64)) return 1;
  if (!tc_make_map_3d(s, &tmK, k, Lk, S, B, Lk, S * Lk, 64, 128)) return 1;
  if (!tc_make_map_3d(s, &tmV, v, Lk, S, B, Lk, S * Lk, 64, 128)) return 1;
  CUtensorMap tmDQ;       // fp32 dq [B][S][Lq]: boxes of 128 rows x 32 channels for the reductions
  {
    cuuint64_t dims[3] = {(cuuint64_t)Lq, (cuuint64_t)S, (cuuint64_t)B};
    cuuint64_t strides[2] = {(cuuint64_t)Lq * 4, (cuuint64_t)S * Lq * 4};
    cuuint32_t box[3] = {32, 128, 1}, estr[3] = {1, 1, 1};
    if (s->encode(&tmDQ, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, dq, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return 1;
  }
  FbParams p;
  p.B = d.B; p.S = d.S; p.hq = d.hq; p.hk = d.hk; p.g = d.g; p.Lq = d.Lq; p.Lk = d.Lk; p.causal = d.causal;
  p.lse = lse; p.delta = delta; p.dq = dq; p.dk = dk; p.dv = dv;
  p.n_tiles = (d.S + 127) / 128;
  p.status = d_status;
  // all exponentials on the transcendental unit measured best here (0.482 ms; 0.488 / 0.500 with one / two of every four
  // pairs on the FMA pipe)
  const int poly = s->attn_poly_bwd < 0 ? 0 : s->attn_poly_bwd;
  if (poly == 0) return launch_fused<0>(s, d, tmQh, tmK, tmV, tmDOh, tmDQ, p, st);
  if (poly == 1) return launch_fused<1>(s, d, tmQh, tmK, tmV, tmDOh, tmDQ, p, st);
  return launch_fused<2>(s, d, tmQh, tmK, tmV, tmDOh, tmDQ, p, st);
}
