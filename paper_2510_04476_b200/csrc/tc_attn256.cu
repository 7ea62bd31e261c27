// Tensor-core kernels, part 7: forward softmax attention in the latent (Eq. 11) for head size 256.
// With d_h = 256 the output accumulator alone takes 256 of the 512 TMEM columns, so a CTA owns ONE 128-row query
// tile of one (sequence, query head) and ping-pongs two score buffers over consecutive key tiles instead of over two
// query tiles: while the softmax warps work on S_j, the tensor core computes S_{j+1} and O += P_{j-1} V_{j-1}.
//
//   warps 0-15 : softmax + epilogue (thread = query row = TMEM lane; warps 4p..4p+3 take score columns [32p, 32p+32))
//   warp  16   : TMA loader: Q once (64 KB), then K and V tiles as 32 KB halves (128 keys x 128 channels) through one
//                5-slot ring in the order K_j[0:128) K_j[128:256) V_j[0:128) V_j[128:256)
//   warp  17   : TMEM owner and MMA issuer
//
// TMEM columns: S0 [0,128) S1 [128,256) O [256,512).  P (bf16) overwrites its own S columns and is the TMEM operand
// of O += P V.  Softmax as in the 64 / 128 kernel: fixed maximum from the norm bound when q and k are normalised,
// online form with a lazy rescale otherwise; row sums over the rounded probabilities.
#include "tc_attn_common.cuh"
#include "tc_kernels.cuh"
#include "tc_ptx.cuh"
#include "tc_state.cuh"

using namespace tc;

namespace {

constexpr int A6_SOFTMAX_WARPS = 16;
constexpr int A6_TMA_WARP = A6_SOFTMAX_WARPS, A6_MMA_WARP = A6_SOFTMAX_WARPS + 1;
constexpr int A6_THREADS = 32 * (A6_SOFTMAX_WARPS + 2);
constexpr int DH6 = 256, BQ6 = 128, BKV6 = 128;
constexpr int GR_BYTES = 128 * 128 * 2;           // one ring granule: 128 rows x 128 channels (two 64-channel boxes)
constexpr int A6_NS = 5;
constexpr int A6_Q_OFF = 0;
constexpr int A6_KV_OFF = 2 * GR_BYTES;
constexpr int A6_BAR_OFF = A6_KV_OFF + A6_NS * GR_BYTES;
constexpr int A6_XCH_OFF = A6_BAR_OFF + 256;
constexpr int A6_TOTAL = A6_XCH_OFF + 2048;

template <int POLY>
__global__ void __launch_bounds__(A6_THREADS, 1)
tc_attn_fwd256_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                      const __grid_constant__ CUtensorMap tmV, AttnParams p) {
  extern __shared__ __align__(1024) unsigned char smem_dyn[];
  unsigned char* smem = smem_dyn;
  if (smem_u32(smem) & 1023u) {
    if (threadIdx.x == 0) atomicCAS(p.status, 0, ST_BAD_SMEM_ALIGNMENT);
    return;
  }
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + A6_BAR_OFF);
  uint64_t* q_full = bars;                    // [1]
  uint64_t* g_full = bars + 1;                // [NS]  granule n of the sequence lives in slot n % NS
  uint64_t* g_empty = g_full + A6_NS;         // [NS]
  uint64_t* s_full = g_empty + A6_NS;         // [2]  MMA -> softmax: S buffer ready
  uint64_t* p_full = s_full + 2;              // [2 buffers][2]  softmax -> MMA: first / second 16 keys of every thread's P
  uint64_t* pv_done = p_full + 4;             // [1]  MMA -> softmax: O += P_j V_j finished (completes once per key tile)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(pv_done + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // work item: heavy (late) query tiles first
  const int per_blk = p.B * p.hq;
  const int blk = p.n_blocks - 1 - (int)(blockIdx.x / per_blk);
  const int rem = blockIdx.x % per_blk;
  const int b = rem / p.hq, hi = rem % p.hq, hj = hi / p.g;
  const int m0 = blk * BQ6;
  const int n_kv_total = (p.S + BKV6 - 1) / BKV6;
  const int n_kv = p.causal ? min(n_kv_total, m0 / BKV6 + 1) : n_kv_total;

  if (threadIdx.x == 0) {
    mbar_init(q_full, 1);
    for (int i = 0; i < A6_NS; ++i) {
      mbar_init(&g_full[i], 1);
      mbar_init(&g_empty[i], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&s_full[i], 1);
      mbar_init(&p_full[2 * i], 512);
      mbar_init(&p_full[2 * i + 1], 512);
    }
    mbar_init(pv_done, 1);
    wait_ctl_init(abort_flag, p.status);
    fence_barrier_init();
    prefetch_tmap(&tmQ);
    prefetch_tmap(&tmK);
    prefetch_tmap(&tmV);
  }
  if (warp == A6_MMA_WARP) {
    tmem_alloc(tmem_slot, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == A6_TMA_WARP) {
    // ---------------------------------------------------------------- TMA loader
    if (lane == 0) {
      mbar_expect_tx(q_full, 2 * GR_BYTES);
#pragma unroll
      for (int c = 0; c < 4; ++c) tma_load_3d(smem + A6_Q_OFF + c * 16384, &tmQ, hi * DH6 + c * 64, m0, b, q_full);
      for (int n = 0; n < 4 * n_kv; ++n) {
        const int j = n >> 2, kind = n & 3, sl = n % A6_NS;
        const uint32_t ph = (n / A6_NS) & 1;
        if (!mbar_wait(&g_empty[sl], ph ^ 1, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_TMA); goto done; }
        mbar_expect_tx(&g_full[sl], GR_BYTES);
#pragma unroll
        for (int c = 0; c < 2; ++c)
          tma_load_3d(smem + A6_KV_OFF + sl * GR_BYTES + c * 16384, (kind & 2) ? &tmV : &tmK,
                      hj * DH6 + (kind & 1) * 128 + c * 64, j * BKV6, b, &g_full[sl]);
      }
    }
  } else if (warp == A6_MMA_WARP) {
    // ---------------------------------------------------------------- MMA issuer (warp-uniform loop, elected lane)
    const bool leader = elect_one();
    const uint32_t idesc = idesc_bf16(128, 0, 0);          // S: N = 128 keys
    const uint32_t idesc_o = idesc_bf16(128, 0, 1);        // O halves: N = 128 channels, V is the MN-major operand
    const uint32_t desc_hi = (uint32_t)(smem_desc_sw128(0, 0, 1024) >> 32);
    const uint32_t q_lo = (smem_u32(smem + A6_Q_OFF) >> 4) | (1u << 16);
    const uint32_t k_lo = (smem_u32(smem + A6_KV_OFF) >> 4) | (1u << 16);
    const uint32_t v_lo = (smem_u32(smem + A6_KV_OFF) >> 4) | ((16384u >> 4) << 16);
    constexpr uint32_t GR16 = GR_BYTES >> 4;
    auto wait_all = [&](uint64_t* bar, uint32_t parity) -> bool {
      return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag));
    };
    auto wait_granule = [&](int n) -> bool { return wait_all(&g_full[n % A6_NS], (n / A6_NS) & 1); };
    auto commit = [&](uint64_t* bar) {
      if (leader) mma_commit(bar);
    };
    auto issue_s = [&](int j) {             // S_{j & 1} = Q K_j^T, 16 k-steps over the two channel halves
      if (leader) {
#pragma unroll
        for (int kk = 0; kk < 16; ++kk) {
          const int g = kk >> 3, k8 = kk & 7;
          const uint32_t off = (uint32_t)(((k8 >> 2) * 16384 + (k8 & 3) * 32) >> 4);
          mma_ss_w(tmem_base + (j & 1) * 128, q_lo + g * GR16 + off, desc_hi, k_lo + ((4 * j + g) % A6_NS) * GR16 + off, desc_hi,
                   idesc, kk != 0);
        }
      }
    };
    auto issue_pv = [&](int j, int hf) {    // O (+)= P_j V_j over the keys of chunk hf, both channel halves
      if (leader) {
#pragma unroll
        for (int gv = 0; gv < 2; ++gv) {
          const uint32_t va = v_lo + ((4 * j + 2 + gv) % A6_NS) * GR16;
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int kk = 2 * i + hf;
            mma_ts_w(tmem_base + 256 + gv * 128, tmem_base + (j & 1) * 128 + (kk >> 1) * 32 + (kk & 1) * 8, va + kk * (2048 >> 4),
                     desc_hi, idesc_o, (j | hf | i) != 0);
          }
        }
      }
    };
    if (n_kv > 0) {
      if (!wait_all(q_full, 0)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
      for (int j = 0; j < 2 && j < n_kv; ++j) {
        if (!wait_granule(4 * j) || !wait_granule(4 * j + 1)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
        tc_fence_after();
        issue_s(j);
        commit(&s_full[j & 1]);
        commit(&g_empty[(4 * j) % A6_NS]);
        commit(&g_empty[(4 * j + 1) % A6_NS]);
      }
    }
    for (int j = 0; j < n_kv; ++j) {
      const int bf = j & 1;
      const uint32_t ph = (j >> 1) & 1;
      if (!wait_all(&p_full[2 * bf], ph)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
      if (!wait_granule(4 * j + 2) || !wait_granule(4 * j + 3)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
      tc_fence_after();
      issue_pv(j, 0);
      if (!wait_all(&p_full[2 * bf + 1], ph)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
      tc_fence_after();
      issue_pv(j, 1);
      commit(&g_empty[(4 * j + 2) % A6_NS]);
      commit(&g_empty[(4 * j + 3) % A6_NS]);
      commit(pv_done);
      if (j + 2 < n_kv) {
        // S_{j+2} goes into the buffer P_j has just been read from (the tensor pipe runs its MMAs in order)
        if (!wait_granule(4 * j + 8) || !wait_granule(4 * j + 9)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
        tc_fence_after();
        issue_s(j + 2);
        commit(&s_full[bf]);
        commit(&g_empty[(4 * j + 8) % A6_NS]);
        commit(&g_empty[(4 * j + 9) % A6_NS]);
      }
    }
  } else {
    // ---------------------------------------------------------------- softmax + epilogue
    const int part = warp >> 2;                      // which 32 score columns of each key tile
    const int row = (warp & 3) * 32 + lane;
    const uint32_t lane_sel = (uint32_t)((warp & 3) * 32) << 16;
    float* xch = reinterpret_cast<float*>(smem + A6_XCH_OFF);      // [4 parts][128 rows]
    auto sync_softmax = [&]() { asm volatile("bar.sync 1, 512;" ::: "memory"); };
    const float c_scale = rsqrtf((float)DH6) * LOG2E_F;
    float m_fixed = 0.f;
    bool fixed = false;
    if (p.temp != nullptr) {
      m_fixed = sqrtf((float)DH6) * __expf(p.temp[hj]) * LOG2E_F * 1.01f;
      fixed = m_fixed <= 56.f;
    }
    const uint64_t scale2 = pack2f(c_scale, c_scale);
    float m_run = fixed ? m_fixed : -INFINITY, l_run = 0.f;
    const uint32_t o_tmem = tmem_base + lane_sel + 256;
    const int tq = m0 + row;
    for (int j = 0; j < n_kv; ++j) {
      const int bf = j & 1;
      const uint32_t s_tmem = tmem_base + lane_sel + bf * 128 + part * 32;   // this thread's 32 S columns
      if (!mbar_wait(&s_full[bf], (j >> 1) & 1, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_SOFTMAX); goto done; }
      tc_fence_after();
      const int k0 = j * BKV6 + part * 32;
      const bool need_mask = (p.causal && j * BKV6 + BKV6 - 1 > m0) || (j * BKV6 + BKV6 > p.S);
      const int lim = p.causal ? min(tq, p.S - 1) : p.S - 1;       // last visible key
      float m_use = m_run;
      if (!fixed) {
        float mx = -INFINITY;
        {
          uint32_t v[32];
          tmem_ld32(s_tmem, v);
          tmem_ld_wait();
#pragma unroll
          for (int c = 0; c < 32; ++c)
            if (!need_mask || k0 + c <= lim) mx = fmaxf(mx, __uint_as_float(v[c]));
        }
        xch[part * 128 + row] = mx;
        sync_softmax();
        mx = fmaxf(fmaxf(xch[row], xch[128 + row]), fmaxf(xch[256 + row], xch[384 + row])) * c_scale;
        sync_softmax();
        const bool grow = mx > m_run + RESCALE_THRESHOLD;        // also true on the first tile
        if (grow) m_use = mx;
        if (m_use == -INFINITY) m_use = 0.f;
        if (j > 0 && __any_sync(0xffffffffu, grow)) {
          // rescale this thread's quarter of the running output (rare); O must not be in use by P_{j-1} V_{j-1}
          if (!mbar_wait(pv_done, (j - 1) & 1, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_SOFTMAX); goto done; }
          tc_fence_after();
          const float alpha = grow ? exp2f(m_run - m_use) : 1.f;
          l_run *= alpha;
#pragma unroll 1
          for (int c = 0; c < DH6 / 64; ++c) {
            uint32_t t[16];
            tmem_ld16(o_tmem + part * (DH6 / 4) + c * 16, t);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 16; ++i) t[i] = __float_as_uint(__uint_as_float(t[i]) * alpha);
            tmem_st16(o_tmem + part * (DH6 / 4) + c * 16, t);
          }
          tmem_st_wait();
        }
        m_run = m_use;
      }
      const uint64_t negm2 = pack2f(-m_use, -m_use);
      uint64_t sum2 = pack2f(0.f, 0.f);
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
        uint32_t v[16], pk[8];
        tmem_ld16(s_tmem + hf * 16, v);
        tmem_ld_wait();
        if (need_mask) {
#pragma unroll
          for (int c = 0; c < 16; ++c)
            if (k0 + hf * 16 + c > lim) v[c] = 0xff800000u;        // -inf
#pragma unroll
          for (int c = 0; c < 2; ++c) exp8<0, false>(&v[8 * c], scale2, negm2, sum2, &pk[4 * c]);
        } else if (fixed) {
#pragma unroll
          for (int c = 0; c < 2; ++c) exp8<POLY, false>(&v[8 * c], scale2, negm2, sum2, &pk[4 * c]);
        } else {
#pragma unroll
          for (int c = 0; c < 2; ++c) exp8<POLY, true>(&v[8 * c], scale2, negm2, sum2, &pk[4 * c]);
        }
        tmem_st8(s_tmem + hf * 8, pk);
        tmem_st_wait();
        tc_fence_before();
        mbar_arrive(&p_full[2 * bf + hf]);
      }
      {
        uint32_t a, b2;
        unpack2u(sum2, a, b2);
        l_run += __uint_as_float(a) + __uint_as_float(b2);
      }
    }
    if (n_kv > 0) {
      sync_softmax();
      xch[part * 128 + row] = l_run;
      sync_softmax();
      const float l_tot = (xch[row] + xch[128 + row]) + (xch[256 + row] + xch[384 + row]);
      if (!mbar_wait(pv_done, (n_kv - 1) & 1, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_EPI); goto done; }
      tc_fence_after();
      const float inv_l = 1.f / l_tot;
      const long long row_g = (long long)b * p.S + tq;
#pragma unroll 1
      for (int c = 0; c < DH6 / 64; ++c) {
        uint32_t t[16];
        const int col = part * (DH6 / 4) + c * 16;
        tmem_ld16(o_tmem + col, t);
        tmem_ld_wait();
        if (tq < p.S) {
          bf16* dst = p.o + row_g * p.Lq + hi * DH6 + col;
#pragma unroll
          for (int i = 0; i < 2; ++i) {
            uint4 w;
            w.x = pack_bf16(__uint_as_float(t[8 * i + 0]) * inv_l, __uint_as_float(t[8 * i + 1]) * inv_l);
            w.y = pack_bf16(__uint_as_float(t[8 * i + 2]) * inv_l, __uint_as_float(t[8 * i + 3]) * inv_l);
            w.z = pack_bf16(__uint_as_float(t[8 * i + 4]) * inv_l, __uint_as_float(t[8 * i + 5]) * inv_l);
            w.w = pack_bf16(__uint_as_float(t[8 * i + 6]) * inv_l, __uint_as_float(t[8 * i + 7]) * inv_l);
            reinterpret_cast<uint4*>(dst)[i] = w;
          }
          if (p.o32) {
            float* d32 = p.o32 + row_g * p.Lq + hi * DH6 + col;
#pragma unroll
            for (int i = 0; i < 4; ++i)
              reinterpret_cast<float4*>(d32)[i] =
                  make_float4(__uint_as_float(t[4 * i]) * inv_l, __uint_as_float(t[4 * i + 1]) * inv_l,
                              __uint_as_float(t[4 * i + 2]) * inv_l, __uint_as_float(t[4 * i + 3]) * inv_l);
          }
        }
      }
      if (part == 0 && tq < p.S) p.lse[((long long)b * p.hq + hi) * p.S + tq] = (m_run + log2f(l_tot)) * LN2_F;
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
  if (warp == A6_MMA_WARP) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

template <int POLY>
int launch_attn256(TcState* s, const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV, const AttnParams& p,
                   unsigned grid, cudaStream_t st) {
  static bool attr_set[TC_MAX_DEVICES] = {};
  if (!attr_set[s->device]) {
    cudaError_t e = cudaFuncSetAttribute(tc_attn_fwd256_kernel<POLY>, cudaFuncAttributeMaxDynamicSharedMemorySize, A6_TOTAL);
    if (e != cudaSuccess) return -(int)e;
    attr_set[s->device] = true;
  }
  tc_attn_fwd256_kernel<POLY><<<grid, A6_THREADS, A6_TOTAL, st>>>(tmQ, tmK, tmV, p);
  cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? 0 : -(int)e;
}

}  // namespace

int tc_attn_fwd256(TcState* s, const CcaDims& d, const bf16* q, const bf16* k, const bf16* v, bf16* o, float* o32, float* lse,
                   const float* temp, int* d_status, cudaStream_t st) {
  if (!s || !s->encode) return 1;
  if (d.dh != 256) return 1;
  CUtensorMap tmQ, tmK, tmV;
  if (!tc_make_map_3d(s, &tmQ, q, (uint64_t)d.Lq, (uint64_t)d.S, (uint64_t)d.B, (uint64_t)d.Lq, (uint64_t)d.S * d.Lq, 64, 128))
    return 1;
  if (!tc_make_map_3d(s, &tmK, k, (uint64_t)d.Lk, (uint64_t)d.S, (uint64_t)d.B, (uint64_t)d.Lk, (uint64_t)d.S * d.Lk, 64, 128))
    return 1;
  if (!tc_make_map_3d(s, &tmV, v, (uint64_t)d.Lk, (uint64_t)d.S, (uint64_t)d.B, (uint64_t)d.Lk, (uint64_t)d.S * d.Lk, 64, 128))
    return 1;
  AttnParams p;
  p.B = d.B; p.S = d.S; p.hq = d.hq; p.hk = d.hk; p.g = d.g; p.Lq = d.Lq; p.Lk = d.Lk; p.causal = d.causal;
  p.o = o; p.o32 = o32; p.lse = lse;
  p.blk0 = 0;
  p.n_blocks = (d.S + BQ6 - 1) / BQ6;
  p.status = d_status;
  p.temp = temp;
  const long long grid = (long long)p.n_blocks * d.B * d.hq;
  if (grid > 0x7fffffffLL) return 1;
  // one exponential per 4 * 256 tensor FLOPs: the transcendental unit has time to spare, no polynomial share
  return launch_attn256<0>(s, tmQ, tmK, tmV, p, (unsigned)grid, st);
}
