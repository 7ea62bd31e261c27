// Tensor-core kernels, part 2: softmax attention in the latent (Eq. 11, softmax line) with grouped kv
// heads, forward.  One CTA owns 256 consecutive query rows of one (sequence, query head) as two
// 128-row tiles that ping-pong: while the softmax warps of one tile work on S = Q K^T, the tensor core
// runs the other tile's MMAs.
//
//   warps 0-3  : softmax + epilogue of query tile 0 (thread = query row = TMEM lane)
//   warps 4-7  : softmax + epilogue of query tile 1
//   warp  8    : TMA loader (Q tiles once, then a 2-stage ring of K and of V tiles)
//   warp  9    : TMEM owner and MMA issuer
//
// TMEM columns: S0 [0,128) S1 [128,256) O0 [256,256+DH) O1 [384,384+DH).  The bf16 probabilities P
// overwrite the first 64 columns of their S tile and feed the P V MMA directly from TMEM.
// Softmax is online with a lazy rescale: the running row maximum only moves (and O is only rescaled)
// when it grows by more than 2^8; with normalised q, k the logits are bounded by sqrt(d_h) * beta, so
// after the first tile this never happens.
#include "tc_kernels.cuh"
#include "tc_ptx.cuh"
#include "tc_state.cuh"

using namespace tc;

namespace {

constexpr int AT_THREADS = 320;
constexpr int BQ = 128, BKV = 128, KV_STAGES = 2;
constexpr float LOG2E_F = 1.4426950408889634f;
constexpr float LN2_F = 0.6931471805599453f;
constexpr float RESCALE_THRESHOLD = 8.0f;      // log2 units

struct AttnParams {
  int B, S, hq, hk, g, Lq, Lk, causal;
  bf16* o;
  float* o32;
  float* lse;
  int n_blocks;       // 256-row blocks per sequence
  int* status;
};

template <int DH>
struct AttnSmem {
  static constexpr int TILE_BYTES = 128 * DH * 2;            // one 128-row tile of Q, K or V
  static constexpr int Q_OFF = 0;
  static constexpr int K_OFF = 2 * TILE_BYTES;
  static constexpr int V_OFF = K_OFF + KV_STAGES * TILE_BYTES;
  static constexpr int BAR_OFF = V_OFF + KV_STAGES * TILE_BYTES;
  // at least 120 KB so that two CTAs (each wanting all 512 TMEM columns) never share an SM
  static constexpr int TOTAL = (BAR_OFF + 512 + 1024) > 122880 ? (BAR_OFF + 512 + 1024) : 122880;
};

TC_DEVINL void fail(volatile int* abort_flag, int* status, int code) {
  *abort_flag = 1;
  atomicCAS(status, 0, code);
}

// K-major operand tile [128 rows][DH] stored as DH/64 swizzled boxes of [128][64]: descriptor of the
// kk-th 16-element slice along the head dimension.
template <int DH>
TC_DEVINL uint64_t kmajor_desc(uint32_t tile_addr, int kk) {
  return smem_desc_sw128(tile_addr + (kk >> 2) * 16384 + (kk & 3) * 32, 16, 1024);
}
// V tile [128 keys][DH] (same storage) used as the MN-major B operand of O += P V: descriptor of the
// kk-th 16-key slice; 64-channel chunks are one box (16384 B) apart.
TC_DEVINL uint64_t v_desc(uint32_t tile_addr, int kk) { return smem_desc_sw128(tile_addr + kk * 2048, 16384, 1024); }

template <int DH>
__global__ void __launch_bounds__(AT_THREADS, 1)
tc_attn_fwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                   const __grid_constant__ CUtensorMap tmV, AttnParams p) {
  using SM = AttnSmem<DH>;
  constexpr int NBOX = DH / 64;
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + SM::BAR_OFF);
  uint64_t* q_full = bars;            // [2]
  uint64_t* k_full = bars + 2;        // [KV_STAGES]
  uint64_t* k_empty = bars + 4;
  uint64_t* v_full = bars + 6;
  uint64_t* v_empty = bars + 8;
  uint64_t* s_full = bars + 10;       // [2]  MMA -> softmax: S tile ready
  uint64_t* p_full = bars + 12;       // [2]  softmax -> MMA: P tile written
  uint64_t* o_done = bars + 14;       // [2]  MMA -> softmax: last P V finished
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 16);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // work item: heavy (late) query blocks first
  const int per_blk = p.B * p.hq;
  const int blk = p.n_blocks - 1 - (int)(blockIdx.x / per_blk);
  const int rem = blockIdx.x % per_blk;
  const int b = rem / p.hq, hi = rem % p.hq, hj = hi / p.g;
  const int n_kv_total = (p.S + BKV - 1) / BKV;
  int n_s[2];
#pragma unroll
  for (int s = 0; s < 2; ++s) {
    const int m0 = blk * 256 + s * BQ;
    if (m0 >= p.S) n_s[s] = 0;
    else n_s[s] = p.causal ? min(n_kv_total, m0 / BKV + 1) : n_kv_total;
  }
  const int n_max = max(n_s[0], n_s[1]);

  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(&q_full[i], 1);
      mbar_init(&k_full[i], 1);
      mbar_init(&k_empty[i], 1);
      mbar_init(&v_full[i], 1);
      mbar_init(&v_empty[i], 1);
      mbar_init(&s_full[i], 1);
      mbar_init(&p_full[i], 128);
      mbar_init(&o_done[i], 1);
    }
    *abort_flag = 0;
    fence_barrier_init();
    prefetch_tmap(&tmQ);
    prefetch_tmap(&tmK);
    prefetch_tmap(&tmV);
  }
  if (warp == 9) {
    tmem_alloc(tmem_slot, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 8) {
    // ---------------------------------------------------------------- TMA loader
    if (lane == 0) {
#pragma unroll
      for (int s = 0; s < 2; ++s) {
        if (n_s[s] == 0) continue;
        mbar_expect_tx(&q_full[s], SM::TILE_BYTES);
#pragma unroll
        for (int c = 0; c < NBOX; ++c)
          tma_load_3d(smem + SM::Q_OFF + s * SM::TILE_BYTES + c * 16384, &tmQ, hi * DH + c * 64, blk * 256 + s * BQ, b,
                      &q_full[s]);
      }
      for (int j = 0; j < n_max; ++j) {
        const int st = j & 1;
        const uint32_t ph = (j >> 1) & 1;
        if (!mbar_wait(&k_empty[st], ph ^ 1, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_TMA); goto done; }
        mbar_expect_tx(&k_full[st], SM::TILE_BYTES);
#pragma unroll
        for (int c = 0; c < NBOX; ++c)
          tma_load_3d(smem + SM::K_OFF + st * SM::TILE_BYTES + c * 16384, &tmK, hj * DH + c * 64, j * BKV, b, &k_full[st]);
        if (!mbar_wait(&v_empty[st], ph ^ 1, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_TMA); goto done; }
        mbar_expect_tx(&v_full[st], SM::TILE_BYTES);
#pragma unroll
        for (int c = 0; c < NBOX; ++c)
          tma_load_3d(smem + SM::V_OFF + st * SM::TILE_BYTES + c * 16384, &tmV, hj * DH + c * 64, j * BKV, b, &v_full[st]);
      }
    }
  } else if (warp == 9) {
    // ---------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      const uint32_t idesc_s = idesc_bf16(BKV, 0, 0);
      const uint32_t idesc_o = idesc_bf16(DH, 0, 1);
      const uint32_t q_addr = smem_u32(smem + SM::Q_OFF), k_addr = smem_u32(smem + SM::K_OFF),
                     v_addr = smem_u32(smem + SM::V_OFF);
      auto issue_s = [&](int s, int j) {      // S_s = Q_s K_j^T
        const uint32_t qa = q_addr + s * SM::TILE_BYTES, ka = k_addr + (j & 1) * SM::TILE_BYTES;
#pragma unroll
        for (int kk = 0; kk < DH / 16; ++kk)
          mma_ss(tmem_base + s * 128, kmajor_desc<DH>(qa, kk), kmajor_desc<DH>(ka, kk), idesc_s, kk != 0);
      };
      auto issue_pv = [&](int s, int j) {     // O_s (+)= P_s V_j
        const uint32_t va = v_addr + (j & 1) * SM::TILE_BYTES;
#pragma unroll
        for (int kk = 0; kk < BKV / 16; ++kk)
          mma_ts(tmem_base + 256 + s * 128, tmem_base + s * 128 + kk * 8, v_desc(va, kk), idesc_o, (j | kk) != 0);
      };
      // prologue: first S tile of each query tile
      if (n_max > 0) {
        if (!mbar_wait(&k_full[0], 0, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
        tc_fence_after();
#pragma unroll
        for (int s = 0; s < 2; ++s) {
          if (n_s[s] == 0) continue;
          if (!mbar_wait(&q_full[s], 0, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
          tc_fence_after();
          issue_s(s, 0);
          mma_commit(&s_full[s]);
        }
      }
      for (int j = 0; j < n_max; ++j) {
        const int st = j & 1;
        const uint32_t ph = (j >> 1) & 1;
        // all S(j) were issued before this point: release K_j when they complete
        mma_commit(&k_empty[st]);
        bool k_next_ready = false;
#pragma unroll
        for (int s = 0; s < 2; ++s) {
          if (j >= n_s[s]) continue;
          if (!mbar_wait(&p_full[s], j & 1, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
          if (!mbar_wait(&v_full[st], ph, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
          tc_fence_after();
          issue_pv(s, j);
          if (j + 1 < n_s[s]) {
            if (!k_next_ready) {
              if (!mbar_wait(&k_full[(j + 1) & 1], ((j + 1) >> 1) & 1, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
              tc_fence_after();
              k_next_ready = true;
            }
            issue_s(s, j + 1);
            mma_commit(&s_full[s]);
          } else {
            mma_commit(&o_done[s]);
          }
        }
        mma_commit(&v_empty[st]);
      }
    }
  } else {
    // ---------------------------------------------------------------- softmax + epilogue
    const int s = warp >> 2;                         // query tile of this warpgroup
    const int row = threadIdx.x & 127;
    const uint32_t lane_sel = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t s_tmem = tmem_base + lane_sel + s * 128;
    const uint32_t o_tmem = tmem_base + lane_sel + 256 + s * 128;
    const int m0 = blk * 256 + s * BQ;
    const int tq = m0 + row;
    const float c_scale = rsqrtf((float)DH) * LOG2E_F;
    float m_run = -INFINITY, l_run = 0.f;
    for (int j = 0; j < n_s[s]; ++j) {
      if (!mbar_wait(&s_full[s], j & 1, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_SOFTMAX); goto done; }
      tc_fence_after();
      uint32_t v[128];
      tmem_ld32(s_tmem + 0, *reinterpret_cast<uint32_t(*)[32]>(&v[0]));
      tmem_ld32(s_tmem + 32, *reinterpret_cast<uint32_t(*)[32]>(&v[32]));
      tmem_ld32(s_tmem + 64, *reinterpret_cast<uint32_t(*)[32]>(&v[64]));
      tmem_ld32(s_tmem + 96, *reinterpret_cast<uint32_t(*)[32]>(&v[96]));
      tmem_ld_wait();
      const int k0 = j * BKV;
      const bool need_mask = (p.causal && k0 + BKV - 1 > m0) || (k0 + BKV > p.S);
      if (need_mask) {
        const int lim = p.causal ? min(tq, p.S - 1) : p.S - 1;     // last visible key
#pragma unroll
        for (int c = 0; c < 128; ++c)
          if (k0 + c > lim) v[c] = 0xff800000u;                    // -inf
      }
      float mx = -INFINITY;
#pragma unroll
      for (int c = 0; c < 128; ++c) mx = fmaxf(mx, __uint_as_float(v[c]));
      mx *= c_scale;
      float m_use = m_run;
      const bool grow = mx > m_run + RESCALE_THRESHOLD;           // also true on the first tile
      if (grow) m_use = mx;
      if (m_use == -INFINITY) m_use = 0.f;
      if (j > 0 && __any_sync(0xffffffffu, grow)) {
        // rescale the running output of this warp's 32 rows (rare)
        const float alpha = grow ? exp2f(m_run - m_use) : 1.f;
        l_run *= alpha;
#pragma unroll 1
        for (int c = 0; c < DH / 32; ++c) {
          uint32_t t[32];
          tmem_ld32(o_tmem + c * 32, t);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 32; ++i) t[i] = __float_as_uint(__uint_as_float(t[i]) * alpha);
          tmem_st32(o_tmem + c * 32, t);
        }
        tmem_st_wait();
      }
      m_run = m_use;
      float sum = 0.f;
      uint32_t pk[64];
#pragma unroll
      for (int c = 0; c < 64; ++c) {
        const float p0 = exp2f(fmaf(__uint_as_float(v[2 * c]), c_scale, -m_use));
        const float p1 = exp2f(fmaf(__uint_as_float(v[2 * c + 1]), c_scale, -m_use));
        sum += p0 + p1;
        pk[c] = pack_bf16(p0, p1);
      }
      l_run += sum;
      tmem_st32(s_tmem + 0, *reinterpret_cast<uint32_t(*)[32]>(&pk[0]));
      tmem_st32(s_tmem + 32, *reinterpret_cast<uint32_t(*)[32]>(&pk[32]));
      tmem_st_wait();
      tc_fence_before();
      mbar_arrive(&p_full[s]);
    }
    if (n_s[s] > 0) {
      if (!mbar_wait(&o_done[s], 0, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_EPI); goto done; }
      tc_fence_after();
      const float inv_l = 1.f / l_run;
      const long long row_g = (long long)b * p.S + tq;
#pragma unroll 1
      for (int c = 0; c < DH / 32; ++c) {
        uint32_t t[32];
        tmem_ld32(o_tmem + c * 32, t);
        tmem_ld_wait();
        if (tq < p.S) {
          bf16* dst = p.o + row_g * p.Lq + hi * DH + c * 32;
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            uint4 w;
            w.x = pack_bf16(__uint_as_float(t[8 * i + 0]) * inv_l, __uint_as_float(t[8 * i + 1]) * inv_l);
            w.y = pack_bf16(__uint_as_float(t[8 * i + 2]) * inv_l, __uint_as_float(t[8 * i + 3]) * inv_l);
            w.z = pack_bf16(__uint_as_float(t[8 * i + 4]) * inv_l, __uint_as_float(t[8 * i + 5]) * inv_l);
            w.w = pack_bf16(__uint_as_float(t[8 * i + 6]) * inv_l, __uint_as_float(t[8 * i + 7]) * inv_l);
            reinterpret_cast<uint4*>(dst)[i] = w;
          }
          if (p.o32) {
            float* d32 = p.o32 + row_g * p.Lq + hi * DH + c * 32;
#pragma unroll
            for (int i = 0; i < 8; ++i)
              reinterpret_cast<float4*>(d32)[i] =
                  make_float4(__uint_as_float(t[4 * i]) * inv_l, __uint_as_float(t[4 * i + 1]) * inv_l,
                              __uint_as_float(t[4 * i + 2]) * inv_l, __uint_as_float(t[4 * i + 3]) * inv_l);
          }
        }
      }
      if (tq < p.S) p.lse[((long long)b * p.hq + hi) * p.S + tq] = (m_run + log2f(l_run)) * LN2_F;
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
  if (warp == 9) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

}  // namespace

int tc_attn_fwd(TcState* s, const CcaDims& d, const bf16* q, const bf16* k, const bf16* v, bf16* o, float* o32,
                float* lse, int* d_status, cudaStream_t st) {
  if (!s || !s->encode) return 1;
  if (d.dh != 64 && d.dh != 128) return 1;
  if (d.Lq % 8 || d.Lk % 8) return 1;
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
  p.n_blocks = (d.S + 255) / 256;
  p.status = d_status;
  const long long grid = (long long)p.n_blocks * d.B * d.hq;
  if (grid > 0x7fffffffLL) return 1;
  cudaError_t e;
  if (d.dh == 128) {
    if (!s->attn_attr_set[1]) {
      e = cudaFuncSetAttribute(tc_attn_fwd_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttnSmem<128>::TOTAL);
      if (e != cudaSuccess) return -(int)e;
      s->attn_attr_set[1] = true;
    }
    tc_attn_fwd_kernel<128><<<(unsigned)grid, AT_THREADS, AttnSmem<128>::TOTAL, st>>>(tmQ, tmK, tmV, p);
  } else {
    if (!s->attn_attr_set[0]) {
      e = cudaFuncSetAttribute(tc_attn_fwd_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttnSmem<64>::TOTAL);
      if (e != cudaSuccess) return -(int)e;
      s->attn_attr_set[0] = true;
    }
    tc_attn_fwd_kernel<64><<<(unsigned)grid, AT_THREADS, AttnSmem<64>::TOTAL, st>>>(tmQ, tmK, tmV, p);
  }
  e = cudaGetLastError();
  return e == cudaSuccess ? 0 : -(int)e;
}
