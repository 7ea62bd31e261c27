// Tensor-core kernels, part 2: softmax attention in the latent (Eq. 11, softmax line) with grouped kv
// heads, forward.  One CTA owns 256 consecutive query rows of one (sequence, query head) as two
// 128-row tiles that ping-pong: while the softmax warps of one tile work on S = Q K^T, the tensor core
// runs the other tile's MMAs.
//
//   warps 0-15 : softmax + epilogue; all of them work on one query tile at a time, alternating between the
//                two tiles (thread = query row = TMEM lane; warps 4p..4p+3 take score columns [32p, 32p+32))
//   warp  16   : TMA loader (Q tiles once, then one ring shared by the K and V tiles)
//   warp  17   : TMEM owner and MMA issuer
//
// TMEM columns: S0 [0,128) S1 [128,256) O0 [256,256+DH) O1 [384,384+DH).  The bf16 probabilities P
// overwrite the first 16 of every 32 columns of their S tile and feed the P V MMA directly from TMEM.
// At d_h = 64 the columns behind each O tile are free, and the row sums of P are taken there by the tensor
// core as well (L0 [320,336) L1 [448,464): P times a block of ones, beside every P V step), which takes three
// of the seven instructions per score pair off the softmax threads.
// Softmax: with L2-normalised q and k (Eq. 11) every logit is bounded by sqrt(d_h) * beta, so that bound
// serves as a fixed row maximum: no max pass, no rescale of O (the kernel falls back to the online form,
// with a lazy rescale when the running maximum grows by more than 2^8, if the latents are not normalised
// or the bound is too loose for fp32).  One score costs 4 d_h tensor FLOPs and one exponential; at
// d_h = 128 the tensor pipe and the 16-per-clock transcendental unit would need the same time, so a
// fixed share of the exponentials is evaluated on the FMA pipe instead (round to integer + cubic for
// 2^f, |f| <= 1/2, relative error 7.5e-5, well under the bf16 rounding of P), two at a time with the
// packed f32x2 instructions.
#include "tc_attn_common.cuh"
#include "tc_kernels.cuh"
#include "tc_ptx.cuh"
#include "tc_state.cuh"

using namespace tc;

namespace {

constexpr int AT_SOFTMAX_WARPS = 16;                 // 2 query tiles x 2 column halves x 4 lane quarters
constexpr int AT_TMA_WARP = AT_SOFTMAX_WARPS, AT_MMA_WARP = AT_SOFTMAX_WARPS + 1;
constexpr int AT_THREADS = 32 * (AT_SOFTMAX_WARPS + 2);
constexpr int BQ = 128, BKV = 128;
template <int DH>
struct AttnSmem {
  static constexpr int TILE_BYTES = 128 * DH * 2;            // one 128-row tile of Q, K or V
  static constexpr int Q_OFF = 0;
  // K and V tiles share one ring, filled and released in the order K_0 V_0 K_1 V_1 ... (that is also the order
  // in which the MMAs finish with them): 5 slots at d_h = 128 fill the shared memory, 2.5 tiles of each ahead
  static constexpr int NSLOT = DH == 128 ? 5 : 8;
  static constexpr int KV_OFF = 2 * TILE_BYTES;
  static constexpr int BAR_OFF = KV_OFF + NSLOT * TILE_BYTES;
  static constexpr int XCH_OFF = BAR_OFF + 256;              // float [2 tiles][2 halves][128 rows]: max / sum exchange
  static constexpr int ONES_OFF = (XCH_OFF + 2048 + 1023) / 1024 * 1024;    // 2 KB of bf16 ones (row sums by MMA)
  static constexpr int USED = DH == 64 ? ONES_OFF + 2048 : XCH_OFF + 2048;
  // no slack for alignment: the kernel checks that its dynamic shared memory starts on a 1024-byte boundary.
  // At least 120 KB so that two CTAs (each wanting all 512 TMEM columns) never share an SM.
  static constexpr int TOTAL = USED > 122880 ? USED : 122880;
};

// K-major operand tile [128 rows][DH] stored as DH/64 swizzled boxes of [128][64]: descriptor of the
// kk-th 16-element slice along the head dimension.
template <int DH>
TC_DEVINL uint64_t kmajor_desc(uint32_t tile_addr, int kk) {
  return smem_desc_sw128(tile_addr + (kk >> 2) * 16384 + (kk & 3) * 32, 16, 1024);
}
// V tile [128 keys][DH] (same storage) used as the MN-major B operand of O += P V: descriptor of the
// kk-th 16-key slice; 64-channel chunks are one box (16384 B) apart.
TC_DEVINL uint64_t v_desc(uint32_t tile_addr, int kk) { return smem_desc_sw128(tile_addr + kk * 2048, 16384, 1024); }


// POLY8: of every 8 score pairs, how many take the polynomial exponential.
template <int DH, int POLY8>
__global__ void __launch_bounds__(AT_THREADS, 1)
tc_attn_fwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                   const __grid_constant__ CUtensorMap tmV, AttnParams p) {
  using SM = AttnSmem<DH>;
  constexpr int NBOX = DH / 64;
  constexpr int NS = SM::NSLOT;
  constexpr bool MSUM = DH == 64;       // row sums of P by the tensor core
  extern __shared__ __align__(1024) unsigned char smem_dyn[];
  unsigned char* smem = smem_dyn;
  if (smem_u32(smem) & 1023u) {       // the swizzled tiles need it; nothing has been set up yet, so just report
    if (threadIdx.x == 0) atomicCAS(p.status, 0, ST_BAD_SMEM_ALIGNMENT);
    return;
  }
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + SM::BAR_OFF);
  uint64_t* q_full = bars;            // [2]
  uint64_t* kv_full = bars + 2;       // [NS]  slot of the n-th tile of the sequence K_0 V_0 K_1 V_1 ...: n % NS
  uint64_t* kv_empty = bars + 2 + NS; // [NS]
  uint64_t* s_full = bars + 2 + 2 * NS;   // [2]  MMA -> softmax: S tile ready
  uint64_t* p_full = s_full + 2;      // [2 tiles][2]  softmax -> MMA: first / second 32 keys of every thread's P written
  uint64_t* o_done = p_full + 4;      // [2]  MMA -> softmax: last P V finished
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(o_done + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // work item: heavy (late) query blocks first
  const int per_blk = p.B * p.hq;
  const int blk = p.blk0 + p.n_blocks - 1 - (int)(blockIdx.x / per_blk);
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
      mbar_init(&s_full[i], 1);
      mbar_init(&p_full[2 * i], AT_SOFTMAX_WARPS);         // one arrival per softmax warp
      mbar_init(&p_full[2 * i + 1], AT_SOFTMAX_WARPS);
      mbar_init(&o_done[i], 1);
    }
    for (int i = 0; i < NS; ++i) {
      mbar_init(&kv_full[i], 1);
      mbar_init(&kv_empty[i], 1);
    }
    wait_ctl_init(abort_flag, p.status);
    fence_barrier_init();
    prefetch_tmap(&tmQ);
    prefetch_tmap(&tmK);
    prefetch_tmap(&tmV);
  }
  if (warp == AT_MMA_WARP) {
    tmem_alloc(tmem_slot, 512);
    tmem_relinquish();
  }
  if (MSUM && warp < AT_SOFTMAX_WARPS) {
    // 16 "channels" of ones for the row-sum MMA: any operand layout reads ones from this block
    reinterpret_cast<uint32_t*>(smem + SM::ONES_OFF)[threadIdx.x] = 0x3F803F80u;
    fence_proxy_async();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == AT_TMA_WARP) {
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
      for (int n = 0; n < 2 * n_max; ++n) {        // n-th tile of K_0 V_0 K_1 V_1 ...
        const int j = n >> 1, sl = n % NS;
        const uint32_t ph = (n / NS) & 1;
        if (!mbar_wait(&kv_empty[sl], ph ^ 1, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_TMA); goto done; }
        mbar_expect_tx(&kv_full[sl], SM::TILE_BYTES);
#pragma unroll
        for (int c = 0; c < NBOX; ++c)
          tma_load_3d(smem + SM::KV_OFF + sl * SM::TILE_BYTES + c * 16384, (n & 1) ? &tmV : &tmK, hj * DH + c * 64, j * BKV, b,
                      &kv_full[sl]);
      }
    }
  } else if (warp == AT_MMA_WARP) {
    // ---------------------------------------------------------------- MMA issuer
    // The whole warp runs the loop (so the address arithmetic stays warp-uniform and cheap); one elected lane
    // issues the MMAs and the commits.
    {
      const bool leader = elect_one();
      const uint32_t idesc_s = idesc_bf16(BKV, 0, 0);
      const uint32_t idesc_o = idesc_bf16(DH, 0, 1);
      const uint32_t idesc_l = idesc_bf16(16, 0, 0);
      const uint32_t ones_lo = (smem_u32(smem + SM::ONES_OFF) >> 4) | (1u << 16);
      // descriptor words: low = address >> 4 | leading offset << 16, high = stride offset, version, swizzle
      const uint32_t desc_hi = (uint32_t)(smem_desc_sw128(0, 0, 1024) >> 32);
      const uint32_t q_lo = (smem_u32(smem + SM::Q_OFF) >> 4) | (1u << 16);
      const uint32_t k_lo = (smem_u32(smem + SM::KV_OFF) >> 4) | (1u << 16);
      const uint32_t v_lo = (smem_u32(smem + SM::KV_OFF) >> 4) | ((16384u >> 4) << 16);   // 64-channel chunks 16 KB apart
      constexpr uint32_t TILE16 = SM::TILE_BYTES >> 4;
      auto wait_all = [&](uint64_t* bar, uint32_t parity) -> bool {
        return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag));
      };
      auto issue_s = [&](int s, int j) {      // S_s = Q_s K_j^T
        const uint32_t qa = q_lo + s * TILE16, ka = k_lo + ((2 * j) % NS) * TILE16;
        if (leader) {
#pragma unroll
          for (int kk = 0; kk < DH / 16; ++kk) {
            const uint32_t off = (uint32_t)(((kk >> 2) * 16384 + (kk & 3) * 32) >> 4);
            mma_ss_w(tmem_base + s * 128, qa + off, desc_hi, ka + off, desc_hi, idesc_s, kk != 0);
          }
        }
      };
      // O_s (+)= P_s V_j over the keys whose P is complete after the softmax threads' chunk hf: each thread owns
      // 32 keys (k-steps 2 part, 2 part + 1) and finishes them 16 at a time, so chunk hf covers k-steps {hf, 2+hf, 4+hf, 6+hf}
      auto issue_pv = [&](int s, int j, int hf) {
        const uint32_t va = v_lo + ((2 * j + 1) % NS) * TILE16;
        if (leader) {
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int kk = 2 * i + hf;
            mma_ts_w(tmem_base + 256 + s * 128, tmem_base + s * 128 + (kk >> 1) * 32 + (kk & 1) * 8, va + kk * (2048 >> 4),
                     desc_hi, idesc_o, (j | hf | i) != 0);
            if (MSUM)
              mma_ts_w(tmem_base + 256 + s * 128 + DH, tmem_base + s * 128 + (kk >> 1) * 32 + (kk & 1) * 8, ones_lo, desc_hi,
                       idesc_l, (j | hf | i) != 0);
          }
        }
      };
      auto commit = [&](uint64_t* bar) {
        if (leader) mma_commit(bar);
      };
      // prologue: first S tile of each query tile
      if (n_max > 0) {
        if (!wait_all(&kv_full[0], 0)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
        tc_fence_after();
#pragma unroll
        for (int s = 0; s < 2; ++s) {
          if (n_s[s] == 0) continue;
          if (!wait_all(&q_full[s], 0)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
          tc_fence_after();
          issue_s(s, 0);
          commit(&s_full[s]);
        }
      }
      for (int j = 0; j < n_max; ++j) {
        const int vsl = (2 * j + 1) % NS;
        const uint32_t vph = ((2 * j + 1) / NS) & 1;
        // all S(j) were issued before this point: release K_j when they complete
        commit(&kv_empty[(2 * j) % NS]);
        bool k_next_ready = false;
#pragma unroll
        for (int s = 0; s < 2; ++s) {
          if (j >= n_s[s]) continue;
          if (!wait_all(&p_full[2 * s], j & 1)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
          if (!wait_all(&kv_full[vsl], vph)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
          tc_fence_after();
          issue_pv(s, j, 0);                 // runs while the softmax threads finish their second 32 keys
          if (!wait_all(&p_full[2 * s + 1], j & 1)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
          tc_fence_after();
          issue_pv(s, j, 1);
          if (j + 1 < n_s[s]) {
            if (!k_next_ready) {
              if (!wait_all(&kv_full[(2 * j + 2) % NS], ((2 * j + 2) / NS) & 1)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
              tc_fence_after();
              k_next_ready = true;
            }
            issue_s(s, j + 1);
            commit(&s_full[s]);
          } else {
            commit(&o_done[s]);
          }
        }
        commit(&kv_empty[vsl]);
      }
    }
  } else {
    // ---------------------------------------------------------------- softmax + epilogue
    // All 16 warps work on one query tile at a time, alternating between the two tiles in the order the MMA
    // warp produces their S: a tile's softmax then takes half as long as with eight warps per tile, which is
    // what bounds the loop (the tile waits for its own softmax and then for its own two MMAs).
    const int part = warp >> 2;                      // which 32 score columns of each KV tile
    const int row = (warp & 3) * 32 + lane;
    const uint32_t lane_sel = (uint32_t)((warp & 3) * 32) << 16;
    float* xch = reinterpret_cast<float*>(smem + SM::XCH_OFF);     // [4 parts][128 rows]
    auto sync_softmax = [&]() { asm volatile("bar.sync 1, 512;" ::: "memory"); };
    const float c_scale = rsqrtf((float)DH) * LOG2E_F;
    // Fixed maximum: |q| = sqrt(d_h), |k| = sqrt(d_h) beta, so the scaled logit (log2 units) is at most
    // sqrt(d_h) beta log2(e); 1 % covers the bf16 rounding of q and k.  Used while 2^(-2 bound) is a normal
    // fp32 number with room to spare.
    float m_fixed = 0.f;
    bool fixed = false;
    if (p.temp != nullptr) {
      m_fixed = sqrtf((float)DH) * __expf(p.temp[hj]) * LOG2E_F * 1.01f;
      fixed = m_fixed <= 56.f;
    }
    const uint64_t scale2 = pack2f(c_scale, c_scale);
    float m_run[2] = {fixed ? m_fixed : -INFINITY, fixed ? m_fixed : -INFINITY}, l_run[2] = {0.f, 0.f};
    for (int j = 0; j < n_max; ++j) {
#pragma unroll
      for (int s = 0; s < 2; ++s) {
        if (j >= n_s[s]) continue;
        const uint32_t s_tmem = tmem_base + lane_sel + s * 128 + part * 32;   // this thread's 32 S columns
        const uint32_t o_tmem = tmem_base + lane_sel + 256 + s * 128;
        const int m0 = blk * 256 + s * BQ;
        const int tq = m0 + row;
        if (!mbar_wait(&s_full[s], j & 1, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_SOFTMAX); goto done; }
        tc_fence_after();
        // this thread's 32 scores, loaded once: one trip to tensor memory per tile
        uint32_t v[32];
        tmem_ld32(s_tmem, v);
        tmem_ld_wait();
        const int k0 = j * BKV + part * 32;            // first key of this thread's columns
        const bool need_mask = (p.causal && j * BKV + BKV - 1 > m0) || (j * BKV + BKV > p.S);
        const int lim = p.causal ? min(tq, p.S - 1) : p.S - 1;       // last visible key
        float m_use = m_run[s];
        if (!fixed) {
          // first pass for the row maximum
          float mx = -INFINITY;
#pragma unroll
          for (int c = 0; c < 32; ++c)
            if (!need_mask || k0 + c <= lim) mx = fmaxf(mx, __uint_as_float(v[c]));
          // the rest of the row belongs to three other threads: exchange through shared memory
          xch[part * 128 + row] = mx;
          sync_softmax();
          mx = fmaxf(fmaxf(xch[row], xch[128 + row]), fmaxf(xch[256 + row], xch[384 + row])) * c_scale;
          sync_softmax();
          const bool grow = mx > m_run[s] + RESCALE_THRESHOLD;        // also true on the first tile
          if (grow) m_use = mx;
          if (m_use == -INFINITY) m_use = 0.f;
          if (j > 0 && __any_sync(0xffffffffu, grow)) {
            // rescale this thread's quarter of the running output (rare)
            const float alpha = grow ? exp2f(m_run[s] - m_use) : 1.f;
            l_run[s] *= alpha;
            if (MSUM && part == 0) {          // the row sum lives beside O: only its first column is read at the end
              uint32_t t[8];
              tmem_ld8(o_tmem + DH, t);
              tmem_ld_wait();
#pragma unroll
              for (int i = 0; i < 8; ++i) t[i] = __float_as_uint(__uint_as_float(t[i]) * alpha);
              tmem_st8(o_tmem + DH, t);
            }
#pragma unroll 1
            for (int c = 0; c < DH / 64; ++c) {
              uint32_t t[16];
              tmem_ld16(o_tmem + part * (DH / 4) + c * 16, t);
              tmem_ld_wait();
#pragma unroll
              for (int i = 0; i < 16; ++i) t[i] = __float_as_uint(__uint_as_float(t[i]) * alpha);
              tmem_st16(o_tmem + part * (DH / 4) + c * 16, t);
            }
            tmem_st_wait();
          }
          m_run[s] = m_use;
        }
        const uint64_t negm2 = pack2f(-m_use, -m_use);
        uint64_t sum2 = pack2f(0.f, 0.f);
        // 16 scores at a time.  The bf16 pairs of P go over the S columns the same thread has already read:
        // part p reads S columns [32p, 32p+32) and writes P into storage columns [32p, 32p+16); after each
        // chunk the MMA warp may start on those keys.
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          uint32_t pk[8];
          if (need_mask) {
#pragma unroll
            for (int c = 0; c < 16; ++c)
              if (k0 + hf * 16 + c > lim) v[hf * 16 + c] = 0xff800000u;        // -inf
#pragma unroll
            exp16<0, false, !MSUM>(&v[hf * 16], scale2, negm2, sum2, pk);
          } else if (fixed) {
            exp16<POLY8, false, !MSUM>(&v[hf * 16], scale2, negm2, sum2, pk);
          } else {
            exp16<POLY8, true, !MSUM>(&v[hf * 16], scale2, negm2, sum2, pk);
          }
          tmem_st8(s_tmem + hf * 8, pk);
          tmem_st_wait();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&p_full[2 * s + hf]);
        }
        if (!MSUM) {
          uint32_t a, b2;
          unpack2u(sum2, a, b2);
          l_run[s] += __uint_as_float(a) + __uint_as_float(b2);
        }
      }
    }
#pragma unroll
    for (int s = 0; s < 2; ++s) {
      if (n_s[s] == 0) continue;
      const uint32_t o_tmem = tmem_base + lane_sel + 256 + s * 128;
      const int tq = blk * 256 + s * BQ + row;
      float l_tot;
      if (!MSUM) {
        // total of the four parts of the row
        sync_softmax();
        xch[part * 128 + row] = l_run[s];
        sync_softmax();
        l_tot = (xch[row] + xch[128 + row]) + (xch[256 + row] + xch[384 + row]);
      }
      if (!mbar_wait(&o_done[s], 0, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_EPI); goto done; }
      tc_fence_after();
      if (MSUM) {
        uint32_t t;
        tmem_ld1(o_tmem + DH, t);
        tmem_ld_wait();
        l_tot = __uint_as_float(t);
      }
      const float inv_l = 1.f / l_tot;
      // The warp's block of O: 32 rows x d_h / 4 columns.  Stored through a shared-memory stage in the tile's own Q
      // buffer (free: every S MMA of the tile finished before its last P V), whole row segments per instruction.
      constexpr int CW = DH / 4;                             // columns per warp
      constexpr int RB = CW * 2;                             // bytes of a bf16 row segment (64 or 32)
      unsigned char* stg = smem + SM::Q_OFF + s * SM::TILE_BYTES + warp * (32 * RB);
      const int row0 = blk * 256 + s * BQ + (warp & 3) * 32;         // first query row of the block
      const int rows_ok = p.S - row0;
      const long long e0 = ((long long)b * p.S + row0) * p.Lq + hi * DH + part * CW;   // element offset of the block
      uint32_t t[CW];
      if (DH == 128) tmem_ld32(o_tmem + part * CW, reinterpret_cast<uint32_t(&)[32]>(t[0]));
      else tmem_ld16(o_tmem + part * CW, reinterpret_cast<uint32_t(&)[16]>(t[0]));
      tmem_ld_wait();
#pragma unroll
      for (int i = 0; i < CW; ++i) t[i] = __float_as_uint(__uint_as_float(t[i]) * inv_l);
      {
        uint32_t w[CW / 2];
#pragma unroll
        for (int i = 0; i < CW / 2; ++i) w[i] = pack_bf16(__uint_as_float(t[2 * i]), __uint_as_float(t[2 * i + 1]));
        warp_store_rows<RB>(stg, w, reinterpret_cast<unsigned char*>(p.o + e0), (long long)p.Lq * 2, rows_ok);
      }
      if (p.o32) {                                            // the fp32 copy for the backward, in two halves
#pragma unroll
        for (int h = 0; h < 2; ++h)
          warp_store_rows<RB>(stg, &t[h * (CW / 2)], reinterpret_cast<unsigned char*>(p.o32 + e0 + h * (CW / 2)),
                              (long long)p.Lq * 4, rows_ok);
      }
      if (part == 0 && tq < p.S) p.lse[((long long)b * p.hq + hi) * p.S + tq] = (m_run[s] + log2f(l_tot)) * LN2_F;
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
  if (warp == AT_MMA_WARP) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

}  // namespace

namespace {
template <int DH, int POLY8>
int launch_attn(TcState* s, const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV, const AttnParams& p,
                unsigned grid, cudaStream_t st) {
  static bool attr_set[TC_MAX_DEVICES] = {};
  if (!attr_set[s->device]) {
    cudaError_t e = cudaFuncSetAttribute(tc_attn_fwd_kernel<DH, POLY8>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         AttnSmem<DH>::TOTAL);
    if (e != cudaSuccess) return -(int)e;
    attr_set[s->device] = true;
  }
  tc_attn_fwd_kernel<DH, POLY8><<<grid, AT_THREADS, AttnSmem<DH>::TOTAL, st>>>(tmQ, tmK, tmV, p);
  cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? 0 : -(int)e;
}
}  // namespace

int tc_attn_fwd(TcState* s, const CcaDims& d, const bf16* q, const bf16* k, const bf16* v, bf16* o, float* o32,
                float* lse, const float* temp, int* d_status, cudaStream_t st, int t_first) {
  if (t_first % 256 || t_first < 0 || t_first >= d.S) return 1;
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
  p.blk0 = t_first / 256;
  p.n_blocks = (d.S - t_first + 255) / 256;
  p.status = d_status;
  const long long grid = (long long)p.n_blocks * d.B * d.hq;
  if (grid > 0x7fffffffLL) return 1;
  // The knob counts eighths of the score pairs that take the polynomial (bit 3: ignore the norm bound).  At d_h = 128
  // the exponential unit and the tensor pipe need the same time and the packed FMA pipe is no faster; at d_h = 64,
  // with the row sums on the tensor core, two of eight measured best (1.256 ms against 1.308 with none and 1.280
  // with three at 4 x 16384 tokens, 8 / 2 heads).
  const int knob = s->attn_poly < 0 ? (d.dh == 128 ? 0 : 2) : s->attn_poly;
  p.temp = (knob & 8) ? nullptr : temp;
  const int poly = knob & 7;
  if (d.dh == 128) {
    if (poly == 0) return launch_attn<128, 0>(s, tmQ, tmK, tmV, p, (unsigned)grid, st);
    if (poly <= 2) return launch_attn<128, 2>(s, tmQ, tmK, tmV, p, (unsigned)grid, st);
    return launch_attn<128, 4>(s, tmQ, tmK, tmV, p, (unsigned)grid, st);
  }
  if (poly == 0) return launch_attn<64, 0>(s, tmQ, tmK, tmV, p, (unsigned)grid, st);
  if (poly <= 2) return launch_attn<64, 2>(s, tmQ, tmK, tmV, p, (unsigned)grid, st);
  if (poly == 3) return launch_attn<64, 3>(s, tmQ, tmK, tmV, p, (unsigned)grid, st);
  return launch_attn<64, 4>(s, tmQ, tmK, tmV, p, (unsigned)grid, st);
}
