// Tensor-core kernels, part 3b: the latent transforms of Eq. 8, 9 and 11 on q and k, forward, with every
// tensor-core operand brought in by TMA.
//
// Eq. 8 applies conv1_seq (depth-wise over the sequence, k_seq taps) and then conv2_seq+ch (d_h x d_h per head,
// k_ch taps) to the packed latent.  Both are linear and causal with zero history, so their composition is one causal
// convolution over the sequence with NT = k_seq + k_ch - 1 taps and a dense d_h x d_h matrix per tap,
//     W_m[o][i] = sum_{j + j' = m} w1[o][i][j] * w0[i][j'],       y2[t] = sum_m W_m qk0[t - (NT-1) + m],
// which a small kernel forms once per forward (compose_conv_weights_kernel, bf16, beside the down-projection).
// The projection's epilogue leaves a bf16 copy of qk0; a work unit (one head, one sequence, 128 consecutive tokens)
// loads rows [t0 - (NT-1), t0 + 128 + ...) of its head's channels with ONE TMA tile of 136 rows (rows before the
// sequence start are filled with zeros: the causal padding), and tap m's operand is that same tile read from row m
// on: the shared-memory descriptor's start address moves down by m rows of 128 bytes, the 128-byte swizzle being a
// function of the address.  No thread touches an operand.
//
//   TMA warp   the head's NT weight tiles when the head changes, one operand tile per unit (ring of stages)
//   MMA warp   acc = sum_m A_m W_m^T into one of NG TMEM accumulators (128 tokens x d_h, fp32)
//   4 NG warps epilogue, thread = token, NG groups of four warps that take every NG-th unit: adds the q-k-mean term
//            of Eq. 9 in fp32 from the fp32 latent, L2 norm * sqrt(d_h) (* exp(temp)), RoPE from the table, bf16
//            store; the norm scale is kept for the backward.  A thread needs 128 bytes of its own token's row at a
//            time (32 fp32 channels, or 16 (cos, sin) pairs); fetched by the thread itself that would be one memory
//            transaction per thread and 16 bytes.  Instead lane 0 of each warp has TMA bring the warp's 32 rows x 128
//            bytes into a private shared-memory slot (two slots per warp, the next box in flight while one is read),
//            and the threads read their rows from there, swizzled, without bank conflicts.
#include "tc_kernels.cuh"
#include "tc_ptx.cuh"
#include "tc_state.cuh"

using namespace tc;

namespace {

// Epilogue groups of four warps (one per TMEM lane quarter), each with a TMEM accumulator of its own, taking every
// NG-th unit: the epilogue is a latency chain (TMA box -> shared memory -> TMEM round trip), so what matters is how many
// units are in flight.  Four groups at head size 64 (4 x 64 TMEM columns), three at 128 (3 x 128; shared memory for the
// boxes' slots and the register file set the limit).
template <int DH, int NT>
struct T2Groups {
  static constexpr int NG = DH == 64 ? 4 : (NT <= 3 ? 3 : 2);
  static constexpr int EPI_WARPS = 4 * NG;
  static constexpr int TMA_WARP = EPI_WARPS, MMA_WARP = EPI_WARPS + 1;
  static constexpr int THREADS = 32 * (EPI_WARPS + 2);
  static constexpr int TMEM_COLS = NG * DH > 256 ? 512 : 256;      // a power of two
};
enum : unsigned { F_CONV1 = 1, F_CONV2 = 2, F_QK_MEAN = 4, F_QK_NORM = 16, F_ROPE = 32 };

template <int DH, int NT>
struct T2Smem {
  static constexpr int ROWS = 136;                       // 128 tokens + up to 6 earlier ones, rounded up to the swizzle period
  static constexpr int BOX = ROWS * 128;                 // one 64-channel box of the operand tile
  static constexpr int A_BYTES = (DH / 64) * BOX;
  static constexpr int WT = DH * DH * 2;                 // one tap's weight tile
  static constexpr int W_BYTES = NT * WT;
  static constexpr int BUDGET = 232448 - 512;            // 227 KB minus barriers
  // per epilogue warp: slots for boxes of 32 rows x 128 bytes, as many as fit beside one operand tile (2..4)
  static constexpr int EPI_WARPS = T2Groups<DH, NT>::EPI_WARPS;
  static constexpr int NSLOT_FIT = (BUDGET - W_BYTES - A_BYTES) / (EPI_WARPS * 4096);
  static constexpr int NSLOT = NSLOT_FIT > 3 ? 3 : NSLOT_FIT;
  static constexpr int SLOT_BYTES = EPI_WARPS * NSLOT * 4096;
  static constexpr int STAGES_FIT = (BUDGET - W_BYTES - SLOT_BYTES) / A_BYTES;
  static constexpr int STAGES = STAGES_FIT > 2 ? 2 : STAGES_FIT;   // one is enough: the contraction of a unit is short
  static_assert(NSLOT >= 2, "box slots do not fit");
  static constexpr int W_OFF = 0;
  static constexpr int A_OFF = W_BYTES;
  static constexpr int SLOT_OFF = A_OFF + STAGES * A_BYTES;
  static constexpr int BAR_OFF = SLOT_OFF + SLOT_BYTES;
  static constexpr int TOTAL = BAR_OFF + 512;
  static_assert(STAGES >= 1, "operand tile does not fit");
  static_assert(NT - 1 <= ROWS - 128, "halo rows");
};

struct T2Params {
  CcaDims d;
  const float* qk0;      // fp32 latent (q-k-mean term)
  const float* temp;
  const float2* rope;
  bf16* q;
  bf16* k;
  float* rnorm;
  int* status;
  int n_tiles, t_first, units_per_head, total_units, cost_q, cost_k;
};

TC_DEVINL void fail(volatile int* abort_flag, int* status, int code) {
  *abort_flag = 1;
  atomicCAS(status, 0, code);
}

struct Unit {
  int h, b, t0;
};
TC_DEVINL Unit unit_of(const T2Params& p, int u) {
  Unit r;
  r.h = u / p.units_per_head;
  const int rem = u % p.units_per_head;
  r.b = rem / p.n_tiles;
  r.t0 = p.t_first + (rem % p.n_tiles) * 128;
  return r;
}

template <int DH, int NT>
__global__ void __launch_bounds__(T2Groups<DH, NT>::THREADS, 1)
tc_transform2_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmW,
                     const __grid_constant__ CUtensorMap tmF, const __grid_constant__ CUtensorMap tmR, const T2Params p) {
  using SM = T2Smem<DH, NT>;
  using GR = T2Groups<DH, NT>;
  constexpr int ST = SM::STAGES, NG = GR::NG;
  extern __shared__ __align__(1024) unsigned char smem[];
  if (smem_u32(smem) & 1023u) {       // the swizzled tiles need it; nothing has been set up yet, so just report
    if (threadIdx.x == 0) atomicCAS(p.status, 0, ST_BAD_SMEM_ALIGNMENT);
    return;
  }
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + SM::BAR_OFF);
  uint64_t* a_full = bars;                 // [ST] TMA -> MMA
  uint64_t* a_empty = bars + ST;           // [ST] MMA -> TMA (commit)
  uint64_t* w_full = bars + 2 * ST;        // TMA -> MMA: the head's weight tiles
  uint64_t* w_empty = w_full + 1;          // MMA -> TMA: every contraction with the previous head's weights is done
  uint64_t* acc_full = w_empty + 1;        // [NG] MMA -> epilogue group (commit)
  uint64_t* acc_empty = acc_full + NG;     // [NG] epilogue group -> MMA (128 arrivals)
  uint64_t* slot_full = acc_empty + NG;    // [epilogue warps][NSLOT] TMA -> the warp's threads
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(slot_full + GR::EPI_WARPS * SM::NSLOT);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const CcaDims& d = p.d;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // contiguous range of units of this CTA, balanced by cost (q-head units first, then kv-head units)
  int u_begin, u_end;
  {
    const long long nq = (long long)d.hq * p.units_per_head, wq = nq * p.cost_q;
    const long long wtot = wq + (long long)d.hk * p.units_per_head * p.cost_k;
    auto unit_at = [&](long long pos) -> int { return (int)(pos < wq ? pos / p.cost_q : nq + (pos - wq) / p.cost_k); };
    u_begin = unit_at(wtot * blockIdx.x / gridDim.x);
    u_end = blockIdx.x + 1 == gridDim.x ? p.total_units : unit_at(wtot * (blockIdx.x + 1) / gridDim.x);
  }

  if (threadIdx.x == 0) {
    for (int s = 0; s < ST; ++s) {
      mbar_init(&a_full[s], 1);
      mbar_init(&a_empty[s], 1);
    }
    mbar_init(w_full, 1);
    mbar_init(w_empty, 1);
    for (int s = 0; s < NG; ++s) {
      mbar_init(&acc_full[s], 1);
      mbar_init(&acc_empty[s], 128);
    }
    for (int s = 0; s < GR::EPI_WARPS * SM::NSLOT; ++s) mbar_init(&slot_full[s], 1);
    wait_ctl_init(abort_flag, p.status);
    fence_barrier_init();
    prefetch_tmap(&tmA);
    prefetch_tmap(&tmW);
    prefetch_tmap(&tmF);
    prefetch_tmap(&tmR);
  }
  if (warp == GR::MMA_WARP) {
    tmem_alloc(tmem_slot, GR::TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == GR::TMA_WARP) {
    // ------------------------------------------------------------------ TMA
    if (lane == 0) {
      int cur_head = -1, wk = 0, it = 0;
      for (int u = u_begin; u < u_end; ++u, ++it) {
        const Unit un = unit_of(p, u);
        if (un.h != cur_head) {
          if (wk > 0 && !mbar_wait(w_empty, (wk - 1) & 1, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_TMA); goto done; }
          mbar_expect_tx(w_full, SM::W_BYTES);
#pragma unroll
          for (int m = 0; m < NT; ++m)
#pragma unroll
            for (int c = 0; c < DH / 64; ++c)
              tma_load_2d(smem + SM::W_OFF + m * SM::WT + c * (DH * 128), &tmW, c * 64, (un.h * NT + m) * DH, w_full);
          cur_head = un.h;
          ++wk;
        }
        const int stage = it % ST;
        if (!mbar_wait(&a_empty[stage], ((it / ST) & 1) ^ 1, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_TMA); goto done; }
        mbar_expect_tx(&a_full[stage], SM::A_BYTES);
#pragma unroll
        for (int c = 0; c < DH / 64; ++c)
          tma_load_3d(smem + SM::A_OFF + stage * SM::A_BYTES + c * SM::BOX, &tmA, un.h * DH + c * 64, un.t0 - (NT - 1), un.b,
                      &a_full[stage]);
      }
    }
  } else if (warp == GR::MMA_WARP) {
    // ------------------------------------------------------------------ MMA issue (whole warp walks, one lane issues)
    const bool leader = elect_one();
    const uint32_t idesc = idesc_bf16(DH, 0, 0);
    auto wait_all = [&](uint64_t* bar, uint32_t parity) -> bool {
      return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag));
    };
    const uint32_t a_base = smem_u32(smem + SM::A_OFF), w_base = smem_u32(smem + SM::W_OFF);
    int cur_head = -1, wk = 0, it = 0;
    for (int u = u_begin; u < u_end; ++u, ++it) {
      const Unit un = unit_of(p, u);
      if (un.h != cur_head) {
        if (wk > 0 && leader) mma_commit(w_empty);
        if (!wait_all(w_full, wk & 1)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
        cur_head = un.h;
        ++wk;
      }
      const int buf = it % NG, stage = it % ST;
      if (!wait_all(&acc_empty[buf], ((it / NG) & 1) ^ 1)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
      if (!wait_all(&a_full[stage], (it / ST) & 1)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
      tc_fence_after();
      if (leader) {
#pragma unroll
        for (int m = 0; m < NT; ++m)
#pragma unroll
          for (int kk = 0; kk < DH / 16; ++kk) {
            // tap m reads the tile from row m on: the start address moves by m rows of 128 bytes
            const uint32_t off_a = stage * SM::A_BYTES + (kk >> 2) * SM::BOX + m * 128 + (kk & 3) * 32;
            const uint32_t off_w = m * SM::WT + (kk >> 2) * (DH * 128) + (kk & 3) * 32;
            mma_ss(tmem_base + buf * DH, smem_desc_sw128(a_base + off_a, 16, 1024), smem_desc_sw128(w_base + off_w, 16, 1024),
                   idesc, (m | kk) != 0);
          }
        mma_commit(&a_empty[stage]);
        mma_commit(&acc_full[buf]);
      }
      __syncwarp();
    }
  } else {
    // ------------------------------------------------------------------ epilogue, thread = token
    constexpr int HALF = DH / 2;
    constexpr int NS = SM::NSLOT;
    const int grp = warp >> 2;                              // units with it % NG == grp, accumulator grp
    const int rho = (warp & 3) * 32 + lane;
    const uint32_t acc = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + grp * DH;
    const bool use_mean = (d.flags & F_QK_MEAN) != 0, use_rope = (d.flags & F_ROPE) != 0;
    unsigned char* my_slots = smem + SM::SLOT_OFF + warp * NS * 4096;
    uint64_t* my_full = slot_full + warp * NS;
    // this thread's 16-byte chunk i of its row in a slot (rows of 128 bytes, 128-byte swizzle)
    uint32_t ch_off[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) ch_off[i] = (uint32_t)lane * 128u + (((uint32_t)i ^ (uint32_t)(lane & 7)) << 4);
    uint32_t nb = 0;                                        // boxes this warp has consumed so far (all units)
    // The boxes of a unit, in the order they are read: for every 32-channel chunk the own rows then the other heads'
    // rows (fp32 latent), then the RoPE table rows, 16 (cos, sin) pairs at a time; rows past the end come as zeros.
    // Box layout of unit u (warp-uniform):
    struct Boxes {
      int h, b, row0, oth_col, per_chunk, n_mean, n_box;
    };
    auto boxes_of = [&](int u) -> Boxes {
      const Unit un = unit_of(p, u);
      const bool is_q = un.h < d.hq;
      const int hj = is_q ? un.h / d.g : un.h - d.hq;
      Boxes x;
      x.h = un.h; x.b = un.b; x.row0 = un.t0 + (warp & 3) * 32;
      x.oth_col = is_q ? d.Lq + hj * DH : hj * d.g * DH;
      x.per_chunk = use_mean ? 1 + (is_q ? 1 : d.g) : 0;
      x.n_mean = (DH / 32) * x.per_chunk;
      x.n_box = x.n_mean + (use_rope ? HALF / 16 : 0);
      return x;
    };
    // Issue cursor (lane 0 acts, every lane tracks): the next box to ask for is box pn of unit pu; it runs NS boxes
    // ahead of the reads, across unit boundaries, so that the slots never sit empty between two units.
    int pu = u_begin + grp, pn = 0;
    uint32_t issued = 0;
    Boxes pbx = pu < u_end ? boxes_of(pu) : Boxes{0, 0, 0, 0, 0, 0, 0};
    auto issue_next = [&]() {
      while (pu < u_end && pn >= pbx.n_box) {               // next unit of this group (units without boxes are skipped)
        pu += NG;
        pn = 0;
        if (pu < u_end) pbx = boxes_of(pu);
      }
      if (pu >= u_end) return;
      if (lane == 0) {
        unsigned char* dst = my_slots + (issued % NS) * 4096;
        uint64_t* bar = &my_full[issued % NS];
        mbar_expect_tx(bar, 4096);
        if (pn < pbx.n_mean) {
          const int c = pn / pbx.per_chunk, j = pn % pbx.per_chunk;
          tma_load_3d(dst, &tmF, (j == 0 ? pbx.h * DH : pbx.oth_col + (j - 1) * DH) + c * 32, pbx.row0, pbx.b, bar);
        } else {
          tma_load_2d(dst, &tmR, (pn - pbx.n_mean) * 32, pbx.row0, bar);
        }
      }
      ++issued;
      ++pn;
    };
    for (int i = 0; i < NS; ++i) issue_next();
    int it = grp;
    for (int u = u_begin + grp; u < u_end; u += NG, it += NG) {
      const Unit un = unit_of(p, u);
      const bool is_q = un.h < d.hq;
      const int hj = is_q ? un.h / d.g : un.h - d.hq;
      const int t = un.t0 + rho;
      const bool valid = t < d.S;
      const long long tok = (long long)un.b * d.S + (valid ? t : 0);
      const int n_oth = is_q ? 1 : d.g;
      const float oth_scale = is_q ? 0.5f : 0.5f / (float)d.g;
      const int per_chunk = use_mean ? 1 + n_oth : 0;
      const int n_mean = (DH / 32) * per_chunk;
      const int n_box = n_mean + (use_rope ? HALF / 16 : 0);
      auto wait_box = [&](int n) -> bool {
        const uint32_t g = nb + (uint32_t)n;
        return mbar_wait(&my_full[g % NS], (g / NS) & 1, abort_flag);
      };
      // Every lane has used a box: its slot takes the next box of the stream.  The TMA write goes through the
      // asynchronous proxy and is not ordered behind shared-memory loads that are still in flight; release_box is
      // therefore called only after the arithmetic that consumes the loaded values has been issued (instructions
      // issue in order, so the values have arrived), and every lane has got there (__syncwarp).
      auto release_box = [&]() {
        __syncwarp();
        if (lane == 0) fence_proxy_async();
        issue_next();
      };
      if (!mbar_wait(&acc_full[grp], (it / NG) & 1, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_EPI); goto done; }
      tc_fence_after();
      // pass 1: pre-norm latent = conv output + mean term (Eq. 9), its squared norm; kept in the accumulator
      float ss = 0.f;
#pragma unroll 1
      for (int c = 0; c < DH / 32; ++c) {
        uint32_t r[32];
        tmem_ld32(acc + c * 32, r);
        if (use_mean) {
          for (int j = 0; j < per_chunk; ++j) {            // j = 0: own rows (weight 1/2), then the other heads' rows
            const int n = c * per_chunk + j;
            if (!wait_box(n)) { fail(abort_flag, p.status, ST_TIMEOUT_EPI); goto done; }
            const unsigned char* src = my_slots + ((nb + n) % NS) * 4096;
            const float wgt = j == 0 ? 0.5f : oth_scale;
            if (j == 0) tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const float4 e = *reinterpret_cast<const float4*>(src + ch_off[i]);
              r[4 * i + 0] = __float_as_uint(fmaf(wgt, e.x, __uint_as_float(r[4 * i + 0])));
              r[4 * i + 1] = __float_as_uint(fmaf(wgt, e.y, __uint_as_float(r[4 * i + 1])));
              r[4 * i + 2] = __float_as_uint(fmaf(wgt, e.z, __uint_as_float(r[4 * i + 2])));
              r[4 * i + 3] = __float_as_uint(fmaf(wgt, e.w, __uint_as_float(r[4 * i + 3])));
            }
            asm volatile("" ::"r"(r[0]), "r"(r[31]) : "memory");      // the sums exist before the slot is handed over
            release_box();
          }
#pragma unroll
          for (int i = 0; i < 32; ++i) ss = fmaf(__uint_as_float(r[i]), __uint_as_float(r[i]), ss);
          tmem_st32(acc + c * 32, r);
        } else {
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 32; ++i) ss = fmaf(__uint_as_float(r[i]), __uint_as_float(r[i]), ss);
        }
      }
      if (use_mean) tmem_st_wait();
      float sc = 1.f;
      if (d.flags & F_QK_NORM) {
        sc = sqrtf((float)DH) * (is_q ? 1.f : __expf(p.temp[hj])) * rsqrtf(ss);
        if (valid) p.rnorm[tok * (d.hq + d.hk) + un.h] = sc;
      }
      // pass 2: scale, rotate the pairs (c, c + d_h/2), store
      bf16* dst = is_q ? p.q + tok * d.Lq + un.h * DH : p.k + tok * d.Lk + hj * DH;
#pragma unroll 1
      for (int c = 0; c < HALF / 16; ++c) {              // one table box = 16 pairs; handled as two halves of 8 pairs
        if (use_rope && !wait_box(n_mean + c)) { fail(abort_flag, p.status, ST_TIMEOUT_EPI); goto done; }
        const unsigned char* src = my_slots + ((nb + n_mean + c) % NS) * 4096;
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          uint32_t ra[8], rb[8];
          tmem_ld8(acc + c * 16 + hf * 8, ra);
          tmem_ld8(acc + HALF + c * 16 + hf * 8, rb);
          float4 cs[4];
          if (use_rope) {
#pragma unroll
            for (int i = 0; i < 4; ++i) cs[i] = *reinterpret_cast<const float4*>(src + ch_off[hf * 4 + i]);   // (cos, sin) x 2
          }
          tmem_ld_wait();
          float lo[8], hi[8];
          if (use_rope) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const float a0 = __uint_as_float(ra[2 * i]) * sc, b0 = __uint_as_float(rb[2 * i]) * sc;
              const float a1 = __uint_as_float(ra[2 * i + 1]) * sc, b1 = __uint_as_float(rb[2 * i + 1]) * sc;
              lo[2 * i] = a0 * cs[i].x - b0 * cs[i].y;
              hi[2 * i] = b0 * cs[i].x + a0 * cs[i].y;
              lo[2 * i + 1] = a1 * cs[i].z - b1 * cs[i].w;
              hi[2 * i + 1] = b1 * cs[i].z + a1 * cs[i].w;
            }
            if (hf == 1) {
              asm volatile("" ::"f"(lo[0]), "f"(hi[7]) : "memory");
              release_box();
            }
          } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              lo[i] = __uint_as_float(ra[i]) * sc;
              hi[i] = __uint_as_float(rb[i]) * sc;
            }
          }
          if (valid) {
            uint4 w;
            w.x = pack_bf16(lo[0], lo[1]);
            w.y = pack_bf16(lo[2], lo[3]);
            w.z = pack_bf16(lo[4], lo[5]);
            w.w = pack_bf16(lo[6], lo[7]);
            reinterpret_cast<uint4*>(dst + c * 16)[hf] = w;
            w.x = pack_bf16(hi[0], hi[1]);
            w.y = pack_bf16(hi[2], hi[3]);
            w.z = pack_bf16(hi[4], hi[5]);
            w.w = pack_bf16(hi[6], hi[7]);
            reinterpret_cast<uint4*>(dst + HALF + c * 16)[hf] = w;
          }
        }
      }
      nb += (uint32_t)n_box;
      tc_fence_before();
      mbar_arrive(&acc_empty[grp]);
    }
  }
done:
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    // let copies and MMAs that are still in flight land before the shared memory and TMEM go away
    const long long c0 = clock64();
    while (clock64() - c0 < 2000000) {}
    __syncthreads();
  }
  if (warp == GR::MMA_WARP) {
    tc_fence_after();
    tmem_dealloc(tmem_base, GR::TMEM_COLS);
  }
}

// W[h][m][o][i] = sum over (conv2 tap j, conv1 tap j') with j + j' = m of w1[h*dh + o][i][j] * w0[h*dh + i][j'].
__global__ void compose_conv_weights_kernel(const bf16* __restrict__ w0, const bf16* __restrict__ w1, bf16* __restrict__ wc,
                                            int heads, int dh, int ks, int kc, int use_conv1) {
  const int nt = (use_conv1 ? ks : 1) + kc - 1;
  const long long n = (long long)heads * nt * dh * dh;
  for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < n; idx += (long long)gridDim.x * blockDim.x) {
    const int i = (int)(idx % dh);
    const int o = (int)((idx / dh) % dh);
    const int m = (int)((idx / ((long long)dh * dh)) % nt);
    const int h = (int)(idx / ((long long)dh * dh * nt));
    const bf16* w1p = w1 + ((size_t)(h * dh + o) * dh + i) * kc;
    float acc = 0.f;
    for (int j = 0; j < kc; ++j) {
      const int jp = m - j;
      if (use_conv1) {
        if (jp >= 0 && jp < ks) acc = fmaf(__bfloat162float(w1p[j]), __bfloat162float(w0[(size_t)(h * dh + i) * ks + jp]), acc);
      } else if (jp == 0) {
        acc = __bfloat162float(w1p[j]);
      }
    }
    wc[idx] = __float2bfloat16(acc);
  }
}

template <int DH, int NT>
int launch_t2(TcState* s, const CcaDims& d, const bf16* qk0b, const bf16* wc, const T2Params& p0, cudaStream_t st) {
  using SM = T2Smem<DH, NT>;
  static bool attr_done[TC_MAX_DEVICES] = {};
  if (!attr_done[s->device]) {
    cudaError_t e = cudaFuncSetAttribute(tc_transform2_kernel<DH, NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, SM::TOTAL);
    if (e != cudaSuccess) return -(int)e;
    attr_done[s->device] = true;
  }
  CUtensorMap tmA, tmW, tmF, tmR;
  if (!tc_make_map_3d(s, &tmA, qk0b, (uint64_t)d.L, (uint64_t)d.S, (uint64_t)d.B, (uint64_t)d.L, (uint64_t)d.S * d.L, 64, SM::ROWS))
    return 1;
  if (!tc_make_map_2d(s, &tmW, wc, (uint64_t)DH, (uint64_t)(d.hq + d.hk) * NT * DH, (uint64_t)DH, 64, DH)) return 1;
  // fp32 boxes of 32 rows x 32 values (128 bytes): the latent [B][S][L] and the RoPE table [S][d_h/2 pairs = d_h floats]
  {
    cuuint64_t dims[3] = {(cuuint64_t)d.L, (cuuint64_t)d.S, (cuuint64_t)d.B};
    cuuint64_t strides[2] = {(cuuint64_t)d.L * 4, (cuuint64_t)d.S * d.L * 4};
    cuuint32_t box[3] = {32, 32, 1}, estr[3] = {1, 1, 1};
    if (s->encode(&tmF, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float*>(p0.qk0), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return 1;
    cuuint64_t rdims[2] = {(cuuint64_t)DH, (cuuint64_t)d.S};
    cuuint64_t rstrides[1] = {(cuuint64_t)DH * 4};
    cuuint32_t rbox[2] = {32, 32}, restr[2] = {1, 1};
    const void* rp = (d.flags & F_ROPE) ? (const void*)p0.rope : (const void*)p0.qk0;      // unused without RoPE
    if (s->encode(&tmR, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(rp), rdims, rstrides, rbox, restr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return 1;
  }
  const int grid = p0.total_units < s->sm_count ? p0.total_units : s->sm_count;
  tc_transform2_kernel<DH, NT><<<grid, T2Groups<DH, NT>::THREADS, SM::TOTAL, st>>>(tmA, tmW, tmF, tmR, p0);
  cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? 0 : -(int)e;
}

}  // namespace

size_t tc_transform2_weight_bytes(const CcaDims& d) {
  const int nt = ((d.flags & F_CONV1) ? d.k_seq : 1) + d.k_ch - 1;
  return (size_t)(d.hq + d.hk) * nt * d.dh * d.dh * 2;
}

int tc_transform2_compose(const CcaDims& d, const bf16* w0, const bf16* w1, bf16* wc, cudaStream_t st) {
  if (!(d.flags & F_CONV2) || !w1 || ((d.flags & F_CONV1) && !w0)) return 1;
  const long long n = (long long)tc_transform2_weight_bytes(d) / 2;
  const unsigned blocks = (unsigned)((n + 255) / 256 > 2048 ? 2048 : (n + 255) / 256);
  compose_conv_weights_kernel<<<blocks, 256, 0, st>>>(w0, w1, wc, d.hq + d.hk, d.dh, d.k_seq, d.k_ch, (d.flags & F_CONV1) ? 1 : 0);
  cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? 0 : -(int)e;
}

bool tc_transform2_covers(const CcaDims& d) {
  if (!(d.flags & F_CONV2)) return false;
  if (d.L % 8 || d.Lq % 8 || d.Lk % 8) return false;
  const int nt = ((d.flags & F_CONV1) ? d.k_seq : 1) + d.k_ch - 1;
  if (d.dh == 128) return nt >= 1 && nt <= 4;
  if (d.dh == 64) return nt >= 1 && nt <= 7;
  return false;
}

int tc_transform2_fwd(TcState* s, const CcaDims& d, const float* qk0, const bf16* qk0b, const bf16* wc, const float* temp,
                      const float2* rope, bf16* q, bf16* k, float* rnorm, int* d_status, cudaStream_t st, int t_first) {
  if (!s || !s->encode || s->sm_count < 1) return 1;
  if (t_first % 128 || t_first < 0 || t_first >= d.S) return 1;
  if (!tc_transform2_covers(d)) return 1;
  if ((reinterpret_cast<uintptr_t>(qk0) & 15) || (reinterpret_cast<uintptr_t>(qk0b) & 15) || (reinterpret_cast<uintptr_t>(wc) & 15) ||
      (reinterpret_cast<uintptr_t>(rope) & 15))
    return 1;
  if (d.L % 4) return 1;
  T2Params p;
  p.d = d; p.qk0 = qk0; p.temp = temp; p.rope = rope; p.q = q; p.k = k; p.rnorm = rnorm; p.status = d_status;
  p.t_first = t_first;
  p.n_tiles = (d.S - t_first + 127) / 128;
  const long long uph = (long long)d.B * p.n_tiles, total = uph * (d.hq + d.hk);
  if (total > 0x7fffffffLL) return 1;
  p.units_per_head = (int)uph;
  p.total_units = (int)total;
  p.cost_q = 4;
  p.cost_k = (d.flags & F_QK_MEAN) ? 3 + d.g : 4;
  const int nt = ((d.flags & F_CONV1) ? d.k_seq : 1) + d.k_ch - 1;
#define T2_CASE(DH_, NT_) \
  if (d.dh == DH_ && nt == NT_) return launch_t2<DH_, NT_>(s, d, qk0b, wc, p, st);
  T2_CASE(128, 1) T2_CASE(128, 2) T2_CASE(128, 3) T2_CASE(128, 4)
  T2_CASE(64, 1) T2_CASE(64, 2) T2_CASE(64, 3) T2_CASE(64, 4) T2_CASE(64, 5) T2_CASE(64, 6) T2_CASE(64, 7)
#undef T2_CASE
  return 1;
}
