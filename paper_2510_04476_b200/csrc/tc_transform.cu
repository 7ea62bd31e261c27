// Tensor-core kernels, part 3: the latent transforms of Eq. 8, 9 and 11 on q and k, forward.
//
// Work unit = (one head, one sequence, 128 consecutive tokens).  A persistent CTA walks a contiguous
// range of units (ordered head-major, so the head's weights are staged once per head) with three roles:
//
//   warps 8-15 producers: read the head's channels of the fp32 latent qk0 with coalesced 128-bit loads,
//              apply conv1_seq (depth-wise, fp32) and write, as bf16 in the 128-byte-swizzled K-major
//              layout the tensor core reads, the k_ch row-shifted copies
//                  A_j[rho] = y1[t0 + rho - (k_ch-1) + j]            (Eq. 8, operand of conv2)
//              and the q-k-mean term of Eq. 9 as two more operand tiles  A_hi + A_lo = mu[t0 + rho]
//              (mu is computed in fp32 and split into a bf16 value and the bf16 of the remainder, so
//              that it enters the sum to ~16 bits: a single bf16 rounding of mu shows up after the norm);
//              the head's conv2 weights as B_j[o][i] = w1[o][i][j] and an identity tile B_mean = I.
//              Once a unit's tiles are complete, the first producer thread issues
//                  acc = sum_j A_j B_j^T + (A_hi + A_lo) I
//              as tcgen05.mma into one of two TMEM accumulators (128 tokens x d_h, K = d_h * (k_ch + 2)).
//   warps 0-7  epilogue, two threads per token (= one TMEM lane), each with half of the rotation pairs: L2 norm * sqrt(d_h) (* exp(temp)),
//              RoPE, bf16 store.  The norm and the rotation pairs (c, c + d_h/2) are local to the thread.
//
// The accumulator is double-buffered, so the epilogue of a unit overlaps the loads of the next one.
#include <type_traits>

#include "tc_kernels.cuh"
#include "tc_ptx.cuh"
#include "tc_state.cuh"

using namespace tc;

namespace {

constexpr int TR_PRODUCERS = 256;
constexpr int TR_EPILOGUE = 256;                    // two threads per token: each takes half of the rotation pairs
constexpr int TR_THREADS = TR_EPILOGUE + TR_PRODUCERS;
constexpr int TR_MMA_WARP = TR_EPILOGUE / 32;       // first producer warp: its lane 0 also issues the MMAs of each unit
enum : unsigned { F_CONV1 = 1, F_CONV2 = 2, F_QK_MEAN = 4, F_QK_NORM = 16, F_ROPE = 32 };

// byte offset of element (row, col) inside a K-major operand tile [rows][DH] stored as DH/64 boxes of
// [rows][64 bf16] with the 128-byte swizzle (16-byte chunk index XOR row mod 8); box_bytes = rows * 128
TC_DEVINL uint32_t sw_off(int row, int col, int box_bytes) {
  return (uint32_t)((col >> 6) * box_bytes + row * 128 + ((((col & 63) >> 3) ^ (row & 7)) << 4) + (col & 7) * 2);
}

template <int DH, int KC>
struct TrSmem {
  static constexpr int NA = KC + 2;              // A tiles: k_ch taps + q-k-mean term (high and low part)
  static constexpr int NB = KC + 1;              // B tiles: k_ch weight taps + identity
  static constexpr int TILE = 128 * DH * 2;      // bytes of one A tile
  static constexpr int BT = DH * DH * 2;         // bytes of one B tile ([DH rows][DH])
  static constexpr int A_OFF = 0;
  static constexpr int B_OFF = NA * TILE;
  static constexpr int BAR_OFF = B_OFF + NB * BT;
  static constexpr int THETA_OFF = BAR_OFF + 128;          // d_h/2 RoPE frequencies (fp32)
  static constexpr int TOTAL = THETA_OFF + 256 + 1024;
};

struct TrParams {
  CcaDims d;
  const float* qk0;
  const bf16* w0;
  const bf16* w1;
  const float* temp;
  const float2* rope;
  bf16* q;
  bf16* k;
  float* rnorm;         // [B*S, hq+hk] norm scale kept for the backward
  int* status;
  int n_tiles;          // 128-token tiles per sequence (of the token range that is processed)
  int t_first;          // first token of that range (0: whole sequences)
  int units_per_head;   // B * n_tiles
  int total_units;
  int cost_q, cost_k;   // relative cost of a unit of a q head / of a kv head (kv units read g more rows)
};

TC_DEVINL void fail(volatile int* abort_flag, int* status, int code) {
  *abort_flag = 1;
  atomicCAS(status, 0, code);
}

template <int DH, int KC>
__global__ void __launch_bounds__(TR_THREADS, 1) tc_transform_fwd_kernel(const TrParams p) {
  using SM = TrSmem<DH, KC>;
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = smem_align1024(smem_dyn);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + SM::BAR_OFF);
  uint64_t* a_full = bars;           // producers -> MMA   (128 arrivals)
  uint64_t* a_empty = bars + 1;      // MMA -> producers   (commit)
  uint64_t* acc_full = bars + 2;     // [2] MMA -> epilogue (commit)
  uint64_t* acc_empty = bars + 4;    // [2] epilogue -> MMA (128 arrivals)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 6);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const CcaDims& d = p.d;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const bool use_mean = (d.flags & F_QK_MEAN) != 0;

  // contiguous range of units of this CTA, balanced by cost (q-head units first, then kv-head units)
  float* theta_s = reinterpret_cast<float*>(smem + SM::THETA_OFF);
  int u_begin, u_end;
  {
    const long long nq = (long long)d.hq * p.units_per_head, wq = nq * p.cost_q;
    const long long wtot = wq + (long long)d.hk * p.units_per_head * p.cost_k;
    auto unit_at = [&](long long pos) -> int {
      return (int)(pos < wq ? pos / p.cost_q : nq + (pos - wq) / p.cost_k);
    };
    u_begin = unit_at(wtot * blockIdx.x / gridDim.x);
    u_end = blockIdx.x + 1 == gridDim.x ? p.total_units : unit_at(wtot * (blockIdx.x + 1) / gridDim.x);
  }
  if (threadIdx.x < DH / 2)      // theta_c = base^(-2c/d_h), as the RoPE table's generator computes it
    theta_s[threadIdx.x] = (float)exp2(-(double)threadIdx.x / (double)(DH / 2) * log2((double)d.rope_base));

  if (threadIdx.x == 0) {
    mbar_init(a_full, TR_PRODUCERS);
    mbar_init(a_empty, 1);
    for (int s = 0; s < 2; ++s) {
      mbar_init(&acc_full[s], 1);
      mbar_init(&acc_empty[s], TR_EPILOGUE);
    }
    wait_ctl_init(abort_flag, p.status);
    fence_barrier_init();
  }
  if (warp == TR_MMA_WARP) {
    tmem_alloc(tmem_slot, 2 * DH);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp >= TR_MMA_WARP) {
    // ------------------------------------------------------------------ producers
    // Thread (cq, rg) owns 4 channels and the operand-tile rows [rg*RPG, (rg+1)*RPG).  Tile j row rho holds
    // y1 of token t0 + rho - (KC-1) + j, so the thread needs y1 at KC-1 tokens before its first row as well
    // (recomputed rather than exchanged), and conv1 needs k_seq-1 raw tokens before that.
    const int pt = threadIdx.x - TR_EPILOGUE;
    constexpr int CG = DH / 4;                   // channel quads per row
    constexpr int RG = TR_PRODUCERS / CG;        // row groups
    constexpr int RPG = 128 / RG;                // tile rows per thread
    static_assert(RPG % 8 == 0 || RPG == 4 || RPG == 2 || RPG == 1, "row batches");
    const int cq = (pt % CG) * 4, rg = pt / CG;
    const int ks = (d.flags & F_CONV1) ? d.k_seq : 1;
    int staged_head = -1;
    int it = 0;
    for (int u = u_begin; u < u_end; ++u, ++it) {
      const int h = u / p.units_per_head, rem = u % p.units_per_head;
      const int b = rem / p.n_tiles, t0 = p.t_first + (rem % p.n_tiles) * 128;
      const bool is_q = h < d.hq;
      const int hj = is_q ? h / d.g : h - d.hq;
      const int ch = h * DH + cq;
      const float* seq = p.qk0 + (long long)b * d.S * d.L;
      const float* col = seq + ch;
      auto load = [&](int tau) -> float4 {
        if (tau < 0 || tau >= d.S) return make_float4(0.f, 0.f, 0.f, 0.f);
        return *reinterpret_cast<const float4*>(col + (long long)tau * d.L);
      };
      // the other operand of the q-k-mean: the kv head's k0 for a q head, the sum of the group's q0 for a kv head
      const float* oth = seq + (is_q ? d.Lq + hj * DH : hj * d.g * DH) + cq;
      const int n_oth = is_q ? 1 : d.g;
      const float oth_scale = is_q ? 0.5f : 0.5f / (float)d.g;
      // conv1 taps in a 4-slot window ending at the current token: slot 3 = current, slot 2 = previous, ...;
      // tap j of the k_seq taps sits in slot 4 - k_seq + j, unused leading slots carry weight 0.
      float wt[4][4];                              // [channel][slot]
#pragma unroll
      for (int c = 0; c < 4; ++c)
#pragma unroll
        for (int sl = 0; sl < 4; ++sl) {
          const int j = sl - (4 - ks);
          wt[c][sl] = (j < 0) ? 0.f : ((d.flags & F_CONV1) ? __bfloat162float(p.w0[(ch + c) * d.k_seq + j]) : 1.f);
        }
      // x = token offset inside the unit; this thread produces y1 at x in [x_first, x_last]
      const int x_first = rg * RPG - (KC - 1);
      float4 win[4];
      float4 halo[KC > 1 ? KC - 1 : 1];
#pragma unroll
      for (int sl = 0; sl < 3; ++sl) win[sl] = (sl >= 4 - ks) ? load(t0 + x_first - 3 + sl) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int i = 0; i < KC - 1; ++i) halo[i] = load(t0 + x_first + i);
      bool waited = false;
      auto emit = [&](int x, const float4& raw, const float4& other) {
        // y1 at token t0 + x from the window, into every tap tile row of this thread that reads it
        const int tau = t0 + x;
        win[3] = raw;
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
            *reinterpret_cast<uint2*>(smem + SM::A_OFF + j * SM::TILE + sw_off(rho, cq, 16384)) = packed;
        }
        if (use_mean && x >= rg * RPG) {
          float m[4] = {fmaf(oth_scale, other.x, 0.5f * raw.x), fmaf(oth_scale, other.y, 0.5f * raw.y),
                        fmaf(oth_scale, other.z, 0.5f * raw.z), fmaf(oth_scale, other.w, 0.5f * raw.w)};
          __nv_bfloat162 h01 = __floats2bfloat162_rn(m[0], m[1]), h23 = __floats2bfloat162_rn(m[2], m[3]);
          uint2 hi, lo;
          hi.x = *reinterpret_cast<uint32_t*>(&h01);
          hi.y = *reinterpret_cast<uint32_t*>(&h23);
          lo.x = pack_bf16(m[0] - __low2float(h01), m[1] - __high2float(h01));
          lo.y = pack_bf16(m[2] - __low2float(h23), m[3] - __high2float(h23));
          *reinterpret_cast<uint2*>(smem + SM::A_OFF + KC * SM::TILE + sw_off(x, cq, 16384)) = hi;
          *reinterpret_cast<uint2*>(smem + SM::A_OFF + (KC + 1) * SM::TILE + sw_off(x, cq, 16384)) = lo;
        }
#pragma unroll
        for (int j = 0; j < 3; ++j) win[j] = win[j + 1];
      };
      // One pass over the thread's rows in batches of CHN rows; NOTH > 0 fixes the number of "other" rows per
      // token at compile time so that all loads of a batch are issued before the first use.
      auto run_rows = [&](auto chn_c, auto noth_c) -> bool {
        constexpr int CHN = decltype(chn_c)::value, NOTH = decltype(noth_c)::value;
#pragma unroll 1
        for (int x0 = rg * RPG; x0 < (rg + 1) * RPG; x0 += CHN) {
          float4 own[CHN], om[CHN];
#pragma unroll
          for (int i = 0; i < CHN; ++i) own[i] = load(t0 + x0 + i);
          if (use_mean) {
            if (NOTH > 0) {
              float4 ot[CHN][NOTH > 0 ? NOTH : 1];
#pragma unroll
              for (int i = 0; i < CHN; ++i)
#pragma unroll
                for (int m = 0; m < NOTH; ++m)
                  ot[i][m] = (t0 + x0 + i < d.S)
                                 ? *reinterpret_cast<const float4*>(oth + (long long)(t0 + x0 + i) * d.L + m * DH)
                                 : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
              for (int i = 0; i < CHN; ++i) {
                om[i] = ot[i][0];
#pragma unroll
                for (int m = 1; m < NOTH; ++m) {
                  om[i].x += ot[i][m].x; om[i].y += ot[i][m].y; om[i].z += ot[i][m].z; om[i].w += ot[i][m].w;
                }
              }
            } else {
#pragma unroll
              for (int i = 0; i < CHN; ++i) om[i] = make_float4(0.f, 0.f, 0.f, 0.f);
              for (int m = 0; m < n_oth; ++m) {
#pragma unroll
                for (int i = 0; i < CHN; ++i) {
                  if (t0 + x0 + i < d.S) {
                    const float4 a = *reinterpret_cast<const float4*>(oth + (long long)(t0 + x0 + i) * d.L + m * DH);
                    om[i].x += a.x; om[i].y += a.y; om[i].z += a.z; om[i].w += a.w;
                  }
                }
              }
            }
          }
          if (!waited) {
            // the loads above are in flight while the previous unit's MMAs finish reading the operand tiles
            if (!mbar_wait(a_empty, (it & 1) ^ 1, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_TMA); return false; }
            waited = true;
          if (h != staged_head) {
            // B_j[o][i] = w1[h*DH + o][i][j]; identity tile once
            const bf16* wsrc = p.w1 + (size_t)h * DH * DH * KC;
            for (int f = pt; f < DH * (DH / 8); f += TR_PRODUCERS) {
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
                *reinterpret_cast<uint4*>(smem + SM::B_OFF + j * SM::BT + sw_off(o, i0, DH * 128)) =
                    *reinterpret_cast<uint4*>(outv);
              }
              if (staged_head < 0) {
                uint4 idv = make_uint4(0u, 0u, 0u, 0u);
                const int e = o - i0;                       // position of the diagonal inside this chunk
                if (e >= 0 && e < 8) {
                  const uint32_t one = (e & 1) ? 0x3F800000u : 0x00003F80u;
                  if ((e >> 1) == 0) idv.x = one;
                  else if ((e >> 1) == 1) idv.y = one;
                  else if ((e >> 1) == 2) idv.z = one;
                  else idv.w = one;
                }
                *reinterpret_cast<uint4*>(smem + SM::B_OFF + KC * SM::BT + sw_off(o, i0, DH * 128)) = idv;
              }
            }
            staged_head = h;
          }
#pragma unroll
            for (int i = 0; i < KC - 1; ++i) emit(x_first + i, halo[i], make_float4(0.f, 0.f, 0.f, 0.f));
          }
#pragma unroll
          for (int i = 0; i < CHN; ++i) emit(x0 + i, own[i], om[i]);
        }
        return true;
      };
      {
        using std::integral_constant;
        bool ok;
        constexpr int C4 = RPG < 4 ? RPG : 4, C2 = RPG < 2 ? RPG : 2;
        constexpr int C1 = 1;
        if (n_oth == 1) ok = run_rows(integral_constant<int, C4>{}, integral_constant<int, 1>{});
        else if (n_oth == 2) ok = run_rows(integral_constant<int, C4>{}, integral_constant<int, 2>{});
        else if (n_oth == 4) ok = run_rows(integral_constant<int, C2>{}, integral_constant<int, 4>{});
        else if (n_oth == 8) ok = run_rows(integral_constant<int, C1>{}, integral_constant<int, 8>{});
        else ok = run_rows(integral_constant<int, C2>{}, integral_constant<int, 0>{});
        if (!ok) goto done;
      }
      fence_proxy_async();          // generic-proxy smem writes -> visible to the tensor core
      mbar_arrive(a_full);
      if (pt == 0) {
        // ---------------------------------------------------------------- MMA issue (one thread)
        const int buf = it & 1;
        if (!mbar_wait(&acc_empty[buf], ((it >> 1) & 1) ^ 1, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
        if (!mbar_wait(a_full, it & 1, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
        tc_fence_after();
        const uint32_t idesc = idesc_bf16(DH, 0, 0);
        const uint32_t a_addr = smem_u32(smem + SM::A_OFF), b_addr = smem_u32(smem + SM::B_OFF);
        const int n_op = use_mean ? SM::NA : KC;
        for (int j = 0; j < n_op; ++j)
#pragma unroll
          for (int kk = 0; kk < DH / 16; ++kk) {
            const uint32_t off_a = (kk >> 2) * 16384 + (kk & 3) * 32;
            const uint32_t off_b = (kk >> 2) * (DH * 128) + (kk & 3) * 32;
            const int jb = j < KC ? j : KC;          // both halves of the mean term multiply the identity
            mma_ss(tmem_base + buf * DH, smem_desc_sw128(a_addr + j * SM::TILE + off_a, 16, 1024),
                   smem_desc_sw128(b_addr + jb * SM::BT + off_b, 16, 1024), idesc, (j | kk) != 0);
          }
        mma_commit(a_empty);
        mma_commit(&acc_full[buf]);
      }
      __syncwarp();
    }
  } else {
    // ------------------------------------------------------------------ epilogue, thread = token
    constexpr int HALF = DH / 2;
    constexpr int NCH = (HALF / 16) / 2;             // 16-pair chunks per thread
    const int rho = threadIdx.x & 127, part = threadIdx.x >> 7;
    const uint32_t lane_sel = (uint32_t)((warp & 3) * 32) << 16;
    int it = 0;
    for (int u = u_begin; u < u_end; ++u, ++it) {
      const int h = u / p.units_per_head, rem = u % p.units_per_head;
      const int b = rem / p.n_tiles, t0 = p.t_first + (rem % p.n_tiles) * 128;
      const bool is_q = h < d.hq;
      const int hj = is_q ? h / d.g : h - d.hq;
      const int buf = it & 1;
      const int t = t0 + rho;
      const bool valid = t < d.S;
      // (cos, sin)(t0 * theta_c) for every channel pair: one table row, the same for all threads.  Issued before
      // the wait so that the latency hides behind it.  The thread's own position is t0 + rho:
      // cos / sin of (t0 + rho) theta follow from the angle-addition formulas with (cos, sin)(rho * theta_c)
      // evaluated here (rho < 128, so the fast sine's argument stays small after one 2 pi reduction).
      float4 cs0[NCH * 8];
      if (d.flags & F_ROPE) {
        const float4* tab0 = reinterpret_cast<const float4*>(p.rope + (long long)t0 * HALF) + part * NCH * 8;
#pragma unroll
        for (int i = 0; i < NCH * 8; ++i) cs0[i] = tab0[i];
      }
      if (!mbar_wait(&acc_full[buf], (it >> 1) & 1, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_EPI); goto done; }
      tc_fence_after();
      const uint32_t acc = tmem_base + lane_sel + buf * DH;
      float sc = 1.f;
      if (d.flags & F_QK_NORM) {
        float ss = 0.f;
#pragma unroll
        for (int c = 0; c < DH / 32; ++c) {
          uint32_t r[32];
          tmem_ld32(acc + c * 32, r);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 32; ++i) ss = fmaf(__uint_as_float(r[i]), __uint_as_float(r[i]), ss);
        }
        sc = sqrtf((float)DH) * (is_q ? 1.f : __expf(p.temp[hj])) * rsqrtf(ss);
        if (valid && part == 0) p.rnorm[((long long)b * d.S + t) * (d.hq + d.hk) + h] = sc;
      }
      const long long tok = (long long)b * d.S + (valid ? t : 0);
      bf16* dst = is_q ? p.q + tok * d.Lq + h * DH : p.k + tok * d.Lk + hj * DH;
      const float rho_f = (float)rho;
#pragma unroll
      for (int cl = 0; cl < NCH; ++cl) {
        const int c = part * NCH + cl;                 // this thread's pairs: channels [16c, 16c+16) and + d_h/2
        uint32_t ra[16], rb[16];
        tmem_ld16(acc + c * 16, ra);
        tmem_ld16(acc + HALF + c * 16, rb);
        tmem_ld_wait();
        float lo[16], hi[16];
        if (d.flags & F_ROPE) {
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            float4 cs;                                                    // (cos, sin) x 2 channels at t0 + rho
            {
              const float4 z = cs0[cl * 8 + i];
              float sr, cr;
              float ang = rho_f * theta_s[c * 16 + 2 * i];
              float n = rintf(ang * 0.15915494309189535f);
              ang = fmaf(n, -6.2831854820251465f, ang);
              ang = fmaf(n, 1.7484555e-7f, ang);
              __sincosf(ang, &sr, &cr);
              cs.x = z.x * cr - z.y * sr;
              cs.y = z.y * cr + z.x * sr;
              ang = rho_f * theta_s[c * 16 + 2 * i + 1];
              n = rintf(ang * 0.15915494309189535f);
              ang = fmaf(n, -6.2831854820251465f, ang);
              ang = fmaf(n, 1.7484555e-7f, ang);
              __sincosf(ang, &sr, &cr);
              cs.z = z.z * cr - z.w * sr;
              cs.w = z.w * cr + z.z * sr;
            }
            const float a0 = __uint_as_float(ra[2 * i]) * sc, b0 = __uint_as_float(rb[2 * i]) * sc;
            const float a1 = __uint_as_float(ra[2 * i + 1]) * sc, b1 = __uint_as_float(rb[2 * i + 1]) * sc;
            lo[2 * i] = a0 * cs.x - b0 * cs.y;
            hi[2 * i] = b0 * cs.x + a0 * cs.y;
            lo[2 * i + 1] = a1 * cs.z - b1 * cs.w;
            hi[2 * i + 1] = b1 * cs.z + a1 * cs.w;
          }
        } else {
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            lo[i] = __uint_as_float(ra[i]) * sc;
            hi[i] = __uint_as_float(rb[i]) * sc;
          }
        }
        if (valid) {
#pragma unroll
          for (int v = 0; v < 2; ++v) {
            uint4 w;
            w.x = pack_bf16(lo[8 * v + 0], lo[8 * v + 1]);
            w.y = pack_bf16(lo[8 * v + 2], lo[8 * v + 3]);
            w.z = pack_bf16(lo[8 * v + 4], lo[8 * v + 5]);
            w.w = pack_bf16(lo[8 * v + 6], lo[8 * v + 7]);
            reinterpret_cast<uint4*>(dst + c * 16)[v] = w;
            w.x = pack_bf16(hi[8 * v + 0], hi[8 * v + 1]);
            w.y = pack_bf16(hi[8 * v + 2], hi[8 * v + 3]);
            w.z = pack_bf16(hi[8 * v + 4], hi[8 * v + 5]);
            w.w = pack_bf16(hi[8 * v + 6], hi[8 * v + 7]);
            reinterpret_cast<uint4*>(dst + HALF + c * 16)[v] = w;
          }
        }
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
  if (warp == TR_MMA_WARP) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 2 * DH);
  }
}

template <int DH, int KC>
int launch_tr(TcState* s, const CcaDims& d, const float* qk0, const bf16* w0, const bf16* w1, const float* temp,
              const float2* rope, bf16* q, bf16* k, float* rnorm, int t_first, int* status, cudaStream_t st) {
  static bool attr_done[TC_MAX_DEVICES] = {};
  using SM = TrSmem<DH, KC>;
  if (!attr_done[s->device]) {
    cudaError_t e = cudaFuncSetAttribute(tc_transform_fwd_kernel<DH, KC>, cudaFuncAttributeMaxDynamicSharedMemorySize, SM::TOTAL);
    if (e != cudaSuccess) return -(int)e;
    attr_done[s->device] = true;
  }
  TrParams p;
  p.d = d; p.qk0 = qk0; p.w0 = w0; p.w1 = w1; p.temp = temp; p.rope = rope; p.q = q; p.k = k; p.rnorm = rnorm; p.status = status;
  p.t_first = t_first;
  p.n_tiles = (d.S - t_first + 127) / 128;
  const long long uph = (long long)d.B * p.n_tiles, total = uph * (d.hq + d.hk);
  if (total > 0x7fffffffLL) return 1;
  p.units_per_head = (int)uph;
  p.total_units = (int)total;
  p.cost_q = 2;
  p.cost_k = (d.flags & F_QK_MEAN) ? 2 + d.g / 2 : 2;
  const int grid = (int)(total < s->sm_count ? total : s->sm_count);
  tc_transform_fwd_kernel<DH, KC><<<grid, TR_THREADS, SM::TOTAL, st>>>(p);
  cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? 0 : -(int)e;
}

}  // namespace

int tc_transform_fwd(TcState* s, const CcaDims& d, const float* qk0, const bf16* w0, const bf16* w1,
                     const float* temp, const float2* rope, bf16* q, bf16* k, float* rnorm, int* d_status,
                     cudaStream_t st, int t_first) {
  if (t_first % 128 || t_first < 0 || t_first >= d.S) return 1;
  if (!s || s->sm_count < 1) return 1;
  if (!(d.flags & F_CONV2)) return 1;                 // no contraction to run: the SIMT kernel is the right tool
  if (d.L % 4 || d.Lq % 8 || d.Lk % 8) return 1;
  if ((reinterpret_cast<uintptr_t>(w1) & 15) || (reinterpret_cast<uintptr_t>(qk0) & 15)) return 1;
  if (d.dh == 128) {
    if (d.k_ch == 1) return launch_tr<128, 1>(s, d, qk0, w0, w1, temp, rope, q, k, rnorm, t_first, d_status, st);
    if (d.k_ch == 2) return launch_tr<128, 2>(s, d, qk0, w0, w1, temp, rope, q, k, rnorm, t_first, d_status, st);
    return 1;
  }
  if (d.dh == 64) {
    if (d.k_ch == 1) return launch_tr<64, 1>(s, d, qk0, w0, w1, temp, rope, q, k, rnorm, t_first, d_status, st);
    if (d.k_ch == 2) return launch_tr<64, 2>(s, d, qk0, w0, w1, temp, rope, q, k, rnorm, t_first, d_status, st);
    if (d.k_ch == 3) return launch_tr<64, 3>(s, d, qk0, w0, w1, temp, rope, q, k, rnorm, t_first, d_status, st);
    if (d.k_ch == 4) return launch_tr<64, 4>(s, d, qk0, w0, w1, temp, rope, q, k, rnorm, t_first, d_status, st);
  }
  return 1;
}
