// Tensor-core kernels, part 6: the large projection GEMMs on CTA pairs.
//   C[M,N] = sum_k A(m,k) B(n,k), A and B K-major or MN-major, bf16 operands, fp32 accumulate; optional split of the
//   k range over several work items whose partial sums are added to a zeroed fp32 output (weight gradients: K = tokens).
// Two CTAs on neighbouring SMs (a cluster of 2) work on one 256 x 256 tile with tcgen05.mma.cta_group::2:
// each CTA loads its own 128 rows of A and only HALF of the B tile (128 of the 256 output columns), the
// tensor cores of both SMs read B from both shared memories.  Per k-block a CTA therefore pulls 32 KB
// through the L2 instead of the 48 KB a stand-alone 128 x 256 tile needs, which is what limited that
// kernel.  Loads use plain TMA (no multicast); only the MMA-completion signal is sent to both CTAs.
//
//   warp 0      : TMA producer, in both CTAs (transaction bytes are counted on the leader CTA's barrier)
//   warp 1      : TMEM owner in both CTAs; in the leader CTA it issues the MMAs for the pair
//   warps 2..5  : epilogue, each CTA drains its own 128 accumulator rows from its own TMEM.  A thread holds one row of
//                 the accumulator (TMEM lane = row), so stored as they are the 32 lanes of a warp would write 16 bytes
//                 each into 32 different rows: 32 partial-sector requests per instruction, which bounded the GEMMs with
//                 a short k loop.  Each warp therefore turns its 32 x 32 block through a private 4 KB shared-memory
//                 stage (swizzled, conflict-free both ways) and stores whole 128-byte (fp32) or 64-byte (bf16) row
//                 segments, 4 or 8 rows per instruction.
#include <cstdio>

#include "tc_kernels.cuh"
#include "tc_ptx.cuh"
#include "tc_state.cuh"

using namespace tc;

namespace {

constexpr int G2_BM = 128;            // rows per CTA (256 per pair)
constexpr int G2_BK = 64;
constexpr int G2_THREADS = 192;

struct G2Params {
  int M, N, K;
  bf16* out_bf16;
  float* out_f32;
  long long ldc;
  int tiles_m, tiles_n, num_kb;     // tiles of 256 x 256
  int a_mn, b_mn;
  int splits, kb_per_split;   // work item = (tile, split)
  int vec_ok;
  int split_L, split_Lk, split_shift, seq_len, row0;   // fused down-projection output (see GemmArgs)
  bf16* out_lat_bf16;
  int* status;
};

template <int BN>
struct G2Smem {
  static constexpr int A_BYTES = G2_BM * G2_BK * 2;          // 16 KB
  static constexpr int B_BYTES = (BN / 2) * G2_BK * 2;       // this CTA's half of the B tile (16 or 12 KB)
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int STAGES = BN == 256 ? 6 : 7;
  static constexpr int BAR_OFFSET = STAGES * STAGE_BYTES;
  static constexpr int EPI_OFFSET = BAR_OFFSET + 256;        // four epilogue warps x 4 KB
  static constexpr int TOTAL = EPI_OFFSET + 4 * 4096 + 1024;
  static_assert(TOTAL <= 232448, "shared memory");
};

TC_DEVINL void fail(volatile int* abort_flag, int* status, int code) {
  *abort_flag = 1;
  atomicCAS(status, 0, code);
}
TC_DEVINL uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
TC_DEVINL void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// 2-D TMA tile load of one CTA of a pair; the bytes are counted on the barrier at the same offset in the
// pair's leader CTA (peer bit of the barrier address cleared)
TC_DEVINL void tma_load_2d_pair(void* dst, const CUtensorMap* map, int c0, int c1, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(c0), "r"(c1), "r"(smem_u32(bar) & 0xFEFFFFFFu)
      : "memory");
}
// D[tmem of both CTAs] (+)= A B over the pair: 256 x N x 16
TC_DEVINL void mma2_ss_w(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi, uint32_t idesc,
                         uint32_t accumulate) {
  const uint32_t z = 0;
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
      "mov.b64 da, {%1, %2};\n\tmov.b64 db, {%3, %4};\n\tsetp.ne.b32 p, %6, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %5, {%7, %7, %7, %7, %7, %7, %7, %7}, p;\n\t}"
      ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate), "r"(z)
      : "memory");
}
// arrive on the barrier at this offset in both CTAs of the pair once all MMAs issued so far have completed
TC_DEVINL void mma2_commit_both(uint64_t* bar) {
  const uint16_t mask = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(smem_u32(bar)), "h"(mask)
               : "memory");
}
// arrive on the barrier at this offset in CTA `rank` of the cluster
TC_DEVINL void mbar_arrive_cta(uint64_t* bar, uint32_t rank) {
  uint32_t remote;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(smem_u32(bar)), "r"(rank));
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(remote) : "memory");
}

template <int BN>
__global__ void __launch_bounds__(G2_THREADS, 1)
tc_gemm2_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, G2Params p) {
  using SM = G2Smem<BN>;
  constexpr int G2_BN = BN, G2_STAGES = SM::STAGES;
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = smem_align1024(smem_dyn);
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + SM::BAR_OFFSET);   // used in the leader CTA
  uint64_t* empty_bar = full_bar + G2_STAGES;                                 // one set per CTA
  uint64_t* acc_full = empty_bar + G2_STAGES;                                 // [2], one set per CTA
  uint64_t* acc_empty = acc_full + 2;                                         // [2], used in the leader CTA
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int num_tiles = p.tiles_m * p.tiles_n * p.splits;       // work items

  if (threadIdx.x == 0) {
    for (int s = 0; s < G2_STAGES; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&acc_full[s], 1);
      mbar_init(&acc_empty[s], 8);          // four epilogue warps of each CTA
    }
    wait_ctl_init(abort_flag, p.status);
    fence_barrier_init();
    prefetch_tmap(&tmA);
    prefetch_tmap(&tmB);
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                       // the peer's barriers exist before anything is sent to them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      for (int tile = pair; tile < num_tiles; tile += n_pairs) {
        const int sp = tile % p.splits, mn = tile / p.splits;
        const int m0 = (mn / p.tiles_n) * (2 * G2_BM) + (int)rank * G2_BM;
        const int n0 = (mn % p.tiles_n) * G2_BN + (int)rank * (G2_BN / 2);
        const int kb_end = min(p.num_kb, (sp + 1) * p.kb_per_split);
        for (int kb = sp * p.kb_per_split; kb < kb_end; ++kb) {
          if (!mbar_wait(&empty_bar[stage], phase ^ 1, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_TMA); goto done; }
          unsigned char* sa = smem + stage * SM::STAGE_BYTES;
          unsigned char* sb = sa + SM::A_BYTES;
          if (rank == 0) mbar_expect_tx(&full_bar[stage], 2 * SM::STAGE_BYTES);
          const int k0 = kb * G2_BK;
          if (!p.a_mn) {
            tma_load_2d_pair(sa, &tmA, k0, m0, &full_bar[stage]);
          } else {
            tma_load_2d_pair(sa, &tmA, m0, k0, &full_bar[stage]);
            tma_load_2d_pair(sa + 8192, &tmA, m0 + 64, k0, &full_bar[stage]);
          }
          if (!p.b_mn) {
            tma_load_2d_pair(sb, &tmB, k0, n0, &full_bar[stage]);
          } else {
#pragma unroll
            for (int c = 0; c < G2_BN / 128; ++c) tma_load_2d_pair(sb + c * 8192, &tmB, n0 + c * 64, k0, &full_bar[stage]);
          }
          if (++stage == G2_STAGES) { stage = 0; phase ^= 1; }
        }
      }
    }
  } else if (warp == 1) {
    if (rank == 0) {
      const bool leader = elect_one();
      // M = 256 over the pair, N = 256
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)p.a_mn << 15) | ((uint32_t)p.b_mn << 16) | ((uint32_t)(G2_BN >> 3) << 17) |
                             ((uint32_t)(256 >> 4) << 24);
      const uint32_t desc_hi = (uint32_t)(smem_desc_sw128(0, 0, 1024) >> 32);
      const uint32_t a_lbo = p.a_mn ? ((8192u >> 4) << 16) : (1u << 16), b_lbo = p.b_mn ? ((8192u >> 4) << 16) : (1u << 16);
      const uint32_t a_step = p.a_mn ? (2048u >> 4) : (32u >> 4), b_step = p.b_mn ? (2048u >> 4) : (32u >> 4);
      const uint32_t smem_lo = smem_u32(smem) >> 4;
      auto wait_all = [&](uint64_t* bar, uint32_t parity) -> bool {
        return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag));
      };
      int stage = 0;
      uint32_t phase = 0;
      int it = 0;
      for (int tile = pair; tile < num_tiles; tile += n_pairs, ++it) {
        const int as = it & 1;
        const uint32_t aphase = (it >> 1) & 1;
        if (!wait_all(&acc_empty[as], aphase ^ 1)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + as * G2_BN;
        const int sp = tile % p.splits;
        const int kb_begin = sp * p.kb_per_split, kb_end = min(p.num_kb, kb_begin + p.kb_per_split);
        for (int kb = kb_begin; kb < kb_end; ++kb) {
          if (!wait_all(&full_bar[stage], phase)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
          tc_fence_after();
          const uint32_t sa = (smem_lo + stage * (SM::STAGE_BYTES >> 4)) | a_lbo;
          const uint32_t sb = (smem_lo + stage * (SM::STAGE_BYTES >> 4) + (SM::A_BYTES >> 4)) | b_lbo;
          if (leader) {
#pragma unroll
            for (int k = 0; k < G2_BK / 16; ++k)
              mma2_ss_w(d_tmem, sa + k * a_step, desc_hi, sb + k * b_step, desc_hi, idesc, (kb != kb_begin) | (k != 0));
            mma2_commit_both(&empty_bar[stage]);
          }
          if (++stage == G2_STAGES) { stage = 0; phase ^= 1; }
        }
        if (leader) mma2_commit_both(&acc_full[as]);
      }
    }
  } else {
    const int q = warp & 3;                       // TMEM lane quarter this warp may access
    unsigned char* stg = smem + SM::EPI_OFFSET + (warp - 2) * 4096;
    // fp32 block: rows of 128 bytes, 16-byte chunk i of row r at chunk i ^ (r & 7)
    auto stage_f32 = [&](const uint32_t (&r)[32]) {
      __syncwarp();                               // the previous block has been read out
#pragma unroll
      for (int i = 0; i < 8; ++i)
        *reinterpret_cast<uint4*>(stg + lane * 128 + ((i ^ (lane & 7)) << 4)) = make_uint4(r[4 * i], r[4 * i + 1], r[4 * i + 2], r[4 * i + 3]);
      __syncwarp();
    };
    // 4 rows x 128 bytes per instruction: lane -> row 4 i + lane / 8, chunk lane % 8
    auto flush_f32 = [&](float* col0, long long ld, int m_first) {
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int rr = 4 * i + (lane >> 3), ch = lane & 7;
        const uint4 v = *reinterpret_cast<const uint4*>(stg + rr * 128 + ((ch ^ (rr & 7)) << 4));
        if (m_first + rr < p.M) *reinterpret_cast<uint4*>(col0 + (long long)(m_first + rr) * ld + ch * 4) = v;
      }
    };
    // bf16 block: rows of 64 bytes, chunk i of row r at chunk i ^ ((r >> 1) & 3)
    auto stage_bf16 = [&](const uint32_t (&r)[32]) {
      __syncwarp();
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        uint4 v;
        v.x = pack_bf16(__uint_as_float(r[8 * i + 0]), __uint_as_float(r[8 * i + 1]));
        v.y = pack_bf16(__uint_as_float(r[8 * i + 2]), __uint_as_float(r[8 * i + 3]));
        v.z = pack_bf16(__uint_as_float(r[8 * i + 4]), __uint_as_float(r[8 * i + 5]));
        v.w = pack_bf16(__uint_as_float(r[8 * i + 6]), __uint_as_float(r[8 * i + 7]));
        *reinterpret_cast<uint4*>(stg + lane * 64 + ((i ^ ((lane >> 1) & 3)) << 4)) = v;
      }
      __syncwarp();
    };
    // 8 rows x 64 bytes per instruction: lane -> row 8 i + lane / 4, chunk lane % 4.  value = true: the value columns of
    // the fused down-projection, stored `late` rows further down inside the same sequence (value shift), a zero row at
    // each sequence start.
    auto flush_bf16 = [&](bf16* col0, long long ld, int m_first, bool value, int late) {
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int rr = 8 * i + (lane >> 2), ch = lane & 3;
        const uint4 v = *reinterpret_cast<const uint4*>(stg + rr * 64 + ((ch ^ ((rr >> 1) & 3)) << 4));
        const int mm = m_first + rr;
        if (mm < p.M) {
          if (!value) {
            *reinterpret_cast<uint4*>(col0 + (long long)mm * ld + ch * 8) = v;
          } else {
            const int t = (mm + p.row0) % p.seq_len;
            if (!late || t + 1 < p.seq_len) *reinterpret_cast<uint4*>(col0 + (long long)(mm + late) * ld + ch * 8) = v;
            if (late && t == 0) *reinterpret_cast<uint4*>(col0 + (long long)mm * ld + ch * 8) = make_uint4(0u, 0u, 0u, 0u);   // x_{-1} = 0
          }
        }
      }
    };
    int it = 0;
    for (int tile = pair; tile < num_tiles; tile += n_pairs, ++it) {
      const int as = it & 1;
      const uint32_t aphase = (it >> 1) & 1;
      const int mn = tile / p.splits;
      const int m0 = (mn / p.tiles_n) * (2 * G2_BM) + (int)rank * G2_BM, n0 = (mn % p.tiles_n) * G2_BN;
      if (!mbar_wait(&acc_full[as], aphase, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_EPI); goto done; }
      tc_fence_after();
      const int m = m0 + q * 32 + lane;
      const int m_base = m0 + q * 32;               // first row of this warp's block
#pragma unroll 1
      for (int c = 0; c < G2_BN / 32; ++c) {
        uint32_t r[32];
        tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + as * G2_BN + c * 32, r);
        tmem_ld_wait();
        const int n = n0 + c * 32;
        if (n >= p.N) continue;                     // (warp-uniform)
        const bool whole = n + 32 <= p.N;
        if (p.split_L > 0) {
          // fused down-projection: latent columns in fp32, value columns in bf16 (second half one token later)
          if (n < p.split_L) {
            stage_f32(r);
            flush_f32(p.out_f32 + n, p.ldc, m_base);
            if (p.out_lat_bf16) {                   // the operand copy the latent-transform kernel loads by TMA
              stage_bf16(r);
              flush_bf16(p.out_lat_bf16 + n, p.split_L, m_base, false, 0);
            }
          } else {
            const int vc = n - p.split_L;
            stage_bf16(r);
            flush_bf16(p.out_bf16 + vc, p.split_Lk, m_base, true, (p.split_shift && vc >= p.split_Lk / 2) ? 1 : 0);
          }
        } else if (p.out_bf16 && p.vec_ok && whole) {
          stage_bf16(r);
          flush_bf16(p.out_bf16 + n, p.ldc, m_base, false, 0);
        } else if (p.out_f32 && p.splits == 1 && p.vec_ok && whole) {
          stage_f32(r);
          flush_f32(p.out_f32 + n, p.ldc, m_base);
        } else if (m < p.M) {
          if (p.out_bf16) {
            bf16* dst = p.out_bf16 + (long long)m * p.ldc + n;
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (n + i < p.N) dst[i] = __float2bfloat16(__uint_as_float(r[i]));
          } else {
            float* dst = p.out_f32 + (long long)m * p.ldc + n;
            if (p.splits > 1) {
              if (p.vec_ok && whole) {
#pragma unroll
                for (int i = 0; i < 8; ++i)
                  asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(dst + 4 * i), "f"(__uint_as_float(r[4 * i])),
                               "f"(__uint_as_float(r[4 * i + 1])), "f"(__uint_as_float(r[4 * i + 2])),
                               "f"(__uint_as_float(r[4 * i + 3]))
                               : "memory");
              } else {
#pragma unroll
                for (int i = 0; i < 32; ++i)
                  if (n + i < p.N) atomicAdd(dst + i, __uint_as_float(r[i]));
              }
            } else {
#pragma unroll
              for (int i = 0; i < 32; ++i)
                if (n + i < p.N) dst[i] = __uint_as_float(r[i]);
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cta(&acc_empty[as], 0);     // the leader CTA's barrier, from either CTA
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
  // neither CTA may leave while the other can still read its shared memory or signal its barriers
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
  }
}

template <int BN>
int launch_pair(TcState* s, const GemmArgs& g, const G2Params& p0, bool a_mn, bool b_mn, long long lda, long long ldb,
                cudaStream_t st) {
  static bool attr_set[TC_MAX_DEVICES] = {};
  using SM = G2Smem<BN>;
  if (!attr_set[s->device]) {
    cudaError_t e = cudaFuncSetAttribute(tc_gemm2_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, SM::TOTAL);
    if (e != cudaSuccess) return -(int)e;
    attr_set[s->device] = true;
  }
  CUtensorMap tmA, tmB;
  bool ok;
  if (!a_mn) ok = tc_make_map_2d(s, &tmA, g.A.p, (uint64_t)g.K, (uint64_t)g.M, (uint64_t)lda, G2_BK, G2_BM);
  else ok = tc_make_map_2d(s, &tmA, g.A.p, (uint64_t)g.M, (uint64_t)g.K, (uint64_t)lda, 64, G2_BK);
  if (!ok) return 1;
  if (!b_mn) ok = tc_make_map_2d(s, &tmB, g.B.p, (uint64_t)g.K, (uint64_t)g.N, (uint64_t)ldb, G2_BK, BN / 2);
  else ok = tc_make_map_2d(s, &tmB, g.B.p, (uint64_t)g.N, (uint64_t)g.K, (uint64_t)ldb, 64, G2_BK);
  if (!ok) return 1;
  G2Params p = p0;
  p.tiles_n = (g.N + BN - 1) / BN;
  // split the k range when that fills the waves of CTA pairs better (fp32 output that the items can add into)
  p.splits = 1;
  if (g.out_f32 && !g.out_bf16 && g.split_L == 0 && g.ldc == g.N && p.num_kb >= 32) {
    const long long mn = (long long)p.tiles_m * p.tiles_n;
    double best = 1e30;
    for (int sp = 1; sp <= 8 && sp * 16 <= p.num_kb; ++sp) {
      const long long waves = (mn * sp + s->pair_clusters - 1) / s->pair_clusters;
      const double c = (double)waves / sp * (1.0 + 0.03 * (sp - 1));
      if (c < best - 1e-9) { best = c; p.splits = sp; }
    }
  }
  p.kb_per_split = (p.num_kb + p.splits - 1) / p.splits;
  p.splits = (p.num_kb + p.kb_per_split - 1) / p.kb_per_split;     // no empty split
  if (p.splits > 1) {
    cudaError_t me = cudaMemsetAsync(g.out_f32, 0, (size_t)g.M * g.N * sizeof(float), st);
    if (me != cudaSuccess) return -(int)me;
  }
  const int tiles = p.tiles_m * p.tiles_n * p.splits;
  const int pairs = tiles < s->pair_clusters ? tiles : s->pair_clusters;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * pairs, 1, 1);
  cfg.blockDim = dim3(G2_THREADS, 1, 1);
  cfg.dynamicSmemBytes = SM::TOTAL;
  cfg.stream = st;
  cudaLaunchAttribute at;
  at.id = cudaLaunchAttributeClusterDimension;
  at.val.clusterDim.x = 2; at.val.clusterDim.y = 1; at.val.clusterDim.z = 1;
  cfg.attrs = &at; cfg.numAttrs = 1;
  cudaError_t e = cudaLaunchKernelEx(&cfg, tc_gemm2_kernel<BN>, tmA, tmB, p);
  return e == cudaSuccess ? 0 : -(int)e;
}

}  // namespace

// Returns 0 if enqueued, 1 if the case is outside this kernel's coverage, -cudaError on failure.
int tc_gemm_pair(TcState* s, const GemmArgs& g, int* d_status, cudaStream_t st) {
  if (g.accumulate) return 1;                       // the one-CTA kernel handles accumulation into the output
  if (!s || !s->encode || !s->use_pairs) return 1;
  if (g.a_row_off != 0) return 1;                                 // no row shift
  const int a_mn = g.A.cs != 1, b_mn = g.B.cs != 1;
  if ((a_mn && g.A.rs != 1) || (b_mn && g.B.rs != 1)) return 1;
  if (a_mn && g.split_L > 0) return 1;
  const long long lda = a_mn ? g.A.cs : g.A.rs, ldb = b_mn ? g.B.cs : g.B.rs;
  if (lda % 8 || ldb % 8) return 1;
  if ((reinterpret_cast<uintptr_t>(g.A.p) & 15) || (reinterpret_cast<uintptr_t>(g.B.p) & 15)) return 1;
  if (g.M < 512 || g.N < 256 || g.K < 64) return 1;
  if (g.split_L > 0) {
    if (g.split_L % 32 || (g.split_Lk / 2) % 32 || g.N != g.split_L + g.split_Lk || g.ldc % 4 || g.split_Lk % 8) return 1;
    if ((reinterpret_cast<uintptr_t>(g.out_f32) & 15) || (reinterpret_cast<uintptr_t>(g.out_bf16) & 15)) return 1;
  }
  if (s->pair_clusters < 0) {
    cudaError_t e = cudaFuncSetAttribute(tc_gemm2_kernel<256>, cudaFuncAttributeMaxDynamicSharedMemorySize, G2Smem<256>::TOTAL);
    if (e != cudaSuccess) return -(int)e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * s->sm_count, 1, 1);
    cfg.blockDim = dim3(G2_THREADS, 1, 1);
    cfg.dynamicSmemBytes = G2Smem<256>::TOTAL;
    cudaLaunchAttribute at;
    at.id = cudaLaunchAttributeClusterDimension;
    at.val.clusterDim.x = 2; at.val.clusterDim.y = 1; at.val.clusterDim.z = 1;
    cfg.attrs = &at; cfg.numAttrs = 1;
    int n = 0;
    e = cudaOccupancyMaxActiveClusters(&n, tc_gemm2_kernel<256>, &cfg);
    s->pair_clusters = (e == cudaSuccess) ? n : 0;
    if (e != cudaSuccess) (void)cudaGetLastError();
  }
  if (s->pair_clusters < 8) return 1;
  G2Params p;
  p.M = g.M; p.N = g.N; p.K = g.K;
  p.out_bf16 = g.out_bf16; p.out_f32 = g.out_f32; p.ldc = g.ldc;
  p.tiles_m = (g.M + 2 * G2_BM - 1) / (2 * G2_BM);
  p.tiles_n = 0;
  p.num_kb = (g.K + G2_BK - 1) / G2_BK;
  p.a_mn = a_mn; p.b_mn = b_mn;
  p.splits = 1; p.kb_per_split = p.num_kb;
  const void* outp = g.out_bf16 ? (const void*)g.out_bf16 : (const void*)g.out_f32;
  const int esz = g.out_bf16 ? 2 : 4;
  p.vec_ok = ((reinterpret_cast<uintptr_t>(outp) & 15) == 0) && ((g.ldc * esz) % 16 == 0);
  p.split_L = g.split_L; p.split_Lk = g.split_Lk; p.split_shift = g.split_shift; p.seq_len = g.seq_len > 0 ? g.seq_len : 1;
  p.row0 = g.row0;
  p.out_lat_bf16 = (g.split_L > 0 && g.split_L % 32 == 0 && !(reinterpret_cast<uintptr_t>(g.out_lat_bf16) & 15)) ? g.out_lat_bf16 : nullptr;
  if (g.out_lat_bf16 && !p.out_lat_bf16) return 1;
  p.status = d_status;
  // tile width: fewer, fuller waves of CTA pairs win (time of a wave is proportional to the tile width)
  auto cost = [&](int bn) {
    const long long tiles = (long long)p.tiles_m * ((g.N + bn - 1) / bn);
    return ((tiles + s->pair_clusters - 1) / s->pair_clusters) * bn;
  };
  // (an MN-major B half of 96 columns would not be a whole number of 64-column swizzle chunks)
  const bool narrow = s->gemm_bn == 192 ? true : s->gemm_bn == 256 ? false : cost(192) < cost(256);
  if (!b_mn && narrow) return launch_pair<192>(s, g, p, a_mn, b_mn, lda, ldb, st);
  return launch_pair<256>(s, g, p, a_mn, b_mn, lda, ldb, st);
}
