// Tensor-core kernels, part 1: persistent warp-specialised GEMM  C[M,N] = sum_k A(m,k) B(n,k)
// on tcgen05 with TMEM accumulators and TMA-fed shared memory (bf16 operands, fp32 accumulate).
//
//   warp 0      : TMA producer (one lane)            -- fills a 4-stage ring of (A, B) k-blocks
//   warp 1      : TMEM owner + MMA issuer (one lane) -- 4 x tcgen05.mma (128 x BN x 16) per k-block
//   warps 2..5  : epilogue -- tcgen05.ld of the finished accumulator, convert, store to global
//
// The accumulator is double-buffered in TMEM (2 x BN columns) so that the epilogue of tile i overlaps
// the main loop of tile i+1.  Every wait is bounded; on expiry the CTA records a status code, lets its
// copies drain, frees its TMEM and returns.
#include "tc_kernels.cuh"

#include <cstdio>
#include <cstdlib>
#include <new>

#include "tc_ptx.cuh"
#include "tc_state.cuh"

using namespace tc;

namespace {

constexpr int GEMM_BM = 128, GEMM_BK = 64, GEMM_STAGES = 4;
constexpr int GEMM_THREADS = 192;

struct TcGemmParams {
  int M, N, K;
  int a_row_off, seq_len;
  bf16* out_bf16;
  float* out_f32;
  long long ldc;
  int tiles_m, tiles_n, num_kb;
  int splits, kb_per_split;   // split-K: work item = (tile, split); partial sums are added atomically (fp32 output)
  int a_mn, b_mn;
  int vec_ok;            // rows of C are 16-byte aligned: vector stores allowed
  int atomic_out;        // add into the fp32 output (split-K partial sums, or the caller's accumulate)
  int* status;
};

template <int BN>
struct GemmSmem {
  static constexpr int A_BYTES = GEMM_BM * GEMM_BK * 2;
  static constexpr int B_BYTES = BN * GEMM_BK * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int BAR_OFFSET = GEMM_STAGES * STAGE_BYTES;
  static constexpr int TOTAL = BAR_OFFSET + 256 + 1024;   // barriers + slack for 1024-byte alignment
};

TC_DEVINL void fail(volatile int* abort_flag, int* status, int code) {
  *abort_flag = 1;
  atomicCAS(status, 0, code);
}

template <int BN>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, TcGemmParams p) {
  using SM = GemmSmem<BN>;
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = smem_align1024(smem_dyn);
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + SM::BAR_OFFSET);
  uint64_t* empty_bar = full_bar + GEMM_STAGES;
  uint64_t* acc_full = empty_bar + GEMM_STAGES;     // [2]
  uint64_t* acc_empty = acc_full + 2;               // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int num_tiles = p.tiles_m * p.tiles_n * p.splits;      // work items

  if (threadIdx.x == 0) {
    for (int s = 0; s < GEMM_STAGES; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&acc_full[s], 1);
      mbar_init(&acc_empty[s], 4);
    }
    wait_ctl_init(abort_flag, p.status);
    fence_barrier_init();
    prefetch_tmap(&tmA);
    prefetch_tmap(&tmB);
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, 2 * BN);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x) {
        const int sp = tile % p.splits, mn = tile / p.splits;
        const int m0 = (mn / p.tiles_n) * GEMM_BM, n0 = (mn % p.tiles_n) * BN;
        const int kb_end = min(p.num_kb, (sp + 1) * p.kb_per_split);
        for (int kb = sp * p.kb_per_split; kb < kb_end; ++kb) {
          if (!mbar_wait(&empty_bar[stage], phase ^ 1, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_TMA); goto done; }
          unsigned char* sa = smem + stage * SM::STAGE_BYTES;
          unsigned char* sb = sa + SM::A_BYTES;
          mbar_expect_tx(&full_bar[stage], SM::STAGE_BYTES);
          const int k0 = kb * GEMM_BK;
          if (!p.a_mn) {
            tma_load_2d(sa, &tmA, k0, m0 + p.a_row_off, &full_bar[stage]);
          } else {
            tma_load_2d(sa, &tmA, m0, k0, &full_bar[stage]);
            tma_load_2d(sa + 8192, &tmA, m0 + 64, k0, &full_bar[stage]);
          }
          if (!p.b_mn) {
            tma_load_2d(sb, &tmB, k0, n0, &full_bar[stage]);
          } else {
#pragma unroll
            for (int c = 0; c < BN / 64; ++c) tma_load_2d(sb + c * 8192, &tmB, n0 + c * 64, k0, &full_bar[stage]);
          }
          if (++stage == GEMM_STAGES) { stage = 0; phase ^= 1; }
        }
      }
    }
  } else if (warp == 1) {
    // The whole warp runs the loop so that the address arithmetic stays warp-uniform; one elected lane issues.
    const bool leader = elect_one();
    const uint32_t idesc = idesc_bf16(BN, p.a_mn, p.b_mn);
    // descriptor words: high = stride offset 1024, version, 128-byte swizzle; low = address >> 4 | leading offset << 16
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
    for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x, ++it) {
      const int as = it & 1;
      const uint32_t aphase = (it >> 1) & 1;
      if (!wait_all(&acc_empty[as], aphase ^ 1)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
      tc_fence_after();
      const uint32_t d_tmem = tmem_base + as * BN;
      const int sp = tile % p.splits;
      const int kb_begin = sp * p.kb_per_split, kb_end = min(p.num_kb, kb_begin + p.kb_per_split);
      for (int kb = kb_begin; kb < kb_end; ++kb) {
        if (!wait_all(&full_bar[stage], phase)) { fail(abort_flag, p.status, ST_TIMEOUT_MMA); goto done; }
        tc_fence_after();
        const uint32_t sa = (smem_lo + stage * (SM::STAGE_BYTES >> 4)) | a_lbo;
        const uint32_t sb = (smem_lo + stage * (SM::STAGE_BYTES >> 4) + (SM::A_BYTES >> 4)) | b_lbo;
        if (leader) {
#pragma unroll
          for (int k = 0; k < GEMM_BK / 16; ++k)
            mma_ss_w(d_tmem, sa + k * a_step, desc_hi, sb + k * b_step, desc_hi, idesc, ((kb - kb_begin) | k) != 0);
          mma_commit(&empty_bar[stage]);
        }
        if (++stage == GEMM_STAGES) { stage = 0; phase ^= 1; }
      }
      if (leader) mma_commit(&acc_full[as]);
    }
  } else {
    const int q = warp & 3;                       // TMEM lane quarter this warp may access
    int it = 0;
    for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x, ++it) {
      const int as = it & 1;
      const uint32_t aphase = (it >> 1) & 1;
      const int mn = tile / p.splits;
      const int m0 = (mn / p.tiles_n) * GEMM_BM, n0 = (mn % p.tiles_n) * BN;
      if (!mbar_wait(&acc_full[as], aphase, abort_flag)) { fail(abort_flag, p.status, ST_TIMEOUT_EPI); goto done; }
      tc_fence_after();
      const int m = m0 + q * 32 + lane;
      bool zero_row = false;
      if (p.a_row_off != 0) {
        const int t = m % p.seq_len + p.a_row_off;
        zero_row = (t < 0) || (t >= p.seq_len);
      }
#pragma unroll 1
      for (int c = 0; c < BN / 32; ++c) {
        uint32_t r[32];
        tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + as * BN + c * 32, r);
        tmem_ld_wait();
        const int n = n0 + c * 32;
        if (m < p.M && n < p.N) {
          if (zero_row) {
#pragma unroll
            for (int i = 0; i < 32; ++i) r[i] = 0u;
          }
          if (p.out_bf16) {
            bf16* dst = p.out_bf16 + (long long)m * p.ldc + n;
            if (p.vec_ok && n + 32 <= p.N) {
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                uint4 v;
                v.x = pack_bf16(__uint_as_float(r[8 * i + 0]), __uint_as_float(r[8 * i + 1]));
                v.y = pack_bf16(__uint_as_float(r[8 * i + 2]), __uint_as_float(r[8 * i + 3]));
                v.z = pack_bf16(__uint_as_float(r[8 * i + 4]), __uint_as_float(r[8 * i + 5]));
                v.w = pack_bf16(__uint_as_float(r[8 * i + 6]), __uint_as_float(r[8 * i + 7]));
                reinterpret_cast<uint4*>(dst)[i] = v;
              }
            } else {
#pragma unroll
              for (int i = 0; i < 32; ++i)
                if (n + i < p.N) dst[i] = __float2bfloat16(__uint_as_float(r[i]));
            }
          } else {
            float* dst = p.out_f32 + (long long)m * p.ldc + n;
            if (p.atomic_out) {
#pragma unroll
              for (int i = 0; i < 32; ++i)
                if (n + i < p.N) atomicAdd(dst + i, __uint_as_float(r[i]));
            } else if (p.vec_ok && n + 32 <= p.N) {
#pragma unroll
              for (int i = 0; i < 8; ++i)
                reinterpret_cast<uint4*>(dst)[i] = make_uint4(r[4 * i], r[4 * i + 1], r[4 * i + 2], r[4 * i + 3]);
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
      if (lane == 0) mbar_arrive(&acc_empty[as]);
    }
  }
done:
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    // let copies and MMAs that are still in flight land before the shared memory and TMEM go away
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000) {}
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 2 * BN);
  }
}

}  // namespace

// 2-D bf16 tensor map: dim0 (contiguous) extent d0, dim1 extent d1 with row pitch ld elements.
bool tc_make_map_2d(TcState* s, CUtensorMap* map, const void* base, uint64_t d0, uint64_t d1, uint64_t ld,
                    uint32_t box0, uint32_t box1) {
  cuuint64_t dims[2] = {d0, d1};
  cuuint64_t strides[1] = {ld * 2};
  cuuint32_t box[2] = {box0, box1};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = s->encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

bool tc_make_map_3d(TcState* s, CUtensorMap* map, const void* base, uint64_t d0, uint64_t d1, uint64_t d2,
                    uint64_t ld1, uint64_t ld2, uint32_t box0, uint32_t box1) {
  cuuint64_t dims[3] = {d0, d1, d2};
  cuuint64_t strides[2] = {ld1 * 2, ld2 * 2};
  cuuint32_t box[3] = {box0, box1, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = s->encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

TcState* tc_create(int sm_count) {
  TcState* s = new (std::nothrow) TcState();
  if (!s) return nullptr;
  s->sm_count = sm_count;
  s->device = 0;
  if (cudaGetDevice(&s->device) != cudaSuccess || s->device < 0 || s->device >= TC_MAX_DEVICES) {
    (void)cudaGetLastError();
    delete s;
    return nullptr;
  }
  s->encode = nullptr;
  s->attr_set_128 = s->attr_set_256 = false;
  s->pair_clusters = -1;
  s->use_pairs = 1;
  if (const char* e = getenv("CCA_GEMM_PAIRS")) s->use_pairs = atoi(e);
  s->gemm_bn = 0;
  if (const char* e = getenv("CCA_GEMM_BN")) s->gemm_bn = atoi(e);
  s->attn_attr_set[0] = s->attn_attr_set[1] = false;
  s->attn_poly = -1;      // -1: per head size (0 at d_h = 128, 2 of 8 at d_h = 64)
  if (const char* e = getenv("CCA_ATTN_POLY")) s->attn_poly = atoi(e);
  s->attn_bwd_fused = 1;
  if (const char* e = getenv("CCA_ATTN_BWD_FUSED")) s->attn_bwd_fused = atoi(e);
  s->attn_poly_bwd = -1;
  if (const char* e = getenv("CCA_ATTN_POLY_BWD")) s->attn_poly_bwd = atoi(e);
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess || !fn) {
    delete s;
    return nullptr;
  }
  s->encode = reinterpret_cast<EncodeTiledFn>(fn);
  return s;
}

void tc_destroy(TcState* s) { delete s; }

int tc_gemm(TcState* s, const GemmArgs& g, int* d_status, cudaStream_t st) {
  if (!s || !s->encode) return 1;
  if (g.M <= 0 || g.N <= 0 || g.K <= 0) return 1;
  const int a_mn = g.A.cs != 1, b_mn = g.B.cs != 1;
  const long long lda = a_mn ? g.A.cs : g.A.rs, ldb = b_mn ? g.B.cs : g.B.rs;
  if ((a_mn && g.A.rs != 1) || (b_mn && g.B.rs != 1)) return 1;
  if (lda % 8 || ldb % 8) return 1;
  if ((reinterpret_cast<uintptr_t>(g.A.p) & 15) || (reinterpret_cast<uintptr_t>(g.B.p) & 15)) return 1;
  if (a_mn && g.a_row_off != 0) return 1;
  if (g.N < 16 || g.M < 1) return 1;
  const int BN = (g.N > 128) ? 256 : 128;
  CUtensorMap tmA, tmB;
  bool ok;
  if (!a_mn) ok = tc_make_map_2d(s, &tmA, g.A.p, (uint64_t)g.K, (uint64_t)g.M, (uint64_t)lda, GEMM_BK, GEMM_BM);
  else ok = tc_make_map_2d(s, &tmA, g.A.p, (uint64_t)g.M, (uint64_t)g.K, (uint64_t)lda, 64, GEMM_BK);
  if (!ok) return 1;
  if (!b_mn) ok = tc_make_map_2d(s, &tmB, g.B.p, (uint64_t)g.K, (uint64_t)g.N, (uint64_t)ldb, GEMM_BK, BN);
  else ok = tc_make_map_2d(s, &tmB, g.B.p, (uint64_t)g.N, (uint64_t)g.K, (uint64_t)ldb, 64, GEMM_BK);
  if (!ok) return 1;
  TcGemmParams p;
  p.M = g.M; p.N = g.N; p.K = g.K;
  p.a_row_off = g.a_row_off; p.seq_len = g.seq_len > 0 ? g.seq_len : 1;
  p.out_bf16 = g.out_bf16; p.out_f32 = g.out_f32; p.ldc = g.ldc;
  p.tiles_m = (g.M + GEMM_BM - 1) / GEMM_BM;
  p.tiles_n = (g.N + BN - 1) / BN;
  p.num_kb = (g.K + GEMM_BK - 1) / GEMM_BK;
  // split-K when the output has too few tiles to fill the machine and the reduction is long (weight gradients)
  p.splits = 1;
  {
    const int mn_tiles = p.tiles_m * p.tiles_n;
    if (g.out_f32 && g.ldc == g.N && g.a_row_off == 0 && mn_tiles * 2 <= s->sm_count && p.num_kb >= 16) {
      int sp = s->sm_count / mn_tiles;
      if (sp > p.num_kb / 8) sp = p.num_kb / 8;
      if (sp > 1) p.splits = sp;
    }
  }
  p.kb_per_split = (p.num_kb + p.splits - 1) / p.splits;
  p.splits = (p.num_kb + p.kb_per_split - 1) / p.kb_per_split;     // no empty split
  if (g.accumulate && !g.out_f32) return 1;
  if (p.splits > 1 && !g.accumulate) {
    cudaError_t me = cudaMemsetAsync(g.out_f32, 0, (size_t)g.M * g.N * sizeof(float), st);
    if (me != cudaSuccess) return -(int)me;
  }
  p.atomic_out = (p.splits > 1 || g.accumulate) ? 1 : 0;
  p.a_mn = a_mn; p.b_mn = b_mn;
  const void* outp = g.out_bf16 ? (const void*)g.out_bf16 : (const void*)g.out_f32;
  const int esz = g.out_bf16 ? 2 : 4;
  p.vec_ok = ((reinterpret_cast<uintptr_t>(outp) & 15) == 0) && ((g.ldc * esz) % 16 == 0);
  p.status = d_status;
  const int tiles = p.tiles_m * p.tiles_n * p.splits;
  const int grid = tiles < s->sm_count ? tiles : s->sm_count;
  cudaError_t e;
  if (BN == 256) {
    if (!s->attr_set_256) {
      e = cudaFuncSetAttribute(tc_gemm_kernel<256>, cudaFuncAttributeMaxDynamicSharedMemorySize, GemmSmem<256>::TOTAL);
      if (e != cudaSuccess) return -(int)e;
      s->attr_set_256 = true;
    }
    tc_gemm_kernel<256><<<grid, GEMM_THREADS, GemmSmem<256>::TOTAL, st>>>(tmA, tmB, p);
  } else {
    if (!s->attr_set_128) {
      e = cudaFuncSetAttribute(tc_gemm_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, GemmSmem<128>::TOTAL);
      if (e != cudaSuccess) return -(int)e;
      s->attr_set_128 = true;
    }
    tc_gemm_kernel<128><<<grid, GEMM_THREADS, GemmSmem<128>::TOTAL, st>>>(tmA, tmB, p);
  }
  e = cudaGetLastError();
  return e == cudaSuccess ? 0 : -(int)e;
}

