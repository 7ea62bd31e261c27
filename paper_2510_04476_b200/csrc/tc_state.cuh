// State shared by the tensor-core launchers: the driver entry point that encodes TMA tensor maps.
#pragma once
#include <cuda.h>

#include "tc_kernels.cuh"

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// cudaFuncSetAttribute is per device; each launcher remembers per device (index = TcState::device) whether its
// kernel has been opted in to its dynamic shared-memory size.
constexpr int TC_MAX_DEVICES = 64;

struct TcState {
  int sm_count;
  int device;             // device the handle was created on (current at tc_create), < TC_MAX_DEVICES
  EncodeTiledFn encode;
  bool attr_set_128, attr_set_256;
  int pair_clusters;      // co-resident CTA pairs of the pair GEMM (-1: not asked yet, 0: unavailable)
  int use_pairs;          // 0 disables the pair GEMM
  int gemm_bn;            // tile width of the pair GEMM: 0 = chosen per shape, 192 or 256 = forced
  bool attn_attr_set[2];
  int attn_poly_bwd;      // the same share in the backward kernels
  int attn_bwd_fused;     // head size 64: the one-kernel attention adjoint (0: the dQ and dK/dV kernels)
  int attn_poly;          // forward: of every 8 score pairs, how many take the polynomial exp2 (-1: per head size)
};

// bf16 tensor maps with 128-byte swizzle.  2-D: dim0 (contiguous) extent d0, dim1 extent d1, row pitch ld
// elements.  3-D adds an outer dimension d2 with pitch ld2 elements.
bool tc_make_map_2d(TcState* s, CUtensorMap* map, const void* base, uint64_t d0, uint64_t d1, uint64_t ld,
                    uint32_t box0, uint32_t box1);
bool tc_make_map_3d(TcState* s, CUtensorMap* map, const void* base, uint64_t d0, uint64_t d1, uint64_t d2,
                    uint64_t ld1, uint64_t ld2, uint32_t box0, uint32_t box1);
