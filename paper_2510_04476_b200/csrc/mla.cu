// MLA baseline (paper Section 2.1, Eq. 3-6): the element-wise step between its projections and the attention.
// The projections run on the library's GEMM kernels and the attention on its attention kernel (host side in
// cca_api.cu); this kernel builds the attention operands of Eq. 6 from the up-projected parts:
//     q[t,i] = [q_nope[t,i], RoPE(q_rope[t,i])],   k[t,i] = [k_nope[t,i], RoPE(k_rope[t])]   (one k_rope for all heads).
#include "common.cuh"

namespace {

// One block per token; items = (head, 8-channel chunk of the head's d_nope + d_rope channels), for q and for k.
__global__ void __launch_bounds__(256) mla_assemble_kernel(int S, int nh, int dn, int dr, const bf16* __restrict__ qn,
                                                           const bf16* __restrict__ qr, const bf16* __restrict__ kn,
                                                           const bf16* __restrict__ kr, const float2* __restrict__ rope,
                                                           bf16* __restrict__ q, bf16* __restrict__ k) {
  const long long tok = blockIdx.x;
  const int t = (int)(tok % S);
  const int dh = dn + dr, half = dr / 2;
  const int chunks = dh / 8, items = 2 * nh * chunks;
  for (int it = threadIdx.x; it < items; it += blockDim.x) {
    const int which = it / (nh * chunks), rem = it % (nh * chunks);
    const int i = rem / chunks, c0 = (rem % chunks) * 8;
    bf16* dst = (which ? k : q) + (tok * nh + i) * dh + c0;
    if (c0 < dn) {
      const bf16* src = (which ? kn : qn) + (tok * nh + i) * dn + c0;
      *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(src);
    } else {
      const bf16* src = which ? kr + tok * dr : qr + (tok * nh + i) * dr;
      const int r0 = c0 - dn;                      // first rope channel of this chunk
      __align__(16) bf16 outv[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const int c = r0 + e, pc = c < half ? c : c - half;      // pair (pc, pc + half)
        const float2 cs = rope[(long long)t * half + pc];
        const float a = __bfloat162float(src[pc]), b = __bfloat162float(src[pc + half]);
        outv[e] = __float2bfloat16(c < half ? a * cs.x - b * cs.y : b * cs.x + a * cs.y);
      }
      *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(outv);
    }
  }
}

}  // namespace

cudaError_t launch_mla_assemble(long long tokens, int S, int nh, int dn, int dr, const bf16* qn, const bf16* qr, const bf16* kn,
                                const bf16* kr, const float2* rope, bf16* q, bf16* k, cudaStream_t st) {
  mla_assemble_kernel<<<(unsigned)tokens, 256, 0, st>>>(S, nh, dn, dr, qn, qr, kn, kr, rope, q, k);
  return cudaGetLastError();
}
