// Pieces shared by the forward attention kernels: launch parameters, the status helper and the exponential of
// eight scores with the rounded row sum.
#pragma once
#include "tc_kernels.cuh"
#include "tc_ptx.cuh"

namespace tc {

constexpr float LOG2E_F = 1.4426950408889634f;
constexpr float LN2_F = 0.6931471805599453f;
constexpr float RESCALE_THRESHOLD = 8.0f;      // log2 units

struct AttnParams {
  int B, S, hq, hk, g, Lq, Lk, causal;
  bf16* o;
  float* o32;
  float* lse;
  int n_blocks;       // query blocks per sequence that this launch covers
  int blk0;           // first of them (0: whole sequences)
  int* status;
  const float* temp;  // log key temperature per kv head if q, k are L2-normalised (Eq. 11), else null
};

TC_DEVINL void fail(volatile int* abort_flag, int* status, int code) {
  *abort_flag = 1;
  atomicCAS(status, 0, code);
}

// Exponentials of 8 consecutive scores (already in registers) -> 4 packed bf16 pairs; adds the rounded
// values to the two running partial sums in `sum2`.  POLY of the 4 pairs go through the
// polynomial.  CLAMP: x may be far below the smallest exponent (online mode); then it is clamped first.
template <int POLY, bool CLAMP>
TC_DEVINL void exp8(const uint32_t* v, uint64_t scale2, uint64_t negm2, uint64_t& sum2, uint32_t* out) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    uint64_t x = fma2(pack2u(v[2 * i], v[2 * i + 1]), scale2, negm2);
    uint64_t e;
    if (i < POLY) {
      if (CLAMP) {
        uint32_t a, b;
        unpack2u(x, a, b);
        x = pack2f(fmaxf(__uint_as_float(a), -120.f), fmaxf(__uint_as_float(b), -120.f));
      }
      e = exp2_poly2(x);
    } else {
      uint32_t a, b;
      unpack2u(x, a, b);
      e = pack2f(ex2f(__uint_as_float(a)), ex2f(__uint_as_float(b)));
    }
    // The row sum is taken over the bf16-rounded probabilities, the values the P V product really uses, so
    // that the weights of a row sum to one whatever the rounding did (with a fixed maximum even the
    // largest probability of a row is rounded).
    uint32_t a, b;
    unpack2u(e, a, b);
    const uint32_t w = pack_bf16(__uint_as_float(a), __uint_as_float(b));
    out[i] = w;
    sum2 = add2(sum2, pack2u(w << 16, w & 0xffff0000u));
  }
}

// The same for 16 consecutive scores -> 8 packed pairs, POLY8 of the 8 pairs through the polynomial.  SUM = false
// leaves the row sum to the caller (the tensor core adds the rounded probabilities against a column of ones).
template <int POLY8, bool CLAMP, bool SUM>
TC_DEVINL void exp16(const uint32_t* v, uint64_t scale2, uint64_t negm2, uint64_t& sum2, uint32_t* out) {
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    uint64_t x = fma2(pack2u(v[2 * i], v[2 * i + 1]), scale2, negm2);
    uint64_t e;
    if (i < POLY8) {
      if (CLAMP) {
        uint32_t a, b;
        unpack2u(x, a, b);
        x = pack2f(fmaxf(__uint_as_float(a), -120.f), fmaxf(__uint_as_float(b), -120.f));
      }
      e = exp2_poly2(x);
    } else {
      uint32_t a, b;
      unpack2u(x, a, b);
      e = pack2f(ex2f(__uint_as_float(a)), ex2f(__uint_as_float(b)));
    }
    uint32_t a, b;
    unpack2u(e, a, b);
    const uint32_t w = pack_bf16(__uint_as_float(a), __uint_as_float(b));
    out[i] = w;
    if (SUM) sum2 = add2(sum2, pack2u(w << 16, w & 0xffff0000u));
  }
}

}  // namespace tc
