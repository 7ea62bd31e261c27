// Decode step: one new token per sequence against the latent KV cache (the KV-cache and decode columns of the
// paper's comparison table).  Everything here is bound by memory traffic -- the weights are read once per step
// and every cached key and value row once per (sequence, kv head) -- so these are plain CUDA kernels laid out
// for coalesced 16-byte accesses, not tcgen05 tiles (the attention uses warp-level tensor-core instructions only to
// keep its instruction count below what the loads need):
//
//   decode_proj_kernel      out[b, n] = sum_k W[n, k] x[b, k] for a few stacked weight segments (Eq. 7, 10; Eq. 11
//                           up-projection; also conv2 of Eq. 8, a contraction over (input channel, tap) per head)
//   decode_conv1_kernel     Eq. 8 conv1 at the tokens conv2 reads, from the caller's history; appends v to the cache,
//                           advances the history and the previous input
//   decode_finalize_kernel  Eq. 9, 11 for the new token of one (sequence, head): q-k-mean, norm, temperature, RoPE at
//                           the sequence's own position; appends k to the cache
//   decode_attn_kernel      softmax(q k^T / sqrt(d_h)) v of the new query over a chunk of the cached keys of one
//                           (sequence, kv head), all its query heads at once; partial results per chunk
//   decode_combine_kernel   merges the chunks' partial results
#include <cstdlib>
#include <cstring>

#include "common.cuh"
#include "decode.cuh"

namespace {

// Programmatic dependent launch: every kernel of the step lets the next one be scheduled as soon as all of its own
// CTAs have started, and waits for the kernel before it (completion and visibility of its writes) before it touches
// global memory.  The wait comes first in every CTA, also in those that return early, so that "kernel N complete"
// always implies "kernel N - 1 complete".
CCA_DEVINL void pdl_enter() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = 0;
  cfg.stream = st;
  cudaLaunchAttribute at;
  at.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &at;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, args...);
}

constexpr unsigned F_CONV1 = 1, F_CONV2 = 2, F_QK_MEAN = 4, F_V_SHIFT = 8, F_QK_NORM = 16, F_ROPE = 32;
constexpr int ST_DECODE_BAD_POSITION = 120;
constexpr float LOG2E = 1.4426950408889634f;

CCA_DEVINL void mma_16816(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
CCA_DEVINL uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// ------------------------------------------------------------------------------------------------ projections
// out[b, n] = sum_k W[n, k] x[b, k]: 16 weight rows per CTA as the rows of m16n8k16 tiles, 32 sequences as four
// column tiles, the inner dimension split over the 8 warps and summed through shared memory.  A lane loads 16
// contiguous bytes of a weight row and of an input row and feeds them to two tensor-core instructions (the inner
// index may be taken in any order as long as both operands agree), so every load is a full 64-byte piece of a row.
constexpr int PJ_WARPS = 8, PJ_ROWS = 16, PJ_NT = 4, PJ_UNR = 4;

struct ProjSeg {
  const bf16* W;     // [rows, K] row-major
  const bf16* X;     // [B, ldx] row-major
  int rows;
  int out_off;       // first output column of this segment
};
struct ProjArgs {
  ProjSeg seg[3];
  int n_seg, K, B;
  int ldx;           // row stride of X in elements
  int x_head_rows;   // > 0: every x_head_rows rows form a head, and head h reads X at column offset h * K
  float* out_f32;    // [B, ldo] (one of the two)
  bf16* out_bf16;
  int ldo;
};

__global__ void __launch_bounds__(PJ_WARPS * 32) decode_proj_kernel(ProjArgs a) {
  pdl_enter();
  __shared__ float red[PJ_WARPS][PJ_ROWS][PJ_NT * 8 + 1];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const int b0 = blockIdx.y * (PJ_NT * 8);
  const int row0 = blockIdx.x * PJ_ROWS;          // first row of this CTA in the stacked row space
  // segments start on multiples of PJ_ROWS in the stacked space (the host pads), so a CTA stays inside one
  int base = 0;
  ProjSeg sg = a.seg[0];
  if (a.n_seg > 1) {
    const int p0 = (a.seg[0].rows + PJ_ROWS - 1) / PJ_ROWS * PJ_ROWS;
    const int p1 = (a.seg[1].rows + PJ_ROWS - 1) / PJ_ROWS * PJ_ROWS;
    if (row0 >= p0 + p1 && a.n_seg > 2) { sg = a.seg[2]; base = p0 + p1; }
    else if (row0 >= p0) { sg = a.seg[1]; base = p0; }
  }
  const int r_lo = row0 - base + g, r_hi = r_lo + 8;
  const bool ok_lo = r_lo < sg.rows, ok_hi = r_hi < sg.rows;
  const bf16* w_lo = sg.W + (size_t)r_lo * a.K + t * 8;
  const bf16* w_hi = sg.W + (size_t)r_hi * a.K + t * 8;
  const bf16* xb = sg.X + (a.x_head_rows > 0 ? (size_t)((row0 - base) / a.x_head_rows) * a.K : 0) + t * 8;
  float acc[PJ_NT][4];
#pragma unroll
  for (int nt = 0; nt < PJ_NT; ++nt)
#pragma unroll
    for (int c = 0; c < 4; ++c) acc[nt][c] = 0.f;
  const int nkb = a.K / 32;
  for (int kb0 = warp; kb0 < nkb; kb0 += PJ_WARPS * PJ_UNR) {
    uint4 wl[PJ_UNR], wh[PJ_UNR], xf[PJ_UNR][PJ_NT];
#pragma unroll
    for (int u = 0; u < PJ_UNR; ++u) {
      const int kb = kb0 + u * PJ_WARPS;
      wl[u] = wh[u] = make_uint4(0, 0, 0, 0);
      if (kb < nkb) {
        if (ok_lo) wl[u] = __ldcs(reinterpret_cast<const uint4*>(w_lo + kb * 32));
        if (ok_hi) wh[u] = __ldcs(reinterpret_cast<const uint4*>(w_hi + kb * 32));
      }
#pragma unroll
      for (int nt = 0; nt < PJ_NT; ++nt) {
        const int seq = b0 + nt * 8 + g;
        xf[u][nt] = make_uint4(0, 0, 0, 0);
        if (kb < nkb && seq < a.B) xf[u][nt] = __ldg(reinterpret_cast<const uint4*>(xb + (size_t)seq * a.ldx + kb * 32));
      }
    }
#pragma unroll
    for (int u = 0; u < PJ_UNR; ++u) {
      const uint32_t a1[4] = {wl[u].x, wh[u].x, wl[u].y, wh[u].y};
      const uint32_t a2[4] = {wl[u].z, wh[u].z, wl[u].w, wh[u].w};
#pragma unroll
      for (int nt = 0; nt < PJ_NT; ++nt) {
        mma_16816(acc[nt], a1, xf[u][nt].x, xf[u][nt].y);
        mma_16816(acc[nt], a2, xf[u][nt].z, xf[u][nt].w);
      }
    }
  }
#pragma unroll
  for (int nt = 0; nt < PJ_NT; ++nt)
#pragma unroll
    for (int c = 0; c < 4; ++c) red[warp][g + 8 * (c >> 1)][nt * 8 + 2 * t + (c & 1)] = acc[nt][c];
  __syncthreads();
  for (int i = threadIdx.x; i < PJ_ROWS * PJ_NT * 8; i += PJ_WARPS * 32) {
    const int row = i % PJ_ROWS, seq = i / PJ_ROWS;
    float v = 0.f;
#pragma unroll
    for (int w = 0; w < PJ_WARPS; ++w) v += red[w][row][seq];
    const int r = row0 - base + row;
    if (r < sg.rows && b0 + seq < a.B) {
      const size_t o = (size_t)(b0 + seq) * a.ldo + sg.out_off + r;
      if (a.out_f32) a.out_f32[o] = v;
      else a.out_bf16[o] = __float2bfloat16(v);
    }
  }
}

// ------------------------------------------------------------------------------------------------ transforms
// Eq. 8, conv1 at the k_ch tokens conv2 reads, for every channel of one sequence; also the value row (Eq. 10),
// the history for the next token and the input the next step's value shift needs.
struct C1Args {
  CcaDims d;
  const float* lat;      // [B, L + Lk]: q0 | k0 | v1 | v2 of the new token
  const bf16* x;         // [B, E] new token
  const bf16* w0;        // [L, k_seq]
  bf16* y1s;             // [B, L * kc]: conv1 output of channel c at tap r in element c * kc + r (conv2 on)
  float* y2;             // [B, L]: written here instead when conv2 is off
  bf16* v_cache;
  float* hist;           // [B, pad, L]
  bf16* x_prev;          // [B, E]
  const int* pos;
  long long S_max;
  int max_len;
  int* status;
};

__global__ void __launch_bounds__(256) decode_conv1_kernel(C1Args a) {
  pdl_enter();
  const CcaDims& d = a.d;
  const int b = blockIdx.y, tid = threadIdx.x;
  const int t = a.pos[b];
  if (t < 0 || t >= a.S_max || t >= a.max_len) {
    if (tid == 0 && blockIdx.x == 0) atomicCAS(a.status, 0, ST_DECODE_BAD_POSITION);
    return;
  }
  const int ld_lat = d.L + d.Lk;
  const int pad = d.k_seq + d.k_ch - 2;
  const int ks = (d.flags & F_CONV1) ? d.k_seq : 1;
  const int kc = (d.flags & F_CONV2) ? d.k_ch : 1;
  const float* lat_b = a.lat + (size_t)b * ld_lat;
  for (int ch = blockIdx.x * 256 + tid; ch < d.L; ch += gridDim.x * 256) {
    float win[8];                                  // tokens t - pad .. t of this channel (pad + 1 <= 7)
#pragma unroll
    for (int r = 0; r < 8; ++r) win[r] = 0.f;
#pragma unroll
    for (int r = 0; r < 7; ++r)
      if (r < pad) win[r] = a.hist[((size_t)b * pad + r) * d.L + ch];
    win[pad] = lat_b[ch];
    for (int r = 0; r < kc; ++r) {
      const int row = pad - (kc - 1) + r;
      float acc;
      if (d.flags & F_CONV1) {
        acc = 0.f;
        for (int j = 0; j < ks; ++j) acc = fmaf(__bfloat162float(a.w0[(size_t)ch * d.k_seq + j]), win[row - (ks - 1) + j], acc);
      } else {
        acc = win[row];
      }
      if (d.flags & F_CONV2) a.y1s[((size_t)b * d.L + ch) * kc + r] = __float2bfloat16(acc);
      else a.y2[(size_t)b * d.L + ch] = acc;
    }
#pragma unroll
    for (int r = 0; r < 7; ++r)
      if (r < pad) a.hist[((size_t)b * pad + r) * d.L + ch] = win[r + 1];
  }
  for (int c = blockIdx.x * 256 + tid; c < d.Lk; c += gridDim.x * 256)
    a.v_cache[((size_t)b * a.S_max + t) * d.Lk + c] = __float2bfloat16(lat_b[d.L + c]);
  for (int c = blockIdx.x * 256 + tid; c < d.E / 8; c += gridDim.x * 256)
    reinterpret_cast<uint4*>(a.x_prev + (size_t)b * d.E)[c] = reinterpret_cast<const uint4*>(a.x + (size_t)b * d.E)[c];
}

// Eq. 9 (q-k-mean) and Eq. 11 (norm, temperature, RoPE at the sequence's own position) for one (sequence, head);
// the query goes to the workspace, the key into the cache.
struct FnArgs {
  CcaDims d;
  const float* lat;
  const float* y2;       // [B, L]: conv output of the new token
  const float* temp;
  float* q;              // [B, Lq]
  bf16* k_cache;
  const int* pos;
  long long S_max;
  int max_len;
};

template <int DH>
__global__ void __launch_bounds__(DH < 128 ? 128 : DH) decode_finalize_kernel(FnArgs a) {
  pdl_enter();
  constexpr int NW = (DH < 128 ? 128 : DH) / 32;      // warps per block
  __shared__ float xh[DH];
  __shared__ float red[NW];
  const CcaDims& d = a.d;
  const int b = blockIdx.y, head = blockIdx.x;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int t = a.pos[b];
  if (t < 0 || t >= a.S_max || t >= a.max_len) return;      // reported by the conv1 kernel
  const bool is_q = head < d.hq;
  const int ch0 = head * DH;                   // first channel of the head in the q0|k0 latent
  const float* lat_b = a.lat + (size_t)b * (d.L + d.Lk);
  float v = 0.f, ssq = 0.f;
  const int c = tid;
  if (c < DH) {
    v = a.y2[(size_t)b * d.L + ch0 + c];
    if (d.flags & F_QK_MEAN) {
      if (is_q) {
        const int j = head / d.g;
        v += 0.5f * (lat_b[ch0 + c] + lat_b[d.Lq + j * DH + c]);
      } else {
        const int j = head - d.hq;
        float sq = 0.f;
        for (int i = 0; i < d.g; ++i) sq += lat_b[(j * d.g + i) * DH + c];
        v += 0.5f * lat_b[ch0 + c] + 0.5f * sq / (float)d.g;
      }
    }
    ssq = v * v;
  }
  if (d.flags & F_QK_NORM) {
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) ssq += __shfl_xor_sync(0xffffffffu, ssq, s);
    if (lane == 0) red[warp] = ssq;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int i = 0; i < NW; ++i) tot += red[i];
    float sc = sqrtf((float)DH) * rsqrtf(tot);
    if (!is_q) sc *= __expf(a.temp[head - d.hq]);
    v *= sc;
  }
  if (c < DH) xh[c] = v;
  __syncthreads();
  if (c >= DH) return;
  if (d.flags & F_ROPE) {
    const int cc = c % (DH / 2);
    const double theta = exp2(-2.0 * (double)cc / (double)DH * log2((double)d.rope_base));
    double sn, cs;
    sincos((double)t * theta, &sn, &cs);
    v = c < DH / 2 ? xh[c] * (float)cs - xh[c + DH / 2] * (float)sn : xh[c] * (float)cs + xh[c - DH / 2] * (float)sn;
  }
  if (is_q) a.q[(size_t)b * d.Lq + ch0 + c] = v;
  else a.k_cache[((size_t)b * a.S_max + t) * d.Lk + (ch0 - d.Lq) + c] = __float2bfloat16(v);
}

// ------------------------------------------------------------------------------------------------ attention
struct AtArgs {
  CcaDims d;
  const float* q;        // [B, Lq]
  const bf16* k_cache;
  const bf16* v_cache;
  const float* temp;     // log key temperature if q, k are normalised, else null
  const int* pos;
  long long S_max;
  int max_len;
  int chunk, splits;
  float* part_o;         // [B, hq, splits, DH]
  float* part_ml;        // [B, hq, splits, 2]
};

constexpr int DA_WARPS = 4;

// Channel that the ci-th value-row element of lane group g is: a lane loads, of every value row, the 16-byte
// pieces that start at channel 8 g (and 64 + 8 g when d_h = 128), or the 8-byte piece at 4 g when d_h = 32, so
// that a warp's load covers whole rows.
template <int DH>
CCA_DEVINL int pv_channel(int g, int ci) {
  if (DH == 32) return g * 4 + ci;
  return (ci >> 3) * 64 + g * 8 + (ci & 7);
}

// One CTA: keys [split * chunk, ...) of sequence b, kv head j, up to 8 NHT of its query heads.  The two
// contractions of a 16-key block run as m16n8k16 tensor-core instructions -- S = Q K^T with the query heads as
// rows (padded to 16), O^T = V^T P^T with the heads as the 8 columns -- so one cached row costs a few
// instructions instead of 4 d_h multiply-adds per head and the kernel's speed is that of its loads.  Keys and
// values go from global memory straight into the operand registers: a contraction does not care about the order
// of its inner index nor about how its output rows are numbered, so each lane takes 16 contiguous bytes per key
// (Q K^T, inner index = channel) and pairs the same channel of two value rows with a byte permute (V^T P^T, inner
// index = key, output row = whichever channel the lane loaded).
template <int DH, int NHT>
__global__ void __launch_bounds__(DA_WARPS * 32) decode_attn_kernel(AtArgs a) {
  pdl_enter();
  constexpr int CB = DH / 32;                  // 32-channel blocks of Q K^T
  constexpr int VW = DH / 16;                  // 32-bit words per lane per value row = 16-channel tiles of O^T
  const CcaDims& d = a.d;
  const int split = blockIdx.x, b = blockIdx.z;
  const int n_grp = (d.g + 8 * NHT - 1) / (8 * NHT);
  const int j = blockIdx.y / n_grp, h0 = (blockIdx.y % n_grp) * 8 * NHT;
  const int nh = min(8 * NHT, d.g - h0);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const int tpos = a.pos[b];
  if (tpos < 0 || tpos >= a.S_max || tpos >= a.max_len) return;     // reported by the transform kernel
  const int n_keys = tpos + 1;
  const int k_begin = split * a.chunk, k_end = min(n_keys, k_begin + a.chunk);
  const float c_scale = rsqrtf((float)DH) * LOG2E;

  // query fragments: rows g and g + 8 of the 16-row operand are heads h0 + g and h0 + g + 8
  uint32_t qa[CB][2][4];
#pragma unroll
  for (int cb = 0; cb < CB; ++cb)
#pragma unroll
    for (int mm = 0; mm < 2; ++mm) {
#pragma unroll
      for (int hi = 0; hi < 2; ++hi) {
        float4 qv = make_float4(0.f, 0.f, 0.f, 0.f);
        if (hi < NHT && g + 8 * hi < nh)
          qv = *reinterpret_cast<const float4*>(a.q + (size_t)b * d.Lq + (size_t)(j * d.g + h0 + g + 8 * hi) * DH + cb * 32 +
                                                t * 8 + mm * 4);
        qa[cb][mm][hi] = pack_bf16x2(qv.x, qv.y);
        qa[cb][mm][2 + hi] = pack_bf16x2(qv.z, qv.w);
      }
    }
  bool fixed = false;
  float m_fixed = 0.f;
  if (a.temp != nullptr) {
    m_fixed = sqrtf((float)DH) * __expf(a.temp[j]) * LOG2E * 1.01f;
    fixed = m_fixed <= 56.f;
  }
  // softmax state of heads g (and g + 8): every lane of group g carries it; the sums are per-lane partials
  float m_row[NHT], l_row[NHT];
#pragma unroll
  for (int hi = 0; hi < NHT; ++hi) { m_row[hi] = fixed ? m_fixed : -INFINITY; l_row[hi] = 0.f; }
  // O^T tiles: o[hi][mt] = {(channel slot g, head 2t), (g, 2t+1), (g + 8, 2t), (g + 8, 2t+1)} of heads 8 hi + ...
  float o[NHT][VW][4];
#pragma unroll
  for (int hi = 0; hi < NHT; ++hi)
#pragma unroll
    for (int mt = 0; mt < VW; ++mt)
#pragma unroll
      for (int c = 0; c < 4; ++c) o[hi][mt][c] = 0.f;

  const bf16* kb = a.k_cache + (size_t)b * a.S_max * d.Lk + j * DH;
  const bf16* vb = a.v_cache + (size_t)b * a.S_max * d.Lk + j * DH;
  for (int k0 = k_begin + warp * 16; k0 < k_end; k0 += DA_WARPS * 16) {
    // ---- loads of the 16-key block
    uint4 kf[2][CB];
#pragma unroll
    for (int ti = 0; ti < 2; ++ti) {
      const int key = k0 + ti * 8 + g;
#pragma unroll
      for (int cb = 0; cb < CB; ++cb) {
        kf[ti][cb] = make_uint4(0, 0, 0, 0);
        if (key < k_end) kf[ti][cb] = __ldcs(reinterpret_cast<const uint4*>(kb + (size_t)key * d.Lk + cb * 32 + t * 8));
      }
    }
    uint32_t vf[4][VW];                        // value rows 2t, 2t+1, 2t+8, 2t+9 of the block
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int key = k0 + 2 * t + (r & 1) + (r >> 1) * 8;
#pragma unroll
      for (int w = 0; w < VW; ++w) vf[r][w] = 0u;
      if (key < k_end) {
        const bf16* vr = vb + (size_t)key * d.Lk;
        if (DH == 32) {
          const uint2 u = __ldcs(reinterpret_cast<const uint2*>(vr + g * 4));
          vf[r][0] = u.x; vf[r][1] = u.y;
        } else {
#pragma unroll
          for (int hf = 0; hf < DH / 64; ++hf) {
            const uint4 u = __ldcs(reinterpret_cast<const uint4*>(vr + hf * 64 + g * 8));
            vf[r][hf * 4 + 0] = u.x; vf[r][hf * 4 + 1] = u.y; vf[r][hf * 4 + 2] = u.z; vf[r][hf * 4 + 3] = u.w;
          }
        }
      }
    }
    // ---- S = Q K^T for the two 8-key tiles: thread (g, t) gets heads g, g + 8 x keys 2t, 2t+1 of each tile
    float sc[2][4];
#pragma unroll
    for (int ti = 0; ti < 2; ++ti) {
#pragma unroll
      for (int c = 0; c < 4; ++c) sc[ti][c] = 0.f;
#pragma unroll
      for (int cb = 0; cb < CB; ++cb) {
        mma_16816(sc[ti], qa[cb][0], kf[ti][cb].x, kf[ti][cb].y);
        mma_16816(sc[ti], qa[cb][1], kf[ti][cb].z, kf[ti][cb].w);
      }
    }
#pragma unroll
    for (int ti = 0; ti < 2; ++ti)
#pragma unroll
      for (int c = 0; c < 2 * NHT; ++c) {
        const int key = k0 + ti * 8 + 2 * t + (c & 1);
        sc[ti][c] = key < k_end ? sc[ti][c] * c_scale : -INFINITY;
      }
    if (!fixed) {
      float mx[NHT];
      bool grow = false;
#pragma unroll
      for (int hi = 0; hi < NHT; ++hi) {
        mx[hi] = fmaxf(fmaxf(sc[0][2 * hi], sc[0][2 * hi + 1]), fmaxf(sc[1][2 * hi], sc[1][2 * hi + 1]));
        mx[hi] = fmaxf(mx[hi], __shfl_xor_sync(0xffffffffu, mx[hi], 1));
        mx[hi] = fmaxf(mx[hi], __shfl_xor_sync(0xffffffffu, mx[hi], 2));
        grow = grow || mx[hi] > m_row[hi];
      }
      if (__any_sync(0xffffffffu, grow)) {
#pragma unroll
        for (int hi = 0; hi < NHT; ++hi) {
          float alpha = 1.f;
          if (mx[hi] > m_row[hi]) {
            alpha = exp2f(m_row[hi] - mx[hi]);                 // 0 while nothing has been seen (m = -inf)
            l_row[hi] *= alpha;
            m_row[hi] = mx[hi];
          }
          // the O^T columns of this lane are heads 2t, 2t+1, whose factors live in lane groups 2t, 2t+1
          const float a0 = __shfl_sync(0xffffffffu, alpha, (2 * t) * 4);
          const float a1 = __shfl_sync(0xffffffffu, alpha, (2 * t + 1) * 4);
#pragma unroll
          for (int mt = 0; mt < VW; ++mt) {
            o[hi][mt][0] *= a0; o[hi][mt][1] *= a1; o[hi][mt][2] *= a0; o[hi][mt][3] *= a1;
          }
        }
      }
    }
    uint32_t pb[NHT][2];                       // P^T operand: keys 2t, 2t+1 (tile 0) and 2t+8, 2t+9 (tile 1) of head g (+ 8)
#pragma unroll
    for (int ti = 0; ti < 2; ++ti)
#pragma unroll
      for (int hi = 0; hi < NHT; ++hi) {
        const float mu = m_row[hi] == -INFINITY ? 0.f : m_row[hi];
        const float p0 = exp2f(sc[ti][2 * hi] - mu), p1 = exp2f(sc[ti][2 * hi + 1] - mu);
        const uint32_t w = pack_bf16x2(p0, p1);
        pb[hi][ti] = w;
        // the sum runs over the rounded weights, the ones the second contraction uses
        l_row[hi] += __uint_as_float(w << 16) + __uint_as_float(w & 0xffff0000u);
      }
    // ---- O^T += V^T P^T
#pragma unroll
    for (int mt = 0; mt < VW; ++mt) {
      uint32_t va[4];
      va[0] = __byte_perm(vf[0][mt], vf[1][mt], 0x5410u);
      va[1] = __byte_perm(vf[0][mt], vf[1][mt], 0x7632u);
      va[2] = __byte_perm(vf[2][mt], vf[3][mt], 0x5410u);
      va[3] = __byte_perm(vf[2][mt], vf[3][mt], 0x7632u);
#pragma unroll
      for (int hi = 0; hi < NHT; ++hi) mma_16816(o[hi][mt], va, pb[hi][0], pb[hi][1]);
    }
  }
  // row sums: the four lanes of a group hold different keys
#pragma unroll
  for (int hi = 0; hi < NHT; ++hi) {
    l_row[hi] += __shfl_xor_sync(0xffffffffu, l_row[hi], 1);
    l_row[hi] += __shfl_xor_sync(0xffffffffu, l_row[hi], 2);
  }
  // merge the warps through shared memory
  __shared__ float sm_o[DA_WARPS][8 * NHT][DH + 1];
  __shared__ float sm_ml[DA_WARPS][8 * NHT][2];
#pragma unroll
  for (int hi = 0; hi < NHT; ++hi)
#pragma unroll
    for (int mt = 0; mt < VW; ++mt)
#pragma unroll
      for (int c = 0; c < 4; ++c)
        sm_o[warp][8 * hi + 2 * t + (c & 1)][pv_channel<DH>(g, 2 * mt + (c >> 1))] = o[hi][mt][c];
  if (t == 0) {
#pragma unroll
    for (int hi = 0; hi < NHT; ++hi) { sm_ml[warp][g + 8 * hi][0] = m_row[hi]; sm_ml[warp][g + 8 * hi][1] = l_row[hi]; }
  }
  __syncthreads();
  for (int i = threadIdx.x; i < nh * DH; i += DA_WARPS * 32) {
    const int h = i / DH, c = i % DH;
    float mn = -INFINITY;
#pragma unroll
    for (int w = 0; w < DA_WARPS; ++w) mn = fmaxf(mn, sm_ml[w][h][0]);
    float lo = 0.f, oo = 0.f;
#pragma unroll
    for (int w = 0; w < DA_WARPS; ++w) {
      const float al = (sm_ml[w][h][0] == -INFINITY) ? 0.f : exp2f(sm_ml[w][h][0] - mn);
      lo += sm_ml[w][h][1] * al;
      oo += sm_o[w][h][c] * al;
    }
    const int hi = j * d.g + h0 + h;
    const size_t pidx = ((size_t)b * d.hq + hi) * a.splits + split;
    a.part_o[pidx * DH + c] = oo;
    if (c == 0) { a.part_ml[pidx * 2] = mn; a.part_ml[pidx * 2 + 1] = lo; }
  }
}

struct CbArgs {
  CcaDims d;
  const float* part_o;
  const float* part_ml;
  const int* pos;
  long long S_max;
  int max_len, splits;
  bf16* o;               // [B, Lq]
};

template <int DH>
__global__ void __launch_bounds__(DH < 64 ? 64 : DH) decode_combine_kernel(CbArgs a) {
  pdl_enter();
  const int hi = blockIdx.x, b = blockIdx.y, c = threadIdx.x;
  const int t = a.pos[b];
  if (t < 0 || t >= a.S_max || t >= a.max_len) return;
  if (c >= DH) return;
  const size_t p0 = ((size_t)b * a.d.hq + hi) * a.splits;
  float mn = -INFINITY;
  for (int s = 0; s < a.splits; ++s) mn = fmaxf(mn, a.part_ml[(p0 + s) * 2]);
  float lo = 0.f, oo = 0.f;
  for (int s = 0; s < a.splits; ++s) {
    const float ms = a.part_ml[(p0 + s) * 2];
    const float al = (ms == -INFINITY) ? 0.f : exp2f(ms - mn);
    lo += a.part_ml[(p0 + s) * 2 + 1] * al;
    oo += a.part_o[(p0 + s) * DH + c] * al;
  }
  a.o[(size_t)b * a.d.Lq + hi * DH + c] = __float2bfloat16(oo / lo);
}

int padded_rows(int rows) { return (rows + PJ_ROWS - 1) / PJ_ROWS * PJ_ROWS; }

cudaError_t launch_proj(const ProjArgs& a, cudaStream_t st) {
  int tot = 0;
  for (int s = 0; s < a.n_seg; ++s) tot += padded_rows(a.seg[s].rows);
  dim3 grid((unsigned)(tot / PJ_ROWS), (unsigned)((a.B + PJ_NT * 8 - 1) / (PJ_NT * 8)));
  return launch_pdl(decode_proj_kernel, grid, dim3(PJ_WARPS * 32), st, a);
}

template <int DH>
cudaError_t launch_attn_dh(const AtArgs& a, cudaStream_t st) {
  const CcaDims& d = a.d;
  if (d.g <= 8) {
    dim3 grid((unsigned)a.splits, (unsigned)d.hk, (unsigned)d.B);
    return launch_pdl(decode_attn_kernel<DH, 1>, grid, dim3(DA_WARPS * 32), st, a);
  } else if constexpr (DH <= 128) {
    dim3 grid((unsigned)a.splits, (unsigned)(d.hk * ((d.g + 15) / 16)), (unsigned)d.B);
    return launch_pdl(decode_attn_kernel<DH, 2>, grid, dim3(DA_WARPS * 32), st, a);
  } else {
    return cudaErrorInvalidValue;          // head size 256: up to 8 query heads per kv head
  }
  return cudaGetLastError();
}

}  // namespace

void decode_plan(const CcaDims& d, int max_len, int sm_count, int* chunk, int* splits) {
  const int n_grp = d.g <= 8 ? 1 : (d.g + 15) / 16;
  const long long base = (long long)d.B * d.hk * n_grp;
  static int per_sm = 0;                                       // CTAs per SM to aim for (CCA_DECODE_CTAS_PER_SM overrides)
  if (per_sm == 0) {
    const char* e = getenv("CCA_DECODE_CTAS_PER_SM");
    per_sm = e ? atoi(e) : 12;
    if (per_sm < 1 || per_sm > 64) per_sm = 12;
  }
  long long want = ((long long)per_sm * sm_count + base - 1) / base;
  if (want < 1) want = 1;
  if (want > 128) want = 128;
  int ch = (int)((max_len + want - 1) / want);
  ch = (ch + 63) / 64 * 64;                                    // the four warps of a CTA take 16 keys each per round
  if (ch < 64) ch = 64;
  *chunk = ch;
  *splits = (max_len + ch - 1) / ch;
}

size_t decode_workspace_bytes(const CcaDims& d, int max_len, int sm_count) {
  int chunk, splits;
  decode_plan(d, max_len, sm_count, &chunk, &splits);
  auto up = [](size_t v) { return (v + 255) / 256 * 256; };
  size_t n = 0;
  n += up((size_t)d.B * (d.L + d.Lk) * 4);             // lat
  n += up((size_t)d.B * d.Lq * 4);                     // q
  n += up((size_t)d.B * d.hq * splits * d.dh * 4);     // partial o
  n += up((size_t)d.B * d.hq * splits * 2 * 4);        // partial (m, l)
  n += up((size_t)d.B * d.Lq * 2);                     // o
  n += up((size_t)d.B * d.L * d.k_ch * 2);             // conv1 output at the taps conv2 reads
  n += up((size_t)d.B * d.L * 4);                      // conv output
  return n;
}

int launch_decode_step(const CcaDims& d, const DecodeWeights& w, const bf16* x, bf16* out, const DecodeState& s,
                       int max_len, void* workspace, int sm_count, int* status, long long* launches, cudaEvent_t ev_attn_begin,
                       cudaEvent_t ev_attn_end, cudaStream_t st) {
  int chunk, splits;
  decode_plan(d, max_len, sm_count, &chunk, &splits);
  auto up = [](size_t v) { return (v + 255) / 256 * 256; };
  unsigned char* p = static_cast<unsigned char*>(workspace);
  float* lat = reinterpret_cast<float*>(p); p += up((size_t)d.B * (d.L + d.Lk) * 4);
  float* q = reinterpret_cast<float*>(p); p += up((size_t)d.B * d.Lq * 4);
  float* part_o = reinterpret_cast<float*>(p); p += up((size_t)d.B * d.hq * splits * d.dh * 4);
  float* part_ml = reinterpret_cast<float*>(p); p += up((size_t)d.B * d.hq * splits * 2 * 4);
  bf16* o = reinterpret_cast<bf16*>(p); p += up((size_t)d.B * d.Lq * 2);
  bf16* y1s = reinterpret_cast<bf16*>(p); p += up((size_t)d.B * d.L * d.k_ch * 2);
  float* y2 = reinterpret_cast<float*>(p);
  cudaError_t e;
  if (d.dh != 32 && d.dh != 64 && d.dh != 128 && d.dh != 256) return 1;
  if (d.E % 32 || d.Lq % 32) return 1;
  if (d.dh == 256 && d.g > 8) return 1;
  // Eq. 7 and Eq. 10: q0 | k0 | v1 from x_t, v2 from x_{t-1}
  ProjArgs pa;
  memset(&pa, 0, sizeof(pa));
  pa.n_seg = 3;
  pa.seg[0] = ProjSeg{w.w_qk, x, d.L, 0};
  pa.seg[1] = ProjSeg{w.w_v1, x, d.Lk / 2, d.L};
  pa.seg[2] = ProjSeg{w.w_v2, (d.flags & F_V_SHIFT) ? s.x_prev : x, d.Lk / 2, d.L + d.Lk / 2};
  pa.K = d.E; pa.B = d.B; pa.ldx = d.E; pa.out_f32 = lat; pa.ldo = d.L + d.Lk;
  if ((e = launch_proj(pa, st)) != cudaSuccess) return -(int)e;
  ++*launches;
  // Eq. 8: conv1 (with the value row, history and previous input), conv2 as a per-head contraction over
  // (input channel, tap); Eq. 9 and the rest of Eq. 11 per head
  const int kc = (d.flags & F_CONV2) ? d.k_ch : 1;
  C1Args c1;
  c1.d = d; c1.lat = lat; c1.x = x; c1.w0 = w.conv0_w; c1.y1s = y1s; c1.y2 = y2; c1.v_cache = s.v_cache;
  c1.hist = s.qk0_hist; c1.x_prev = s.x_prev; c1.pos = s.pos; c1.S_max = s.S_max; c1.max_len = max_len; c1.status = status;
  if ((e = launch_pdl(decode_conv1_kernel, dim3((unsigned)((d.L + 255) / 256), (unsigned)d.B), dim3(256), st, c1)) != cudaSuccess)
    return -(int)e;
  ++*launches;
  if (d.flags & F_CONV2) {
    ProjArgs pc;
    memset(&pc, 0, sizeof(pc));
    pc.n_seg = 1;
    pc.seg[0] = ProjSeg{w.conv1_w, y1s, d.L, 0};
    pc.K = d.dh * kc; pc.B = d.B; pc.ldx = d.L * kc; pc.x_head_rows = d.dh; pc.out_f32 = y2; pc.ldo = d.L;
    if ((e = launch_proj(pc, st)) != cudaSuccess) return -(int)e;
    ++*launches;
  }
  FnArgs fa;
  fa.d = d; fa.lat = lat; fa.y2 = y2; fa.temp = w.temp; fa.q = q; fa.k_cache = s.k_cache; fa.pos = s.pos;
  fa.S_max = s.S_max; fa.max_len = max_len;
  {
    dim3 grid((unsigned)(d.hq + d.hk), (unsigned)d.B);
    switch (d.dh) {
      case 32: e = launch_pdl(decode_finalize_kernel<32>, grid, dim3(128), st, fa); break;
      case 64: e = launch_pdl(decode_finalize_kernel<64>, grid, dim3(128), st, fa); break;
      case 128: e = launch_pdl(decode_finalize_kernel<128>, grid, dim3(128), st, fa); break;
      default: e = launch_pdl(decode_finalize_kernel<256>, grid, dim3(256), st, fa); break;
    }
    if (e != cudaSuccess) return -(int)e;
    ++*launches;
  }
  AtArgs aa;
  aa.d = d; aa.q = q; aa.k_cache = s.k_cache; aa.v_cache = s.v_cache;
  aa.temp = (d.flags & F_QK_NORM) ? w.temp : nullptr;
  aa.pos = s.pos; aa.S_max = s.S_max; aa.max_len = max_len; aa.chunk = chunk; aa.splits = splits;
  aa.part_o = part_o; aa.part_ml = part_ml;
  if (ev_attn_begin && (e = cudaEventRecord(ev_attn_begin, st)) != cudaSuccess) return -(int)e;
  switch (d.dh) {
    case 32: e = launch_attn_dh<32>(aa, st); break;
    case 64: e = launch_attn_dh<64>(aa, st); break;
    case 128: e = launch_attn_dh<128>(aa, st); break;
    case 256: e = launch_attn_dh<256>(aa, st); break;
    default: return 1;
  }
  if (e != cudaSuccess) return -(int)e;
  ++*launches;
  if (ev_attn_end && (e = cudaEventRecord(ev_attn_end, st)) != cudaSuccess) return -(int)e;
  CbArgs ca;
  ca.d = d; ca.part_o = part_o; ca.part_ml = part_ml; ca.pos = s.pos; ca.S_max = s.S_max; ca.max_len = max_len;
  ca.splits = splits; ca.o = o;
  {
    dim3 grid((unsigned)d.hq, (unsigned)d.B);
    switch (d.dh) {
      case 32: e = launch_pdl(decode_combine_kernel<32>, grid, dim3(64), st, ca); break;
      case 64: e = launch_pdl(decode_combine_kernel<64>, grid, dim3(64), st, ca); break;
      case 128: e = launch_pdl(decode_combine_kernel<128>, grid, dim3(128), st, ca); break;
      case 256: e = launch_pdl(decode_combine_kernel<256>, grid, dim3(256), st, ca); break;
      default: return 1;
    }
    if (e != cudaSuccess) return -(int)e;
    ++*launches;
  }
  // Eq. 11, up-projection
  ProjArgs pb;
  memset(&pb, 0, sizeof(pb));
  pb.n_seg = 1;
  pb.seg[0] = ProjSeg{w.w_o, o, d.E, 0};
  pb.K = d.Lq; pb.B = d.B; pb.ldx = d.Lq; pb.out_bf16 = out; pb.ldo = d.E;
  if ((e = launch_proj(pb, st)) != cudaSuccess) return -(int)e;
  ++*launches;
  return 0;
}
