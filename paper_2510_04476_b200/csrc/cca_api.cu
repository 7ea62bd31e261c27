// C ABI of the CCA library: handle, validation, metadata, workspace layout, forward / backward drivers.
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>

#include "../../include/cca.h"
#include "common.cuh"
#include "decode.cuh"
#include "tc_kernels.cuh"
#include "tc_ptx.cuh"

struct cca_handle {
  cca_config cfg;
  int device;
  int impl;               // 0 = SIMT only, 1 = tensor-core kernels where available
  int sm_count;
  int* d_status;          // device status word (64 bytes)
  int last_cuda;
  long long launches;
  TcState* tc;            // tensor-map cache etc. (may be null if unavailable)
  cudaEvent_t ev_attn_begin, ev_attn_end;   // optional, recorded around the attention kernel
  cudaStream_t side;                        // the RoPE table is computed here, beside the down-projection
  cudaEvent_t ev_fork, ev_join;
  // cca_forward_host, chunked: copies in and out run on their own streams beside the compute
  cudaStream_t s_in, s_out;
  cudaEvent_t ev_chunk[2][64];              // [arrived / computed][chunk]
  int n_ev;                                 // events created so far
  cudaEvent_t stage_ev[CCA_N_STAGE_EVENTS]; // optional, recorded at the stage boundaries of forward and backward
  // what the last cca_forward kept for a backward: cca_backward refuses anything else
  const void* saved_ws;
  int64_t saved_B, saved_S;
};

namespace {

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct Layout {
  size_t qk0, q, k, v, o, lse, rope, rnorm, w_all, y1s, y2, qk0b, wc, saved_end;
  size_t o32, d_o, delta, dq, dk, dv, dlat, dy1, total_end;
  size_t u_s, u_dp, u_p, u_ds, u_dy1s;   // head size 256: scratch of the unfused adjoints
  int u_rows;                            // query rows per chunk of the unfused attention adjoint
  size_t u_ld;                           // row stride (keys) of its score chunks
};

CcaDims make_dims(const cca_config& c, int64_t B, int64_t S);

Layout make_layout(const cca_config& c, int64_t B, int64_t S) {
  Layout l;
  const size_t T = (size_t)B * S;
  const size_t Lq = (size_t)c.n_q_heads * c.head_dim, Lk = (size_t)c.n_kv_heads * c.head_dim, L = Lq + Lk;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  l.qk0 = take(T * L * 4);     // fp32: a small pre-norm latent would amplify a bf16 rounding here
  l.q = take(T * Lq * 2);
  l.k = take(T * Lk * 2);
  l.v = take(T * Lk * 2);
  l.o = take(T * Lq * 2);
  l.lse = take((size_t)B * c.n_q_heads * S * 4);
  l.rope = take((size_t)S * (c.head_dim / 2) * 8);
  l.rnorm = take(T * (size_t)(c.n_q_heads + c.n_kv_heads) * 4);   // norm scale of every (token, head)
  l.w_all = take((L + Lk) * (size_t)c.d_model * 2);                // [W_qk; W_v1; W_v2] stacked
  // unfused latent transforms (head sizes the fused kernel does not cover): conv1 taps and conv output
  l.y1s = l.y2 = off;
  if (c.head_dim > 128) {
    l.y1s = take(T * L * (size_t)c.k_ch * 2);
    l.y2 = take(T * L * 4);
  }
  // operands of the TMA-fed latent-transform kernel: a bf16 copy of qk0 and the composed conv weights
  l.qk0b = l.wc = off;
  {
    CcaDims dd = make_dims(c, B, S);
    if (tc_transform2_covers(dd)) {
      l.qk0b = take(T * L * 2);
      l.wc = take(tc_transform2_weight_bytes(dd));
    }
  }
  l.saved_end = off;
  l.o32 = take(T * Lq * 4);
  l.d_o = take(T * Lq * 2);
  l.delta = take((size_t)B * c.n_q_heads * S * 4);
  l.dq = take(T * Lq * 4);
  l.dk = take(T * Lk * 4);
  l.dv = take(T * Lk * 4);
  l.dlat = take(T * (L + Lk) * 2);
  l.dy1 = take(T * L * 4);
  l.u_s = l.u_dp = l.u_p = l.u_ds = l.u_dy1s = off;
  l.u_rows = 2048;
  l.u_ld = align_up((size_t)S, 128);
  if (c.head_dim > 128) {
    l.u_s = take((size_t)l.u_rows * l.u_ld * 4);
    l.u_dp = take((size_t)l.u_rows * l.u_ld * 4);
    l.u_p = take((size_t)l.u_rows * l.u_ld * 2);
    l.u_ds = take((size_t)l.u_rows * l.u_ld * 2);
    l.u_dy1s = take(T * L * (size_t)c.k_ch * 4);
  }
  l.total_end = off;
  return l;
}

CcaDims make_dims(const cca_config& c, int64_t B, int64_t S) {
  CcaDims d;
  d.B = (int)B; d.S = (int)S; d.E = c.d_model;
  d.hq = c.n_q_heads; d.hk = c.n_kv_heads; d.dh = c.head_dim; d.g = c.n_q_heads / c.n_kv_heads;
  d.Lq = d.hq * d.dh; d.Lk = d.hk * d.dh; d.L = d.Lq + d.Lk;
  d.k_seq = c.k_seq; d.k_ch = c.k_ch; d.causal = c.causal; d.flags = c.flags; d.rope_base = c.rope_base;
  return d;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

// True if three row blocks of `row_bytes` wide rows already lie one after the other in memory (a then b then c).
bool adjacent(const void* a, const void* b, const void* c, size_t rows_a, size_t rows_b, size_t row_bytes) {
  const char* pa = (const char*)a;
  return pa && (const char*)b == pa + rows_a * row_bytes && (const char*)c == pa + (rows_a + rows_b) * row_bytes;
}

int check_sizes(const cca_handle* h, int64_t B, int64_t S, bool need_device = false) {
  if (!h || B < 1 || S < 1) return CCA_ERR_INVALID_ARG;
  if (need_device && h->device < 0) return CCA_ERR_INVALID_ARG;
  if (B * S > (int64_t)1 << 30 || S > (int64_t)1 << 24) return CCA_ERR_UNSUPPORTED;
  return CCA_OK;
}

#define CU(call)                                   \
  do {                                             \
    cudaError_t e_ = (call);                       \
    if (e_ != cudaSuccess) {                       \
      h->last_cuda = (int)e_;                      \
      return CCA_ERR_CUDA;                         \
    }                                              \
  } while (0)

#define STAGE(idx)                                                         \
  do {                                                                     \
    if (h->stage_ev[idx]) CU(cudaEventRecord(h->stage_ev[idx], st));       \
  } while (0)

GemmOperand kmajor(const void* p, long long ld) { return GemmOperand{(const bf16*)p, ld, 1}; }
GemmOperand mmajor(const void* p, long long ld) { return GemmOperand{(const bf16*)p, 1, ld}; }

// One contraction: tensor-core kernel if it is enabled and covers the case, else the SIMT kernel.
int run_gemm(cca_handle* h, const GemmArgs& g, cudaStream_t st) {
  if (h->impl >= 1 && h->tc) {
    int r = tc_gemm_pair(h->tc, g, h->d_status, st);
    if (r == 1) r = tc_gemm(h->tc, g, h->d_status, st);
    if (r == 0) { h->launches++; return CCA_OK; }
    if (r < 0) { h->last_cuda = -r; return CCA_ERR_CUDA; }
  }
  CU(launch_gemm_simt(g, st));
  h->launches++;
  return CCA_OK;
}

int run_attention_fwd(cca_handle* h, const CcaDims& d, const bf16* q, const bf16* k, const bf16* v, bf16* o,
                      float* o32, float* lse, const float* temp, cudaStream_t st) {
  if (h->ev_attn_begin) CU(cudaEventRecord(h->ev_attn_begin, st));
  bool done = false;
  if (h->impl >= 1 && h->tc) {
    int r = d.dh == 256 ? tc_attn_fwd256(h->tc, d, q, k, v, o, o32, lse, temp, h->d_status, st)
                        : tc_attn_fwd(h->tc, d, q, k, v, o, o32, lse, temp, h->d_status, st);
    if (r == 0) done = true;
    if (r < 0) { h->last_cuda = -r; return CCA_ERR_CUDA; }
  }
  if (!done) CU(launch_attn_fwd_simt(d, q, k, v, o, o32, lse, st));
  h->launches++;
  if (h->ev_attn_end) CU(cudaEventRecord(h->ev_attn_end, st));
  return CCA_OK;
}

}  // namespace

extern "C" {

const char* cca_status_string(int s) {
  switch (s) {
    case CCA_OK: return "ok";
    case CCA_ERR_INVALID_ARG: return "invalid argument";
    case CCA_ERR_UNSUPPORTED: return "unsupported shape or device";
    case CCA_ERR_ALIGNMENT: return "pointer not 16-byte aligned";
    case CCA_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case CCA_ERR_CUDA: return "CUDA error";
    case CCA_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
    case CCA_ERR_STATIC_WORKSPACE_EXCEEDED: return "problem needs more than the built-in static workspace";
    default: return "unknown status";
  }
}

static int validate_config(const cca_config* c) {
  if (!c) return CCA_ERR_INVALID_ARG;
  if (c->d_model < 1 || c->n_q_heads < 1 || c->n_kv_heads < 1 || c->head_dim < 1 || c->compression < 1)
    return CCA_ERR_INVALID_ARG;
  if ((int64_t)c->compression * c->n_q_heads * c->head_dim != c->d_model) return CCA_ERR_INVALID_ARG;
  if (c->n_q_heads % c->n_kv_heads != 0) return CCA_ERR_INVALID_ARG;
  if (((int64_t)c->n_kv_heads * c->head_dim) % 2 != 0) return CCA_ERR_INVALID_ARG;
  if (c->k_seq < 1 || c->k_ch < 1) return CCA_ERR_INVALID_ARG;
  if (c->flags & ~(uint32_t)CCA_ALL_STAGES) return CCA_ERR_INVALID_ARG;
  if ((c->flags & CCA_ROPE) && !(c->rope_base > 0.f)) return CCA_ERR_INVALID_ARG;
  if (c->k_seq > 4 || c->k_ch > 4) return CCA_ERR_UNSUPPORTED;
  if (c->head_dim != 32 && c->head_dim != 64 && c->head_dim != 128 && c->head_dim != 256) return CCA_ERR_UNSUPPORTED;
  if (c->n_q_heads > 64) return CCA_ERR_UNSUPPORTED;
  if (c->d_model % 8 != 0) return CCA_ERR_UNSUPPORTED;
  return CCA_OK;
}

int cca_init(const cca_config* cfg, int device, cca_handle** out) {
  if (!out) return CCA_ERR_INVALID_ARG;
  *out = nullptr;
  int v = validate_config(cfg);
  if (v != CCA_OK) return v;
  cudaDeviceProp prop;
  prop.multiProcessorCount = 0;
  if (device >= 0) {
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || device >= ndev) return CCA_ERR_CUDA;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return CCA_ERR_CUDA;
    if (prop.major != 10) return CCA_ERR_UNSUPPORTED;
    if (cudaSetDevice(device) != cudaSuccess) return CCA_ERR_CUDA;
  } else if (device != -1) {
    return CCA_ERR_INVALID_ARG;
  }
  cca_handle* h = new (std::nothrow) cca_handle();
  if (!h) return CCA_ERR_INVALID_ARG;
  h->cfg = *cfg;
  h->device = device;
  h->impl = 1;
  h->sm_count = prop.multiProcessorCount;
  h->last_cuda = 0;
  h->launches = 0;
  h->d_status = nullptr;
  h->tc = nullptr;
  h->ev_attn_begin = h->ev_attn_end = nullptr;
  h->side = nullptr; h->ev_fork = h->ev_join = nullptr;
  h->s_in = h->s_out = nullptr; h->n_ev = 0;
  h->saved_ws = nullptr; h->saved_B = h->saved_S = 0;
  for (int i = 0; i < CCA_N_STAGE_EVENTS; ++i) h->stage_ev[i] = nullptr;
  if (device >= 0) {
    if (cudaMalloc(&h->d_status, 64) != cudaSuccess || cudaMemset(h->d_status, 0, 64) != cudaSuccess) {
      if (h->d_status) cudaFree(h->d_status);
      delete h;
      return CCA_ERR_CUDA;
    }
    h->tc = tc_create(h->sm_count);
    if (cudaStreamCreateWithFlags(&h->side, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&h->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&h->ev_join, cudaEventDisableTiming) != cudaSuccess) {
      (void)cudaGetLastError();
      h->side = nullptr;                      // everything then runs on the caller's stream
    }
  }
  *out = h;
  return CCA_OK;
}

int cca_destroy(cca_handle* h) {
  if (!h) return CCA_ERR_INVALID_ARG;
  if (h->tc) tc_destroy(h->tc);
  if (h->s_in) cudaStreamDestroy(h->s_in);
  if (h->s_out) cudaStreamDestroy(h->s_out);
  for (int i = 0; i < h->n_ev; ++i) {
    cudaEventDestroy(h->ev_chunk[0][i]);
    cudaEventDestroy(h->ev_chunk[1][i]);
  }
  if (h->side) {
    cudaStreamDestroy(h->side);
    cudaEventDestroy(h->ev_fork);
    cudaEventDestroy(h->ev_join);
  }
  if (h->d_status) cudaFree(h->d_status);
  delete h;
  return CCA_OK;
}

int cca_set_impl(cca_handle* h, int impl) {
  if (!h) return -1;
  int old = h->impl;
  h->impl = impl;
  return old;
}

int cca_set_attention_events(cca_handle* h, void* ev_begin, void* ev_end) {
  if (!h) return CCA_ERR_INVALID_ARG;
  h->ev_attn_begin = (cudaEvent_t)ev_begin;
  h->ev_attn_end = (cudaEvent_t)ev_end;
  return CCA_OK;
}

int cca_set_stage_events(cca_handle* h, void* const* events, int n) {
  if (!h || (events && n != CCA_N_STAGE_EVENTS)) return CCA_ERR_INVALID_ARG;
  for (int i = 0; i < CCA_N_STAGE_EVENTS; ++i) h->stage_ev[i] = events ? (cudaEvent_t)events[i] : nullptr;
  return CCA_OK;
}

int64_t cca_launch_count(const cca_handle* h) { return h ? h->launches : -1; }
int cca_last_cuda_error(const cca_handle* h) { return h ? h->last_cuda : -1; }

int cca_last_status(cca_handle* h, int* device_status) {
  if (!h || !device_status || h->device < 0) return CCA_ERR_INVALID_ARG;
  int host[16];
  CU(cudaMemcpy(host, h->d_status, 64, cudaMemcpyDeviceToHost));
  *device_status = host[0];
  if (host[0] != 0) {
    cudaMemset(h->d_status, 0, 4);           // word 0 only: word 1 is the wait limit
    return CCA_ERR_DEVICE_TIMEOUT;
  }
  return CCA_OK;
}

int cca_set_wait_limit(cca_handle* h, int64_t sm_cycles) {
  if (!h || h->device < 0 || sm_cycles < 0) return CCA_ERR_INVALID_ARG;
  long long k = sm_cycles == 0 ? 0 : (sm_cycles + 1023) / 1024;      // 0 = default
  if (k != 0 && k < tc::WAIT_KCYCLES_MIN) k = tc::WAIT_KCYCLES_MIN;
  if (k > 0x7fffffffLL) k = 0x7fffffffLL;
  const int word = (int)k;
  CU(cudaSetDevice(h->device));
  CU(cudaMemcpy(h->d_status + 1, &word, 4, cudaMemcpyHostToDevice));
  return CCA_OK;
}

namespace {
// One CTA whose only wait is on a barrier that nothing arrives at: the wait runs into the handle's limit, the
// kernel records ST_TIMEOUT_PROBE and returns.  Nothing traps, nothing spins without a bound.
__global__ void wait_probe_kernel(int* status) {
  __shared__ uint64_t bar;
  __shared__ int ctl[2];
  if (threadIdx.x == 0) {
    tc::mbar_init(&bar, 1);
    tc::wait_ctl_init(ctl, status);
    tc::fence_barrier_init();
  }
  __syncthreads();
  if (!tc::mbar_wait(&bar, 0, ctl)) {
    ctl[0] = 1;
    atomicCAS(status, 0, (int)tc::ST_TIMEOUT_PROBE);
  }
}
}  // namespace

int cca_wait_selftest(cca_handle* h, void* cuda_stream) {
  if (!h || h->device < 0) return CCA_ERR_INVALID_ARG;
  CU(cudaSetDevice(h->device));
  wait_probe_kernel<<<1, 64, 0, (cudaStream_t)cuda_stream>>>(h->d_status);
  CU(cudaGetLastError());
  h->launches++;
  return CCA_OK;
}

int cca_describe(const cca_handle* h, int64_t B, int64_t S, cca_layout* out) {
  int r = check_sizes(h, B, S);
  if (r != CCA_OK) return r;
  if (!out) return CCA_ERR_INVALID_ARG;
  const cca_config& c = h->cfg;
  memset(out, 0, sizeof(*out));
  const int64_t E = c.d_model, dh = c.head_dim;
  const int64_t Lq = (int64_t)c.n_q_heads * dh, Lk = (int64_t)c.n_kv_heads * dh, L = Lq + Lk, T = B * S;
  out->L_q = Lq;
  out->L_k = Lk;
  out->g = c.n_q_heads / c.n_kv_heads;
  out->total_padding = c.k_seq + c.k_ch - 2;
  out->v_shift_split = Lk / 2;
  for (int i = 0; i < 64; ++i) out->q_to_kv_head[i] = i < c.n_q_heads ? i / out->g : -1;
  out->conv_params = L * c.k_seq + L * dh * c.k_ch;
  out->params = E * Lq + 2 * E * Lk + Lq * E + out->conv_params;
  out->kv_cache_elems = 2 * B * S * Lk;
  const int64_t proj = 2 * T * E * (Lq + 2 * Lk) + 2 * T * Lq * E;
  out->fwd_flops = proj + 4 * B * S * S * Lq + 2 * T * out->conv_params;
  out->fwd_flops_causal = proj + 2 * B * S * S * Lq + 2 * T * out->conv_params;
  out->decode_flops = 2 * B * E * (Lq + 2 * Lk) + 2 * B * Lq * E + 4 * B * S * Lq + 2 * B * out->conv_params;
  Layout l = make_layout(c, B, S);
  out->off_qk0 = (int64_t)l.qk0; out->off_q = (int64_t)l.q; out->off_k = (int64_t)l.k; out->off_v = (int64_t)l.v;
  out->off_o = (int64_t)l.o; out->off_lse = (int64_t)l.lse; out->off_rope = (int64_t)l.rope;
  out->off_rnorm = (int64_t)l.rnorm;
  out->saved_bytes = (int64_t)l.saved_end;
  out->total_bytes = (int64_t)l.total_end;
  return CCA_OK;
}

int cca_workspace_size(const cca_handle* h, int64_t B, int64_t S, int need_backward, size_t* bytes) {
  int r = check_sizes(h, B, S);
  if (r != CCA_OK) return r;
  if (!bytes) return CCA_ERR_INVALID_ARG;
  Layout l = make_layout(h->cfg, B, S);
  *bytes = need_backward ? l.total_end : l.saved_end;
  return CCA_OK;
}

int cca_attention_forward(cca_handle* h, const void* q, const void* k, const void* v, void* o, float* lse, int64_t B,
                          int64_t S, void* cuda_stream) {
  int r = check_sizes(h, B, S, true);
  if (r != CCA_OK) return r;
  if (!q || !k || !v || !o || !lse) return CCA_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || !aligned16(lse)) return CCA_ERR_ALIGNMENT;
  CU(cudaSetDevice(h->device));
  CcaDims d = make_dims(h->cfg, B, S);
  // q and k come from the caller: nothing is known about their norms
  return run_attention_fwd(h, d, (const bf16*)q, (const bf16*)k, (const bf16*)v, (bf16*)o, nullptr, lse, nullptr,
                           (cudaStream_t)cuda_stream);
}

int cca_decode_workspace_size(const cca_handle* h, int64_t B, int64_t max_len, size_t* bytes) {
  int r = check_sizes(h, B, max_len);
  if (r != CCA_OK) return r;
  if (!bytes) return CCA_ERR_INVALID_ARG;
  CcaDims d = make_dims(h->cfg, B, 1);
  *bytes = decode_workspace_bytes(d, (int)max_len, h->sm_count > 0 ? h->sm_count : 148);
  return CCA_OK;
}

int cca_decode_step(cca_handle* h, const cca_weights* w, const void* x, void* out, const cca_decode_state* s,
                    int64_t max_len, void* workspace, size_t workspace_bytes, int64_t B, void* cuda_stream) {
  int r = check_sizes(h, B, max_len, true);
  if (r != CCA_OK) return r;
  if (!w || !x || !out || !s || !workspace) return CCA_ERR_INVALID_ARG;
  if (!w->w_qk || !w->w_v1 || !w->w_v2 || !w->w_o) return CCA_ERR_INVALID_ARG;
  const cca_config& c = h->cfg;
  if ((c.flags & CCA_CONV1) && !w->conv0_w) return CCA_ERR_INVALID_ARG;
  if ((c.flags & CCA_CONV2) && !w->conv1_w) return CCA_ERR_INVALID_ARG;
  if ((c.flags & CCA_QK_NORM) && !w->temp) return CCA_ERR_INVALID_ARG;
  const int pad = c.k_seq + c.k_ch - 2;
  if (!s->k_cache || !s->v_cache || !s->x_prev || !s->pos || (pad > 0 && !s->qk0_hist)) return CCA_ERR_INVALID_ARG;
  if (max_len > s->S_max || s->S_max > (int64_t)1 << 24) return CCA_ERR_INVALID_ARG;
  if (!c.causal) return CCA_ERR_UNSUPPORTED;
  CcaDims d = make_dims(c, B, 1);
  if (d.Lk % 8 || d.E % 32 || d.Lq % 32) return CCA_ERR_UNSUPPORTED;
  if (!aligned16(x) || !aligned16(out) || !aligned16(w->w_qk) || !aligned16(w->w_v1) || !aligned16(w->w_v2) ||
      !aligned16(w->w_o) || !aligned16(s->k_cache) || !aligned16(s->v_cache) || !aligned16(s->x_prev) ||
      (reinterpret_cast<uintptr_t>(workspace) & 255))
    return CCA_ERR_ALIGNMENT;
  if (workspace_bytes < decode_workspace_bytes(d, (int)max_len, h->sm_count)) return CCA_ERR_WORKSPACE_TOO_SMALL;
  CU(cudaSetDevice(h->device));
  DecodeWeights dw{(const bf16*)w->w_qk, (const bf16*)w->w_v1, (const bf16*)w->w_v2, (const bf16*)w->w_o,
                   (const bf16*)w->conv0_w, (const bf16*)w->conv1_w, (const float*)w->temp};
  DecodeState ds{(bf16*)s->k_cache, (bf16*)s->v_cache, (float*)s->qk0_hist, (bf16*)s->x_prev, s->pos, s->S_max};
  int rr = launch_decode_step(d, dw, (const bf16*)x, (bf16*)out, ds, (int)max_len, workspace, h->sm_count, h->d_status,
                              &h->launches, h->ev_attn_begin, h->ev_attn_end, (cudaStream_t)cuda_stream);
  if (rr < 0) { h->last_cuda = -rr; return CCA_ERR_CUDA; }
  if (rr > 0) return CCA_ERR_UNSUPPORTED;
  return CCA_OK;
}

int cca_decode_state_from_prefill(cca_handle* h, const void* x, const void* workspace, size_t workspace_bytes,
                                  int64_t B, int64_t S, const cca_decode_state* s, void* cuda_stream) {
  int r = check_sizes(h, B, S, true);
  if (r != CCA_OK) return r;
  if (!x || !workspace || !s) return CCA_ERR_INVALID_ARG;
  const cca_config& c = h->cfg;
  const int pad = c.k_seq + c.k_ch - 2;
  if (!s->k_cache || !s->v_cache || !s->x_prev || (pad > 0 && !s->qk0_hist) || S > s->S_max) return CCA_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(s->k_cache) || !aligned16(s->v_cache) || !aligned16(s->x_prev) ||
      (pad > 0 && !aligned16(s->qk0_hist)) || (reinterpret_cast<uintptr_t>(workspace) & 255))
    return CCA_ERR_ALIGNMENT;
  Layout l = make_layout(c, B, S);
  if (workspace_bytes < l.saved_end) return CCA_ERR_WORKSPACE_TOO_SMALL;
  CU(cudaSetDevice(h->device));
  cudaStream_t st = (cudaStream_t)cuda_stream;
  CcaDims d = make_dims(c, B, S);
  const char* ws = (const char*)workspace;
  const size_t row_k = (size_t)d.Lk * 2;
  for (int64_t b = 0; b < B; ++b) {
    CU(cudaMemcpyAsync((char*)s->k_cache + (size_t)b * s->S_max * row_k, ws + l.k + (size_t)b * S * row_k, (size_t)S * row_k,
                       cudaMemcpyDeviceToDevice, st));
    CU(cudaMemcpyAsync((char*)s->v_cache + (size_t)b * s->S_max * row_k, ws + l.v + (size_t)b * S * row_k, (size_t)S * row_k,
                       cudaMemcpyDeviceToDevice, st));
  }
  // previous input: the last token of every sequence (rows S-1 of x, one strided copy)
  CU(cudaMemcpy2DAsync(s->x_prev, (size_t)d.E * 2, (const char*)x + (size_t)(S - 1) * d.E * 2, (size_t)S * d.E * 2,
                       (size_t)d.E * 2, (size_t)B, cudaMemcpyDeviceToDevice, st));
  if (pad > 0) {
    const size_t row = (size_t)d.L * 4;
    const int64_t n = S < pad ? S : pad;
    CU(cudaMemsetAsync(s->qk0_hist, 0, (size_t)B * pad * row, st));
    CU(cudaMemcpy2DAsync((char*)s->qk0_hist + (size_t)(pad - n) * row, (size_t)pad * row,
                         ws + l.qk0 + (size_t)(S - n) * row, (size_t)S * row, (size_t)n * row, (size_t)B,
                         cudaMemcpyDeviceToDevice, st));
  }
  return CCA_OK;
}

int cca_forward(cca_handle* h, const cca_weights* w, const void* x, void* out, void* workspace,
                size_t workspace_bytes, int64_t B, int64_t S, int save_for_backward, void* cuda_stream) {
  int r = check_sizes(h, B, S, true);
  if (r != CCA_OK) return r;
  if (!w || !x || !out || !workspace) return CCA_ERR_INVALID_ARG;
  if (!w->w_qk || !w->w_v1 || !w->w_v2 || !w->w_o) return CCA_ERR_INVALID_ARG;
  const cca_config& c = h->cfg;
  if ((c.flags & CCA_CONV1) && !w->conv0_w) return CCA_ERR_INVALID_ARG;
  if ((c.flags & CCA_CONV2) && !w->conv1_w) return CCA_ERR_INVALID_ARG;
  if ((c.flags & CCA_QK_NORM) && !w->temp) return CCA_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(out) || !aligned16(w->w_qk) || !aligned16(w->w_v1) || !aligned16(w->w_v2) ||
      !aligned16(w->w_o) || (reinterpret_cast<uintptr_t>(workspace) & 255))
    return CCA_ERR_ALIGNMENT;
  Layout l = make_layout(c, B, S);
  if (workspace_bytes < (save_for_backward ? l.total_end : l.saved_end)) return CCA_ERR_WORKSPACE_TOO_SMALL;
  h->saved_ws = nullptr;                       // set again below once everything is enqueued
  CU(cudaSetDevice(h->device));
  cudaStream_t st = (cudaStream_t)cuda_stream;
  CcaDims d = make_dims(c, B, S);
  const int T = d.B * d.S;
  char* ws = (char*)workspace;
  float* qk0 = (float*)(ws + l.qk0);
  bf16* q = (bf16*)(ws + l.q);
  bf16* k = (bf16*)(ws + l.k);
  bf16* v = (bf16*)(ws + l.v);
  bf16* o = (bf16*)(ws + l.o);
  float* lse = (float*)(ws + l.lse);
  float2* rope = (float2*)(ws + l.rope);
  float* rnorm = (float*)(ws + l.rnorm);
  // fp32 copy of o for the backward's delta = rowsum(dO * O)
  float* o32 = save_for_backward ? (float*)(ws + l.o32) : nullptr;

  STAGE(CCA_EV_FWD_BEGIN);
  // The RoPE table and the composed conv weights do not depend on x: they are computed on a side stream while the
  // down-projection runs.
  const bool use_t2 = h->impl >= 1 && h->tc && tc_transform2_covers(d) && w->conv1_w;
  bf16* qk0b = use_t2 ? (bf16*)(ws + l.qk0b) : nullptr;
  bf16* wc = use_t2 ? (bf16*)(ws + l.wc) : nullptr;
  bool forked = false;
  if ((c.flags & CCA_ROPE) || use_t2) {
    cudaStream_t ss = st;
    if (h->side) {
      CU(cudaEventRecord(h->ev_fork, st));
      CU(cudaStreamWaitEvent(h->side, h->ev_fork, 0));
      ss = h->side;
      forked = true;
    }
    if (c.flags & CCA_ROPE) {
      CU(launch_rope_table(rope, d.S, d.dh, c.rope_base, ss));
      h->launches++;
    }
    if (use_t2) {
      int cr = tc_transform2_compose(d, (const bf16*)w->conv0_w, (const bf16*)w->conv1_w, wc, ss);
      if (cr < 0) { h->last_cuda = -cr; return CCA_ERR_CUDA; }
      if (cr != 0) return CCA_ERR_INVALID_ARG;
      h->launches++;
    }
    if (forked) CU(cudaEventRecord(h->ev_join, h->side));
  }
  // the three down-projection weights stacked (also the B operand of the input gradient in the backward)
  // (no copy if the caller keeps them adjacent in that order already)
  const bf16* w_all = (const bf16*)w->w_qk;
  if (!adjacent(w->w_qk, w->w_v1, w->w_v2, d.L, d.Lk / 2, (size_t)d.E * 2)) {
    bf16* ws_all = (bf16*)(ws + l.w_all);
    CU(cudaMemcpyAsync(ws_all, w->w_qk, (size_t)d.L * d.E * 2, cudaMemcpyDeviceToDevice, st));
    CU(cudaMemcpyAsync(ws_all + (size_t)d.L * d.E, w->w_v1, (size_t)(d.Lk / 2) * d.E * 2, cudaMemcpyDeviceToDevice, st));
    CU(cudaMemcpyAsync(ws_all + (size_t)(d.L + d.Lk / 2) * d.E, w->w_v2, (size_t)(d.Lk / 2) * d.E * 2,
                       cudaMemcpyDeviceToDevice, st));
    w_all = ws_all;
  }
  GemmArgs g{};
  bool fused = false;
  if (h->impl >= 1 && h->tc) {
    // Eq. 7 and Eq. 10 in one contraction: [qk0 | v1 | v2] = x [W_qk; W_v1; W_v2]^T, the v2 columns stored one token later
    g.A = kmajor(x, d.E); g.B = kmajor(w_all, d.E);
    g.M = T; g.N = d.L + d.Lk; g.K = d.E; g.a_row_off = 0; g.seq_len = d.S;
    g.out_bf16 = v; g.out_f32 = qk0; g.ldc = d.L;
    g.split_L = d.L; g.split_Lk = d.Lk; g.split_shift = (c.flags & CCA_V_SHIFT) ? 1 : 0;
    g.out_lat_bf16 = (use_t2 && d.L % 32 == 0) ? qk0b : nullptr;
    int pr = tc_gemm_pair(h->tc, g, h->d_status, st);
    if (pr < 0) { h->last_cuda = -pr; return CCA_ERR_CUDA; }
    if (pr == 0) { fused = true; h->launches++; }
  }
  const bool have_qk0b = fused && g.out_lat_bf16 != nullptr;
  if (!fused) {
    // Eq. 7: packed q/k down-projection
    g = GemmArgs{};
    g.A = kmajor(x, d.E); g.B = kmajor(w->w_qk, d.E);
    g.M = T; g.N = d.L; g.K = d.E; g.a_row_off = 0; g.seq_len = d.S;
    g.out_bf16 = nullptr; g.out_f32 = qk0; g.ldc = d.L;
    if ((r = run_gemm(h, g, st)) != CCA_OK) return r;
    // Eq. 10: value halves from x_t and x_{t-1}
    g.B = kmajor(w->w_v1, d.E); g.N = d.Lk / 2; g.out_f32 = nullptr; g.out_bf16 = v; g.ldc = d.Lk;
    if ((r = run_gemm(h, g, st)) != CCA_OK) return r;
    g.B = kmajor(w->w_v2, d.E); g.out_bf16 = v + d.Lk / 2;
    g.a_row_off = (c.flags & CCA_V_SHIFT) ? -1 : 0;
    if ((r = run_gemm(h, g, st)) != CCA_OK) return r;
  }
  // Eq. 8, 9, 11: convs, q-k-mean, norm, temperature, RoPE
  if (forked) CU(cudaStreamWaitEvent(st, h->ev_join, 0));
  STAGE(CCA_EV_FWD_PROJ);
  if (d.dh > 128) {
    // unfused: conv1 at the taps conv2 reads, conv2 as one contraction per head over (input channel, tap), then the
    // per-(token, head) stages
    bf16* y1s = (bf16*)(ws + l.y1s);
    float* y2 = (float*)(ws + l.y2);
    CU(launch_conv1_taps(d, qk0, (const bf16*)w->conv0_w, y1s, y2, st));
    h->launches++;
    if (c.flags & CCA_CONV2) {
      const int kd = d.dh * c.k_ch;
      for (int hh = 0; hh < d.hq + d.hk; ++hh) {
        GemmArgs gc{};
        gc.A = kmajor(y1s + (size_t)hh * kd, (long long)d.L * c.k_ch);
        gc.B = kmajor((const bf16*)w->conv1_w + (size_t)hh * d.dh * kd, kd);
        gc.M = T; gc.N = d.dh; gc.K = kd; gc.seq_len = d.S; gc.out_f32 = y2 + (size_t)hh * d.dh; gc.ldc = d.L;
        if ((r = run_gemm(h, gc, st)) != CCA_OK) return r;
      }
    }
    CU(launch_finalize(d, qk0, y2, w->temp, rope, q, k, rnorm, st));
    h->launches++;
  } else if (h->impl >= 1 && !(c.flags & (CCA_CONV1 | CCA_CONV2)) && (d.dh == 64 || d.dh == 128)) {
    // no convolution at all (the plain GQA / MHA configurations): the per-(token, head) stages read qk0 directly
    CU(launch_finalize(d, qk0, qk0, w->temp, rope, q, k, rnorm, st));
    h->launches++;
  } else {
    bool done = false;
    if (have_qk0b) {
      int tr = tc_transform2_fwd(h->tc, d, qk0, qk0b, wc, w->temp, rope, q, k, rnorm, h->d_status, st);
      if (tr == 0) done = true;
      if (tr < 0) { h->last_cuda = -tr; return CCA_ERR_CUDA; }
    }
    if (!done && h->impl >= 1 && h->tc) {
      int tr = tc_transform_fwd(h->tc, d, qk0, (const bf16*)w->conv0_w, (const bf16*)w->conv1_w, w->temp, rope, q, k,
                                rnorm, h->d_status, st);
      if (tr == 0) done = true;
      if (tr < 0) { h->last_cuda = -tr; return CCA_ERR_CUDA; }
    }
    if (!done)
      CU(launch_transform_fwd(d, qk0, (const bf16*)w->conv0_w, (const bf16*)w->conv1_w, w->temp, rope, q, k, rnorm, st));
    h->launches++;
  }
  STAGE(CCA_EV_FWD_TRANSFORM);
  // Eq. 11: attention in the latent
  // with the norm stage on, the logits are bounded by sqrt(d_h) exp(temp): the kernel may use that as the row maximum
  if ((r = run_attention_fwd(h, d, q, k, v, o, o32, lse, (c.flags & CCA_QK_NORM) ? w->temp : nullptr, st)) != CCA_OK)
    return r;
  STAGE(CCA_EV_FWD_ATTN);
  // Eq. 11: up-projection
  g = GemmArgs{};
  g.A = kmajor(o, d.Lq); g.B = kmajor(w->w_o, d.Lq);
  g.M = T; g.N = d.E; g.K = d.Lq; g.a_row_off = 0; g.seq_len = d.S;
  g.out_bf16 = (bf16*)out; g.ldc = d.E;
  if ((r = run_gemm(h, g, st)) != CCA_OK) return r;
  STAGE(CCA_EV_FWD_END);
  if (save_for_backward) { h->saved_ws = workspace; h->saved_B = B; h->saved_S = S; }
  return CCA_OK;
}

// Tokens [t_begin, t_end) of one causal sequence of S_total tokens whose earlier tokens have been through this function
// (or cca_forward) with the same workspace: see the header.
int cca_forward_chunk(cca_handle* h, const cca_weights* w, const void* x_chunk, void* out_chunk, void* workspace,
                      size_t workspace_bytes, int64_t S_total, int64_t t_begin, int64_t t_end, void* cuda_stream) {
  int r = check_sizes(h, 1, S_total, true);
  if (r != CCA_OK) return r;
  if (!w || !x_chunk || !out_chunk || !workspace) return CCA_ERR_INVALID_ARG;
  if (!w->w_qk || !w->w_v1 || !w->w_v2 || !w->w_o) return CCA_ERR_INVALID_ARG;
  if (t_begin < 0 || t_begin >= t_end || t_end > S_total || t_begin % 256) return CCA_ERR_INVALID_ARG;
  const cca_config& c = h->cfg;
  if ((c.flags & CCA_CONV1) && !w->conv0_w) return CCA_ERR_INVALID_ARG;
  if (!w->conv1_w || ((c.flags & CCA_QK_NORM) && !w->temp)) return CCA_ERR_INVALID_ARG;
  // the tensor-core kernels only: causal, fused conv2, head size 64 or 128, at least 512 tokens per chunk
  if (!c.causal || !(c.flags & CCA_CONV2) || (c.head_dim != 64 && c.head_dim != 128) || h->impl < 1 || !h->tc ||
      t_end - t_begin < 512)
    return CCA_ERR_UNSUPPORTED;
  if (!aligned16(x_chunk) || !aligned16(out_chunk) || !aligned16(w->w_qk) || !aligned16(w->w_v1) || !aligned16(w->w_v2) ||
      !aligned16(w->w_o) || (reinterpret_cast<uintptr_t>(workspace) & 255))
    return CCA_ERR_ALIGNMENT;
  Layout l = make_layout(c, 1, S_total);
  if (workspace_bytes < l.saved_end) return CCA_ERR_WORKSPACE_TOO_SMALL;
  CU(cudaSetDevice(h->device));
  cudaStream_t st = (cudaStream_t)cuda_stream;
  CcaDims d = make_dims(c, 1, t_end);            // the sequence as far as it exists now
  const int M = (int)(t_end - t_begin);
  char* ws = (char*)workspace;
  float* qk0 = (float*)(ws + l.qk0);
  bf16* q = (bf16*)(ws + l.q);
  bf16* k = (bf16*)(ws + l.k);
  bf16* v = (bf16*)(ws + l.v);
  bf16* o = (bf16*)(ws + l.o);
  float* lse = (float*)(ws + l.lse);
  float2* rope = (float2*)(ws + l.rope);
  float* rnorm = (float*)(ws + l.rnorm);
  if (t_begin == 0 && (c.flags & CCA_ROPE)) {
    CU(launch_rope_table(rope, (int)S_total, d.dh, c.rope_base, st));
    h->launches++;
  }
  const bf16* w_all = (const bf16*)w->w_qk;
  if (!adjacent(w->w_qk, w->w_v1, w->w_v2, d.L, d.Lk / 2, (size_t)d.E * 2)) {
    bf16* ws_all = (bf16*)(ws + l.w_all);
    CU(cudaMemcpyAsync(ws_all, w->w_qk, (size_t)d.L * d.E * 2, cudaMemcpyDeviceToDevice, st));
    CU(cudaMemcpyAsync(ws_all + (size_t)d.L * d.E, w->w_v1, (size_t)(d.Lk / 2) * d.E * 2, cudaMemcpyDeviceToDevice, st));
    CU(cudaMemcpyAsync(ws_all + (size_t)(d.L + d.Lk / 2) * d.E, w->w_v2, (size_t)(d.Lk / 2) * d.E * 2,
                       cudaMemcpyDeviceToDevice, st));
    w_all = ws_all;
  }
  // Eq. 7 and Eq. 10 for the chunk's rows; the value-shifted half of row t_end goes to the next chunk's first row
  GemmArgs g{};
  g.A = kmajor(x_chunk, d.E); g.B = kmajor(w_all, d.E);
  g.M = M; g.N = d.L + d.Lk; g.K = d.E; g.seq_len = (int)S_total; g.row0 = (int)t_begin;
  g.out_bf16 = v + (size_t)t_begin * d.Lk; g.out_f32 = qk0 + (size_t)t_begin * d.L; g.ldc = d.L;
  g.split_L = d.L; g.split_Lk = d.Lk; g.split_shift = (c.flags & CCA_V_SHIFT) ? 1 : 0;
  // the TMA-fed transform kernel where it covers the configuration: bf16 copy of the chunk's qk0 rows, composed weights
  const bool use_t2 = tc_transform2_covers(d) && d.L % 32 == 0;
  bf16* qk0b = (bf16*)(ws + l.qk0b);
  bf16* wc = (bf16*)(ws + l.wc);
  if (use_t2) {
    g.out_lat_bf16 = qk0b + (size_t)t_begin * d.L;
    int cr = tc_transform2_compose(d, (const bf16*)w->conv0_w, (const bf16*)w->conv1_w, wc, st);
    if (cr < 0) { h->last_cuda = -cr; return CCA_ERR_CUDA; }
    if (cr != 0) return CCA_ERR_INVALID_ARG;
    h->launches++;
  }
  int pr = tc_gemm_pair(h->tc, g, h->d_status, st);
  if (pr < 0) { h->last_cuda = -pr; return CCA_ERR_CUDA; }
  if (pr != 0) return CCA_ERR_UNSUPPORTED;
  h->launches++;
  int tr = use_t2 ? tc_transform2_fwd(h->tc, d, qk0, qk0b, wc, w->temp, rope, q, k, rnorm, h->d_status, st, (int)t_begin)
                  : tc_transform_fwd(h->tc, d, qk0, (const bf16*)w->conv0_w, (const bf16*)w->conv1_w, w->temp, rope, q, k,
                                     rnorm, h->d_status, st, (int)t_begin);
  if (tr < 0) { h->last_cuda = -tr; return CCA_ERR_CUDA; }
  if (tr != 0) return CCA_ERR_UNSUPPORTED;
  h->launches++;
  if (h->ev_attn_begin) CU(cudaEventRecord(h->ev_attn_begin, st));
  int ar = tc_attn_fwd(h->tc, d, q, k, v, o, nullptr, lse, (c.flags & CCA_QK_NORM) ? w->temp : nullptr, h->d_status, st,
                       (int)t_begin);
  if (ar < 0) { h->last_cuda = -ar; return CCA_ERR_CUDA; }
  if (ar != 0) return CCA_ERR_UNSUPPORTED;
  h->launches++;
  if (h->ev_attn_end) CU(cudaEventRecord(h->ev_attn_end, st));
  g = GemmArgs{};
  g.A = kmajor(o + (size_t)t_begin * d.Lq, d.Lq); g.B = kmajor(w->w_o, d.Lq);
  g.M = M; g.N = d.E; g.K = d.Lq; g.seq_len = M;
  g.out_bf16 = (bf16*)out_chunk; g.ldc = d.E;
  return run_gemm(h, g, st);
}

int cca_forward_host(cca_handle* h, const cca_weights* w, const void* x_host, void* out_host, void* workspace,
                     size_t workspace_bytes, int64_t B, int64_t S, void* cuda_stream) {
  int r = check_sizes(h, B, S, true);
  if (r != CCA_OK) return r;
  if (!x_host || !out_host || !workspace) return CCA_ERR_INVALID_ARG;
  Layout l = make_layout(h->cfg, B, S);
  const size_t act = align_up((size_t)B * S * h->cfg.d_model * 2, 256);
  if (workspace_bytes < l.saved_end + 2 * act) return CCA_ERR_WORKSPACE_TOO_SMALL;
  CU(cudaSetDevice(h->device));
  cudaStream_t st = (cudaStream_t)cuda_stream;
  char* xs = (char*)workspace + l.saved_end;
  char* os = xs + act;
  // One causal sequence that the tensor-core kernels cover: chunks of the sequence go through the copy engines and
  // the kernels as a pipeline (tokens in on one stream, compute on the caller's, results out on a third), since a
  // chunk needs nothing of the tokens after it.
  const cca_config& c = h->cfg;
  const int64_t CH = 2048;
  if (B == 1 && S >= 2 * CH && S % CH == 0 && S / CH <= 64 && c.causal && (c.flags & CCA_CONV2) &&
      (c.head_dim == 64 || c.head_dim == 128) && h->impl >= 1 && h->tc) {
    if (!h->s_in) {
      if (cudaStreamCreateWithFlags(&h->s_in, cudaStreamNonBlocking) != cudaSuccess ||
          cudaStreamCreateWithFlags(&h->s_out, cudaStreamNonBlocking) != cudaSuccess) {
        (void)cudaGetLastError();
        if (h->s_in) cudaStreamDestroy(h->s_in);
        h->s_in = h->s_out = nullptr;
      }
    }
    const int n_ch = (int)(S / CH);
    while (h->s_in && h->n_ev < n_ch) {
      if (cudaEventCreateWithFlags(&h->ev_chunk[0][h->n_ev], cudaEventDisableTiming) != cudaSuccess) break;
      if (cudaEventCreateWithFlags(&h->ev_chunk[1][h->n_ev], cudaEventDisableTiming) != cudaSuccess) {
        cudaEventDestroy(h->ev_chunk[0][h->n_ev]);
        break;
      }
      h->n_ev++;
    }
    if (h->s_in && h->n_ev >= n_ch) {
      const size_t row = (size_t)c.d_model * 2;
      // the copy streams start after whatever the caller's stream has queued so far
      CU(cudaEventRecord(h->ev_chunk[1][0], st));
      CU(cudaStreamWaitEvent(h->s_in, h->ev_chunk[1][0], 0));
      CU(cudaStreamWaitEvent(h->s_out, h->ev_chunk[1][0], 0));
      for (int i = 0; i < n_ch; ++i) {
        const size_t off = (size_t)i * CH * row;
        CU(cudaMemcpyAsync(xs + off, (const char*)x_host + off, (size_t)CH * row, cudaMemcpyHostToDevice, h->s_in));
        CU(cudaEventRecord(h->ev_chunk[0][i], h->s_in));
        CU(cudaStreamWaitEvent(st, h->ev_chunk[0][i], 0));
        r = cca_forward_chunk(h, w, xs + off, os + off, workspace, l.saved_end, S, (int64_t)i * CH, (int64_t)(i + 1) * CH,
                              cuda_stream);
        if (r != CCA_OK) return r;
        CU(cudaEventRecord(h->ev_chunk[1][i], st));
        CU(cudaStreamWaitEvent(h->s_out, h->ev_chunk[1][i], 0));
        CU(cudaMemcpyAsync((char*)out_host + off, os + off, (size_t)CH * row, cudaMemcpyDeviceToHost, h->s_out));
      }
      CU(cudaStreamSynchronize(h->s_out));
      CU(cudaStreamSynchronize(st));
      return CCA_OK;
    }
  }
  CU(cudaMemcpyAsync(xs, x_host, (size_t)B * S * h->cfg.d_model * 2, cudaMemcpyHostToDevice, st));
  r = cca_forward(h, w, xs, os, workspace, l.saved_end, B, S, 0, cuda_stream);
  if (r != CCA_OK) return r;
  CU(cudaMemcpyAsync(out_host, os, (size_t)B * S * h->cfg.d_model * 2, cudaMemcpyDeviceToHost, st));
  CU(cudaStreamSynchronize(st));
  return CCA_OK;
}

int cca_backward(cca_handle* h, const cca_weights* w, const void* x, const void* d_out, void* workspace,
                 size_t workspace_bytes, void* d_x, const cca_weight_grads* gr, int64_t B, int64_t S,
                 void* cuda_stream) {
  int r = check_sizes(h, B, S, true);
  if (r != CCA_OK) return r;
  if (!w || !x || !d_out || !workspace || !d_x || !gr) return CCA_ERR_INVALID_ARG;
  if (!w->w_qk || !w->w_v1 || !w->w_v2 || !w->w_o) return CCA_ERR_INVALID_ARG;
  if (!gr->d_w_qk || !gr->d_w_v1 || !gr->d_w_v2 || !gr->d_w_o || !gr->d_conv0_w || !gr->d_conv1_w || !gr->d_temp)
    return CCA_ERR_INVALID_ARG;
  const cca_config& c = h->cfg;
  if ((c.flags & CCA_CONV1) && !w->conv0_w) return CCA_ERR_INVALID_ARG;
  if ((c.flags & CCA_CONV2) && !w->conv1_w) return CCA_ERR_INVALID_ARG;
  if ((c.flags & CCA_QK_NORM) && !w->temp) return CCA_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(d_out) || !aligned16(d_x) || !aligned16(w->w_qk) || !aligned16(w->w_v1) ||
      !aligned16(w->w_v2) || !aligned16(w->w_o) || !aligned16(gr->d_w_qk) || !aligned16(gr->d_w_v1) ||
      !aligned16(gr->d_w_v2) || !aligned16(gr->d_w_o) || (reinterpret_cast<uintptr_t>(workspace) & 255))
    return CCA_ERR_ALIGNMENT;
  Layout l = make_layout(c, B, S);
  if (workspace_bytes < l.total_end) return CCA_ERR_WORKSPACE_TOO_SMALL;
  // the workspace must be the one the last cca_forward(..., save_for_backward = 1) filled for this B and S:
  // without it the fp32 copy of o (and hence delta and every gradient) would be read from unwritten memory
  if (h->saved_ws != workspace || h->saved_B != B || h->saved_S != S) return CCA_ERR_INVALID_ARG;
  CU(cudaSetDevice(h->device));
  cudaStream_t st = (cudaStream_t)cuda_stream;
  CcaDims d = make_dims(c, B, S);
  const int T = d.B * d.S;
  char* ws = (char*)workspace;
  const float* qk0 = (const float*)(ws + l.qk0);
  const bf16* q = (const bf16*)(ws + l.q);
  const bf16* k = (const bf16*)(ws + l.k);
  const bf16* v = (const bf16*)(ws + l.v);
  const bf16* o = (const bf16*)(ws + l.o);
  const float* lse = (const float*)(ws + l.lse);
  const float2* rope = (const float2*)(ws + l.rope);
  const float* rnorm = (const float*)(ws + l.rnorm);
  const float* o32 = (const float*)(ws + l.o32);
  bf16* d_o = (bf16*)(ws + l.d_o);
  float* delta = (float*)(ws + l.delta);
  float* dq = (float*)(ws + l.dq);
  float* dk = (float*)(ws + l.dk);
  float* dv = (float*)(ws + l.dv);
  bf16* dlat = (bf16*)(ws + l.dlat);
  // the stacked down-projection weights: the caller's own if they are adjacent, else the forward's copy
  const bf16* w_all = adjacent(w->w_qk, w->w_v1, w->w_v2, d.L, d.Lk / 2, (size_t)d.E * 2) ? (const bf16*)w->w_qk
                                                                                         : (const bf16*)(ws + l.w_all);
  const long long ldl = d.L + d.Lk;

  STAGE(CCA_EV_BWD_BEGIN);
  CU(cudaMemsetAsync(gr->d_conv0_w, 0, (size_t)d.L * c.k_seq * 4, st));
  CU(cudaMemsetAsync(gr->d_conv1_w, 0, (size_t)d.L * d.dh * c.k_ch * 4, st));
  CU(cudaMemsetAsync(gr->d_temp, 0, (size_t)d.hk * 4, st));
  // up-projection adjoint: d_o = d_out W_o ; d_W_o = d_out^T o
  GemmArgs g{};
  g.A = kmajor(d_out, d.E); g.B = mmajor(w->w_o, d.Lq);
  g.M = T; g.N = d.Lq; g.K = d.E; g.seq_len = d.S; g.out_bf16 = d_o; g.ldc = d.Lq;
  if ((r = run_gemm(h, g, st)) != CCA_OK) return r;
  STAGE(CCA_EV_BWD_DO);
  g = GemmArgs{};
  g.A = mmajor(d_out, d.E); g.B = mmajor(o, d.Lq);
  g.M = d.E; g.N = d.Lq; g.K = T; g.seq_len = d.S; g.out_f32 = gr->d_w_o; g.ldc = d.Lq;
  if ((r = run_gemm(h, g, st)) != CCA_OK) return r;
  STAGE(CCA_EV_BWD_DWO);
  // attention adjoint
  CU(launch_attn_delta(d, o32, d_o, delta, st));
  h->launches++;
  STAGE(CCA_EV_BWD_DELTA);
  {
    if (h->ev_attn_begin) CU(cudaEventRecord(h->ev_attn_begin, st));
    bool done = false;
    if (d.dh > 128) {
      // Head size 256: the adjoint as plain contractions over chunks of query rows of one (sequence, query head) at a
      // time.  S = Q K^T and dP = dO V^T (fp32), P and dS / sqrt(d_h) (bf16, element-wise), then dQ = dS K,
      // dV += P^T dO, dK += dS^T Q, the latter two accumulated over chunks and over the g heads of a group.
      float* s32 = (float*)(ws + l.u_s);
      float* dp32 = (float*)(ws + l.u_dp);
      bf16* pb = (bf16*)(ws + l.u_p);
      bf16* dsb = (bf16*)(ws + l.u_ds);
      const long long ld = (long long)l.u_ld;
      CU(cudaMemsetAsync(dk, 0, (size_t)T * d.Lk * 4, st));
      CU(cudaMemsetAsync(dv, 0, (size_t)T * d.Lk * 4, st));
      for (int b = 0; b < d.B; ++b)
        for (int i = 0; i < d.hq; ++i) {
          const int j = i / d.g;
          const bf16* kj = k + (size_t)b * d.S * d.Lk + (size_t)j * d.dh;
          const bf16* vj = v + (size_t)b * d.S * d.Lk + (size_t)j * d.dh;
          const float* lse_i = lse + ((size_t)b * d.hq + i) * d.S;
          const float* delta_i = delta + ((size_t)b * d.hq + i) * d.S;
          for (int m0 = 0; m0 < d.S; m0 += l.u_rows) {
            const int rows = d.S - m0 < l.u_rows ? d.S - m0 : l.u_rows;
            const int n_keys = d.causal ? m0 + rows : d.S;
            const size_t qoff = ((size_t)b * d.S + m0) * d.Lq + (size_t)i * d.dh;
            GemmArgs ga{};
            ga.A = kmajor(q + qoff, d.Lq); ga.B = kmajor(kj, d.Lk);
            ga.M = rows; ga.N = n_keys; ga.K = d.dh; ga.seq_len = rows; ga.out_f32 = s32; ga.ldc = ld;
            if ((r = run_gemm(h, ga, st)) != CCA_OK) return r;
            ga.A = kmajor(d_o + qoff, d.Lq); ga.B = kmajor(vj, d.Lk); ga.out_f32 = dp32;
            if ((r = run_gemm(h, ga, st)) != CCA_OK) return r;
            CU(launch_pds(s32, dp32, ld, lse_i, delta_i, m0, rows, n_keys, d.S, d.causal, d.dh, pb, dsb, st));
            h->launches++;
            ga = GemmArgs{};
            ga.A = kmajor(dsb, ld); ga.B = mmajor(kj, d.Lk);
            ga.M = rows; ga.N = d.dh; ga.K = n_keys; ga.seq_len = rows; ga.out_f32 = dq + qoff; ga.ldc = d.Lq;
            if ((r = run_gemm(h, ga, st)) != CCA_OK) return r;
            ga = GemmArgs{};
            ga.A = mmajor(pb, ld); ga.B = mmajor(d_o + qoff, d.Lq);
            ga.M = n_keys; ga.N = d.dh; ga.K = rows; ga.seq_len = n_keys; ga.ldc = d.Lk; ga.accumulate = 1;
            ga.out_f32 = dv + (size_t)b * d.S * d.Lk + (size_t)j * d.dh;
            if ((r = run_gemm(h, ga, st)) != CCA_OK) return r;
            ga.A = mmajor(dsb, ld); ga.B = mmajor(q + qoff, d.Lq);
            ga.out_f32 = dk + (size_t)b * d.S * d.Lk + (size_t)j * d.dh;
            if ((r = run_gemm(h, ga, st)) != CCA_OK) return r;
          }
        }
      done = true;
    }
    if (!done && h->impl >= 1 && h->tc) {
      int tr = tc_attn_bwd(h->tc, d, q, k, v, d_o, lse, delta, dq, dk, dv, h->d_status, st);
      if (tr == 0) done = true;
      if (tr < 0) { h->last_cuda = -tr; return CCA_ERR_CUDA; }
    }
    if (!done) CU(launch_attn_bwd_simt(d, q, k, v, o32, d_o, lse, delta, dq, dk, dv, st));
    h->launches += 2;
    if (h->ev_attn_end) CU(cudaEventRecord(h->ev_attn_end, st));
  }
  STAGE(CCA_EV_BWD_ATTN);
  // latent-transform adjoints
  CU(launch_transform_bwd_norm(d, q, k, rnorm, w->temp, rope, dq, dk, gr->d_temp, st));
  STAGE(CCA_EV_BWD_NORM);
  {
    bool done = false;
    if (d.dh > 128) {
      // Head size 256: conv2's adjoint as one contraction per head on the stored conv1 taps (the forward's y1s),
      // dy1s = d_hat W_head and d_conv1_w[head] = d_hat^T y1s, then the taps folded back onto their tokens.
      float* dy1 = (float*)(ws + l.dy1);
      if (c.flags & CCA_CONV2) {
        bf16* dhat = dlat;                      // the latent-gradient buffer is free until conv1's adjoint writes it
        const bf16* y1s = (const bf16*)(ws + l.y1s);
        float* dy1s = (float*)(ws + l.u_dy1s);
        const int kd = d.dh * c.k_ch;
        CU(launch_cast_dhat(d, dq, dk, dhat, nullptr, st));
        for (int hh = 0; hh < d.hq + d.hk; ++hh) {
          GemmArgs gc{};
          gc.A = kmajor(dhat + (size_t)hh * d.dh, d.L);
          gc.B = mmajor((const bf16*)w->conv1_w + (size_t)hh * d.dh * kd, kd);
          gc.M = T; gc.N = kd; gc.K = d.dh; gc.seq_len = d.S; gc.out_f32 = dy1s + (size_t)hh * kd; gc.ldc = (long long)d.L * c.k_ch;
          if ((r = run_gemm(h, gc, st)) != CCA_OK) return r;
          gc = GemmArgs{};
          gc.A = mmajor(dhat + (size_t)hh * d.dh, d.L);
          gc.B = mmajor(y1s + (size_t)hh * kd, (long long)d.L * c.k_ch);
          gc.M = d.dh; gc.N = kd; gc.K = T; gc.seq_len = d.S; gc.out_f32 = gr->d_conv1_w + (size_t)hh * d.dh * kd; gc.ldc = kd;
          if ((r = run_gemm(h, gc, st)) != CCA_OK) return r;
        }
        CU(launch_taps_adjoint(d, dy1s, dy1, st));
      } else {
        CU(launch_cast_dhat(d, dq, dk, nullptr, dy1, st));
      }
      STAGE(CCA_EV_BWD_CONV2);
      CU(launch_conv1_adjoint(d, dy1, dq, dk, qk0, (const bf16*)w->conv0_w, dlat, ldl, gr->d_conv0_w, st));
      done = true;
    }
    if (!done && h->impl >= 1 && h->tc) {
      float* dy1 = (float*)(ws + l.dy1);
      int tr = tc_transform_bwd(h->tc, d, qk0, (const bf16*)w->conv0_w, (const bf16*)w->conv1_w, dq, dk, dy1,
                                gr->d_conv1_w, h->d_status, st);
      if (tr < 0) { h->last_cuda = -tr; return CCA_ERR_CUDA; }
      if (tr == 0) {
        STAGE(CCA_EV_BWD_CONV2);
        CU(launch_conv1_adjoint(d, dy1, dq, dk, qk0, (const bf16*)w->conv0_w, dlat, ldl, gr->d_conv0_w, st));
        done = true;
      }
    }
    if (!done) {
      CU(launch_transform_bwd_conv(d, qk0, (const bf16*)w->conv0_w, (const bf16*)w->conv1_w, dq, dk, dlat, ldl,
                                   gr->d_conv0_w, st));
      CU(launch_transform_bwd_w1(d, qk0, (const bf16*)w->conv0_w, dq, dk, gr->d_conv1_w, st));
    }
  }
  STAGE(CCA_EV_BWD_CONV1);
  CU(launch_pack_dv(d, dv, dlat, ldl, st));
  h->launches += 4;
  STAGE(CCA_EV_BWD_PACK);
  // down-projection adjoints: parameter gradients
  g = GemmArgs{};
  g.A = mmajor(dlat, ldl); g.B = mmajor(x, d.E);
  g.M = d.L; g.N = d.E; g.K = T; g.seq_len = d.S; g.out_f32 = gr->d_w_qk; g.ldc = d.E;
  if (adjacent(gr->d_w_qk, gr->d_w_v1, gr->d_w_v2, d.L, d.Lk / 2, (size_t)d.E * 4)) {
    // the three gradients are one [L + L_k, E] block for the caller: one contraction writes them all
    g.M = d.L + d.Lk;
    if ((r = run_gemm(h, g, st)) != CCA_OK) return r;
  } else {
    if ((r = run_gemm(h, g, st)) != CCA_OK) return r;
    g.A = mmajor(dlat + d.L, ldl); g.M = d.Lk / 2; g.out_f32 = gr->d_w_v1;
    if ((r = run_gemm(h, g, st)) != CCA_OK) return r;
    g.A = mmajor(dlat + d.L + d.Lk / 2, ldl); g.out_f32 = gr->d_w_v2;
    if ((r = run_gemm(h, g, st)) != CCA_OK) return r;
  }
  STAGE(CCA_EV_BWD_DW);
  // input gradient: d_x = [d_qk0, d_v1, d_v2 moved one token earlier] [W_qk; W_v1; W_v2] (stacked by the forward)
  g = GemmArgs{};
  g.A = kmajor(dlat, ldl); g.B = mmajor(w_all, d.E);
  g.M = T; g.N = d.E; g.K = (int)ldl; g.seq_len = d.S; g.out_bf16 = (bf16*)d_x; g.ldc = d.E;
  if ((r = run_gemm(h, g, st)) != CCA_OK) return r;
  STAGE(CCA_EV_BWD_END);
  return CCA_OK;
}

// ---- MLA baseline ---------------------------------------------------------------------------------
namespace {
struct MlaLayout {
  size_t cq, ckv, kr, qn, qr, kn, q, k, v, o, lse, rope, end;
};
MlaLayout make_mla_layout(const cca_config& c, const cca_mla_dims& m, int64_t B, int64_t S) {
  MlaLayout l;
  const size_t T = (size_t)B * S, nh = c.n_q_heads, dh = c.head_dim;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  l.cq = take(T * m.d_cq * 2);
  l.ckv = take(T * m.d_ckv * 2);
  l.kr = take(T * m.d_rope * 2);
  l.qn = take(T * nh * m.d_nope * 2);
  l.qr = take(T * nh * m.d_rope * 2);
  l.kn = take(T * nh * m.d_nope * 2);
  l.q = take(T * nh * dh * 2);
  l.k = take(T * nh * dh * 2);
  l.v = take(T * nh * dh * 2);
  l.o = take(T * nh * dh * 2);
  l.lse = take((size_t)B * nh * S * 4);
  l.rope = take((size_t)S * (m.d_rope / 2) * 8);
  l.end = off;
  return l;
}
int check_mla(const cca_handle* h, const cca_mla_dims* m) {
  if (!h || !m) return CCA_ERR_INVALID_ARG;
  const cca_config& c = h->cfg;
  if (m->d_nope < 8 || m->d_rope < 8 || m->d_ckv < 8 || m->d_cq < 8) return CCA_ERR_INVALID_ARG;
  if (m->d_nope + m->d_rope != c.head_dim || c.n_q_heads != c.n_kv_heads) return CCA_ERR_INVALID_ARG;
  if (m->d_nope % 8 || m->d_rope % 16 || m->d_ckv % 8 || m->d_cq % 8) return CCA_ERR_UNSUPPORTED;
  return CCA_OK;
}
}  // namespace

int cca_mla_workspace_size(const cca_handle* h, const cca_mla_dims* m, int64_t B, int64_t S, size_t* bytes) {
  int r = check_sizes(h, B, S);
  if (r != CCA_OK) return r;
  if ((r = check_mla(h, m)) != CCA_OK) return r;
  if (!bytes) return CCA_ERR_INVALID_ARG;
  *bytes = make_mla_layout(h->cfg, *m, B, S).end;
  return CCA_OK;
}

int cca_mla_forward(cca_handle* h, const cca_mla_dims* m, const cca_mla_weights* w, const void* x, void* out, void* workspace,
                    size_t workspace_bytes, int64_t B, int64_t S, void* cuda_stream) {
  int r = check_sizes(h, B, S, true);
  if (r != CCA_OK) return r;
  if ((r = check_mla(h, m)) != CCA_OK) return r;
  if (!w || !x || !out || !workspace) return CCA_ERR_INVALID_ARG;
  if (!w->w_dq || !w->w_dkv || !w->w_uq || !w->w_uqr || !w->w_uk || !w->w_uv || !w->w_kr || !w->w_o) return CCA_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(out) || !aligned16(w->w_dq) || !aligned16(w->w_dkv) || !aligned16(w->w_uq) ||
      !aligned16(w->w_uqr) || !aligned16(w->w_uk) || !aligned16(w->w_uv) || !aligned16(w->w_kr) || !aligned16(w->w_o) ||
      (reinterpret_cast<uintptr_t>(workspace) & 255))
    return CCA_ERR_ALIGNMENT;
  const cca_config& c = h->cfg;
  MlaLayout l = make_mla_layout(c, *m, B, S);
  if (workspace_bytes < l.end) return CCA_ERR_WORKSPACE_TOO_SMALL;
  CU(cudaSetDevice(h->device));
  cudaStream_t st = (cudaStream_t)cuda_stream;
  CcaDims d = make_dims(c, B, S);
  const int T = d.B * d.S, nh = d.hq, dn = m->d_nope, dr = m->d_rope, E = d.E;
  char* ws = (char*)workspace;
  bf16 *cq = (bf16*)(ws + l.cq), *ckv = (bf16*)(ws + l.ckv), *kr = (bf16*)(ws + l.kr), *qn = (bf16*)(ws + l.qn);
  bf16 *qr = (bf16*)(ws + l.qr), *kn = (bf16*)(ws + l.kn), *q = (bf16*)(ws + l.q), *k = (bf16*)(ws + l.k);
  bf16 *v = (bf16*)(ws + l.v), *o = (bf16*)(ws + l.o);
  float* lse = (float*)(ws + l.lse);
  float2* rope = (float2*)(ws + l.rope);
  STAGE(CCA_EV_FWD_BEGIN);
  CU(launch_rope_table(rope, d.S, dr, c.rope_base > 0.f ? c.rope_base : 10000.f, st));
  h->launches++;
  auto gemm = [&](const void* a, long long lda, const void* bw, int N, int K, bf16* dst) -> int {
    GemmArgs g{};
    g.A = kmajor(a, lda); g.B = kmajor(bw, K);
    g.M = T; g.N = N; g.K = K; g.seq_len = d.S; g.out_bf16 = dst; g.ldc = N;
    return run_gemm(h, g, st);
  };
  // Eq. 3: the two latents (and the shared key's RoPE part straight from x, Eq. 6)
  if ((r = gemm(x, E, w->w_dq, m->d_cq, E, cq)) != CCA_OK) return r;
  if ((r = gemm(x, E, w->w_dkv, m->d_ckv, E, ckv)) != CCA_OK) return r;
  if ((r = gemm(x, E, w->w_kr, dr, E, kr)) != CCA_OK) return r;
  // Eq. 4 and Eq. 6: per-head up-projections
  if ((r = gemm(cq, m->d_cq, w->w_uq, nh * dn, m->d_cq, qn)) != CCA_OK) return r;
  if ((r = gemm(cq, m->d_cq, w->w_uqr, nh * dr, m->d_cq, qr)) != CCA_OK) return r;
  if ((r = gemm(ckv, m->d_ckv, w->w_uk, nh * dn, m->d_ckv, kn)) != CCA_OK) return r;
  if ((r = gemm(ckv, m->d_ckv, w->w_uv, nh * d.dh, m->d_ckv, v)) != CCA_OK) return r;
  STAGE(CCA_EV_FWD_PROJ);
  CU(launch_mla_assemble(T, d.S, nh, dn, dr, qn, qr, kn, kr, rope, q, k, st));
  h->launches++;
  STAGE(CCA_EV_FWD_TRANSFORM);
  if ((r = run_attention_fwd(h, d, q, k, v, o, nullptr, lse, nullptr, st)) != CCA_OK) return r;
  STAGE(CCA_EV_FWD_ATTN);
  if ((r = gemm(o, d.Lq, w->w_o, E, d.Lq, (bf16*)out)) != CCA_OK) return r;
  STAGE(CCA_EV_FWD_END);
  return CCA_OK;
}

// ---- forward without any caller-provided or allocated workspace ---------------------------------
// The scratch of cca_forward_static: one array in the library's device image.  Every GPU that loads the
// library reserves these bytes until the process exits.  In host code `g_static_ws` is only a handle for
// cudaGetSymbolAddress, never a pointer a kernel may be given.
static __device__ __align__(256) unsigned char g_static_ws[CCA_STATIC_WORKSPACE_BYTES];

namespace {
constexpr int kMaxStaticDevices = 64;
std::mutex g_static_mu;
void* g_static_ptr[kMaxStaticDevices];     // device address of g_static_ws on each device, once resolved
}  // namespace

int cca_forward_static(cca_handle* h, const cca_weights* w, const void* x, void* out, int64_t B, int64_t S,
                       void* cuda_stream) {
  int r = check_sizes(h, B, S, true);
  if (r != CCA_OK) return r;
  if (h->device >= kMaxStaticDevices) return CCA_ERR_UNSUPPORTED;
  Layout l = make_layout(h->cfg, B, S);
  if (l.saved_end > (size_t)CCA_STATIC_WORKSPACE_BYTES) return CCA_ERR_STATIC_WORKSPACE_EXCEEDED;
  CU(cudaSetDevice(h->device));
  void* ws = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_static_mu);
    if (!g_static_ptr[h->device]) {
      // set-up, once per device, with that device current: resolve the array's address on this device
      void* p = nullptr;
      CU(cudaGetSymbolAddress(&p, g_static_ws));
      if (!p || (reinterpret_cast<uintptr_t>(p) & 255)) return CCA_ERR_ALIGNMENT;
      g_static_ptr[h->device] = p;
    }
    ws = g_static_ptr[h->device];
  }
  // Every region of the forward workspace is written in full before it is read, so the previous call's
  // contents need no clearing.  Passing exactly the forward-only size keeps the fp32 copy of o off.
  return cca_forward(h, w, x, out, ws, l.saved_end, B, S, 0, cuda_stream);
}

}  // extern "C"
