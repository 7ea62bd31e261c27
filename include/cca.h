/*
 * cca.h -- C ABI of the B200 (sm_100a) Compressed Convolutional Attention block.
 *
 * One block = down-projection of x to latent q/k/v, the latent transforms on q and k
 * (two causal convolutions, q-k-mean, L2 norm with key temperature, RoPE), value-shift,
 * causal softmax attention with grouped kv heads inside the latent, up-projection; the
 * matching backward; chunked prefill and the decode step against the latent KV cache.  The
 * method is the paper's Section 2.2 (Eq. 7-11) and Listing A.1.
 *
 * Conventions
 *   - Every pointer named "device" is CUDA device memory on the handle's device, owned by the
 *     caller.  The library allocates nothing on the device except a 64-byte status word per
 *     handle; cca_forward / cca_backward / cca_decode_step never allocate, never synchronise,
 *     never fall back to the CPU.  All work is enqueued on the caller's stream (the forward
 *     computes its RoPE table on a stream of the handle's own, joined back before it is used).
 *   - Activations are row-major [B, S, width] (the paper's listing is [S, B, width]; sequences
 *     are independent so the result is the same).  bf16 = 16-bit brain float, raw bits.
 *   - Linear weights are [out, in] row-major, like torch.nn.Linear.
 *   - Every function returns a cca_status code; nothing throws, aborts or traps.
 */
#ifndef CCA_H_
#define CCA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  CCA_OK = 0,
  CCA_ERR_INVALID_ARG = 1,         /* null pointer, non-positive size, inconsistent config   */
  CCA_ERR_UNSUPPORTED = 2,         /* shape outside kernel coverage, or device is not sm_100 */
  CCA_ERR_ALIGNMENT = 3,           /* a device pointer is not 16-byte aligned                */
  CCA_ERR_WORKSPACE_TOO_SMALL = 4,
  CCA_ERR_CUDA = 5,                /* a CUDA call failed; see cca_last_cuda_error            */
  CCA_ERR_DEVICE_TIMEOUT = 6,      /* a bounded device-side wait expired (cca_last_status)   */
  CCA_ERR_STATIC_WORKSPACE_EXCEEDED = 7  /* cca_forward_static: B, S need more than the built-in scratch */
} cca_status;

/* Optional stages (rows of the paper's ablation tables; all on = the method of Eq. 7-11). */
enum {
  CCA_CONV1 = 1,     /* conv1_seq: depth-wise causal conv over the sequence, Eq. 8          */
  CCA_CONV2 = 2,     /* conv2_seq+ch: head-wise grouped causal conv, Eq. 8                  */
  CCA_QK_MEAN = 4,   /* q-k-mean, Eq. 9                                                     */
  CCA_V_SHIFT = 8,   /* value-shift, Eq. 10 (off: both value halves read x_t)               */
  CCA_QK_NORM = 16,  /* L2 norm * sqrt(d_h), keys also * exp(temp), Eq. 11                  */
  CCA_ROPE = 32,     /* rotary embedding on the normalised latents, Eq. 11                  */
  CCA_ALL_STAGES = 63
};

/* The paper's parameters (notation table). */
typedef struct {
  int32_t d_model;      /* E                                                                */
  int32_t n_q_heads;    /* h_q;  L_q = h_q * head_dim = E / C1                              */
  int32_t n_kv_heads;   /* h_k;  L_k = h_k * head_dim = E / C2;  h_q % h_k == 0, L_k even   */
  int32_t head_dim;     /* d_h, latent per-head size: 32, 64, 128, 256                      */
  int32_t compression;  /* C = C1; checked: E == C * h_q * d_h                              */
  int32_t k_seq;        /* taps of conv1_seq (1..4)                                         */
  int32_t k_ch;         /* taps of conv2_seq+ch (1..4)                                      */
  int32_t causal;       /* attention mask only; the convs and value-shift are always causal */
  uint32_t flags;       /* CCA_* stage bits                                                 */
  float rope_base;      /* RoPE base, e.g. 10000                                            */
} cca_config;

/* Parameters, all device pointers.  q rows of w_qk come first, then k rows (Listing A.1).
 * Layout hint: the library contracts x with the stacked matrix [w_qk; w_v1; w_v2].  If the three already lie one
 * after the other in memory in that order (w_v1 == w_qk + L*E elements, w_v2 == w_v1 + (L_k/2)*E) it reads them in
 * place; otherwise every forward first copies them into the workspace (12.6 MB at the 16k prefill shape). */
typedef struct {
  const void* w_qk;     /* bf16 [L_q + L_k, E]   packed q/k down-projection, Eq. 7          */
  const void* w_v1;     /* bf16 [L_k/2, E]       value projection of x_t, Eq. 10            */
  const void* w_v2;     /* bf16 [L_k/2, E]       value projection of x_{t-1}, Eq. 10        */
  const void* w_o;      /* bf16 [E, L_q]         up-projection, Eq. 11                      */
  const void* conv0_w;  /* bf16 [L, k_seq]       depth-wise taps, last tap = current token  */
  const void* conv1_w;  /* bf16 [L, d_h, k_ch]   (out channel, in channel in head, tap)     */
  const float* temp;    /* fp32 [h_k]            log of the key temperature beta            */
} cca_weights;

/* Parameter gradients, fp32 device buffers of the parameters' shapes; overwritten.  If d_w_qk, d_w_v1, d_w_v2 lie one
 * after the other in memory (one [L + L_k, E] block) a single contraction writes all three. */
typedef struct {
  float* d_w_qk;
  float* d_w_v1;
  float* d_w_v2;
  float* d_w_o;
  float* d_conv0_w;
  float* d_conv1_w;
  float* d_temp;
} cca_weight_grads;

/* Shape and indexing metadata (integers only).  Offsets are bytes into the workspace. */
typedef struct {
  int64_t L_q, L_k, g;              /* latent widths and query heads per kv head            */
  int64_t total_padding;            /* k_seq + k_ch - 2 tokens of causal history (listing)  */
  int64_t v_shift_split;            /* first channel of the value latent fed by x_{t-1}     */
  int64_t q_to_kv_head[64];         /* q head i reads kv head floor(i / g); -1 beyond h_q   */
  int64_t conv_params;              /* L*k_seq + L*d_h*k_ch                                 */
  int64_t params;                   /* 2E^2/C1 + 2E^2/C2 + conv (comparison table)          */
  int64_t kv_cache_elems;           /* 2*B*S*E/C2                                           */
  int64_t fwd_flops;                /* (1/C1+1/C2)*4BSE^2 + 4BES^2/C1 + conv                */
  int64_t fwd_flops_causal;         /* same with the S^2 term halved                        */
  int64_t decode_flops;             /* (1/C1+1/C2)*4BE^2 + 4BES/C1 + conv                   */
  /* saved activations (written by cca_forward, read by cca_backward) */
  int64_t off_qk0, off_q, off_k, off_v, off_o, off_lse, off_rope;
  int64_t saved_bytes;              /* forward-only workspace size                          */
  int64_t total_bytes;              /* forward + backward workspace size                    */
  int64_t off_rnorm;                /* fp32 [B*S, h_q+h_k]: norm scale sqrt(d_h)[*beta]/|x| kept for the backward */
} cca_layout;

typedef struct cca_handle cca_handle;

/* Validate the configuration for `device`, create a handle.  Paper: Eq. 7-11 parameters.
 * Errors: INVALID_ARG (null, E != C*h_q*d_h, h_q % h_k, odd L_k, bad kernel sizes),
 * UNSUPPORTED (head_dim not in {32,64,128,256}, h_q > 64, device not compute capability 10.x),
 * CUDA.  device = -1 makes a host-only handle: cca_describe and cca_workspace_size work, every
 * compute entry point returns INVALID_ARG. */
int cca_init(const cca_config* cfg, int device, cca_handle** out);
int cca_destroy(cca_handle* h);

/* Fill `out` for batch B and sequence length S.  Pure host arithmetic; follows the CCGQA row
 * of the paper's comparison table and the padding / grouping / concat rules of Listing A.1. */
int cca_describe(const cca_handle* h, int64_t B, int64_t S, cca_layout* out);

/* Bytes of caller-owned device workspace needed (need_backward != 0 adds backward scratch). */
int cca_workspace_size(const cca_handle* h, int64_t B, int64_t S, int need_backward, size_t* bytes);

/* Forward of the whole block, Eq. 7-11: out = W_o [ softmax(q k^T / sqrt(d_h)) v ]_heads.
 *   x   device bf16 [B,S,E] (read), out device bf16 [B,S,E] (written).
 *   workspace: device, 256-byte aligned, >= cca_workspace_size(h, B, S, save_for_backward, ..).  On return
 *   (stream order) it holds qk0 (fp32), q, k, v, o (bf16), lse and the norm scales (fp32) at the cca_layout offsets.
 *   save_for_backward != 0: an fp32 copy of o is kept as well (the backward's delta = rowsum(dO * O) needs it) and
 *   the handle remembers (workspace, B, S); keep the workspace untouched until cca_backward.  With 0 nothing beyond
 *   saved_bytes is touched and a later cca_backward on this workspace is refused.
 * Errors: INVALID_ARG, ALIGNMENT, WORKSPACE_TOO_SMALL, CUDA. */
int cca_forward(cca_handle* h, const cca_weights* w, const void* x, void* out,
                void* workspace, size_t workspace_bytes, int64_t B, int64_t S, int save_for_backward,
                void* cuda_stream);

/* Backward of the block: given d_out = dLoss/d out (device bf16 [B,S,E]) and the workspace
 * left by cca_forward(..., save_for_backward = 1, ..) for the same x, weights, B and S, writes d_x (device bf16
 * [B,S,E]) and every field of `grads` (fp32, overwritten).  The paper prints no backward; this is the exact
 * adjoint of Eq. 7-11.  Errors as cca_forward (weights and gradient buffers 16-byte aligned; the conv weights and
 * temp non-null when their stage is on); INVALID_ARG also when `workspace`, B, S are not those of this handle's
 * last forward with save_for_backward set (nothing is launched). */
int cca_backward(cca_handle* h, const cca_weights* w, const void* x, const void* d_out,
                 void* workspace, size_t workspace_bytes, void* d_x,
                 const cca_weight_grads* grads, int64_t B, int64_t S, void* cuda_stream);

/* Chunked prefill of one causal sequence: tokens [t_begin, t_end) of a sequence of S_total tokens, given that the
 * tokens before t_begin have been through this function (or cca_forward) with the same workspace, which holds their
 * latents.  Eq. 7-11 are causal, so a chunk needs nothing of the tokens after it: out_chunk equals rows
 * [t_begin, t_end) of cca_forward on the whole sequence.  x_chunk, out_chunk: device bf16 [t_end - t_begin, E].
 * workspace: as for cca_forward(1, S_total) without the backward part; nothing is kept for a backward (the
 * log-sum-exp region is scratch here).  Chunks are processed in order of position on one stream.
 * Limits: t_begin a multiple of 256, at least 512 tokens per chunk, causal = 1, conv2 on, head_dim 64 or 128, the
 * tensor-core kernels enabled; otherwise UNSUPPORTED (use cca_forward).  Errors: as cca_forward. */
int cca_forward_chunk(cca_handle* h, const cca_weights* w, const void* x_chunk, void* out_chunk, void* workspace,
                      size_t workspace_bytes, int64_t S_total, int64_t t_begin, int64_t t_end, void* cuda_stream);

/* Same block, host buffers: copies x (host, ideally pinned) to a staging area inside the
 * workspace, runs cca_forward, copies out back to `out_host`, and synchronises the stream.
 * workspace must be >= cca_workspace_size(h, B, S, 0, ..) + 2 * round_up(B*S*E*2, 256) bytes; nothing is kept
 * for a backward.  One long causal sequence (B = 1, S a multiple of 2048) goes through as a pipeline of
 * cca_forward_chunk calls with the copies on two streams of the handle's own (created on the first such call), so
 * that the transfers in both directions overlap the compute. */
int cca_forward_host(cca_handle* h, const cca_weights* w, const void* x_host, void* out_host,
                     void* workspace, size_t workspace_bytes, int64_t B, int64_t S,
                     void* cuda_stream);

/* Forward for callers that cannot allocate device memory.  (The paper has no counterpart: this is a
 * deployment variant of cca_forward, same arithmetic, same kernels.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- a serving process whose device memory
 * was handed in full to another allocator at start-up, a plug-in that is only lent a stream and its
 * input/output buffers, a latency-critical loop that must not take the device-wide synchronisation an
 * allocation implies.  Such a caller has nowhere to get the workspace cca_forward asks for.  Here the
 * workspace is a fixed array of CCA_STATIC_WORKSPACE_BYTES inside the library's device image, so the
 * caller passes only x, out and the weights.  The function calls no cudaMalloc / cudaFree and no
 * allocating library routine.
 *
 *   - Limit: cca_workspace_size(h, B, S, 0, &n) must give n <= CCA_STATIC_WORKSPACE_BYTES, otherwise
 *     CCA_ERR_STATIC_WORKSPACE_EXCEEDED is returned and nothing is enqueued.  (32 MiB holds, for
 *     example, 4096 tokens of an 8 x 64 / 2 x 64 latent, or 2048 tokens of a 16 x 64 / 4 x 64 one.)
 *   - Cost: every GPU on which the library is loaded holds those bytes until the process exits.
 *   - The first call on a device looks up the array's device address (once, under a lock, with that
 *     device current).  Make that first call before any stream capture begins.
 *   - One array per device, shared by every handle and every call, holding whatever the last call
 *     left.  The forward overwrites each region before reading it, so nothing is cleared.  Two calls
 *     whose kernels can overlap on the GPU (different streams without an ordering between them) race
 *     on it: order them.  No activations are kept for cca_backward.
 * x, out: device bf16 [B,S,E] as in cca_forward.  Errors: as cca_forward, plus the one above. */
#define CCA_STATIC_WORKSPACE_BYTES (32u << 20)
int cca_forward_static(cca_handle* h, const cca_weights* w, const void* x, void* out, int64_t B, int64_t S,
                       void* cuda_stream);

/* Attention stage alone (Eq. 11, third line) on latents already in the workspace layout:
 * q [B,S,h_q,d_h], k, v [B,S,h_k,d_h] bf16 device -> o bf16 [B,S,h_q,d_h], lse fp32 [B,h_q,S]. */
int cca_attention_forward(cca_handle* h, const void* q, const void* k, const void* v, void* o,
                          float* lse, int64_t B, int64_t S, void* cuda_stream);

/* ---- Decode: one new token per sequence against the latent KV cache ------------------------------
 * The paper's comparison table gives the cache (2 B S E / C2 numbers: the latent keys and values) and the
 * decode FLOPs of the block; this is that step.  Besides the cache the block's definition needs, of the
 * past, the pre-convolution q0|k0 of the last k_seq + k_ch - 2 tokens (Eq. 8: the two causal convs' halo)
 * and the previous token's input (Eq. 10: half of the value channels come from x_{t-1}).  All of it is
 * caller-owned device memory described by cca_decode_state; the library keeps nothing between steps. */
typedef struct {
  void* k_cache;        /* bf16 [B, S_max, L_k]: keys after norm, temperature and RoPE (Eq. 11), row = position */
  void* v_cache;        /* bf16 [B, S_max, L_k]: values (Eq. 10)                                                */
  void* qk0_hist;       /* fp32 [B, k_seq + k_ch - 2, L]: q0|k0 (Eq. 7) of the last tokens, oldest first; all
                           zeros before a sequence's first token; may be null when k_seq = k_ch = 1           */
  void* x_prev;         /* bf16 [B, E]: previous token's input; zeros before a sequence's first token          */
  const int32_t* pos;   /* int32 [B], device: position of each sequence's new token = tokens already cached;
                           read, never written (the caller advances it after the step)                         */
  int64_t S_max;        /* capacity of both caches in tokens                                                    */
} cca_decode_state;

/* Bytes of device workspace one decode step needs for B sequences of at most max_len tokens (the new
 * token included).  The size depends on the device's SM count (the key range is split over the SMs); a
 * host-only handle assumes 148. */
int cca_decode_workspace_size(const cca_handle* h, int64_t B, int64_t max_len, size_t* bytes);

/* One decode step, Eq. 7-11 for a single new token per sequence: x device bf16 [B,E] (read), out device
 * bf16 [B,E] (written).  Sequence b's token sits at position pos[b]; it attends to cached positions
 * 0..pos[b]-1 and to itself.  On return (stream order) row pos[b] of both caches holds the new key and
 * value, qk0_hist and x_prev are advanced by one token.  max_len: host-side bound, pos[b] < max_len <=
 * S_max for every b; it sizes the launch.  A sequence whose pos[b] is outside [0, min(max_len, S_max)) is
 * skipped (its caches, history and output row are left untouched or undefined, nothing is written out of
 * bounds) and the device status word becomes 120, which cca_last_status reports.
 * Needs causal = 1, L_k a multiple of 8, E and L_q multiples of 32 (at head_dim = 256 at most 8 query heads per
 * kv head); otherwise UNSUPPORTED.  No allocation, no synchronisation.
 * Errors: INVALID_ARG, UNSUPPORTED, ALIGNMENT, WORKSPACE_TOO_SMALL, CUDA. */
int cca_decode_step(cca_handle* h, const cca_weights* w, const void* x, void* out, const cca_decode_state* state,
                    int64_t max_len, void* workspace, size_t workspace_bytes, int64_t B, void* cuda_stream);

/* Hand-over from a prefill: fills `state` (caches rows 0..S-1, history, previous input) from x [B,S,E] and
 * the workspace cca_forward left for it, so that the next cca_decode_step continues at pos[b] = S.  Copies
 * only (stream order); state->pos is not read.  Errors: INVALID_ARG (S > S_max, null), ALIGNMENT (x, the caches,
 * x_prev, qk0_hist 16-byte, workspace 256-byte), WORKSPACE_TOO_SMALL, CUDA. */
int cca_decode_state_from_prefill(cca_handle* h, const void* x, const void* workspace, size_t workspace_bytes,
                                  int64_t B, int64_t S, const cca_decode_state* state, void* cuda_stream);

/* ---- MLA baseline --------------------------------------------------------------------------------
 * Multi-Latent Attention as the paper's Section 2.1 defines it (Eq. 3-6), one of the methods its kernel study compares
 * CCA with, run on this library's GEMM and attention kernels: forward only.  C_KV = x W_DKV, C_Q = x W_DQ (Eq. 3);
 * per-head q, k, v up-projected from the latents (Eq. 4); a RoPE part per query head from C_Q and ONE RoPE key part from
 * x shared by every head, concatenated behind the position-free parts (Eq. 6); causal softmax attention per head with
 * scale 1 / sqrt(d_nope + d_rope); output projection.
 * The handle describes the attention: n_q_heads = n_kv_heads = n_h, head_dim = d_nope + d_rope (also the value head
 * size), d_model = E, causal; its stage flags are not used.  All weights bf16 device, [out, in] row-major. */
typedef struct {
  int32_t d_nope, d_rope;   /* per-head sizes of the position-free and the RoPE part (multiples of 8 / 16)        */
  int32_t d_ckv, d_cq;      /* widths of the shared KV latent (E / c_kv) and of the query latent (E / c_q)        */
} cca_mla_dims;
typedef struct {
  const void* w_dq;     /* [d_cq, E]               Eq. 3 */
  const void* w_dkv;    /* [d_ckv, E]              Eq. 3 */
  const void* w_uq;     /* [n_h * d_nope, d_cq]    Eq. 4 */
  const void* w_uqr;    /* [n_h * d_rope, d_cq]    Eq. 6 */
  const void* w_uk;     /* [n_h * d_nope, d_ckv]   Eq. 4 */
  const void* w_uv;     /* [n_h * head_dim, d_ckv] Eq. 4 */
  const void* w_kr;     /* [d_rope, E]             Eq. 6 */
  const void* w_o;      /* [E, n_h * head_dim]           */
} cca_mla_weights;
int cca_mla_workspace_size(const cca_handle* h, const cca_mla_dims* m, int64_t B, int64_t S, size_t* bytes);
/* x, out: device bf16 [B,S,E].  workspace: device, 256-byte aligned, >= cca_mla_workspace_size; on return it holds the
 * latents and q, k, v, o ([B,S,n_h,head_dim] bf16) and lse.  Errors: INVALID_ARG (null, sizes that do not add up to
 * the handle's head_dim, n_q_heads != n_kv_heads), UNSUPPORTED, ALIGNMENT, WORKSPACE_TOO_SMALL, CUDA. */
int cca_mla_forward(cca_handle* h, const cca_mla_dims* m, const cca_mla_weights* w, const void* x, void* out, void* workspace,
                    size_t workspace_bytes, int64_t B, int64_t S, void* cuda_stream);

/* Select kernel implementations: 0 = plain SIMT kernels, 1 = tcgen05/TMA kernels where they
 * exist (default).  Returns the previous value. */
int cca_set_impl(cca_handle* h, int impl);

/* Profiling hook: two cudaEvent_t (or null to clear) that every later attention stage records on the
 * caller's stream immediately before and after its kernel: the forward attention kernel in cca_forward, the decode
 * attention kernel in cca_decode_step, the two attention-adjoint kernels (dQ, dK/dV) together in cca_backward,
 * which therefore overwrites what the forward of the same step recorded. */
int cca_set_attention_events(cca_handle* h, void* ev_begin, void* ev_end);

/* Profiling hook, finer: CCA_N_STAGE_EVENTS cudaEvent_t (or null to clear) that cca_forward and cca_backward record on
 * the caller's stream at their stage boundaries, so that the time between two consecutive events is one stage:
 * forward   BEGIN | down-projection (Eq. 7, 10) | PROJ | latent transforms (Eq. 8, 9, 11) | TRANSFORM | attention
 *           (Eq. 11) | ATTN | up-projection | END;
 * backward  BEGIN | d_o = d_out W_o | DO | d_W_o | DWO | delta | DELTA | attention adjoint | ATTN | norm / RoPE
 *           adjoint | NORM | conv2 adjoint | CONV2 | conv1 and q-k-mean adjoint | CONV1 | value-unshift | PACK |
 *           down-projection weight gradients | DW | d_x | END.
 * Events the configuration's path does not reach (CONV2 without the tensor-core conv2 adjoint) are not recorded.
 * Recording costs a little stream time: time whole steps without it. */
enum {
  CCA_EV_FWD_BEGIN = 0, CCA_EV_FWD_PROJ, CCA_EV_FWD_TRANSFORM, CCA_EV_FWD_ATTN, CCA_EV_FWD_END,
  CCA_EV_BWD_BEGIN, CCA_EV_BWD_DO, CCA_EV_BWD_DWO, CCA_EV_BWD_DELTA, CCA_EV_BWD_ATTN, CCA_EV_BWD_NORM, CCA_EV_BWD_CONV2,
  CCA_EV_BWD_CONV1, CCA_EV_BWD_PACK, CCA_EV_BWD_DW, CCA_EV_BWD_END, CCA_N_STAGE_EVENTS
};
int cca_set_stage_events(cca_handle* h, void* const* events, int n);

/* Number of kernel launches the library has enqueued through this handle so far. */
int64_t cca_launch_count(const cca_handle* h);

/* After the caller has synchronised the stream: copies the device status word.  0 = no error;
 * otherwise the code written by a kernel whose bounded wait expired (101..105 by role, 109 from
 * cca_wait_selftest; or 120: a decode step met a position outside its cache).  Returns
 * CCA_ERR_DEVICE_TIMEOUT if it is non-zero, and clears the word. */
int cca_last_status(cca_handle* h, int* device_status);

/* Limit of every bounded device-side wait of this handle's kernels, in SM clock cycles (about 0.5 ns each).
 * 0 restores the default (4e9, about 2 s).  Values below 2^21 cycles (about 1 ms) are raised to that: the waits
 * of a healthy kernel last microseconds, and a limit they could reach would turn a slow tile into an error.
 * A kernel whose wait runs out records a status code, lets its copies in flight land, frees its tensor memory
 * and returns; nothing traps.  Synchronous (one small copy to the device).  Errors: INVALID_ARG, CUDA. */
int cca_set_wait_limit(cca_handle* h, int64_t sm_cycles);

/* Enqueues one 64-thread kernel whose only wait is on a barrier that nothing ever arrives at, so that the wait
 * runs into the handle's limit: after the caller synchronises, cca_last_status returns CCA_ERR_DEVICE_TIMEOUT
 * with status 109, and the handle stays usable.  A check of the error path, not part of the method. */
int cca_wait_selftest(cca_handle* h, void* cuda_stream);

/* Last CUDA runtime error code seen by this handle, and its string. */
int cca_last_cuda_error(const cca_handle* h);
const char* cca_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* CCA_H_ */
