/*
 * sol.h - C ABI of the action-conditioned batched decode step for B200 (sm_100a).
 *
 * One new token per sequence is pushed through a frozen Llama-shaped decoder
 * layer.  Every sequence i carries its own efficiency action, the paper's
 * tuple (kappa, rho, q) (Method, "Actions and controlled compute"), passed as
 * three int32 arrays of length B:
 *
 *   r_permille[i]  attention keep-rate r = kappa, in 1/1000, 0..1000
 *   p_permille[i]  MLP prune rate     p = 1 - rho, in 1/1000, 0..1000
 *   bits[i]        activation bit-width b = q, 2..8 or 16 (16 = bf16 passthrough)
 *
 * Conventions for every call:
 *   - returns a sol_status_t; never throws, never traps the device;
 *   - unless a parameter says "host", every pointer is DEVICE memory owned by
 *     the caller, 16-byte aligned, valid until the work enqueued on `stream`
 *     has finished; the library allocates no device memory on these calls
 *     (scratch comes from the caller's workspace `ws`);
 *   - work is enqueued on `stream` (a cudaStream_t); the call does not wait
 *     for it;
 *   - bf16 tensors are raw 16-bit patterns; matrices are row-major;
 *   - argument errors are detected on the host before anything is launched.
 */
#ifndef SOL_H_
#define SOL_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t sol_status_t;
#define SOL_OK 0
#define SOL_ERR_INVALID_ARG 1         /* null pointer, negative size, rate or bit-width out of range */
#define SOL_ERR_UNSUPPORTED 2         /* a shape this build has no kernel for (see sol_shape_t) */
#define SOL_ERR_WORKSPACE_TOO_SMALL 3 /* ws_bytes < sol_workspace_bytes(...) */
#define SOL_ERR_CUDA 4                /* a CUDA runtime call failed; see sol_last_cuda_error() */
#define SOL_ERR_DEVICE_TIMEOUT 5      /* a bounded device-side wait gave up (reported by sol_read_device_status) */

typedef struct CUstream_st *sol_stream_t; /* a cudaStream_t */

/* Layer geometry.  Supported: head_dim 64 or 128; page_size 64;
 * n_q_heads a multiple of n_kv_heads (at most 8 query heads per kv head);
 * d_model (<= 8192) and n_q_heads*head_dim multiples of 256; d_ff a multiple
 * of 32, at most 49152; batch 1..128; at most 768 pages (49152 tokens) per
 * sequence.  Anything else: SOL_ERR_UNSUPPORTED (sol_workspace_bytes: 0). */
typedef struct sol_shape {
  int32_t d_model, n_q_heads, n_kv_heads, head_dim, d_ff, page_size;
  float rms_eps;
  float rope_theta;         /* 0 disables the rotary embedding */
  int32_t n_sink, n_window; /* always-attended first / last tokens (the paper's sink and window
                               tokens, Method, "Policy inputs and architecture"); the task's
                               default is 0 and 1: only the newest token is forced */
  int32_t quant_placement;  /* where bits[i] acts in a layer: SOL_QUANT_PROJ_INPUTS (0, the task's default) on the
                               inputs of the QKV and gate/up projections, widths 2..8 and 16; SOL_QUANT_MLP_OUTPUT
                               (1, the paper's: appendix "Activation quantization", "What is quantized") on the MLP
                               output before the residual add, widths 2..15, 16 and more: unchanged; the
                               projections then read bf16 rows */
  int32_t mlp_prune;        /* what p_permille[i] prunes in a layer: SOL_PRUNE_INTERMEDIATE (0, the task's default) the
                               intermediate channels with the smallest |silu(g) u|; SOL_PRUNE_MLP_INPUT (1, the
                               paper's: appendix "Structured MLP activation pruning") the input channels of the MLP
                               block with the smallest |x|: ceil((1 - p) d_model) survive (ties: lower index), the
                               rest of the normalised row is zeroed before the quantizer; the attention input is
                               not pruned and every intermediate channel is kept */
  int32_t token_select;     /* how r_permille[i] picks the keys a step attends to: SOL_SELECT_TOKENS (0, the task's
                               default) the ceil(r T) tokens with the largest q.k summed over the query group, per
                               (sequence, kv head); SOL_SELECT_QUEST_PAGES (1, the paper's: appendix "Token sparsity
                               via Quest") pages of quest_page_size contiguous tokens, scored per QUERY head by the
                               bound q_pos.m+ + q_neg.m- from the per-dimension extrema of each page's keys; every
                               head keeps its ceil(ceil(r T) / quest_page_size) best pages (ties: lower page; the
                               pages that hold a forced token are always among them) and attends to all keys of
                               its pages and to nothing else.  Needs sol_kv_t.quest_meta */
  int32_t quest_page_size;  /* 4, 8, 16, 32 or 64, and at least n_q_heads / n_kv_heads, when token_select is
                               SOL_SELECT_QUEST_PAGES (ignored otherwise) */
} sol_shape_t;
#define SOL_QUANT_PROJ_INPUTS 0
#define SOL_QUANT_MLP_OUTPUT 1
#define SOL_PRUNE_INTERMEDIATE 0
#define SOL_PRUNE_MLP_INPUT 1
#define SOL_SELECT_TOKENS 0
#define SOL_SELECT_QUEST_PAGES 1

/* Paged bf16 KV cache of one layer.  Pools: [num_pages][n_kv_heads][page_size][head_dim].
 * page_table: int32 [B][max_pages_per_seq], physical page of each logical page.
 * seq_lens:   int32 [B], valid tokens of each sequence INCLUDING the newest one. */
typedef struct sol_kv {
  void *k_pool, *v_pool;
  const int32_t *page_table;
  const int32_t *seq_lens;
  int32_t max_pages_per_seq, num_pages;
  void *quest_meta; /* SOL_SELECT_QUEST_PAGES only (else unused, may be NULL): device, bf16
                       [num_pages][n_kv_heads][page_size / quest_page_size][2][head_dim]: for every block of
                       quest_page_size tokens of a cache page the per-dimension maximum of its keys, then the negated
                       minimum, over the tokens the sequence has (sol_quest_meta_bytes, sol_quest_build_meta).
                       sol_decode_layer / sol_decode_step update the block of the token they append */
} sol_kv_t;

/* Weight matrices are PACKED once at load time (sol_pack_weights) into the order the tensor cores read
 * them, so that the kernels stream each matrix with large contiguous copies.  Kinds and their row-major
 * bf16 sources:
 *   SOL_W_QKV      [(n_q+2 n_kv)*head_dim][d_model]   rows: q heads, then k heads, then v heads
 *   SOL_W_O        [d_model][n_q*head_dim]
 *   SOL_W_GATE_UP  two matrices [d_ff][d_model] (gate, up), packed into one
 *   SOL_W_DOWN     W_down transposed, [d_ff][d_model]: row j is intermediate channel j, so a pruned
 *                  channel is a row that is not read
 * The packed size depends on the shape and, for SOL_W_GATE_UP, on the SM count of the current device:
 * pack on the device that runs the layer. */
#define SOL_W_QKV 0
#define SOL_W_O 1
#define SOL_W_GATE_UP 2
#define SOL_W_DOWN 3
/* Bytes of the packed form of a matrix; 0 if the shape or kind is unsupported. */
size_t sol_packed_weight_bytes(const sol_shape_t *shape, int32_t kind);
/* Packs src0 (and src1: the up matrix when kind is SOL_W_GATE_UP, else NULL) into dst (dst_bytes >=
 * sol_packed_weight_bytes), all device pointers, 16-byte aligned; enqueued on `stream`.  A pure
 * permutation of 16-byte pieces (tiles that reach past the matrix are padded with zeros). */
sol_status_t sol_pack_weights(const sol_shape_t *shape, int32_t kind, const void *src0, const void *src1, void *dst,
                              size_t dst_bytes, sol_stream_t stream);

/* Packed bf16 weights of one layer (see sol_pack_weights) and the RMSNorm gains. */
typedef struct sol_layer_weights {
  const void *w_qkv;     /* packed SOL_W_QKV */
  const void *w_o;       /* packed SOL_W_O */
  const void *w_gate_up; /* packed SOL_W_GATE_UP */
  const void *w_down;    /* packed SOL_W_DOWN */
  const void *gamma1;    /* [d_model] RMSNorm gain before attention */
  const void *gamma2;    /* [d_model] RMSNorm gain before the MLP */
} sol_layer_weights_t;

/* Optional taps on sol_decode_layer; any pointer may be NULL.  They exist so a
 * checker can compare each stage on the inputs that stage really saw. */
typedef struct sol_layer_trace {
  float *xn1;           /* [B][d_model] normalised attention input (float32) */
  int8_t *codes1;       /* [B][d_model] */
  float *scales1;       /* [B] */
  float *q_rot;         /* [B][n_q][head_dim] rotated queries (float32) */
  int32_t *kept_idx;    /* [B][n_kv][max_pages_per_seq*page_size] ascending */
  int32_t *kept_cnt;    /* [B][n_kv] */
  float *attn_out;      /* [B][n_q][head_dim] */
  float *h_mid;         /* [B][d_model] residual stream after attention (float32) */
  float *xn2;           /* [B][d_model] */
  int8_t *codes2;       /* [B][d_model] */
  float *scales2;       /* [B] */
  float *t;             /* [B][d_ff] silu(g)*u before pruning (float32) */
  int32_t *kept_ch;     /* [B][d_ff] ascending */
  int32_t *kept_ch_cnt; /* [B] */
  float *h_out;         /* [B][d_model] float32 copy of the output */
  float *z;             /* SOL_QUANT_MLP_OUTPUT only: [B][d_model] MLP output before the quantizer (float32) */
  int16_t *z_codes;     /* SOL_QUANT_MLP_OUTPUT only: [B][d_model] its codes (0 for 16 bits) */
  float *z_scales;      /* SOL_QUANT_MLP_OUTPUT only: [B] */
  float *xm2;           /* SOL_PRUNE_MLP_INPUT only: [B][d_model] the MLP input after the channel gating (float32) */
} sol_layer_trace_t;

const char *sol_status_string(sol_status_t s);
const char *sol_last_cuda_error(void); /* text of the last CUDA error seen by this thread's calls */

/* Bytes of scratch that any call below needs for batches up to max_batch and
 * contexts up to max_pages_per_seq pages.  0 if the shape is unsupported.
 * The offsets inside the workspace depend on the batch of each call.  Results
 * do not depend on what earlier calls left behind (every counter a call needs
 * is cleared by the call itself), but stale "row is live" flags of a call with
 * another batch size can cost extra weight reads: pass the workspace through
 * sol_workspace_init again when the batch size changes. */
size_t sol_workspace_bytes(const sol_shape_t *shape, int32_t max_batch, int32_t max_pages_per_seq);

/* Must be called once per workspace before its first use (and may be called
 * again to clear the device status words).  Enqueues a memset on `stream`. */
sol_status_t sol_workspace_init(void *ws, size_t ws_bytes, sol_stream_t stream);

/* Per-token symmetric activation quantizer (appendix "Activation
 * quantization", "Quantizer"): a = max_j |x_j|, s = a / q_max with
 * q_max = 2^(b-1) - 1, code_j = clip(rne(x_j / s), -q_max, q_max); both
 * divisions IEEE float32, rounding to nearest-even.  Row i uses bits[i].
 *   x_bf16 [B][d] in; codes int8 [B][d] and scales float32 [B] out.
 *   bits[i] == 16: codes of that row are 0, scale is 1 (passthrough).
 *   An all-zero row gives scale 0 and codes 0.
 *   xhat_bf16 (optional, [B][d]): the value the next matmul consumes, before
 *   the scale is applied: the codes as bf16 numbers, or x itself for 16 bits.
 * d must be a multiple of 8.  Needs no workspace. */
sol_status_t sol_quant_act(const void *x_bf16, int32_t B, int32_t d, const int32_t *bits, int8_t *codes,
                           float *scales, void *xhat_bf16, sol_stream_t stream);

/* The same quantizer with int16 codes, for widths 2..15 (the paper's action tables use up to 15 bits);
 * bits[i] >= 16: codes 0, scale 1.  No operand output. */
sol_status_t sol_quant_act_wide(const void *x_bf16, int32_t B, int32_t d, const int32_t *bits, int16_t *codes,
                                float *scales, sol_stream_t stream);

/* Page extrema for SOL_SELECT_QUEST_PAGES (the paper's appendix "Token sparsity via Quest": m+ = max_j k_j,
 * m- = -min_j k_j over the keys of a page).  sol_quest_meta_bytes: size of sol_kv_t.quest_meta for a pool of
 * num_pages pages (0: unsupported shape).  sol_quest_build_meta: fills quest_meta for every token the B
 * sequences of `kv` hold (seq_lens counts them), e.g. after a prefill; blocks past a sequence's last token
 * are left alone, the block that holds it takes its extrema over the tokens that exist.  Pointers: device;
 * errors as for the other calls. */
size_t sol_quest_meta_bytes(const sol_shape_t *shape, int32_t num_pages);
sol_status_t sol_quest_build_meta(const sol_shape_t *shape, const sol_kv_t *kv, int32_t B, sol_stream_t stream);

/* Decode attention with a per-sequence keep-rate (appendix "Token sparsity",
 * "Budgeted token selection": budget ceil(kappa*K_t) clamped to [0, K_t];
 * selection by exact token-level top-k instead of the paper's page bounds).
 * For each (sequence, kv-head): keep k = max(ceil(r*T), forced) tokens, the
 * forced ones plus those with the largest q.k summed over the query group
 * (ties: lower index); softmax over the kept tokens only; only kept V rows
 * are read.
 *   q_bf16 [B][n_q][head_dim] (already rotated); out_bf16 same shape.
 *   kept_idx (optional) int32 [B][n_kv][max_pages_per_seq*page_size], the
 *   kept token indices of each (sequence, kv-head) in ascending order;
 *   kept_cnt (optional) int32 [B][n_kv].
 * With shape->token_select == SOL_SELECT_QUEST_PAGES the selection is the paper's (see sol_shape_t): per QUERY
 * head; K and V rows are read only for pages that some head of the kv-head's group keeps; kv->quest_meta must
 * be current.  kept_idx then holds int32 [B][n_q][max_pages_per_seq*page_size/quest_page_size]: the kept PAGE
 * indices of each query head in ascending order (no larger than the token form, since quest_page_size is at
 * least the number of query heads per kv head); kept_cnt is int32 [B][n_q].
 * The cache is only read. */
sol_status_t sol_sparse_decode_attn(const sol_shape_t *shape, const void *q_bf16, const sol_kv_t *kv, int32_t B,
                                    const int32_t *r_permille, void *out_bf16, int32_t *kept_idx,
                                    int32_t *kept_cnt, void *ws, size_t ws_bytes, sol_stream_t stream);

/* The same attention for callers that cannot provide a workspace (the paper has
 * no counterpart: this entry exists for hosts that may not allocate).  A serving
 * process that handed all of its device memory to a pool at start-up, a plugin
 * inside a runtime that owns the allocator, or a loop that must never reach
 * cudaMalloc / cudaFree can call this instead of sol_sparse_decode_attn: the
 * scratch is a fixed array of SOL_STATIC_SCRATCH_BYTES inside the library
 * image, present on every GPU that loads the library until the process exits.
 * The call allocates nothing.
 *   Inputs and outputs as sol_sparse_decode_attn (SOL_SELECT_TOKENS only); kept_idx / kept_cnt optional.
 *   status_out (optional, DEVICE int32[8]) receives the status words of this
 *   call (layout as sol_read_device_status) by a copy enqueued on `stream`.
 *   Limit: B * n_kv * (max_pages_per_seq * 64 * (4 G + 12) + 24 KiB) bytes plus small
 *   terms must fit the array (for 4 query / 2 kv heads of 64: batch 4 with contexts
 *   up to about 25 thousand tokens); a larger problem is refused with
 *   SOL_ERR_WORKSPACE_TOO_SMALL before anything is launched.
 *   The first call on each device looks up the array's device address (with
 *   that device current); make that first call outside any stream capture.
 *   All calls on a device share the one array and it keeps the previous call's
 *   contents (the status words are cleared at the start of each call): two
 *   calls whose GPU work can overlap (different streams or threads) race. */
#define SOL_STATIC_SCRATCH_BYTES (4u << 20)
sol_status_t sol_sparse_decode_attn_static(const sol_shape_t *shape, const void *q_bf16, const sol_kv_t *kv,
                                           int32_t B, const int32_t *r_permille, void *out_bf16, int32_t *kept_idx,
                                           int32_t *kept_cnt, int32_t *status_out, sol_stream_t stream);

/* SwiGLU MLP with a per-token prune rate (count mirrors the paper's
 * m = ceil(rho*d), "Per-token channel selection"; the pruned axis is the
 * intermediate one): t_j = silu(W_g x)_j (W_u x)_j, keep the
 * m = ceil((1-p) d_ff) channels with the largest |t_j| (ties: lower index),
 * out = sum over kept j of t_j * W_down[j, :].  Blocks of W_down rows that no
 * token of the batch keeps are not read.
 *   x_bf16 [B][d_model]; w_gate_up, w_down: packed SOL_W_GATE_UP / SOL_W_DOWN;
 *   out_bf16 [B][d_model] (no residual added);
 *   kept_ch (optional) int32 [B][d_ff] ascending; kept_ch_cnt (optional) [B]. */
sol_status_t sol_pruned_swiglu_mlp(const sol_shape_t *shape, const void *x_bf16, const void *w_gate_up,
                                   const void *w_down, int32_t B, const int32_t *p_permille,
                                   void *out_bf16, int32_t *kept_ch, int32_t *kept_ch_cnt, void *ws,
                                   size_t ws_bytes, sol_stream_t stream);

/* One decoder layer under per-sequence actions: RMSNorm, quantize(b), QKV,
 * rotary embedding at position T-1, append k/v (bf16) to the cache at
 * position T-1, sparse attention(r), output projection + residual, RMSNorm,
 * quantize(b), pruned SwiGLU MLP(p) + residual.  The caller has already
 * reserved the page slot of the newest token and seq_lens counts it.
 *   h_in_bf16 [B][d_model] in; h_out_bf16 [B][d_model] out; trace optional. */
sol_status_t sol_decode_layer(const sol_shape_t *shape, const sol_layer_weights_t *w, const sol_kv_t *kv, int32_t B,
                              const void *h_in_bf16, void *h_out_bf16, const int32_t *r_permille,
                              const int32_t *p_permille, const int32_t *bits, const sol_layer_trace_t *trace,
                              void *ws, size_t ws_bytes, sol_stream_t stream);

/* n_layers layers with the same action in every layer (the paper broadcasts
 * one action tuple over all layers of a decode step).  `layers` and `kvs` are
 * HOST arrays of n_layers structs (holding device pointers).  The residual
 * stream stays in float32 between layers.  h_out_f32 is optional. */
sol_status_t sol_decode_step(const sol_shape_t *shape, int32_t n_layers, const sol_layer_weights_t *layers,
                             const sol_kv_t *kvs, int32_t B, const void *h_in_bf16, void *h_out_bf16,
                             float *h_out_f32, const int32_t *r_permille, const int32_t *p_permille,
                             const int32_t *bits, void *ws, size_t ws_bytes, sol_stream_t stream);

/* sol_decode_step with the taps of sol_decode_layer on every layer: `traces` is a HOST array of
 * n_layers structs (or NULL); layer l fills traces[l].  traces[l].h_out is the float32 residual
 * stream that layer l+1 reads, so a checker can compare every layer on the input it really saw. */
sol_status_t sol_decode_step_traced(const sol_shape_t *shape, int32_t n_layers, const sol_layer_weights_t *layers,
                                    const sol_kv_t *kvs, int32_t B, const void *h_in_bf16, void *h_out_bf16,
                                    float *h_out_f32, const int32_t *r_permille, const int32_t *p_permille,
                                    const int32_t *bits, const sol_layer_trace_t *traces, void *ws, size_t ws_bytes,
                                    sol_stream_t stream);

/* Periodic KV-cache refresh (Background, paragraph "Episodes and control horizon"): a fully dense pass
 * (keep-rate 1, prune rate 0, 16 bits) over the last n_tokens already-known tokens of every
 * sequence that rebuilds their keys and values in all layers; no token is sampled.  Token i of
 * the span attends to the whole context before it and to tokens 0..i of the span (causal).
 *   kvs[l].seq_lens  device [B]: lengths INCLUDING the span; each must be >= n_tokens (a shorter
 *                    sequence raises the bad-action bit of the device status word and leaves
 *                    that sequence's cache undefined)
 *   h_in_bf16        device [B][n_tokens][d_model]: the layer-0 inputs of the span, oldest first
 *   h_out_bf16       optional device [B][n_tokens][d_model]: the last layer's outputs
 * 1 <= n_tokens <= 128.  The rows of floor(128 / n_tokens) sequences go through the layers
 * together; the workspace must hold sol_workspace_bytes(shape, min(B, 128 / n_tokens) * n_tokens,
 * max_pages_per_seq).  In the Quest mode the page extrema of the rewritten blocks are rebuilt.
 * `layers`, `kvs`: HOST arrays of n_layers structs as in sol_decode_step. */
sol_status_t sol_kv_refresh(const sol_shape_t *shape, int32_t n_layers, const sol_layer_weights_t *layers,
                            const sol_kv_t *kvs, int32_t B, int32_t n_tokens, const void *h_in_bf16,
                            void *h_out_bf16, void *ws, size_t ws_bytes, sol_stream_t stream);

/* The same step for a caller whose per-step data lives on the HOST: h_in,
 * the three action arrays, seq_lens and h_out are host pointers (pinned
 * memory makes the copies of h_in and h_out asynchronous; the four int32
 * arrays are read during the call and travel as kernel parameters).  They
 * land in staging areas inside the workspace, the step runs with
 * kvs[l].seq_lens replaced by the staged copy, and the result is copied back;
 * the call returns after the stream has been synchronised.  Weights, pools and
 * page tables stay on the device.  Because the call synchronises, it also reads the workspace's
 * error word and returns SOL_ERR_DEVICE_TIMEOUT if a bounded device-side wait gave up. */
sol_status_t sol_decode_step_host(const sol_shape_t *shape, int32_t n_layers, const sol_layer_weights_t *layers,
                                  const sol_kv_t *kvs, int32_t B, const void *h_in_bf16_host,
                                  void *h_out_bf16_host, const int32_t *r_permille_host,
                                  const int32_t *p_permille_host, const int32_t *bits_host,
                                  const int32_t *seq_lens_host, void *ws, size_t ws_bytes, sol_stream_t stream);

/* Device status words of a workspace, copied to HOST out[8] after waiting for
 * `stream`:  out[0] bit mask of errors raised by kernels (bit 0: a bounded
 * wait timed out -> SOL_ERR_DEVICE_TIMEOUT is returned; bit 1: a page-table
 * entry was out of range and the access was skipped; bit 2: a bit-width outside
 * 2..8 and 16 was met and treated as 16), out[1] token
 * selections whose near-threshold candidate list overflowed and fell back to
 * float32 ordering, out[2] the same for channel selections, out[3] token
 * candidates re-scored in float64, out[4] channel candidates re-scored. */
sol_status_t sol_read_device_status(const void *ws, int32_t *out_host8, sol_stream_t stream);

/* Self-check of the time-out reporting (no counterpart in the paper): launches one CTA that waits, with a
 * limit of a few thousand polls, on a barrier nothing arrives at; the wait gives up, raises bit 0 of
 * the status words of `ws` (>= 256 bytes, initialised) and the kernel returns.  A following
 * sol_read_device_status must then return SOL_ERR_DEVICE_TIMEOUT; sol_workspace_init clears the bit. */
sol_status_t sol_selftest_wait_timeout(void *ws, sol_stream_t stream);

/* Per-kernel timing for benchmarks.  While enabled, every kernel launch of
 * this library is bracketed by CUDA events on its stream.  sol_timing_collect
 * synchronises the device and fills HOST arrays, one entry per kernel name:
 * returns the number of entries (at most max_entries).  Not thread-safe. */
typedef struct sol_kernel_time {
  char name[48];
  int32_t launches;
  float total_ms;
} sol_kernel_time_t;
void sol_timing_enable(int32_t on);
int32_t sol_timing_collect(sol_kernel_time_t *out_host, int32_t max_entries);

/* Kernels launched by this library since the last reset (reset != 0 clears). */
int64_t sol_launch_count(int32_t reset);

#ifdef __cplusplus
}
#endif
#endif /* SOL_H_ */
