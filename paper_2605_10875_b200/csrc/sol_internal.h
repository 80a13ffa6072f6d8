// Host-side declarations shared by the .cu files of the library: the launch
// wrapper (launch counting + optional per-kernel event timing) and the
// launchers of each kernel family.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>

#include "../../include/sol.h"

namespace sol {

// ---- launch bookkeeping (sol_api.cu) ---------------------------------------
void note_launch_begin(const char* name, cudaStream_t st);
void note_launch_end(cudaStream_t st);
bool record_cuda_error(cudaError_t e, const char* where);  // true if e != success
bool take_cuda_failure();  // true if a CUDA call of this thread failed since the last check; clears the mark

// Every kernel is launched with programmatic stream serialization: it may start while the kernel
// before it in the stream is still running, does its set-up (and, for the GEMMs, starts streaming
// weights), and calls pdl_wait() before it touches anything an earlier kernel produced.
#define SOL_LAUNCH(name, kernel, grid, block, smem, st, ...)                                   \
  do {                                                                                         \
    ::sol::note_launch_begin(name, st);                                                        \
    cudaLaunchConfig_t sol_cfg_;                                                               \
    memset(&sol_cfg_, 0, sizeof(sol_cfg_));                                                    \
    sol_cfg_.gridDim = grid;                                                                   \
    sol_cfg_.blockDim = block;                                                                 \
    sol_cfg_.dynamicSmemBytes = smem;                                                          \
    sol_cfg_.stream = st;                                                                      \
    cudaLaunchAttribute sol_attr_[1];                                                          \
    sol_attr_[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;                      \
    sol_attr_[0].val.programmaticStreamSerializationAllowed = 1;                               \
    sol_cfg_.attrs = sol_attr_;                                                                \
    sol_cfg_.numAttrs = 1;                                                                     \
    ::sol::record_cuda_error(cudaLaunchKernelEx(&sol_cfg_, kernel, __VA_ARGS__), name);        \
    ::sol::note_launch_end(st);                                                                \
  } while (0)

int sm_count();
// Raises a kernel's dynamic shared memory limit to at least `bytes` on the current device
// (remembered per device and kernel, so repeated calls cost a table lookup).
void ensure_dynamic_smem(const void* kernel, int bytes);
constexpr int MAX_PAGES_PER_SEQ = 768;  // 49152 tokens: the selection kernel keeps one float per token in shared memory

// ---- quantizer / RMSNorm (sol_quant.cu) ------------------------------------
// One token per CTA.  The row is in[B][d] (bf16 or float32) plus, when `part` is given, the ksplit
// partial sums part[z][B][d] of a split-K projection (the output projection: in is the residual).
// gamma == nullptr: no norm.  Outputs (each optional): sum_out float32 [B][d] (the row before the
// norm), a_op bf16 [B][d] (codes as bf16, or x as bf16 for 16 bits), scale [B], xn float32 [B][d],
// codes int8 [B][d].
struct NormQuantArgs {
  const void* in;
  bool in_f32;
  const float* part;
  int ksplit;
  size_t part_stride;  // floats between two partials; 0: B * d
  float* sum_out;
  const void* gamma_bf16;
  float eps;
  const int32_t* bits;
  int B, d;
  void* a_op;
  int a_op_rows;     // 0: a_op is a plain [B][d] matrix; otherwise the packed operand layout with this many rows
  float* scale;
  float* xn;
  int8_t* codes;
  int16_t* codes16;  // optional: int16 codes (widths up to 15 bits where no operand is produced)
  const int32_t* gate_p_permille;  // optional [B]: input-channel gating of the MLP block before the quantizer
  float* xm;         // optional tap of the gated row
  int* status;
  uint32_t* clear;   // optional: [B][clear_words] words zeroed, row by row, for the kernels that follow
  int clear_words;
  int32_t* zero_flags;  // optional: n_zero_flags words zeroed by the grid as a whole (the down projection's live flags,
  int n_zero_flags;     // when this kernel also stands in for the reduction of the previous layer's down projection)
};
void launch_norm_quant(const NormQuantArgs& a, cudaStream_t st);

// The paper's placement of the quantizer: out = resid + fake_quant(sum of the down projection's partials),
// per token at bits[row] (2..15; 16: unchanged).  Also clears the n_live "granule is live" flags.
struct QuantOutArgs {
  const float* partial;  // [chunks][Mpad][d]
  int chunks, M, Mpad, d;
  const void* resid;
  int resid_f32;
  const int32_t* bits;
  void* out_bf16;
  float* out_f32;
  float* out_f32_b;
  float* z_tap;       // optional [M][d]: the MLP output before the quantizer
  int16_t* z_codes;   // optional [M][d]
  float* z_scale;     // optional [M]
  int32_t* live;
  int n_live;
  int* status;
};
void launch_quant_out(const QuantOutArgs& a, cudaStream_t st);

// ---- packed operand layouts ---------------------------------------------------
// Every tensor-core operand is stored the way the MMA reads it from shared memory, so that a stage of the
// GEMM pipelines is one or two large contiguous bulk copies: 64-wide k chunks of rows, each row 128 bytes
// whose 16-byte pieces are permuted by (piece ^ (row & 7)) (the 128-byte swizzle of the K-major operand
// layout).
//   weights [N][K]      -> [tile][chunk][R rows][128 B]; the gate and up matrices share one packed matrix whose
//                          rows alternate gate_c, up_c (so a channel's two sums sit in neighbouring
//                          accumulator lanes)
//   W_down_t [ff][d]    -> [128-column slab][64-channel block][2 column halves][64 channels][128 B] (the
//                          MN-major operand)
//   activations [M][K]  -> [chunk][n_rows][128 B]
struct NKGeom {
  int N, K;     // packed rows in all (gate/up: 2 ff), contraction length
  int R;        // rows per tile (a multiple of 8, at most 128)
  int tiles, chunks;
};
inline NKGeom nk_geom_plain(int N, int K) {
  NKGeom g;
  g.N = N;
  g.K = K;
  g.R = N >= 128 ? 128 : (N + 7) / 8 * 8;
  g.tiles = (N + g.R - 1) / g.R;
  g.chunks = K / 64;
  return g;
}
// channels per tile: the fewest waves of CTAs that keep a tile within 64 channels (128 accumulator lanes)
inline NKGeom nk_geom_gate_up(int ff, int K, int sms) {
  int c = 64;
  for (int w = 1; w <= 64; ++w) {
    c = ((ff + sms * w - 1) / (sms * w) + 3) / 4 * 4;
    if (c <= 64) break;
  }
  NKGeom g;
  g.N = 2 * ff;
  g.K = K;
  g.R = 2 * c;
  g.tiles = (ff + c - 1) / c;
  g.chunks = K / 64;
  return g;
}
inline size_t nk_packed_bytes(const NKGeom& g) { return (size_t)g.tiles * g.chunks * g.R * 128; }
inline size_t down_packed_bytes(int ff, int d) { return (size_t)(d / 128) * ((ff + 63) / 64) * 16384; }
// byte offset of 16-byte piece q (elements 8 q .. 8 q + 7 of a chunk) of packed row n in chunk `chunk`
__host__ __device__ inline size_t nk_piece_offset(int R, int chunks, int n, int chunk, int q) {
  const int r = n % R;
  return (((size_t)(n / R) * chunks + chunk) * R + r) * 128 + (size_t)((q ^ (r & 7)) * 16);
}
// byte offset of the piece that holds elements 8 kp .. 8 kp + 7 of row m of a packed activation operand
__host__ __device__ inline size_t act_piece_offset(int n_rows, int m, int kp) {
  return ((size_t)(kp >> 3) * n_rows + m) * 128 + (size_t)(((kp & 7) ^ (m & 7)) * 16);
}
int pad_rows(int B);  // rows of an activation operand block: the batch padded to 16, 32, 64 or 128

// ---- weight-streaming GEMMs (sol_gemm.cu) ----------------------------------
// EPI_PARTIAL: split-K; out0 is [ksplit][M][N] raw partial sums (no scale, no residual), summed by the
// consumer kernel.  EPI_SWIGLU: whole K per CTA; g, u and t = silu(g) u with the row scale applied.
enum GemmEpilogue { EPI_PARTIAL = 0, EPI_SWIGLU = 2 };
// K slices launch_gemm_nk uses for an [N][K] weight matrix in EPI_PARTIAL mode (<= NK_MAX_KSPLIT).
constexpr int NK_MAX_KSPLIT = 16;
int nk_ksplit(int N, int K);
struct GemmNK {
  const char* name;       // kernel name for the per-kernel timing table
  const void* a;          // packed activation operand, n_b * Mpad rows (high rows, then low rows when n_b == 2)
  int n_b;                // 1, or 2: the product uses the sum of the two row blocks
  const void* w;          // packed weights (EPI_SWIGLU: the gate/up matrix)
  int M, K, N;            // EPI_SWIGLU: N = ff
  const float* row_scale; // EPI_SWIGLU: [M] or nullptr
  float* out0;            // EPI_PARTIAL: [ksplit][M][N]; EPI_SWIGLU: g [M][N]
  float* out1;            // EPI_SWIGLU: u
  float* out2;            // EPI_SWIGLU: t = silu(g) * u
  uint32_t* sel;          // EPI_SWIGLU: [M][CH_SEL_WORDS] histogram of |t| and max |g|, |u| per token (pre-cleared)
  const int32_t* sel_p_permille;  // EPI_SWIGLU, optional: [M] prune rates; tokens that keep all or no channels need no histogram
  int* status;
};
void launch_gemm_nk(const GemmNK& p, GemmEpilogue epi, cudaStream_t st);

struct GemmDown {
  const void* t;     // packed masked activations: 2 Mpad rows (high parts, then low parts), K = ff
  const float* t_f32;         // [M][ff] unmasked t and
  const unsigned char* keep;  // [M][ff] keep mask: the small-batch kernel reads these instead of the packed operand
  const void* w;     // packed W_down_t
  const int32_t* live;  // [ff/32] non-zero if any token keeps a channel of the granule
  int M, ff, d;
  float* partial;    // [chunks][Mpad][d]
  int chunks;        // as returned by down_chunks()
  int* status;
};
int down_chunks(int ff, int d);
void launch_gemm_down(const GemmDown& p, cudaStream_t st);
// out = resid + sum over chunks of partial; out_bf16 / out_f32 optional.
// Also clears the n_live "granule is live" flags, which every reader has finished with by then.
void launch_reduce_out(const float* partial, int chunks, int M, int Mpad, int d, const void* resid, int resid_f32,
                       void* out_bf16, float* out_f32, float* out_f32_b, int32_t* live, int n_live, cudaStream_t st);
// One-time packing of a weight matrix (kinds as in sol.h); src1 is the up matrix of the gate/up pair.
void launch_pack_weights(const sol_shape_t& s, int kind, const void* src0, const void* src1, void* dst, cudaStream_t st);

// ---- attention (sol_attn.cu) ------------------------------------------------
// Kept tokens per pass-2 chunk: 32 KB of V rows.
inline int attn_split_len(int head_dim) { return head_dim == 64 ? 256 : 128; }
inline int attn_splits(int head_dim, int max_pages, int page_size) {
  const int len = attn_split_len(head_dim);
  const int s = (max_pages * page_size + len - 1) / len;
  return s < 1 ? 1 : s;
}
// CTAs per row of the token selection: one per 2048 tokens.
inline int attn_select_segs(int max_pages, int page_size) {
  const int s = (max_pages * page_size + 2047) / 2048;
  return s < 1 ? 1 : s;
}
constexpr int ATTN_ITEM_CHUNKS = 64;  // chunks of attn_split_len kept tokens per pass-2 work item at most
constexpr int PAGE = 64;  // tokens of a cache page
// words of AttnArgs::work_ctr
enum : int { WC_ITEMS = 0, WC_NEXT = 1, WC_CPI = 2, WC_DONE = 4 };

struct AttnArgs {
  sol_shape_t shape;
  sol_kv_t kv;
  int B;
  int span_tokens;  // 0, or: the rows are B / span_tokens spans of consecutive tokens (KV refresh): dense causal attention
  const int32_t* r_permille;
  // inputs of the query preparation: either the split-K partial sums of the QKV projection (layer
  // path: rotate q and k, append k and v) or bf16 q [B][Hq][hd] (stand-alone path: no rotation, no append)
  const float* qkv_f32;   // [qkv_ksplit][B][ldq]
  int ldq;
  int qkv_ksplit;
  const float* qkv_scale; // [B] quantizer scale applied to the summed rows
  const void* q_bf16;
  // scratch (attn_scratch_layout)
  float* q_rot;         // [B][Hq][hd]
  void* q_split;        // bf16 [B][Hkv][HG*16][hd]
  float* logits;        // [B][Hkv][Tmax][G]
  float* sigma;         // [B][Hkv][Tmax]
  uint32_t* row_hist;   // [B][Hkv][4096] histogram of a row's scores (rows that span several selection CTAs)
  uint32_t* row_ctl;    // [B][Hkv][8] selection state of a row
  uint32_t* seg_pub;    // [B][Hkv][segments] kept count of each 2048-token segment of the row (| ready bit)
  int32_t* cand_idx;    // [B][Hkv][1024] tokens between the selection's edges
  float* cand_val;      // [B][Hkv][1024] their scores
  int32_t* list_idx;    // [B][Hkv][Tmax] token index of every kept token, in the order pass 2 reads them
  int32_t* kept_idx_out; // optional: the caller's [B][Hkv][Tmax] array for the ascending index list
  int32_t* kept_cnt;    // [B][Hkv]
  uint32_t* kept_row;   // same layout as kept_idx: cache row (page table applied) of every kept token,
                        // 0xffffffff: bad page
  float* part;          // [B][Hkv][S][G][hd + 2]
  int splits;           // S = ceil(Tmax / attn_split_len(hd))
  int32_t* plan;        // [3][132] cumulative page / segment counts over the batch: the flat work lists of pass 1 and
                        // of the selection, written by the query preparation
  int32_t* work_items;  // [B*Hkv*S][2] pass-2 work list (item code, kept count), filled by the selection
  int32_t* work_ctr;    // [4 + B*Hkv]: items emitted, next item to claim, chunks per item, unused; then the finished
                        // items of every (sequence, kv-head)
  // outputs (each optional)
  float* out_f32;    // [B][Hq][hd]
  void* out_bf16;    // [B][Hq][hd]
  void* out_hi;      // packed operand of the output projection: 2 out_rows rows (bf16 high parts, then low parts)
  void* out_lo;      // unused
  int out_rows;
  // SOL_SELECT_QUEST_PAGES (launch_quest_selection)
  unsigned char* page_mask;   // scratch [B][Hkv][Tmax / 4]: per Quest page, bit h = query head h of the group keeps it
  uint32_t* quest_keys;       // scratch [B][Hq][Tmax / S]: float32 bound of every page as a sortable key
  uint32_t* quest_err;        // scratch [B][Hq]: largest rounding-error bound of the row's scores (float bits)
  unsigned char* quest_hmask; // scratch [B][Hq][Tmax / S]: 1 = the query head keeps the page
  uint16_t* quest_qsplit;     // scratch [B][Hkv][ceil(G / 4) * 16][2 hd] bf16: sign-split queries as a tensor-core operand
  float* quest_l1;            // scratch [B][Hq]: |q|_1
  int* quest_order;           // scratch [B]: the sequences, longest first
  int32_t* quest_pages_out;   // optional: the caller's [B][Hq][Tmax / S] kept pages of every query head, ascending
  int32_t* quest_cnt_out;     // optional: [B][Hq]
  int* status;
};
// Quest page extrema of the cache (all pages of the B sequences, or only the block of each sequence's newest token).
void launch_quest_meta(const sol_shape_t& sh, const sol_kv_t& kv, int B, bool all, int* status, cudaStream_t st);
// ... the cache pages that hold the last n_tail tokens of each sequence.
void launch_quest_meta_tail(const sol_shape_t& sh, const sol_kv_t& kv, int B, int n_tail, int* status, cudaStream_t st);
// Page scores and selection per query head, union token list + pass-2 work items per (sequence, kv-head), then the
// logits of the listed tokens (minus infinity for the heads that did not pick the token's page).
void launch_quest_selection(const AttnArgs& a, bool update_meta, cudaStream_t st);
// Attention over the Quest selection's token lists in one pass (sol_quest_attend.cu), after launch_quest_selection.
void launch_quest_attend(const AttnArgs& a, cudaStream_t st);
// Dense causal attention of spans of n_tok consecutive tokens per sequence, after the query preparation (sol_span.cu).
void launch_span_attention(const AttnArgs& a, int n_tok, cudaStream_t st);

// Offsets of the attention scratch inside a buffer, starting at `at` (a multiple of 256).
struct AttnScratch {
  size_t q_rot, q_split, logits, sigma, row_hist, row_ctl, seg_pub, cand_idx, cand_val, kept_idx, kept_cnt, kept_row, part, plan, work_items, work_ctr, page_mask, quest_keys, quest_err, quest_hmask, quest_qsplit, quest_l1, quest_order, end;
  int splits;
};
inline AttnScratch attn_scratch_layout(const sol_shape_t& s, int B, int max_pages, size_t at) {
  AttnScratch L;
  const size_t Hq = s.n_q_heads, Hkv = s.n_kv_heads, hd = s.head_dim, G = Hq / Hkv, HG = (G + 3) / 4;
  const size_t Tmax = (size_t)max_pages * s.page_size, BK = (size_t)B * Hkv;
  L.splits = attn_splits(s.head_dim, max_pages, s.page_size);
  auto take = [&](size_t bytes) {
    const size_t o = at;
    at += (bytes + 255) / 256 * 256;
    return o;
  };
  L.q_rot = take(B * Hq * hd * 4);
  L.q_split = take(BK * HG * 16 * hd * 2);
  L.logits = take(BK * Tmax * G * 4);
  L.sigma = take(BK * Tmax * 4);
  L.row_hist = take(BK * 4096 * 4);
  L.row_ctl = take(BK * 8 * 4);
  L.seg_pub = take(BK * (size_t)attn_select_segs(max_pages, s.page_size) * 4);
  L.cand_idx = take(BK * 1024 * 4);
  L.cand_val = take(BK * 1024 * 4);
  L.kept_idx = take(BK * Tmax * 4);
  L.kept_cnt = take(BK * 4);
  L.kept_row = take(BK * Tmax * 4);
  L.part = take(BK * L.splits * G * (hd + 2) * 4);
  L.plan = take(3 * 132 * 4);
  L.work_items = take(BK * L.splits * 8);
  L.work_ctr = take((4 + BK) * 4);
  const bool quest = s.token_select == SOL_SELECT_QUEST_PAGES;
  L.page_mask = take(quest ? BK * (Tmax / 4) : 0);
  L.quest_keys = take(quest ? (size_t)B * Hq * (Tmax / s.quest_page_size) * 4 : 0);
  L.quest_err = take(quest ? (size_t)B * Hq * 4 : 0);
  L.quest_hmask = take(quest ? (size_t)B * Hq * (Tmax / s.quest_page_size) : 0);
  L.quest_qsplit = take(quest ? (size_t)B * Hkv * ((Hq / Hkv + 3) / 4) * 16 * 2 * hd * 2 : 0);
  L.quest_l1 = take(quest ? (size_t)B * Hq * 4 : 0);
  L.quest_order = take(quest ? (size_t)B * 4 : 0);
  L.end = at;
  return L;
}
// kept_idx / kept_cnt: the caller's arrays, or nullptr to use the scratch.
inline void attn_scratch_bind(AttnArgs& a, void* base, const AttnScratch& L, int32_t* kept_idx, int32_t* kept_cnt) {
  unsigned char* b = static_cast<unsigned char*>(base);
  a.q_rot = reinterpret_cast<float*>(b + L.q_rot);
  a.q_split = b + L.q_split;
  a.logits = reinterpret_cast<float*>(b + L.logits);
  a.sigma = reinterpret_cast<float*>(b + L.sigma);
  a.row_hist = reinterpret_cast<uint32_t*>(b + L.row_hist);
  a.row_ctl = reinterpret_cast<uint32_t*>(b + L.row_ctl);
  a.seg_pub = reinterpret_cast<uint32_t*>(b + L.seg_pub);
  a.cand_idx = reinterpret_cast<int32_t*>(b + L.cand_idx);
  a.cand_val = reinterpret_cast<float*>(b + L.cand_val);
  a.list_idx = reinterpret_cast<int32_t*>(b + L.kept_idx);
  a.kept_idx_out = kept_idx;
  a.kept_cnt = kept_cnt ? kept_cnt : reinterpret_cast<int32_t*>(b + L.kept_cnt);
  a.kept_row = reinterpret_cast<uint32_t*>(b + L.kept_row);
  a.part = reinterpret_cast<float*>(b + L.part);
  a.plan = reinterpret_cast<int32_t*>(b + L.plan);
  a.work_items = reinterpret_cast<int32_t*>(b + L.work_items);
  a.work_ctr = reinterpret_cast<int32_t*>(b + L.work_ctr);
  a.page_mask = b + L.page_mask;
  a.quest_keys = reinterpret_cast<uint32_t*>(b + L.quest_keys);
  a.quest_err = reinterpret_cast<uint32_t*>(b + L.quest_err);
  a.quest_hmask = b + L.quest_hmask;
  a.quest_qsplit = reinterpret_cast<uint16_t*>(b + L.quest_qsplit);
  a.quest_l1 = reinterpret_cast<float*>(b + L.quest_l1);
  a.quest_order = reinterpret_cast<int*>(b + L.quest_order);
  a.quest_pages_out = nullptr;
  a.quest_cnt_out = nullptr;
  a.splits = L.splits;
}
void launch_attention(const AttnArgs& a, cudaStream_t st);

// ---- MLP channel selection (sol_mlp.cu) -------------------------------------
struct ChannelSelectArgs {
  int B, d, ff;
  const int32_t* p_permille;
  const float* g;      // [B][ff]
  const float* u;
  const float* t;
  const void* a_op;    // packed MLP input operand (pad_rows(B) rows)
  const float* scale;  // [B]
  const void* w_gate_up;  // packed gate/up weights
  uint32_t* sel;       // [B][CH_SEL_WORDS] filled by the gate/up epilogue
  double* cand_val;    // [B][CH_CAND_CAP]
  int32_t* cand_idx;   // [B][CH_CAND_CAP]
  unsigned char* keep; // [B][ff] 1 = kept
  int32_t* scratch_idx; // [B][ff] scratch of the single-CTA path
  int32_t* kept_ch;    // optional [B][ff]: ascending list, written only when requested
  int32_t* kept_cnt;   // [B]
  void* t_op;          // packed operand of the down projection: 2 pad_rows(B) rows (bf16 high parts, then low parts)
  int32_t* live;       // [ff/32], all zero on entry (cleared by reduce_out after the down projection)
  int* status;
};
void launch_channel_select(const ChannelSelectArgs& a, cudaStream_t st);

}  // namespace sol
