// C ABI of the library: argument validation, workspace layout, and the
// composition of the kernels into attention, MLP, layer and step calls.
#include <atomic>
#include <cstdio>
#include <cstring>
#include <map>
#include <mutex>
#include <string>
#include <vector>

#include "sol_common.cuh"
#include "sol_internal.h"

namespace sol {

// ---------------------------------------------------------------------------
// launch bookkeeping
// ---------------------------------------------------------------------------
static std::atomic<long long> g_launches{0};
static bool g_timing = false;
struct TimedLaunch {
  const char* name;
  cudaEvent_t e0, e1;
};
static std::vector<TimedLaunch> g_timed;
static thread_local char tl_cuda_error[256] = "";
static thread_local bool tl_cuda_failed = false;

bool record_cuda_error(cudaError_t e, const char* where) {
  if (e == cudaSuccess) return false;
  snprintf(tl_cuda_error, sizeof(tl_cuda_error), "%s: %s", where, cudaGetErrorString(e));
  tl_cuda_failed = true;
  return true;
}

bool take_cuda_failure() {
  const bool f = tl_cuda_failed;
  tl_cuda_failed = false;
  return f;
}

void note_launch_begin(const char* name, cudaStream_t st) {
  g_launches.fetch_add(1, std::memory_order_relaxed);
  if (g_timing) {
    TimedLaunch t;
    t.name = name;
    cudaEventCreate(&t.e0);
    cudaEventCreate(&t.e1);
    cudaEventRecord(t.e0, st);
    g_timed.push_back(t);
  }
}

void note_launch_end(cudaStream_t st) {
  if (g_timing) cudaEventRecord(g_timed.back().e1, st);
  record_cuda_error(cudaGetLastError(), "kernel launch");
}

int sm_count() {
  static int cached[64] = {0};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev < 0 || dev >= 64) dev = 0;
  if (cached[dev] == 0) {
    int n = 0;
    cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
    cached[dev] = n > 0 ? n : 148;
  }
  return cached[dev];
}

void ensure_dynamic_smem(const void* kernel, int bytes) {
  struct Entry { int dev; const void* fn; int bytes; };
  static Entry table[256];
  static int n = 0;
  static std::mutex mu;
  int dev = 0;
  cudaGetDevice(&dev);
  std::lock_guard<std::mutex> lock(mu);
  for (int i = 0; i < n; ++i) {
    if (table[i].dev == dev && table[i].fn == kernel) {
      if (table[i].bytes >= bytes) return;
      record_cuda_error(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes), "smem attribute");
      table[i].bytes = bytes;
      return;
    }
  }
  record_cuda_error(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes), "smem attribute");
  if (n < 256) table[n++] = Entry{dev, kernel, bytes};
}

// ---------------------------------------------------------------------------
// workspace layout
// ---------------------------------------------------------------------------
struct Layout {
  size_t status, zero_p, stage_h_in, stage_act, stage_h_out, a_op, scale, qkv, attn_hi, attn_lo, attn_f32, h_mid, o_part, g, u, t, t_hi, t_lo, kept_ch, kept_ch_cnt, live, ch_sel, ch_cand_val, ch_cand_idx, ch_keep, down_part,
      h_a, h_b, refresh_tab, refresh_act, total;
  AttnScratch attn;
  int chunks, Mpad, Tmax;
};

static bool shape_ok(const sol_shape_t* s) {
  if (!s) return false;
  if (s->head_dim != 64 && s->head_dim != 128) return false;
  if (s->page_size != 64) return false;
  if (s->n_kv_heads <= 0 || s->n_q_heads <= 0 || s->n_q_heads % s->n_kv_heads) return false;
  if (s->n_q_heads / s->n_kv_heads > 8) return false;
  if (s->d_model <= 0 || s->d_model % 256 || s->d_model > 8192) return false;
  if ((s->n_q_heads * s->head_dim) % 256) return false;
  if (s->d_ff <= 0 || s->d_ff % 32 || s->d_ff > 49152) return false;
  if (s->n_sink < 0 || s->n_window < 0) return false;
  if (s->quant_placement != SOL_QUANT_PROJ_INPUTS && s->quant_placement != SOL_QUANT_MLP_OUTPUT) return false;
  if (s->mlp_prune != SOL_PRUNE_INTERMEDIATE && s->mlp_prune != SOL_PRUNE_MLP_INPUT) return false;
  if (s->token_select != SOL_SELECT_TOKENS && s->token_select != SOL_SELECT_QUEST_PAGES) return false;
  if (s->token_select == SOL_SELECT_QUEST_PAGES) {
    const int S = s->quest_page_size;
    if (S != 4 && S != 8 && S != 16 && S != 32 && S != 64) return false;
    if (S < s->n_q_heads / s->n_kv_heads) return false;  // the callers' page lists fit the token lists' arrays
  }
  return true;
}
// the page extrema are there when the shape asks for them
static bool quest_ok(const sol_shape_t* s, const sol_kv_t* kv) {
  return s->token_select != SOL_SELECT_QUEST_PAGES || kv->quest_meta != nullptr;
}

static Layout make_layout(const sol_shape_t& s, int B, int max_pages) {
  Layout L;
  memset(&L, 0, sizeof(L));
  const size_t d = s.d_model, Hq = s.n_q_heads, Hkv = s.n_kv_heads, hd = s.head_dim, ff = s.d_ff;
  const size_t Nqkv = (Hq + 2 * Hkv) * hd;
  const size_t Mpad = pad_rows(B), Tmax = (size_t)max_pages * s.page_size;
  L.Mpad = (int)Mpad;
  L.Tmax = (int)Tmax;
  L.chunks = down_chunks((int)ff, (int)d);
  size_t at = 0;
  auto take = [&](size_t bytes) {
    const size_t o = at;
    at += (bytes + 255) / 256 * 256;
    return o;
  };
  L.status = take(256);
  L.zero_p = take(128 * 4);  // per-sequence prune rates of zero (never written after the workspace is initialised)
  L.stage_h_in = take(B * d * 2);
  L.stage_act = take(4 * (size_t)B * 4);
  L.stage_h_out = take(B * d * 2);
  L.a_op = take(Mpad * d * 2);
  L.scale = take(Mpad * 4);
  L.qkv = take((size_t)NK_MAX_KSPLIT * B * Nqkv * 4);  // split-K partial sums of the QKV projection
  L.attn = attn_scratch_layout(s, B, max_pages, at);
  at = L.attn.end;
  L.attn_hi = take(2 * Mpad * Hq * hd * 2);  // packed operand: high rows and low rows of every chunk side by side
  L.attn_lo = take(256);
  L.attn_f32 = take(B * Hq * hd * 4);
  L.h_mid = take(B * d * 4);
  L.o_part = take((size_t)NK_MAX_KSPLIT * B * d * 4);  // split-K partial sums of the output projection
  L.g = take(B * ff * 4);
  L.u = take(B * ff * 4);
  L.t = take(B * ff * 4);
  const size_t ffc = (ff + 63) / 64 * 64;  // the packed operand is written in whole 64-channel chunks
  L.t_hi = take(2 * Mpad * ffc * 2);       // high rows and low rows of every chunk side by side
  L.t_lo = take(256);
  L.kept_ch = take(B * ff * 4);
  L.kept_ch_cnt = take((size_t)B * 4);
  L.live = take(ff / 32 * 4);
  L.ch_sel = take((size_t)B * CH_SEL_WORDS * 4);
  L.ch_cand_val = take((size_t)B * CH_CAND_CAP * 8);
  L.ch_cand_idx = take((size_t)B * CH_CAND_CAP * 4);
  L.ch_keep = take((size_t)B * ff);
  L.down_part = take((size_t)L.chunks * Mpad * d * 4);
  L.h_a = take(B * d * 4);
  L.h_b = take(B * d * 4);
  L.refresh_tab = take((size_t)B * max_pages * 4);  // sol_kv_refresh: a page-table row per refreshed token
  L.refresh_act = take(4 * (size_t)B * 4);           // ... its length and the dense action
  L.total = at;
  return L;
}

template <typename T>
static T* at(void* ws, size_t off) {
  return reinterpret_cast<T*>(static_cast<unsigned char*>(ws) + off);
}

static sol_status_t finish() {
  if (tl_cuda_failed) {
    tl_cuda_failed = false;
    return SOL_ERR_CUDA;
  }
  return SOL_OK;
}

static bool kv_ok(const sol_kv_t* kv) {
  return kv && kv->k_pool && kv->v_pool && kv->page_table && kv->seq_lens && kv->max_pages_per_seq > 0 &&
         kv->num_pages > 0;
}

// ---------------------------------------------------------------------------
// compositions
// ---------------------------------------------------------------------------
static void run_attention(const sol_shape_t& s, const Layout& L, void* ws, const sol_kv_t& kv, int B,
                          const int32_t* r_permille, const float* qkv, int ldq, int qkv_ksplit, const float* qkv_scale,
                          const void* q_bf16, void* out_bf16,
                          float* out_f32, bool want_split, int32_t* kept_idx, int32_t* kept_cnt, cudaStream_t st,
                          int span_tokens = 0) {
  AttnArgs a;
  a.shape = s;
  a.kv = kv;
  a.B = B;
  a.span_tokens = span_tokens;
  a.r_permille = r_permille;
  a.qkv_f32 = qkv;
  a.ldq = ldq;
  a.qkv_ksplit = qkv_ksplit;
  a.qkv_scale = qkv_scale;
  a.q_bf16 = q_bf16;
  const bool quest = s.token_select == SOL_SELECT_QUEST_PAGES;
  attn_scratch_bind(a, ws, L.attn, quest ? nullptr : kept_idx, quest ? nullptr : kept_cnt);
  if (quest) {  // the callers' arrays take the kept pages of every query head
    a.quest_pages_out = kept_idx;
    a.quest_cnt_out = kept_cnt;
  }
  a.out_f32 = out_f32;
  a.out_bf16 = out_bf16;
  a.out_hi = want_split ? at<void>(ws, L.attn_hi) : nullptr;  // packed, high and low parts
  a.out_lo = nullptr;
  a.out_rows = L.Mpad;
  a.status = at<int>(ws, L.status);
  launch_attention(a, st);
}

// What a layer leaves to the first RMSNorm kernel of the next one when it skips its own reduction: the partial
// sums of its down projection, the residual they are added to, and the live flags to clear.
struct LayerCarry {
  const float* resid;
  const float* part;
  int chunks;
  size_t stride;
  int32_t* live;
  int n_live;
};

// a_op (packed) / scale in the workspace hold the MLP input operand.
static void run_mlp(const sol_shape_t& s, const Layout& L, void* ws, int B, const void* w_gate_up, const void* w_down,
                    const int32_t* p_permille, const void* resid, int resid_f32, void* out_bf16,
                    float* out_f32, float* out_f32_b, float* t_trace, int32_t* kept_ch, int32_t* kept_ch_cnt,
                    cudaStream_t st, const int32_t* out_bits = nullptr, const sol_layer_trace_t* tr = nullptr,
                    LayerCarry* carry_out = nullptr) {
  int* status = at<int>(ws, L.status);
  GemmNK gu;
  memset(&gu, 0, sizeof(gu));
  gu.a = at<void>(ws, L.a_op);
  gu.n_b = 1;
  gu.w = w_gate_up;
  gu.M = B;
  gu.K = s.d_model;
  gu.N = s.d_ff;
  gu.row_scale = at<float>(ws, L.scale);
  gu.out0 = at<float>(ws, L.g);
  gu.out1 = at<float>(ws, L.u);
  gu.out2 = t_trace ? t_trace : at<float>(ws, L.t);
  gu.sel = at<uint32_t>(ws, L.ch_sel);
  gu.sel_p_permille = p_permille;
  gu.status = status;
  launch_gemm_nk(gu, EPI_SWIGLU, st);

  ChannelSelectArgs cs;
  cs.B = B;
  cs.d = s.d_model;
  cs.ff = s.d_ff;
  cs.p_permille = p_permille;
  cs.g = gu.out0;
  cs.u = gu.out1;
  cs.t = gu.out2;
  cs.a_op = at<void>(ws, L.a_op);
  cs.scale = at<float>(ws, L.scale);
  cs.w_gate_up = w_gate_up;
  cs.sel = at<uint32_t>(ws, L.ch_sel);
  cs.cand_val = at<double>(ws, L.ch_cand_val);
  cs.cand_idx = at<int32_t>(ws, L.ch_cand_idx);
  cs.keep = at<unsigned char>(ws, L.ch_keep);
  cs.scratch_idx = at<int32_t>(ws, L.kept_ch);
  cs.kept_ch = kept_ch;
  cs.kept_cnt = kept_ch_cnt ? kept_ch_cnt : at<int32_t>(ws, L.kept_ch_cnt);
  cs.t_op = at<void>(ws, L.t_hi);
  cs.live = at<int32_t>(ws, L.live);
  cs.status = status;
  launch_channel_select(cs, st);

  GemmDown dn;
  dn.t = cs.t_op;
  dn.t_f32 = cs.t;
  dn.keep = cs.keep;
  dn.w = w_down;
  dn.live = cs.live;
  dn.M = B;
  dn.ff = s.d_ff;
  dn.d = s.d_model;
  dn.partial = at<float>(ws, L.down_part);
  dn.chunks = down_chunks(s.d_ff, s.d_model);
  dn.status = status;
  launch_gemm_down(dn, st);
  if (out_bits != nullptr) {  // the paper's placement: the MLP output is quantized before the residual add
    QuantOutArgs q;
    memset(&q, 0, sizeof(q));
    q.partial = dn.partial; q.chunks = dn.chunks; q.M = B; q.Mpad = pad_rows(B); q.d = s.d_model;
    q.resid = resid; q.resid_f32 = resid_f32; q.bits = out_bits;
    q.out_bf16 = out_bf16; q.out_f32 = out_f32; q.out_f32_b = out_f32_b;
    q.z_tap = tr ? tr->z : nullptr; q.z_codes = tr ? tr->z_codes : nullptr; q.z_scale = tr ? tr->z_scales : nullptr;
    q.live = cs.live; q.n_live = s.d_ff / 32; q.status = status;
    launch_quant_out(q, st);
    return;
  }
  if (carry_out != nullptr) {  // the next layer's first RMSNorm kernel adds the partial sums to the residual
    carry_out->resid = static_cast<const float*>(resid);
    carry_out->part = dn.partial;
    carry_out->chunks = dn.chunks;
    carry_out->stride = (size_t)pad_rows(B) * s.d_model;
    carry_out->live = cs.live;
    carry_out->n_live = s.d_ff / 32;
    return;
  }
  launch_reduce_out(dn.partial, dn.chunks, B, pad_rows(B), s.d_model, resid, resid_f32, out_bf16, out_f32, out_f32_b,
                    cs.live, s.d_ff / 32, st);
}

static void run_layer(const sol_shape_t& s, const Layout& L, void* ws, const sol_layer_weights_t& w,
                      const sol_kv_t& kv, int B, const void* h_in, bool in_f32, void* h_out_bf16, float* h_out_f32,
                      const int32_t* r, const int32_t* p, const int32_t* bits, const sol_layer_trace_t* tr,
                      cudaStream_t st, const LayerCarry* carry_in = nullptr, LayerCarry* carry_out = nullptr,
                      int span_tokens = 0) {
  int* status = at<int>(ws, L.status);
  const int d = s.d_model, Hq = s.n_q_heads, Hkv = s.n_kv_heads, hd = s.head_dim;
  const int Nqkv = (Hq + 2 * Hkv) * hd;
  float* scale = at<float>(ws, L.scale);
  const bool out_quant = s.quant_placement == SOL_QUANT_MLP_OUTPUT;
  const int32_t* in_bits = out_quant ? nullptr : bits;  // no width: the rows go through as bf16

  NormQuantArgs n1;
  memset(&n1, 0, sizeof(n1));
  if (carry_in != nullptr) {  // the previous layer left its down projection unreduced: h_in = its residual + the partials
    n1.in = carry_in->resid; n1.in_f32 = true; n1.part = carry_in->part; n1.ksplit = carry_in->chunks;
    n1.part_stride = carry_in->stride; n1.zero_flags = carry_in->live; n1.n_zero_flags = carry_in->n_live;
    n1.sum_out = at<float>(ws, L.h_a);
    h_in = n1.sum_out;
    in_f32 = true;
  } else {
    n1.in = h_in; n1.in_f32 = in_f32;
  }
  n1.gamma_bf16 = w.gamma1; n1.eps = s.rms_eps; n1.bits = in_bits; n1.B = B; n1.d = d;
  n1.a_op = at<void>(ws, L.a_op); n1.a_op_rows = L.Mpad; n1.scale = scale; n1.xn = tr ? tr->xn1 : nullptr;
  n1.codes = tr ? tr->codes1 : nullptr;
  n1.status = status;
  launch_norm_quant(n1, st);
  if (tr && tr->scales1) cudaMemcpyAsync(tr->scales1, scale, sizeof(float) * B, cudaMemcpyDeviceToDevice, st);

  // QKV projection, split over K: raw partial sums, summed and scaled by the kernel that rotates and appends
  GemmNK q;
  memset(&q, 0, sizeof(q));
  q.name = "gemm_qkv";
  q.a = at<void>(ws, L.a_op);
  q.n_b = 1;
  q.w = w.w_qkv;
  q.M = B;
  q.K = d;
  q.N = Nqkv;
  q.out0 = at<float>(ws, L.qkv);
  q.status = status;
  launch_gemm_nk(q, EPI_PARTIAL, st);

  run_attention(s, L, ws, kv, B, r, at<float>(ws, L.qkv), Nqkv, nk_ksplit(Nqkv, d), scale, nullptr, nullptr,
                tr ? tr->attn_out : nullptr, true, tr ? tr->kept_idx : nullptr, tr ? tr->kept_cnt : nullptr, st,
                span_tokens);
  if (tr && tr->q_rot)
    cudaMemcpyAsync(tr->q_rot, at<float>(ws, L.attn.q_rot), sizeof(float) * B * Hq * hd, cudaMemcpyDeviceToDevice, st);

  // output projection, split over K; the second RMSNorm kernel adds the partial sums to the residual
  GemmNK o;
  memset(&o, 0, sizeof(o));
  o.name = "gemm_out_proj";
  o.a = at<void>(ws, L.attn_hi);
  o.n_b = 2;
  o.w = w.w_o;
  o.M = B;
  o.K = Hq * hd;
  o.N = d;
  o.out0 = at<float>(ws, L.o_part);
  o.status = status;
  launch_gemm_nk(o, EPI_PARTIAL, st);

  NormQuantArgs n2;
  memset(&n2, 0, sizeof(n2));
  n2.in = h_in; n2.in_f32 = in_f32; n2.part = at<float>(ws, L.o_part); n2.ksplit = nk_ksplit(d, Hq * hd);
  n2.sum_out = at<float>(ws, L.h_mid);
  n2.gamma_bf16 = w.gamma2; n2.eps = s.rms_eps; n2.bits = in_bits; n2.B = B; n2.d = d;
  n2.a_op = at<void>(ws, L.a_op); n2.a_op_rows = L.Mpad; n2.scale = scale; n2.xn = tr ? tr->xn2 : nullptr;
  n2.codes = tr ? tr->codes2 : nullptr;
  n2.status = status;
  const bool gate_inputs = s.mlp_prune == SOL_PRUNE_MLP_INPUT;
  if (gate_inputs) {  // the paper's MLP pruning: p gates the input channels, every intermediate channel is kept
    n2.gate_p_permille = p;
    n2.xm = tr ? tr->xm2 : nullptr;
  }
  n2.clear = at<uint32_t>(ws, L.ch_sel);
  n2.clear_words = CH_SEL_WORDS;
  launch_norm_quant(n2, st);
  if (tr && tr->h_mid)
    cudaMemcpyAsync(tr->h_mid, at<float>(ws, L.h_mid), sizeof(float) * B * d, cudaMemcpyDeviceToDevice, st);
  if (tr && tr->scales2) cudaMemcpyAsync(tr->scales2, scale, sizeof(float) * B, cudaMemcpyDeviceToDevice, st);

  run_mlp(s, L, ws, B, w.w_gate_up, w.w_down, gate_inputs ? at<int32_t>(ws, L.zero_p) : p, at<float>(ws, L.h_mid), 1,
          h_out_bf16, h_out_f32,
          tr ? tr->h_out : nullptr, tr ? tr->t : nullptr, tr ? tr->kept_ch : nullptr, tr ? tr->kept_ch_cnt : nullptr,
          st, out_quant ? bits : nullptr, tr, carry_out);
}

static bool weights_ok(const sol_layer_weights_t* w) {
  return w && w->w_qkv && w->w_o && w->w_gate_up && w->w_down && w->gamma1 && w->gamma2;
}

}  // namespace sol

using namespace sol;

// ---------------------------------------------------------------------------
// exported entry points
// ---------------------------------------------------------------------------
extern "C" {

const char* sol_status_string(sol_status_t s) {
  switch (s) {
    case SOL_OK: return "ok";
    case SOL_ERR_INVALID_ARG: return "invalid argument";
    case SOL_ERR_UNSUPPORTED: return "unsupported shape";
    case SOL_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case SOL_ERR_CUDA: return "CUDA error";
    case SOL_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
    default: return "unknown status";
  }
}

const char* sol_last_cuda_error(void) { return tl_cuda_error; }

size_t sol_workspace_bytes(const sol_shape_t* shape, int32_t max_batch, int32_t max_pages_per_seq) {
  if (!shape_ok(shape) || max_batch < 1 || max_batch > 128 || max_pages_per_seq < 1 ||
      max_pages_per_seq > MAX_PAGES_PER_SEQ)
    return 0;
  return make_layout(*shape, max_batch, max_pages_per_seq).total;
}

sol_status_t sol_workspace_init(void* ws, size_t ws_bytes, sol_stream_t stream) {
  if (!ws || ws_bytes < 256) return SOL_ERR_INVALID_ARG;
  if (record_cuda_error(cudaMemsetAsync(ws, 0, ws_bytes, (cudaStream_t)stream), "workspace memset"))
    return finish();
  return SOL_OK;
}

sol_status_t sol_quant_act(const void* x_bf16, int32_t B, int32_t d, const int32_t* bits, int8_t* codes,
                           float* scales, void* xhat_bf16, sol_stream_t stream) {
  if (!x_bf16 || !bits || !codes || !scales || B < 0 || d <= 0) return SOL_ERR_INVALID_ARG;
  if (d % 8 || d > 8192) return SOL_ERR_UNSUPPORTED;
  if (B == 0) return SOL_OK;
  NormQuantArgs n;
  memset(&n, 0, sizeof(n));
  n.in = x_bf16; n.bits = bits; n.B = B; n.d = d; n.a_op = xhat_bf16; n.scale = scales; n.codes = codes;
  launch_norm_quant(n, (cudaStream_t)stream);
  return finish();
}

sol_status_t sol_quant_act_wide(const void* x_bf16, int32_t B, int32_t d, const int32_t* bits, int16_t* codes,
                                float* scales, sol_stream_t stream) {
  if (!x_bf16 || !bits || !codes || !scales || B < 0 || d <= 0) return SOL_ERR_INVALID_ARG;
  if (d % 8 || d > 8192) return SOL_ERR_UNSUPPORTED;
  if (B == 0) return SOL_OK;
  NormQuantArgs n;
  memset(&n, 0, sizeof(n));
  n.in = x_bf16; n.bits = bits; n.B = B; n.d = d; n.scale = scales; n.codes16 = codes;
  launch_norm_quant(n, (cudaStream_t)stream);
  return finish();
}

size_t sol_quest_meta_bytes(const sol_shape_t* shape, int32_t num_pages) {
  if (!shape_ok(shape) || shape->token_select != SOL_SELECT_QUEST_PAGES || num_pages <= 0) return 0;
  return (size_t)num_pages * shape->n_kv_heads * (PAGE / shape->quest_page_size) * 2 * shape->head_dim * 2;
}

sol_status_t sol_quest_build_meta(const sol_shape_t* shape, const sol_kv_t* kv, int32_t B, sol_stream_t stream) {
  if (!shape || !kv_ok(kv) || B < 0) return SOL_ERR_INVALID_ARG;
  if (!shape_ok(shape) || shape->token_select != SOL_SELECT_QUEST_PAGES || kv->max_pages_per_seq > MAX_PAGES_PER_SEQ)
    return SOL_ERR_UNSUPPORTED;
  if (!kv->quest_meta) return SOL_ERR_INVALID_ARG;
  if (B == 0) return SOL_OK;
  // a bad page id is reported through the status words of a workspace; this call has none, so such pages are
  // skipped here and found by the attention call
  static int* sink = nullptr;
  if (!sink && record_cuda_error(cudaMalloc(&sink, 64), "sol_quest_build_meta")) return finish();
  launch_quest_meta(*shape, *kv, B, true, sink, (cudaStream_t)stream);
  return finish();
}

sol_status_t sol_sparse_decode_attn(const sol_shape_t* shape, const void* q_bf16, const sol_kv_t* kv, int32_t B,
                                    const int32_t* r_permille, void* out_bf16, int32_t* kept_idx, int32_t* kept_cnt,
                                    void* ws, size_t ws_bytes, sol_stream_t stream) {
  if (!shape || !q_bf16 || !kv_ok(kv) || !r_permille || !out_bf16 || !ws || B < 0) return SOL_ERR_INVALID_ARG;
  if (!shape_ok(shape) || B > 128 || kv->max_pages_per_seq > MAX_PAGES_PER_SEQ) return SOL_ERR_UNSUPPORTED;
  if (!quest_ok(shape, kv)) return SOL_ERR_INVALID_ARG;
  if (B == 0) return SOL_OK;
  const Layout L = make_layout(*shape, B, kv->max_pages_per_seq);
  if (ws_bytes < L.total) return SOL_ERR_WORKSPACE_TOO_SMALL;
  run_attention(*shape, L, ws, *kv, B, r_permille, nullptr, 0, 0, nullptr, q_bf16, out_bf16, nullptr, false, kept_idx,
                kept_cnt, (cudaStream_t)stream);
  return finish();
}

sol_status_t sol_pruned_swiglu_mlp(const sol_shape_t* shape, const void* x_bf16, const void* w_gate_up,
                                   const void* w_down, int32_t B, const int32_t* p_permille, void* out_bf16,
                                   int32_t* kept_ch, int32_t* kept_ch_cnt, void* ws, size_t ws_bytes,
                                   sol_stream_t stream) {
  if (!shape || !x_bf16 || !w_gate_up || !w_down || !p_permille || !out_bf16 || !ws || B < 0)
    return SOL_ERR_INVALID_ARG;
  if (!shape_ok(shape) || B > 128) return SOL_ERR_UNSUPPORTED;
  if (B == 0) return SOL_OK;
  const Layout L = make_layout(*shape, B, 1);
  if (ws_bytes < L.total) return SOL_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t st = (cudaStream_t)stream;
  // bf16 passthrough into the padded, packed operand buffer, scale 1
  NormQuantArgs n;
  memset(&n, 0, sizeof(n));
  n.in = x_bf16; n.B = B; n.d = shape->d_model; n.a_op = at<void>(ws, L.a_op); n.a_op_rows = L.Mpad;
  n.scale = at<float>(ws, L.scale);
  n.clear = at<uint32_t>(ws, L.ch_sel);
  n.clear_words = CH_SEL_WORDS;
  launch_norm_quant(n, st);
  run_mlp(*shape, L, ws, B, w_gate_up, w_down, p_permille, nullptr, 0, out_bf16, nullptr, nullptr, nullptr,
          kept_ch, kept_ch_cnt, st);
  return finish();
}

size_t sol_packed_weight_bytes(const sol_shape_t* shape, int32_t kind) {
  if (!shape_ok(shape)) return 0;
  const int d = shape->d_model, qo = shape->n_q_heads * shape->head_dim;
  const int nqkv = (shape->n_q_heads + 2 * shape->n_kv_heads) * shape->head_dim;
  switch (kind) {
    case SOL_W_QKV: return nk_packed_bytes(nk_geom_plain(nqkv, d));
    case SOL_W_O: return nk_packed_bytes(nk_geom_plain(d, qo));
    case SOL_W_GATE_UP: return nk_packed_bytes(nk_geom_gate_up(shape->d_ff, d, sm_count()));
    case SOL_W_DOWN: return down_packed_bytes(shape->d_ff, d);
    default: return 0;
  }
}

sol_status_t sol_pack_weights(const sol_shape_t* shape, int32_t kind, const void* src0, const void* src1, void* dst,
                              size_t dst_bytes, sol_stream_t stream) {
  if (!shape || !src0 || !dst || kind < SOL_W_QKV || kind > SOL_W_DOWN || (kind == SOL_W_GATE_UP && !src1))
    return SOL_ERR_INVALID_ARG;
  const size_t need = sol_packed_weight_bytes(shape, kind);
  if (need == 0) return SOL_ERR_UNSUPPORTED;
  if (dst_bytes < need) return SOL_ERR_WORKSPACE_TOO_SMALL;
  launch_pack_weights(*shape, kind, src0, src1, dst, (cudaStream_t)stream);
  return finish();
}

static sol_status_t check_actions_host_side(const sol_shape_t* shape, int32_t B) {
  if (!shape_ok(shape) || B > 128) return SOL_ERR_UNSUPPORTED;
  return SOL_OK;
}

sol_status_t sol_decode_layer(const sol_shape_t* shape, const sol_layer_weights_t* w, const sol_kv_t* kv, int32_t B,
                              const void* h_in_bf16, void* h_out_bf16, const int32_t* r_permille,
                              const int32_t* p_permille, const int32_t* bits, const sol_layer_trace_t* trace,
                              void* ws, size_t ws_bytes, sol_stream_t stream) {
  if (!shape || !weights_ok(w) || !kv_ok(kv) || !h_in_bf16 || !h_out_bf16 || !r_permille || !p_permille || !bits ||
      !ws || B < 0)
    return SOL_ERR_INVALID_ARG;
  sol_status_t s = check_actions_host_side(shape, B);
  if (s != SOL_OK) return s;
  if (kv->max_pages_per_seq > MAX_PAGES_PER_SEQ) return SOL_ERR_UNSUPPORTED;
  if (!quest_ok(shape, kv)) return SOL_ERR_INVALID_ARG;
  if (B == 0) return SOL_OK;
  const Layout L = make_layout(*shape, B, kv->max_pages_per_seq);
  if (ws_bytes < L.total) return SOL_ERR_WORKSPACE_TOO_SMALL;
  run_layer(*shape, L, ws, *w, *kv, B, h_in_bf16, false, h_out_bf16, nullptr, r_permille, p_permille, bits, trace,
            (cudaStream_t)stream);
  return finish();
}

static sol_status_t decode_step_impl(const sol_shape_t* shape, int32_t n_layers, const sol_layer_weights_t* layers,
                                     const sol_kv_t* kvs, const int32_t* seq_lens_override, int32_t B,
                                     const void* h_in_bf16, void* h_out_bf16, float* h_out_f32, const int32_t* r,
                                     const int32_t* p, const int32_t* bits, void* ws, const Layout& L,
                                     cudaStream_t st, const sol_layer_trace_t* traces = nullptr) {
  const void* h = h_in_bf16;
  bool in_f32 = false;
  // Between two layers the reduction of the down projection (partials + residual) is left to the next layer's
  // first RMSNorm kernel, which reads the row anyway: one launch less per layer.  Not with per-layer taps and not
  // when the MLP output goes through the quantizer first.
  const bool may_defer = traces == nullptr && shape->quant_placement != SOL_QUANT_MLP_OUTPUT;
  LayerCarry carry[2];
  bool have = false;
  for (int l = 0; l < n_layers; ++l) {
    sol_kv_t kv = kvs[l];
    if (seq_lens_override) kv.seq_lens = seq_lens_override;
    const bool last = l == n_layers - 1;
    const bool defer = may_defer && !last;
    float* out32 = last ? h_out_f32 : at<float>(ws, (l & 1) ? L.h_b : L.h_a);
    run_layer(*shape, L, ws, layers[l], kv, B, h, in_f32, last ? h_out_bf16 : nullptr, out32, r, p, bits,
              traces ? &traces[l] : nullptr, st, have ? &carry[(l + 1) & 1] : nullptr, defer ? &carry[l & 1] : nullptr);
    have = defer;
    h = out32;
    in_f32 = true;
  }
  return finish();
}

static sol_status_t step_args_ok(const sol_shape_t* shape, int32_t n_layers, const sol_layer_weights_t* layers,
                                 const sol_kv_t* kvs, int32_t B, int* max_pages) {
  if (!shape || n_layers < 1 || !layers || !kvs || B < 0) return SOL_ERR_INVALID_ARG;
  if (!shape_ok(shape) || B > 128) return SOL_ERR_UNSUPPORTED;
  int mp = 0;
  for (int l = 0; l < n_layers; ++l) {
    if (!weights_ok(&layers[l]) || !kv_ok(&kvs[l]) || !quest_ok(shape, &kvs[l])) return SOL_ERR_INVALID_ARG;
    if (kvs[l].max_pages_per_seq > mp) mp = kvs[l].max_pages_per_seq;
  }
  if (mp > MAX_PAGES_PER_SEQ) return SOL_ERR_UNSUPPORTED;
  *max_pages = mp;
  return SOL_OK;
}

sol_status_t sol_decode_step(const sol_shape_t* shape, int32_t n_layers, const sol_layer_weights_t* layers,
                             const sol_kv_t* kvs, int32_t B, const void* h_in_bf16, void* h_out_bf16,
                             float* h_out_f32, const int32_t* r_permille, const int32_t* p_permille,
                             const int32_t* bits, void* ws, size_t ws_bytes, sol_stream_t stream) {
  int mp = 0;
  sol_status_t s = step_args_ok(shape, n_layers, layers, kvs, B, &mp);
  if (s != SOL_OK) return s;
  if (!h_in_bf16 || !h_out_bf16 || !r_permille || !p_permille || !bits || !ws) return SOL_ERR_INVALID_ARG;
  if (B == 0) return SOL_OK;
  const Layout L = make_layout(*shape, B, mp);
  if (ws_bytes < L.total) return SOL_ERR_WORKSPACE_TOO_SMALL;
  return decode_step_impl(shape, n_layers, layers, kvs, nullptr, B, h_in_bf16, h_out_bf16, h_out_f32, r_permille,
                          p_permille, bits, ws, L, (cudaStream_t)stream);
}

sol_status_t sol_decode_step_traced(const sol_shape_t* shape, int32_t n_layers, const sol_layer_weights_t* layers,
                                    const sol_kv_t* kvs, int32_t B, const void* h_in_bf16, void* h_out_bf16,
                                    float* h_out_f32, const int32_t* r_permille, const int32_t* p_permille,
                                    const int32_t* bits, const sol_layer_trace_t* traces, void* ws, size_t ws_bytes,
                                    sol_stream_t stream) {
  int mp = 0;
  sol_status_t s = step_args_ok(shape, n_layers, layers, kvs, B, &mp);
  if (s != SOL_OK) return s;
  if (!h_in_bf16 || !h_out_bf16 || !r_permille || !p_permille || !bits || !ws) return SOL_ERR_INVALID_ARG;
  if (B == 0) return SOL_OK;
  const Layout L = make_layout(*shape, B, mp);
  if (ws_bytes < L.total) return SOL_ERR_WORKSPACE_TOO_SMALL;
  return decode_step_impl(shape, n_layers, layers, kvs, nullptr, B, h_in_bf16, h_out_bf16, h_out_f32, r_permille,
                          p_permille, bits, ws, L, (cudaStream_t)stream, traces);
}

// ---------------------------------------------------------------------------
// KV refresh: the last n_tokens tokens of every sequence go through the layers again as rows of one batch,
// row (s, i) with the page table of sequence s and the length T_s - n_tokens + 1 + i, under the dense action.
// Every row appends its key and value at its own position before any row's attention reads the cache (the
// append is a kernel of its own, ahead of the attention), so row i sees the refreshed entries of rows < i: the
// causal pass the paper describes.  The projections and the MLP are the decode step's kernels; the attention of
// spans up to 16 tokens is the span kernel's (sol_span.cu).
// ---------------------------------------------------------------------------
__global__ void refresh_expand_kernel(const int32_t* __restrict__ table, const int32_t* __restrict__ seq_lens, int mp,
                                      int n_tok, int rows, int32_t* __restrict__ out_table,
                                      int32_t* __restrict__ out_act, int* __restrict__ status) {
  const int row = blockIdx.x, s = row / n_tok, i = row - s * n_tok;
  for (int j = threadIdx.x; j < mp; j += blockDim.x) out_table[(size_t)row * mp + j] = table[(size_t)s * mp + j];
  if (threadIdx.x == 0) {
    int len = seq_lens[s] - n_tok + 1 + i;
    if (len < 1) {  // a sequence shorter than the refreshed span: reported, and the row kept inside the cache
      atomicOr(status + ST_ERR, ERR_BAD_ACTION);
      len = 1;
    }
    out_act[row] = 1000;             // keep-rate
    out_act[rows + row] = 0;         // prune rate
    out_act[2 * rows + row] = 16;    // bit-width
    out_act[3 * rows + row] = len;   // length of the row's context, its own token included
  }
}

sol_status_t sol_kv_refresh(const sol_shape_t* shape, int32_t n_layers, const sol_layer_weights_t* layers,
                            const sol_kv_t* kvs, int32_t B, int32_t n_tokens, const void* h_in_bf16,
                            void* h_out_bf16, void* ws, size_t ws_bytes, sol_stream_t stream) {
  int mp = 0;
  sol_status_t s = step_args_ok(shape, n_layers, layers, kvs, B, &mp);
  if (s != SOL_OK) return s;
  if (!h_in_bf16 || !ws || n_tokens < 1) return SOL_ERR_INVALID_ARG;
  if (n_tokens > 128) return SOL_ERR_UNSUPPORTED;
  if (B == 0) return SOL_OK;
  sol_shape_t dense = *shape;
  dense.token_select = SOL_SELECT_TOKENS;  // every token is kept: no page bounds are needed, and the rows of a
  dense.quest_page_size = 0;               // sequence would race for the extrema of the block they share
  const int per = 128 / n_tokens;          // sequences per pass
  const int rows_max = (B < per ? B : per) * n_tokens;
  if (ws_bytes < make_layout(dense, rows_max, mp).total) return SOL_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t st = (cudaStream_t)stream;
  const size_t row_bytes = (size_t)shape->d_model * 2;
  for (int s0 = 0; s0 < B; s0 += per) {
    const int ns = B - s0 < per ? B - s0 : per, rows = ns * n_tokens;
    const Layout L = make_layout(dense, rows, mp);
    int32_t* tab = at<int32_t>(ws, L.refresh_tab);
    int32_t* act = at<int32_t>(ws, L.refresh_act);
    const void* h = static_cast<const unsigned char*>(h_in_bf16) + (size_t)s0 * n_tokens * row_bytes;
    void* out = h_out_bf16 ? static_cast<unsigned char*>(h_out_bf16) + (size_t)s0 * n_tokens * row_bytes : nullptr;
    bool in_f32 = false;
    const int32_t* prev_table = nullptr;
    const int32_t* prev_lens = nullptr;
    int prev_mp = 0;
    for (int l = 0; l < n_layers; ++l) {
      sol_kv_t kv = kvs[l];
      if (kv.page_table != prev_table || kv.seq_lens != prev_lens || kv.max_pages_per_seq != prev_mp) {
        // a plain launch: it starts after everything before it on the stream has ended, and the layer's first
        // kernel after it
        refresh_expand_kernel<<<rows, 128, 0, st>>>(kv.page_table + (size_t)s0 * kv.max_pages_per_seq, kv.seq_lens + s0,
                                                    kv.max_pages_per_seq, n_tokens, rows, tab, act, at<int>(ws, L.status));
        if (record_cuda_error(cudaGetLastError(), "refresh: page-table rows")) return finish();
        prev_table = kv.page_table; prev_lens = kv.seq_lens; prev_mp = kv.max_pages_per_seq;
      }
      kv.page_table = tab;
      kv.seq_lens = act + 3 * rows;
      const bool last = l == n_layers - 1;
      float* out32 = at<float>(ws, (l & 1) ? L.h_b : L.h_a);
      // up to 16 tokens per sequence are the rows of one tensor-core tile of the span attention, which reads a
      // sequence's cache once for all of them; longer spans go through the decode step's attention row by row
      run_layer(dense, L, ws, layers[l], kv, rows, h, in_f32, last ? out : nullptr, last && out ? nullptr : out32, act,
                act + rows, act + 2 * rows, nullptr, st, nullptr, nullptr, n_tokens <= 16 ? n_tokens : 0);
      h = out32;
      in_f32 = true;
    }
    if (shape->token_select == SOL_SELECT_QUEST_PAGES) {  // the extrema of the blocks that hold refreshed keys
      for (int l = 0; l < n_layers; ++l) {
        sol_kv_t kv = kvs[l];
        kv.page_table += (size_t)s0 * kv.max_pages_per_seq;
        kv.seq_lens += s0;
        launch_quest_meta_tail(*shape, kv, ns, n_tokens, at<int>(ws, L.status), st);
      }
    }
  }
  return finish();
}

// The per-sequence actions and lengths of a step (at most 128 sequences) travel as kernel parameters:
// one launch instead of four small host-to-device copies, and the values are taken at the call.
struct StepActions {
  int32_t v[4][128];  // keep-rate, prune rate, bit-width, sequence length
};
__global__ void upload_actions_kernel(const StepActions a, int B, int32_t* __restrict__ dst) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < 4 * B) dst[i] = a.v[i / B][i % B];
}

sol_status_t sol_decode_step_host(const sol_shape_t* shape, int32_t n_layers, const sol_layer_weights_t* layers,
                                  const sol_kv_t* kvs, int32_t B, const void* h_in_bf16_host, void* h_out_bf16_host,
                                  const int32_t* r_permille_host, const int32_t* p_permille_host,
                                  const int32_t* bits_host, const int32_t* seq_lens_host, void* ws, size_t ws_bytes,
                                  sol_stream_t stream) {
  int mp = 0;
  sol_status_t s = step_args_ok(shape, n_layers, layers, kvs, B, &mp);
  if (s != SOL_OK) return s;
  if (!h_in_bf16_host || !h_out_bf16_host || !r_permille_host || !p_permille_host || !bits_host || !seq_lens_host ||
      !ws)
    return SOL_ERR_INVALID_ARG;
  for (int i = 0; i < B; ++i) {
    if (r_permille_host[i] < 0 || r_permille_host[i] > 1000 || p_permille_host[i] < 0 || p_permille_host[i] > 1000)
      return SOL_ERR_INVALID_ARG;
    const int b = bits_host[i];
    const int b_max = shape->quant_placement == SOL_QUANT_MLP_OUTPUT ? 15 : 8;  // operand codes are exact bf16 numbers up to 8 bits
    if (!(b == 16 || (b >= 2 && b <= b_max))) return (b >= 9 && b <= 15) ? SOL_ERR_UNSUPPORTED : SOL_ERR_INVALID_ARG;
    if (seq_lens_host[i] < 1 || seq_lens_host[i] > mp * shape->page_size) return SOL_ERR_INVALID_ARG;
  }
  if (B == 0) return SOL_OK;
  const Layout L = make_layout(*shape, B, mp);
  if (ws_bytes < L.total) return SOL_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t st = (cudaStream_t)stream;
  const size_t hb = (size_t)B * shape->d_model * 2, ab = (size_t)B * 4;
  int32_t* act = at<int32_t>(ws, L.stage_act);
  bool bad = false;
  bad |= record_cuda_error(cudaMemcpyAsync(at<void>(ws, L.stage_h_in), h_in_bf16_host, hb, cudaMemcpyHostToDevice, st), "h2d h_in");
  {
    StepActions sa;
    memcpy(sa.v[0], r_permille_host, ab);
    memcpy(sa.v[1], p_permille_host, ab);
    memcpy(sa.v[2], bits_host, ab);
    memcpy(sa.v[3], seq_lens_host, ab);
    upload_actions_kernel<<<(4 * B + 127) / 128, 128, 0, st>>>(sa, B, act);
    bad |= record_cuda_error(cudaGetLastError(), "upload of the actions");
  }
  if (bad) return finish();
  s = decode_step_impl(shape, n_layers, layers, kvs, act + 3 * B, B, at<void>(ws, L.stage_h_in),
                       at<void>(ws, L.stage_h_out), nullptr, act, act + B, act + 2 * B, ws, L, st);
  if (s != SOL_OK) return s;
  record_cuda_error(cudaMemcpyAsync(h_out_bf16_host, at<void>(ws, L.stage_h_out), hb, cudaMemcpyDeviceToHost, st), "d2h h_out");
  // the call synchronises anyway, so it also reads the error word of the workspace: a wait that gave up is
  // reported here instead of leaving a result built from skipped stores
  int32_t err_word = 0;
  record_cuda_error(cudaMemcpyAsync(&err_word, at<int32_t>(ws, L.status) + ST_ERR, sizeof(int32_t), cudaMemcpyDeviceToHost, st),
                    "status copy");
  record_cuda_error(cudaStreamSynchronize(st), "stream synchronize");
  s = finish();
  if (s != SOL_OK) return s;
  return (err_word & ERR_TIMEOUT) ? SOL_ERR_DEVICE_TIMEOUT : SOL_OK;
}

sol_status_t sol_read_device_status(const void* ws, int32_t* out_host8, sol_stream_t stream) {
  if (!ws || !out_host8) return SOL_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  if (record_cuda_error(cudaMemcpyAsync(out_host8, ws, sizeof(int32_t) * ST_WORDS, cudaMemcpyDeviceToHost, st), "status copy"))
    return finish();
  if (record_cuda_error(cudaStreamSynchronize(st), "stream synchronize")) return finish();
  return (out_host8[ST_ERR] & ERR_TIMEOUT) ? SOL_ERR_DEVICE_TIMEOUT : SOL_OK;
}

// One CTA waits on an mbarrier that nothing ever arrives at; the bounded wait gives up after a few thousand
// polls, raises the time-out bit of the workspace's status words and the kernel returns.
__global__ void selftest_wait_kernel(int* status) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    fence_mbar_init();
  }
  __syncthreads();
  if (threadIdx.x == 0) mbar_wait(&bar, 0, status, 4096);
}

sol_status_t sol_selftest_wait_timeout(void* ws, sol_stream_t stream) {
  if (!ws) return SOL_ERR_INVALID_ARG;
  selftest_wait_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(at<int>(ws, 0));
  record_cuda_error(cudaGetLastError(), "self-test launch");
  return finish();
}

void sol_timing_enable(int32_t on) {
  g_timing = on != 0;
  if (!g_timing) {
    for (auto& t : g_timed) {
      cudaEventDestroy(t.e0);
      cudaEventDestroy(t.e1);
    }
    g_timed.clear();
  }
}

int32_t sol_timing_collect(sol_kernel_time_t* out_host, int32_t max_entries) {
  cudaDeviceSynchronize();
  std::map<std::string, std::pair<int, float>> agg;
  std::vector<std::string> order;
  for (auto& t : g_timed) {
    float ms = 0.f;
    cudaEventElapsedTime(&ms, t.e0, t.e1);
    auto it = agg.find(t.name);
    if (it == agg.end()) {
      agg[t.name] = {1, ms};
      order.push_back(t.name);
    } else {
      it->second.first += 1;
      it->second.second += ms;
    }
    cudaEventDestroy(t.e0);
    cudaEventDestroy(t.e1);
  }
  g_timed.clear();
  int n = 0;
  for (auto& name : order) {
    if (n >= max_entries || !out_host) break;
    memset(&out_host[n], 0, sizeof(sol_kernel_time_t));
    strncpy(out_host[n].name, name.c_str(), sizeof(out_host[n].name) - 1);
    out_host[n].launches = agg[name].first;
    out_host[n].total_ms = agg[name].second;
    ++n;
  }
  return n;
}

int64_t sol_launch_count(int32_t reset) {
  const long long v = g_launches.load();
  if (reset) g_launches.store(0);
  return v;
}

}  // extern "C"
