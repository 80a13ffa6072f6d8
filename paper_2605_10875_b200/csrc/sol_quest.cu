// The paper's own token sparsity: Quest page selection per query head (appendix on efficiency actions,
// "Token sparsity via Quest": "Budgeted token selection", "Quest masking in LLaMA attention", "Granularity").
//
//   quest_meta    per block of S tokens of a cache page: the per-dimension maximum of its keys (m+) and the
//                 negated minimum (m-), as bf16 (extrema of bf16 numbers are bf16 numbers).  Either for every
//                 page of the sequences (after a prefill) or only for the block of each sequence's newest token
//                 (after a decode step's append).
//   quest_select  one CTA per (sequence, kv-head): for each query head of the group the bound
//                 q_pos.m+ + q_neg.m- of every page in float64 (a page costs 2/S of its keys' bytes), an exact
//                 radix select of the head's ceil(b_t / S) best pages on the 64-bit keys (forced pages first,
//                 ties to the lower page), then the union of the heads' pages as the row's token list, its
//                 pass-2 work items, and a byte per page that says which heads keep it.
//   quest_logits  q.k of every listed token for the G heads (K rows are read only for pages in the union),
//                 minus infinity for the heads that did not keep the token's page: pass 2 (attn_gather) then
//                 weighs a token with zero for those heads, which is the paper's additive mask.
#include <math.h>

#include "sol_common.cuh"
#include "sol_internal.h"

namespace sol {

// bf16 elements before the extrema of block qb of (physical page, kv-head): m+ [hd], then m- [hd]
__host__ __device__ inline size_t quest_meta_offset(int page, int kvh, int qb, int Hkv, int S, int hd) {
  return ((((size_t)page * Hkv + kvh) * (PAGE / S)) + qb) * 2 * hd;
}

// ============================================================================
// quest_meta
// ============================================================================
struct QuestMetaDev {
  sol_kv_t kv;
  int Hkv, hd, S, all;
  int* status;
};

constexpr int QM_THREADS = 128;

__global__ void __launch_bounds__(QM_THREADS) quest_meta_kernel(const QuestMetaDev p) {
  const int b = blockIdx.z, kvh = blockIdx.y;
  pdl_trigger();
  pdl_wait();  // the newest key is written by the kernel before this one
  const int T = min(max(p.kv.seq_lens[b], 0), p.kv.max_pages_per_seq * PAGE);
  if (T <= 0) return;
  const int lp = p.all ? (int)blockIdx.x : (T - 1) / PAGE;  // logical cache page
  if (lp * PAGE >= T) return;
  const int page = p.kv.page_table[(size_t)b * p.kv.max_pages_per_seq + lp];
  if (page < 0 || page >= p.kv.num_pages) {
    if (threadIdx.x == 0) atomicOr(p.status + ST_ERR, ERR_BAD_PAGE);
    return;
  }
  const int half = p.hd / 2, nblk = PAGE / p.S;
  const uint32_t* rows = reinterpret_cast<const uint32_t*>(static_cast<const uint16_t*>(p.kv.k_pool) +
                                                           ((size_t)page * p.Hkv + kvh) * PAGE * p.hd);
  uint32_t* meta = reinterpret_cast<uint32_t*>(static_cast<uint16_t*>(p.kv.quest_meta));
  const int newest = ((T - 1) % PAGE) / p.S;
  for (int w = threadIdx.x; w < nblk * half; w += QM_THREADS) {
    const int qb = w / half, dp = w - qb * half;  // block of the page, pair of dimensions
    if (!p.all && qb != newest) continue;
    const int t0 = lp * PAGE + qb * p.S;
    if (t0 >= T) continue;
    const int n = min(p.S, T - t0);
    float mx0 = -INFINITY, mx1 = -INFINITY, mn0 = INFINITY, mn1 = INFINITY;
    for (int j = 0; j < n; ++j) {
      const uint32_t u = rows[(size_t)(qb * p.S + j) * half + dp];
      const float lo = bf16_lo(u), hi = bf16_hi(u);
      mx0 = fmaxf(mx0, lo);
      mn0 = fminf(mn0, lo);
      mx1 = fmaxf(mx1, hi);
      mn1 = fminf(mn1, hi);
    }
    const size_t o = quest_meta_offset(page, kvh, qb, p.Hkv, p.S, p.hd) / 2;  // in 32-bit words
    meta[o + dp] = pack_bf16(mx0, mx1);
    meta[o + half + dp] = pack_bf16(-mn0, -mn1);
  }
}

void launch_quest_meta(const sol_shape_t& sh, const sol_kv_t& kv, int B, bool all, int* status, cudaStream_t st) {
  QuestMetaDev d;
  d.kv = kv; d.Hkv = sh.n_kv_heads; d.hd = sh.head_dim; d.S = sh.quest_page_size; d.all = all ? 1 : 0; d.status = status;
  const dim3 grid(all ? kv.max_pages_per_seq : 1, sh.n_kv_heads, B);
  SOL_LAUNCH("quest_meta", quest_meta_kernel, grid, dim3(QM_THREADS), 0, st, d);
}

// ============================================================================
// quest_select
// ============================================================================
struct QuestSelDev {
  sol_shape_t sh;
  sol_kv_t kv;
  const int32_t* r_permille;
  int Tmax, S, splits, split_len, Pstride, Prow;
  const float* q_rot;       // [B][Hq][hd]
  unsigned char* page_mask; // [B][Hkv][Pstride]
  int32_t* list_idx;        // [B][Hkv][Tmax]
  uint32_t* list_row;
  int32_t* kept_cnt;        // [B][Hkv] tokens listed
  int32_t* pages_out;       // optional [B][Hq][Prow]
  int32_t* cnt_out;         // optional [B][Hq]
  int32_t* work_items;
  int32_t* work_ctr;
  int* status;
};

constexpr int QS_THREADS = 256;

// Monotone 64-bit key of a double (larger value, larger key); never the all-ones key, which marks forced pages.
__device__ __forceinline__ unsigned long long quest_key(double s) {
  const long long bits = __double_as_longlong(s + 0.0);  // -0 becomes +0
  const unsigned long long k = bits < 0 ? ~(unsigned long long)bits : (unsigned long long)bits | 0x8000000000000000ull;
  return k == ~0ull ? k - 1 : k;
}

// Exclusive prefix of v over the block (threads in index order) and the block total; `buf` holds one int per warp.
__device__ __forceinline__ int quest_block_scan(int v, int& total, int* buf) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int x = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += x;
  }
  __syncthreads();  // buf may still be read from the previous call
  if (lane == 31) buf[warp] = incl;
  __syncthreads();
  int before = 0, tot = 0;
#pragma unroll
  for (int w = 0; w < QS_THREADS / 32; ++w) {
    const int x = buf[w];
    if (w < warp) before += x;
    tot += x;
  }
  total = tot;
  return before + incl - v;
}

__global__ void __launch_bounds__(QS_THREADS) quest_select_kernel(const QuestSelDev p) {
  extern __shared__ __align__(16) unsigned char qsm[];
  const int kvh = blockIdx.x, b = blockIdx.y, tid = threadIdx.x;
  const int Hkv = p.sh.n_kv_heads, Hq = p.sh.n_q_heads, G = Hq / Hkv, hd = p.sh.head_dim, S = p.S;
  const int bk = b * Hkv + kvh;
  unsigned long long* keys = reinterpret_cast<unsigned long long*>(qsm);        // [Prow]
  double* qpos = reinterpret_cast<double*>(qsm + (size_t)p.Prow * 8);            // [hd]
  double* qneg = qpos + hd;                                                      // [hd]
  unsigned char* mask = reinterpret_cast<unsigned char*>(qneg + hd);             // [Prow]
  __shared__ int hist[256];
  __shared__ int scan_buf[QS_THREADS / 32];
  __shared__ unsigned long long s_prefix;
  __shared__ int s_remaining, s_item0;
  pdl_trigger();
  pdl_wait();

  const int T = min(max(p.kv.seq_lens[b], 0), p.kv.max_pages_per_seq * PAGE);
  const int P = (T + S - 1) / S;
  // pages that hold a forced token: the first n_sink tokens, the last n_window
  const int n_sink = min(max(p.sh.n_sink, 0), T), n_win = min(max(p.sh.n_window, 0), T);
  const int lo_pages = n_sink > 0 ? (n_sink - 1) / S + 1 : 0;    // pages [0, lo_pages)
  const int hi_first = n_win > 0 ? (T - n_win) / S : P;            // pages [hi_first, P)
  const int n_forced = hi_first >= lo_pages ? lo_pages + (P - hi_first) : P;
  const int r = min(max(p.r_permille[b], 0), 1000);
  const int budget = min(T, (int)(((long long)r * T + 999) / 1000));
  const int n_keep = min(P, max((budget + S - 1) / S, n_forced));
  const int32_t* table = p.kv.page_table + (size_t)b * p.kv.max_pages_per_seq;
  const uint16_t* meta = static_cast<const uint16_t*>(p.kv.quest_meta);

  for (int pg = tid; pg < P; pg += QS_THREADS) mask[pg] = 0;

  for (int h = 0; h < G; ++h) {
    const int head = kvh * G + h;
    __syncthreads();  // keys, qpos, qneg of the previous head are not read any more
    for (int d = tid; d < hd; d += QS_THREADS) {
      const double q = (double)p.q_rot[((size_t)b * Hq + head) * hd + d];
      qpos[d] = q >= 0.0 ? fabs(q) : 0.0;
      qneg[d] = q >= 0.0 ? 0.0 : fabs(q);
    }
    __syncthreads();
    // ---- the bound of every page, as a key ----
    for (int pg = tid; pg < P; pg += QS_THREADS) {
      const bool forced = pg < lo_pages || pg >= hi_first;
      unsigned long long key = ~0ull;
      if (!forced) {
        const int tok = pg * S, page = table[tok / PAGE];
        double s = 0.0;
        if (page >= 0 && page < p.kv.num_pages) {
          const uint4* mp = reinterpret_cast<const uint4*>(meta + quest_meta_offset(page, kvh, (tok % PAGE) / S, Hkv, S, hd));
          const int pieces = hd / 8;
          for (int c = 0; c < pieces; ++c) {
            const uint4 a = mp[c], m = mp[pieces + c];
            const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, mw[4] = {m.x, m.y, m.z, m.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const int d = c * 8 + 2 * e;
              s += qpos[d] * (double)bf16_lo(aw[e]) + qneg[d] * (double)bf16_lo(mw[e]);
              s += qpos[d + 1] * (double)bf16_hi(aw[e]) + qneg[d + 1] * (double)bf16_hi(mw[e]);
            }
          }
        } else {
          atomicOr(p.status + ST_ERR, ERR_BAD_PAGE);
          s = -INFINITY;
        }
        key = quest_key(s);
      }
      keys[pg] = key;
    }
    // ---- the n_keep-th largest key: eight passes over the key's bytes, most significant first ----
    if (tid == 0) {
      s_prefix = 0ull;
      s_remaining = n_keep;
    }
    for (int pass = 7; pass >= 0 && n_keep < P; --pass) {
      hist[tid] = 0;  // QS_THREADS == 256 bins
      __syncthreads();
      const unsigned long long prefix = s_prefix;
      const int shift = 8 * pass;
      for (int pg = tid; pg < P; pg += QS_THREADS) {
        const unsigned long long k = keys[pg];
        if (pass == 7 || (k >> (shift + 8)) == (prefix >> (shift + 8))) atomicAdd(&hist[(int)((k >> shift) & 255ull)], 1);
      }
      __syncthreads();
      if (tid == 0) {
        int rem = s_remaining, dgt = 255;
        for (; dgt > 0; --dgt) {
          if (hist[dgt] >= rem) break;
          rem -= hist[dgt];
        }
        s_prefix = prefix | ((unsigned long long)dgt << shift);
        s_remaining = rem;
      }
      __syncthreads();
    }
    __syncthreads();
    const unsigned long long tau = s_prefix;  // keys above tau are kept, and the first s_remaining keys equal to it
    const int n_equal = s_remaining;
    const bool all_pages = n_keep >= P;
    // ---- mark the head's pages; write its ascending page list ----
    int seen_equal = 0, written = 0;
    int32_t* out = p.pages_out ? p.pages_out + ((size_t)b * Hq + head) * p.Prow : nullptr;
    for (int base = 0; base < P; base += QS_THREADS) {
      const int pg = base + tid;
      const unsigned long long k = pg < P ? keys[pg] : 0ull;
      const bool eq = pg < P && !all_pages && k == tau;
      int tot_eq;
      const int rank_eq = quest_block_scan(eq ? 1 : 0, tot_eq, scan_buf);
      const bool sel = pg < P && (all_pages || k > tau || (eq && seen_equal + rank_eq < n_equal));
      seen_equal += tot_eq;
      int tot_sel;
      const int pos = quest_block_scan(sel ? 1 : 0, tot_sel, scan_buf);
      if (sel) {
        mask[pg] |= (unsigned char)(1u << h);
        if (out) out[written + pos] = pg;
      }
      written += tot_sel;
    }
    if (tid == 0 && p.cnt_out) p.cnt_out[(size_t)b * Hq + head] = written;
  }
  __syncthreads();

  // ---- the row's token list: every token of a page some head keeps, ascending ----
  const size_t row = (size_t)bk * p.Tmax;
  int n_list = 0;
  for (int base = 0; base < P; base += QS_THREADS) {
    const int pg = base + tid;
    const unsigned char m = pg < P ? mask[pg] : 0;
    if (pg < P) p.page_mask[(size_t)bk * p.Pstride + pg] = m;
    const int ntok = m ? min(S, T - pg * S) : 0;
    int tot;
    const int off = quest_block_scan(ntok, tot, scan_buf);
    if (ntok > 0) {
      const int tok = pg * S, page = table[tok / PAGE];
      const bool ok = page >= 0 && page < p.kv.num_pages;
      const uint32_t r0 = (uint32_t)((page * Hkv + kvh) * PAGE + (tok % PAGE));
      for (int j = 0; j < ntok; ++j) {
        p.list_idx[row + n_list + off + j] = tok + j;
        p.list_row[row + n_list + off + j] = ok ? r0 + j : 0xffffffffu;
      }
    }
    n_list += tot;
  }
  if (tid == 0) p.kept_cnt[bk] = n_list;

  // Pass-2 work items of this (sequence, kv-head): runs of `cpi` chunks of split_len listed tokens (at least one
  // item, so that the output is always written)
  const int cpi = p.work_ctr[WC_CPI];
  const int chunks = max(1, (n_list + p.split_len - 1) / p.split_len);
  const int ns_items = (chunks + cpi - 1) / cpi;
  __syncthreads();
  if (tid == 0) s_item0 = atomicAdd(p.work_ctr + WC_ITEMS, ns_items);
  __syncthreads();
  const int item0 = s_item0;
  for (int i = tid; i < ns_items; i += QS_THREADS) {
    p.work_items[2 * (item0 + i)] = bk * p.splits + i * cpi;  // first chunk of the item
    p.work_items[2 * (item0 + i) + 1] = n_list;
  }
}

// ============================================================================
// quest_logits
// ============================================================================
struct QuestLogitDev {
  sol_kv_t kv;
  int Hq, Hkv, G, hd, Tmax, S, Pstride;
  const float* q_rot;
  const int32_t* list_idx;
  const uint32_t* list_row;
  const int32_t* kept_cnt;
  const unsigned char* page_mask;
  float* logits;  // [B][Hkv][Tmax][G]
};

constexpr int QL_THREADS = 256;
constexpr int QL_CHUNK = 1024;  // listed tokens per CTA

template <int HD, int GMAX>
__global__ void __launch_bounds__(QL_THREADS) quest_logits_kernel(const QuestLogitDev p) {
  constexpr int LPT = HD / 8;     // lanes per token: 16 bytes of the key row each
  constexpr int TPW = 32 / LPT;   // tokens per warp and pass
  const int kvh = blockIdx.y, b = blockIdx.z, bk = b * p.Hkv + kvh;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, sub = lane % LPT;
  pdl_trigger();
  pdl_wait();
  const int cnt = p.kept_cnt[bk];
  const int n0 = blockIdx.x * QL_CHUNK;
  if (n0 >= cnt) return;
  const int n1 = min(cnt, n0 + QL_CHUNK);
  float q[GMAX][8];
#pragma unroll
  for (int h = 0; h < GMAX; ++h) {
#pragma unroll
    for (int e = 0; e < 8; ++e) q[h][e] = h < p.G ? p.q_rot[((size_t)b * p.Hq + kvh * p.G + h) * HD + sub * 8 + e] : 0.f;
  }
  const size_t row = (size_t)bk * p.Tmax;
  const uint16_t* kp = static_cast<const uint16_t*>(p.kv.k_pool);
  for (int nb = n0 + warp * TPW; nb < n1; nb += (QL_THREADS / 32) * TPW) {
    const int n = nb + lane / LPT;
    const bool have = n < n1;
    int j = 0;
    uint32_t r = 0xffffffffu;
    if (have) {
      j = p.list_idx[row + n];
      r = p.list_row[row + n];
    }
    float dot[GMAX];
#pragma unroll
    for (int h = 0; h < GMAX; ++h) dot[h] = 0.f;
    if (r != 0xffffffffu) {
      const uint4 kv8 = *reinterpret_cast<const uint4*>(kp + (size_t)r * HD + sub * 8);
      const uint32_t w[4] = {kv8.x, kv8.y, kv8.z, kv8.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float k0 = bf16_lo(w[e]), k1 = bf16_hi(w[e]);
#pragma unroll
        for (int h = 0; h < GMAX; ++h) dot[h] = fmaf(q[h][2 * e + 1], k1, fmaf(q[h][2 * e], k0, dot[h]));
      }
    }
#pragma unroll
    for (int h = 0; h < GMAX; ++h) {
#pragma unroll
      for (int o = 1; o < LPT; o <<= 1) dot[h] += __shfl_xor_sync(0xffffffffu, dot[h], o);
    }
    if (have && sub == 0) {
      const unsigned m = r != 0xffffffffu ? p.page_mask[(size_t)bk * p.Pstride + j / p.S] : 0u;
      float* dst = p.logits + (row + j) * p.G;
#pragma unroll
      for (int h = 0; h < GMAX; ++h)
        if (h < p.G) dst[h] = ((m >> h) & 1u) ? dot[h] : -INFINITY;
    }
  }
}

void launch_quest_selection(const AttnArgs& a, cudaStream_t st) {
  const sol_shape_t& sh = a.shape;
  const int Hq = sh.n_q_heads, Hkv = sh.n_kv_heads, hd = sh.head_dim, G = Hq / Hkv, S = sh.quest_page_size;
  const int Tmax = a.kv.max_pages_per_seq * PAGE;

  QuestSelDev d;
  d.sh = sh; d.kv = a.kv; d.r_permille = a.r_permille; d.Tmax = Tmax; d.S = S; d.splits = a.splits;
  d.split_len = attn_split_len(hd); d.Pstride = Tmax / 4; d.Prow = Tmax / S;
  d.q_rot = a.q_rot; d.page_mask = a.page_mask; d.list_idx = a.list_idx; d.list_row = a.kept_row;
  d.kept_cnt = a.kept_cnt; d.pages_out = a.quest_pages_out; d.cnt_out = a.quest_cnt_out;
  d.work_items = a.work_items; d.work_ctr = a.work_ctr; d.status = a.status;
  const int smem = d.Prow * 8 + 2 * hd * 8 + d.Prow + 16;
  ensure_dynamic_smem(reinterpret_cast<const void*>(&quest_select_kernel), smem);
  SOL_LAUNCH("quest_select", quest_select_kernel, dim3(Hkv, a.B), dim3(QS_THREADS), smem, st, d);

  QuestLogitDev l;
  l.kv = a.kv; l.Hq = Hq; l.Hkv = Hkv; l.G = G; l.hd = hd; l.Tmax = Tmax; l.S = S; l.Pstride = d.Pstride;
  l.q_rot = a.q_rot; l.list_idx = a.list_idx; l.list_row = a.kept_row; l.kept_cnt = a.kept_cnt;
  l.page_mask = a.page_mask; l.logits = a.logits;
  const dim3 grid((Tmax + QL_CHUNK - 1) / QL_CHUNK, Hkv, a.B);
  if (hd == 64) {
    if (G <= 4) SOL_LAUNCH("quest_logits", (quest_logits_kernel<64, 4>), grid, dim3(QL_THREADS), 0, st, l);
    else SOL_LAUNCH("quest_logits", (quest_logits_kernel<64, 8>), grid, dim3(QL_THREADS), 0, st, l);
  } else {
    if (G <= 4) SOL_LAUNCH("quest_logits", (quest_logits_kernel<128, 4>), grid, dim3(QL_THREADS), 0, st, l);
    else SOL_LAUNCH("quest_logits", (quest_logits_kernel<128, 8>), grid, dim3(QL_THREADS), 0, st, l);
  }
}

}  // namespace sol
