// The paper's own token sparsity: Quest page selection per query head (appendix on efficiency actions,
// "Token sparsity via Quest": "Budgeted token selection", "Quest masking in LLaMA attention", "Granularity").
//
//   quest_meta    per block of S tokens of a cache page: the per-dimension maximum of its keys (m+) and the
//                 negated minimum (m-), as bf16 (extrema of bf16 numbers are bf16 numbers).  For every page of
//                 the sequences (after a prefill) or for the pages of a refreshed span.
//   quest_query   per (sequence, kv-head): the extrema of the block of the key a decode step appended, the G
//                 heads' queries split by sign as a tensor-core operand, their 1-norms; the sequences by length.
//   quest_score   the bound q_pos.m+ + q_neg.m- of every page for every query head, in float32, as sortable keys,
//                 with a bound of its rounding error (a page costs 2/S of its keys' bytes), on the tensor cores.
//   quest_select  one CTA per (sequence, query head): an exact selection of the head's ceil(b_t / S) best pages: radix
//                 select on the float32 keys, float64 bounds for the few pages within the error window of the
//                 threshold (forced pages first, ties to the lower page); a byte per page: kept or not.
//   quest_list    one CTA per (sequence, kv-head): the union of the group's heads' pages as the row's token list
//                 and a byte per page that says which heads keep it.
// The attention over the lists (keys and values read only for pages in the union, the paper's additive mask for
// the heads that did not keep a page) is sol_quest_attend.cu.
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
  int Hkv, hd, S, all;  // all: 0 the block of the newest token, 1 every page, 2 the pages of the last n_tail tokens
  int n_tail;
  int* status;
};

constexpr int QM_THREADS = 128;

// The extrema of the blocks of one cache page of (sequence b, kv-head kvh): all its blocks, or only the one that
// holds the newest token.  For a block of QM_THREADS threads.
__device__ __forceinline__ void quest_meta_page(const QuestMetaDev& p, int b, int kvh, int lp_all) {
  const int T = min(max(p.kv.seq_lens[b], 0), p.kv.max_pages_per_seq * PAGE);
  if (T <= 0) return;
  const int lp = p.all == 1 ? lp_all : (T - 1) / PAGE - (p.all == 2 ? lp_all : 0);  // logical cache page
  if (lp < 0 || lp * PAGE >= T) return;
  if (p.all == 2 && (lp + 1) * PAGE <= T - p.n_tail) return;  // wholly before the tail
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

__global__ void __launch_bounds__(QM_THREADS) quest_meta_kernel(const QuestMetaDev p) {
  pdl_trigger();
  pdl_wait();  // the newest key is written by the kernel before this one
  quest_meta_page(p, blockIdx.z, blockIdx.y, blockIdx.x);
}

void launch_quest_meta_tail(const sol_shape_t& sh, const sol_kv_t& kv, int B, int n_tail, int* status, cudaStream_t st) {
  QuestMetaDev d;
  d.kv = kv; d.Hkv = sh.n_kv_heads; d.hd = sh.head_dim; d.S = sh.quest_page_size; d.all = 2; d.n_tail = n_tail; d.status = status;
  const dim3 grid((n_tail + PAGE - 1) / PAGE + 1, sh.n_kv_heads, B);  // n_tail tokens touch that many cache pages at most
  SOL_LAUNCH("quest_meta", quest_meta_kernel, grid, dim3(QM_THREADS), 0, st, d);
}

void launch_quest_meta(const sol_shape_t& sh, const sol_kv_t& kv, int B, bool all, int* status, cudaStream_t st) {
  QuestMetaDev d;
  d.kv = kv; d.Hkv = sh.n_kv_heads; d.hd = sh.head_dim; d.S = sh.quest_page_size; d.all = all ? 1 : 0; d.n_tail = 0; d.status = status;
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
  int Tmax, S, Pstride, Prow;
  const float* q_rot;       // [B][Hq][hd]
  const uint32_t* keys;     // [B][Hq][Prow] float32 bounds as keys (quest_score)
  const uint32_t* err;      // [B][Hq] largest error bound of the row, float bits
  const int* order;         // [B] the sequences, longest first (quest_query)
  unsigned char* hmask;     // [B][Hq][Prow] 1 = the head keeps the page (quest_select -> quest_list)
  unsigned char* page_mask; // [B][Hkv][Pstride]
  int32_t* list_idx;        // [B][Hkv][Tmax]
  uint32_t* list_row;
  int32_t* kept_cnt;        // [B][Hkv] tokens listed
  int32_t* pages_out;       // optional [B][Hq][Prow]
  int32_t* cnt_out;         // optional [B][Hq]
  int* status;
};

constexpr int QS_THREADS = 256;

// Monotone 64-bit key of a double (larger value, larger key); never the all-ones key, which marks forced pages.
__device__ __forceinline__ unsigned long long quest_key(double s) {
  const long long bits = __double_as_longlong(s + 0.0);  // -0 becomes +0
  const unsigned long long k = bits < 0 ? ~(unsigned long long)bits : (unsigned long long)bits | 0x8000000000000000ull;
  return k == ~0ull ? k - 1 : k;
}

// Exclusive prefix of v over a block of NTHR threads (in index order) and the block total; `buf` holds one int per warp.
template <int NTHR = 256>
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
  for (int w = 0; w < NTHR / 32; ++w) {
    const int x = buf[w];
    if (w < warp) before += x;
    tot += x;
  }
  total = tot;
  return before + incl - v;
}

constexpr int QS_CAND_CAP = 1024;  // pages per head whose bound is taken again in float64

// Monotone 32-bit key of a float; never the all-ones key (forced pages).
__device__ __forceinline__ uint32_t quest_key32(float s) {
  const uint32_t bits = __float_as_uint(s + 0.0f);
  const uint32_t k = (bits & 0x80000000u) ? ~bits : bits | 0x80000000u;
  return k == 0xffffffffu ? k - 1 : k;
}
__device__ __forceinline__ float quest_key32_value(uint32_t k) {
  return __uint_as_float((k & 0x80000000u) ? k & 0x7fffffffu : ~k);
}

// The `need`-th largest of n keys in shared memory (0 < need <= n): byte-wise radix passes, most significant
// first.  Leaves the key in *s_prefix and, in *s_remaining, how many keys EQUAL to it belong to the `need`
// largest (keys above it all do).  The lanes of a warp with the same digit add to the histogram once: the
// scores of a row share their upper bytes, so most keys of a pass fall into one or two bins.
template <typename KeyT, int NTHR>
__device__ __forceinline__ void quest_radix_threshold(const KeyT* keys, int n, int need, int* hist,
                                                      unsigned long long* s_prefix, int* s_remaining) {
  const int tid = threadIdx.x;
  if (tid == 0) {
    *s_prefix = 0ull;
    *s_remaining = need;
  }
  for (int pass = (int)sizeof(KeyT) - 1; pass >= 0; --pass) {
    for (int i = tid; i < 256; i += NTHR) hist[i] = 0;
    __syncthreads();
    const unsigned long long prefix = *s_prefix;
    const int shift = 8 * pass;
    const bool top = pass == (int)sizeof(KeyT) - 1;
    for (int base = 0; base < n; base += NTHR) {
      const int i = base + tid;
      const unsigned long long k = i < n ? (unsigned long long)keys[i] : 0ull;
      const bool in = i < n && (top || (k >> (shift + 8)) == (prefix >> (shift + 8)));
      // Most keys share their upper bytes and few survive to the lower ones, so a warp's 32 keys are mostly all in
      // one bin (one addition for the warp) or nearly all out (a handful of additions that cannot collide much);
      // only a mixed warp pays for the match.
      const unsigned act = __ballot_sync(0xffffffffu, in);
      if (act == 0u) continue;
      const int dgt = in ? (int)((k >> shift) & 255ull) : 256 + (tid & 31);  // lanes without a key match nobody
      if (__popc(act) <= 4) {
        if (in) atomicAdd(&hist[dgt], 1);
        continue;
      }
      const int lead = __ffs(act) - 1;
      const int d0 = __shfl_sync(0xffffffffu, dgt, lead);
      if (__ballot_sync(0xffffffffu, in && dgt == d0) == act) {
        if ((tid & 31) == lead) atomicAdd(&hist[d0], __popc(act));
        continue;
      }
      const unsigned same = __match_any_sync(0xffffffffu, dgt);
      if (in && (tid & 31) == __ffs(same) - 1) atomicAdd(&hist[dgt], __popc(same));
    }
    __syncthreads();
    if (tid < 32) {
      // the digit whose bin holds the rem-th key counted from the top: lane l owns bins 255 - 8 l .. 248 - 8 l
      const int rem0 = *s_remaining;
      int mine = 0;
#pragma unroll
      for (int q = 0; q < 8; ++q) mine += hist[255 - 8 * tid - q];
      int incl = mine;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int x = __shfl_up_sync(0xffffffffu, incl, o);
        if (tid >= o) incl += x;
      }
      const int before = incl - mine;  // keys in the bins above this lane's
      if (before < rem0 && rem0 <= incl) {
        int rem = rem0 - before, dgt = 255 - 8 * tid;
        for (int q = 0; q < 7; ++q, --dgt) {
          if (hist[dgt] >= rem) break;
          rem -= hist[dgt];
        }
        *s_prefix = prefix | ((unsigned long long)dgt << shift);
        *s_remaining = rem;
      }
    }
    __syncthreads();
  }
}

struct QuestScoreDev {
  sol_shape_t sh;
  sol_kv_t kv;
  int S, Prow, B;
  const float* q_rot;  // [B][Hq][hd]
  uint32_t* keys;      // [B][Hq][Prow]
  uint32_t* err;       // [B][Hq] float bits, zeroed by quest_query_kernel
  uint16_t* qsplit;    // [B][Hkv][ceil(G / 4) * 16][2 hd] bf16: the sign-split queries as an operand
  float* l1;           // [B][Hq]: |q|_1
  int* order;          // [B]: the sequences, longest first
  int update_meta;     // 1: quest_query_kernel first takes the extrema of the block with the step's new key
  int* status;
};

// ---- the pages' bounds on the tensor cores ----
// A page's extrema are one row of 2 hd bf16 numbers (m+, then -m-), and the bound is its dot product with the
// query split by sign, [max(q, 0) ; max(-q, 0)]: the scoring pass over again with the extrema as keys.
//
// quest_query_kernel, a CTA per (sequence, kv-head): the G heads' sign-split queries, each as three bf16 parts
// (exact to 2^-24), laid out as the N side of m16n8k16 (head t of a group of four: hi in row 2t, mid in row
// 2t + 1, lo in row 8 + 2t of 16 rows of 2 hd), the heads' |q|_1, and the row's error bounds reset to zero.
//
// quest_score_mma_kernel: a warp takes 16 consecutive pages of a (sequence, kv-head) as the M side (their rows
// come by bulk copies, one per cache page they lie in; a lane each, so that the table look-ups go side by side)
// and reads the N side's fragments from the operand above while the rows travel.  Units of 64 pages are numbered
// along the batch.  Error bound of a row's scores: (terms + 2) 2^-24 |q|_1 max|m| for the float32 sums plus
// 2^-23 |q|_1 max|m| for the split, with max|m| over the row's extrema (taken from the fragments on the way).
// (Building the operand in shared memory inside the scoring kernel, once per (sequence, kv-head) a CTA met, took
// 39 us on the ragged batch where this takes less: the build and its barriers stood between the units.)
constexpr int QSM_WARPS = 4;
constexpr int QQ_THREADS = 128;

__global__ void __launch_bounds__(QQ_THREADS) quest_query_kernel(const QuestScoreDev p) {
  extern __shared__ __align__(16) unsigned char qqsm[];
  uint16_t* qs = reinterpret_cast<uint16_t*>(qqsm);  // [HG * 16][2 hd]
  __shared__ float s_l1[8];
  const int kvh = blockIdx.x, b = blockIdx.y, tid = threadIdx.x, lane = tid & 31;
  const int Hkv = p.sh.n_kv_heads, Hq = p.sh.n_q_heads, G = Hq / Hkv, hd = p.sh.head_dim, HD2 = 2 * hd;
  const int rows = ((G + 3) / 4) * 16;
  pdl_trigger();
  for (int i = tid * 8; i < rows * HD2; i += QQ_THREADS * 8) *reinterpret_cast<uint4*>(qs + i) = make_uint4(0u, 0u, 0u, 0u);
  if (tid < 8) s_l1[tid] = 0.f;
  __syncthreads();
  pdl_wait();  // the rotated queries come from the kernel before; the scratch below may still be read until then
  if (p.update_meta) {  // the step's new key is in the cache: the extrema of its block
    QuestMetaDev m;
    m.kv = p.kv; m.Hkv = Hkv; m.hd = hd; m.S = p.S; m.all = 0; m.n_tail = 0; m.status = p.status;
    quest_meta_page(m, b, kvh, 0);
  }
  for (int i = tid; i < G * hd; i += QQ_THREADS) {
    const int gi = i / hd, d = i - gi * hd;
    const float q = p.q_rot[((size_t)b * Hq + kvh * G + gi) * hd + d];
    const float v = fabsf(q);
    const int e = q >= 0.f ? d : hd + d;  // the half of the operand row that meets m+ or -m-
    const uint16_t hi = f2bf(v);
    const float r1 = v - bf2f(hi);
    const uint16_t mid = f2bf(r1);
    uint16_t* base = qs + (size_t)((gi >> 2) * 16) * HD2;
    const int tt = gi & 3;
    base[(2 * tt) * HD2 + e] = hi;
    base[(2 * tt + 1) * HD2 + e] = mid;
    base[(8 + 2 * tt) * HD2 + e] = f2bf(r1 - bf2f(mid));
    float sum = v;  // a warp's 32 dimensions belong to one head (head_dim is a multiple of 32)
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    if (lane == 0) atomicAdd(&s_l1[gi], sum);
  }
  __syncthreads();
  uint4* dst = reinterpret_cast<uint4*>(p.qsplit + (size_t)(b * Hkv + kvh) * rows * HD2);
  for (int i = tid; i < rows * HD2 / 8; i += QQ_THREADS) dst[i] = reinterpret_cast<const uint4*>(qs)[i];
  if (tid < G) {
    p.l1[(size_t)b * Hq + kvh * G + tid] = s_l1[tid];
    p.err[(size_t)b * Hq + kvh * G + tid] = 0u;
  }
  // the first CTA also ranks the sequences by length: the selection starts its longest rows first, so that none
  // of them begins when the others are about to end
  if (blockIdx.x == 0 && blockIdx.y == 0 && tid < p.B) {
    const int mine = p.kv.seq_lens[tid];
    int rank = 0;
    for (int j = 0; j < p.B; ++j) {
      const int other = p.kv.seq_lens[j];
      rank += (other > mine || (other == mine && j < tid)) ? 1 : 0;
    }
    p.order[rank] = tid;
  }
}

template <int HD2, int HG>
__global__ void __launch_bounds__(QSM_WARPS * 32) quest_score_mma_kernel(const QuestScoreDev p) {
  extern __shared__ __align__(128) unsigned char qssm[];
  constexpr int TILE_BYTES = 16 * HD2 * 2;
  uint64_t* bars = reinterpret_cast<uint64_t*>(qssm + QSM_WARPS * TILE_BYTES);
  __shared__ int s_cum[QSM_WARPS * 32 + 1], s_wsum[QSM_WARPS];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, tid = threadIdx.x;
  const int Hkv = p.sh.n_kv_heads, Hq = p.sh.n_q_heads, G = Hq / Hkv, hd = HD2 / 2, S = p.S;
  const int B = p.B;
  pdl_trigger();
  int my_incl = 0;
  if (tid < B) {
    const int T = min(max(p.kv.seq_lens[tid], 0), p.kv.max_pages_per_seq * PAGE);
    my_incl = ((T + S - 1) / S + 16 * QSM_WARPS - 1) / (16 * QSM_WARPS);
  }
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int x = __shfl_up_sync(0xffffffffu, my_incl, o);
    if (lane >= o) my_incl += x;
  }
  if (lane == 31) s_wsum[warp] = my_incl;
  if (tid == 0) {
    for (int i = 0; i < QSM_WARPS; ++i) mbar_init(&bars[i], 1);
    fence_mbar_init();
    s_cum[0] = 0;
  }
  __syncthreads();
  for (int w = 0; w < warp; ++w) my_incl += s_wsum[w];
  s_cum[tid + 1] = my_incl;
  __syncthreads();
  const int n_units = s_cum[B] * Hkv;
  if ((int)blockIdx.x >= n_units) return;
  pdl_wait();
  const int g = lane >> 2, t = lane & 3;
  constexpr int KS = HD2 / 32;
  const int npk = PAGE / S;                        // pages per cache page
  const int rpc = npk < 16 ? npk : 16;             // rows per bulk copy
  uint32_t phase = 0;
  bool dead = false;
#pragma unroll 1
  for (int u = blockIdx.x; u < n_units; u += gridDim.x) {
    const int key = u / Hkv;
    const int b = __syncthreads_count(tid < B && my_incl <= key);
    const int first = s_cum[b], n_groups = s_cum[b + 1] - first;
    const int rem = u - first * Hkv;
    const int kvh = rem / n_groups, grp = rem - kvh * n_groups;
    const int T = min(max(p.kv.seq_lens[b], 0), p.kv.max_pages_per_seq * PAGE);
    const int P = (T + S - 1) / S;
    const int pg0 = (grp * QSM_WARPS + warp) * 16;
    if (dead || pg0 >= P) continue;
    const int n_sink = min(max(p.sh.n_sink, 0), T), n_win = min(max(p.sh.n_window, 0), T);
    const int lo_pages = n_sink > 0 ? (n_sink - 1) / S + 1 : 0;
    const int hi_first = n_win > 0 ? (T - n_win) / S : P;
    unsigned char* tile = qssm + warp * TILE_BYTES;
    const int nrow = min(16, P - pg0);
    if (lane == 0) mbar_expect_tx(&bars[warp], nrow * HD2 * 2);
    __syncwarp();
    {
      const int r0 = lane * rpc;
      if (r0 < nrow) {
        const int tok = (pg0 + r0) * S, page = p.kv.page_table[(size_t)b * p.kv.max_pages_per_seq + tok / PAGE];
        const bool ok = page >= 0 && page < p.kv.num_pages;
        if (!ok) atomicOr(p.status + ST_ERR, ERR_BAD_PAGE);
        const int n = min(rpc, nrow - r0);
        bulk_g2s(tile + (size_t)r0 * HD2 * 2,
                 static_cast<const uint16_t*>(p.kv.quest_meta) + quest_meta_offset(ok ? page : 0, kvh, (tok % PAGE) / S, Hkv, S, hd),
                 n * HD2 * 2, &bars[warp]);
      }
    }
    const uint16_t* qop = p.qsplit + (size_t)(b * Hkv + kvh) * (HG * 16) * HD2;
    uint4 qf[KS][2];
#pragma unroll
    for (int sx = 0; sx < KS; ++sx) {
      qf[sx][0] = __ldg(reinterpret_cast<const uint4*>(qop + (size_t)g * HD2 + sx * 32 + t * 8));
      qf[sx][1] = __ldg(reinterpret_cast<const uint4*>(qop + (size_t)(8 + g) * HD2 + sx * 32 + t * 8));
    }
    if (!mbar_wait(&bars[warp], phase, p.status)) {
      dead = true;
      continue;
    }
    phase ^= 1;
    const uint32_t tb = smem_u32(tile);
    const bool v0 = g < nrow, v1 = g + 8 < nrow;  // rows beyond the sequence's pages hold whatever the tile held before
    uint4 ka[KS][2];
    uint32_t am = 0u;  // largest magnitudes of this lane's elements, two bf16 patterns side by side
#pragma unroll
    for (int sx = 0; sx < KS; ++sx) {
      ka[sx][0] = v0 ? lds128(tb + g * (HD2 * 2) + (sx * 32 + t * 8) * 2) : make_uint4(0u, 0u, 0u, 0u);
      ka[sx][1] = v1 ? lds128(tb + (g + 8) * (HD2 * 2) + (sx * 32 + t * 8) * 2) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
      for (int x = 0; x < 2; ++x) {
        am = __vmaxu2(am, ka[sx][x].x & 0x7fff7fffu);
        am = __vmaxu2(am, ka[sx][x].y & 0x7fff7fffu);
        am = __vmaxu2(am, ka[sx][x].z & 0x7fff7fffu);
        am = __vmaxu2(am, ka[sx][x].w & 0x7fff7fffu);
      }
    }
#pragma unroll
    for (int hg = 0; hg < HG; ++hg) {
      float d0[4] = {0.f, 0.f, 0.f, 0.f}, d1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int sx = 0; sx < KS; ++sx) {
        mma_bf16(d0, ka[sx][0].x, ka[sx][1].x, ka[sx][0].y, ka[sx][1].y, qf[sx][0].x, qf[sx][0].y);
        mma_bf16(d0, ka[sx][0].z, ka[sx][1].z, ka[sx][0].w, ka[sx][1].w, qf[sx][0].z, qf[sx][0].w);
        mma_bf16(d1, ka[sx][0].x, ka[sx][1].x, ka[sx][0].y, ka[sx][1].y, qf[sx][1].x, qf[sx][1].y);
        mma_bf16(d1, ka[sx][0].z, ka[sx][1].z, ka[sx][0].w, ka[sx][1].w, qf[sx][1].z, qf[sx][1].w);
      }
      if (hg + 1 < HG) {  // the next four heads' fragments (more than four heads per kv-head is the rare case)
#pragma unroll
        for (int sx = 0; sx < KS; ++sx) {
          qf[sx][0] = __ldg(reinterpret_cast<const uint4*>(qop + (size_t)((hg + 1) * 16 + g) * HD2 + sx * 32 + t * 8));
          qf[sx][1] = __ldg(reinterpret_cast<const uint4*>(qop + (size_t)((hg + 1) * 16 + 8 + g) * HD2 + sx * 32 + t * 8));
        }
      }
      const float s0 = d0[0] + (d0[1] + d1[0]);  // page pg0 + g
      const float s1 = d0[2] + (d0[3] + d1[2]);  // page pg0 + g + 8
      const int head = hg * 4 + t;
      if (head < G) {
        uint32_t* dst = p.keys + ((size_t)b * Hq + kvh * G + head) * p.Prow;
        const int pa = pg0 + g, pb = pg0 + g + 8;
        if (v0) dst[pa] = (pa < lo_pages || pa >= hi_first) ? 0xffffffffu : quest_key32(s0);
        if (v1) dst[pb] = (pb < lo_pages || pb >= hi_first) ? 0xffffffffu : quest_key32(s1);
      }
    }
    am = max(am & 0xffffu, am >> 16);
    am = __reduce_max_sync(0xffffffffu, am);
    if (lane < G) {
      const float amax = __uint_as_float(am << 16);
      const float w = ((float)(3 * HD2 + 2) * 5.9604644775390625e-08f + 1.1920928955078125e-07f) * 1.001f *
                      p.l1[(size_t)b * Hq + kvh * G + lane] * amax;
      atomicMax(p.err + (size_t)b * Hq + kvh * G + lane, __float_as_uint(w));  // non-negative floats order like their bits
    }
    __syncwarp();
  }
}

template <int HD2, int HG>
static void launch_quest_score_mma(const QuestScoreDev& d, int Hkv, cudaStream_t st) {
  const int smem = QSM_WARPS * 16 * HD2 * 2 + QSM_WARPS * 8 + 32;
  const long long upper = (long long)((d.Prow + 16 * QSM_WARPS - 1) / (16 * QSM_WARPS)) * Hkv * d.B;
  const long long resident = (long long)sm_count() * (HD2 == 128 ? 24 : 12);  // twice what the shared memory lets stay on an SM
  ensure_dynamic_smem(reinterpret_cast<const void*>(&quest_score_mma_kernel<HD2, HG>), smem);
  SOL_LAUNCH("quest_score", (quest_score_mma_kernel<HD2, HG>), dim3((unsigned)(upper < resident ? upper : resident)), dim3(QSM_WARPS * 32), smem, st, d);
}

// Selection of one query head, in two precisions.  The bound of every page is first summed in float32 (two
// fused multiply-adds per dimension: the score and the sum of the terms' magnitudes, which bounds the rounding
// error of the score); the n_keep-th largest float32 score tau is found by radix select; with w the largest
// error bound of the row, a page above tau + 2 w is certainly among the n_keep best exact scores and one below
// tau - 2 w certainly is not (the k-th largest of a set of numbers moves by at most w when each number moves by
// at most w).  Only the pages in between are scored again in float64 (the widening of the extrema to float64
// is the slow instruction: all pages in float64 took 400 us for a row of 2048 pages) and the missing ones are
// taken from them by a second radix select on the 64-bit keys, ties to the lower page.
// QSEL_THREADS: 128 where a row has up to 4096 pages (a row of the median sequence has 256: eight warps mostly
// waited for each other), 256 for longer rows (small page sizes).
constexpr int QSEL_RANK_MAX = 256;  // candidates up to which ranking by counting beats a second radix select

template <int QSEL_THREADS>
__global__ void __launch_bounds__(QSEL_THREADS) quest_select_kernel(const QuestSelDev p) {
  extern __shared__ __align__(16) unsigned char qsm[];
  const int tid = threadIdx.x, head = blockIdx.x;  // one query head per CTA
  const int Hkv = p.sh.n_kv_heads, Hq = p.sh.n_q_heads, G = Hq / Hkv, hd = p.sh.head_dim, S = p.S;
  const int kvh = head / G;
  unsigned long long* cand_key = reinterpret_cast<unsigned long long*>(qsm);             // [QS_CAND_CAP]
  float* qf = reinterpret_cast<float*>(cand_key + QS_CAND_CAP);                           // [hd] the head's query (16-byte aligned)
  uint32_t* keys = reinterpret_cast<uint32_t*>(qf + hd);                                  // [Prow]
  int* cand_idx = reinterpret_cast<int*>(keys + p.Prow);                                  // [QS_CAND_CAP]
  unsigned char* cand_sel = reinterpret_cast<unsigned char*>(cand_idx + QS_CAND_CAP);     // [QS_CAND_CAP]
  unsigned char* pflag = cand_sel + QS_CAND_CAP;                                          // [Prow] 1 = the head keeps the page
  __shared__ int hist[256];
  __shared__ int scan_buf[QSEL_THREADS / 32];
  __shared__ unsigned long long s_prefix;
  __shared__ int s_remaining, s_ncand, s_cin;
  pdl_trigger();
  pdl_wait();
  const int b = p.order[blockIdx.y];  // longest sequences first

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
  auto page_meta = [&](int pg, bool& ok) {
    const int tok = pg * S, page = table[tok / PAGE];
    ok = page >= 0 && page < p.kv.num_pages;
    return reinterpret_cast<const uint4*>(meta + quest_meta_offset(ok ? page : 0, kvh, (tok % PAGE) / S, Hkv, S, hd));
  };

  for (int i = tid; i < hd; i += QSEL_THREADS) qf[i] = p.q_rot[((size_t)b * Hq + head) * hd + i];
  {  // the float32 keys of this head's bounds (quest_score)
    const uint32_t* src = p.keys + ((size_t)b * Hq + head) * p.Prow;
    for (int pg = tid; pg < P; pg += QSEL_THREADS) keys[pg] = src[pg];
  }
  if (tid == 0) {
    s_ncand = 0;
    s_cin = 0;
  }
  __syncthreads();
  const bool all_pages = n_keep >= P;
  uint32_t tau32 = 0u;
  int rem32 = 0;
  if (!all_pages && n_keep > 0) {
    quest_radix_threshold<uint32_t, QSEL_THREADS>(keys, P, n_keep, hist, &s_prefix, &s_remaining);
    tau32 = (uint32_t)s_prefix;
    rem32 = s_remaining;
  }
  __syncthreads();  // s_prefix, s_remaining are rewritten below
  const float w = __uint_as_float(p.err[(size_t)b * Hq + head]);  // the row's largest error bound for this head
  const bool only_forced = tau32 == 0xffffffffu || n_keep == 0;  // the budget is met by the forced pages alone
  const double tau = only_forced || all_pages ? 0.0 : (double)quest_key32_value(tau32);
  const double hi = tau + 2.002 * (double)w, lo = tau - 2.002 * (double)w;
  auto classify = [&](int pg, bool& in, bool& cand) {
    const uint32_t k = keys[pg];
    const double v = (double)quest_key32_value(k);
    in = k == 0xffffffffu || v > hi;
    cand = !in && v >= lo;
  };
  // ---- the pages above hi are kept; those between lo and hi are listed (in no order: the lanes take their
  //      slots by a counter, which spares a block-wide scan per 256 pages) ----
  int n_cand = 0, c_in = 0;
  bool overflow = false;
  if (all_pages || only_forced) {
    for (int pg = tid; pg < P; pg += QSEL_THREADS) pflag[pg] = (all_pages || keys[pg] == 0xffffffffu) ? 1 : 0;
  } else {
    int my_in = 0;
    for (int pg = tid; pg < P; pg += QSEL_THREADS) {
      bool in, cand;
      classify(pg, in, cand);
      my_in += in ? 1 : 0;
      pflag[pg] = in ? 1 : 0;
      if (cand) {
        const int slot = atomicAdd(&s_ncand, 1);
        if (slot < QS_CAND_CAP) cand_idx[slot] = pg;
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) my_in += __shfl_xor_sync(0xffffffffu, my_in, o);
    if ((tid & 31) == 0 && my_in) atomicAdd(&s_cin, my_in);
    __syncthreads();
    n_cand = s_ncand;
    c_in = s_cin;
    overflow = n_cand > QS_CAND_CAP;
    if (overflow && tid == 0) atomicAdd(p.status + ST_TOK_OVERFLOW, 1);
    if (n_cand > QSEL_RANK_MAX && !overflow) {
      // a long list goes through the radix select below, whose tie rule (the lower page first) reads the list
      // in page order: listed again, by ordered scans
      int at = 0;
      for (int base = 0; base < P; base += QSEL_THREADS) {
        const int pg = base + tid;
        bool in = false, cand = false;
        if (pg < P) classify(pg, in, cand);
        int tot;
        const int pos = quest_block_scan<QSEL_THREADS>(cand ? 1 : 0, tot, scan_buf);
        if (cand) cand_idx[at + pos] = pg;
        at += tot;
      }
      __syncthreads();
    }
  }
  const bool refine = !all_pages && !only_forced && !overflow && n_cand > 0;
  if (refine) {
    // ---- exact bounds of the candidates: a group of hd/4 lanes per candidate, one piece of the extrema per
    //      lane, float64 partial sums added up over the group ----
    {
      const int lane = tid & 31, warp = tid >> 5;
      const int LPG = hd / 4, GPW = 32 / LPG, sub = lane % LPG, grp = lane / LPG;
      const bool minus = sub >= hd / 8;
      const int d0 = (minus ? sub - hd / 8 : sub) * 8;
      const float* q = qf + d0;
      const int stride = (QSEL_THREADS / 32) * GPW;
      for (int c0 = 0; c0 < n_cand; c0 += stride) {  // block-uniform trip count
        const int c = c0 + warp * GPW + grp;
        bool ok = true;
        uint4 piece = make_uint4(0u, 0u, 0u, 0u);
        if (c < n_cand) {
          const uint4* mp = page_meta(cand_idx[c], ok);
          if (ok) piece = mp[sub];
        }
        const uint32_t w4[4] = {piece.x, piece.y, piece.z, piece.w};
        double sd = 0.0;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float q0 = q[2 * e], q1 = q[2 * e + 1];
          if ((q0 < 0.f) == minus) sd = fma((double)fabsf(q0), (double)bf16_lo(w4[e]), sd);
          if ((q1 < 0.f) == minus) sd = fma((double)fabsf(q1), (double)bf16_hi(w4[e]), sd);
        }
        for (int o = 1; o < LPG; o <<= 1) sd += __shfl_xor_sync(0xffffffffu, sd, o);
        if (sub == 0 && c < n_cand) cand_key[c] = quest_key(ok ? sd : -INFINITY);
      }
    }
    if (tid == 0) atomicAdd(p.status + ST_TOK_REFINED, n_cand);
    __syncthreads();
    const int need2 = min(max(n_keep - c_in, 0), n_cand);
    if (n_cand <= QSEL_RANK_MAX) {
      // a short list: a candidate is kept when fewer than need2 others come before it (larger key, or the
      // same key and a lower page)
      for (int c = tid; c < n_cand; c += QSEL_THREADS) {
        const unsigned long long mine = cand_key[c];
        const int my_pg = cand_idx[c];
        int rank = 0;
        for (int x = 0; x < n_cand; ++x) {
          const unsigned long long k = cand_key[x];
          rank += (k > mine || (k == mine && cand_idx[x] < my_pg)) ? 1 : 0;
        }
        if (rank < need2) pflag[my_pg] = 1;
      }
    } else {
      unsigned long long tau64 = ~0ull;  // need2 == 0: no candidate key reaches this
      int rem64 = 0;
      if (need2 > 0) {
        quest_radix_threshold<unsigned long long, QSEL_THREADS>(cand_key, n_cand, need2, hist, &s_prefix, &s_remaining);
        tau64 = s_prefix;
        rem64 = s_remaining;
      }
      // the candidates that are kept, ties in page order
      int seen = 0;
      for (int base = 0; base < n_cand; base += QSEL_THREADS) {
        const int c = base + tid;
        const unsigned long long k = c < n_cand ? cand_key[c] : 0ull;
        const bool eq = c < n_cand && k == tau64;
        int tot;
        const int rank = quest_block_scan<QSEL_THREADS>(eq ? 1 : 0, tot, scan_buf);
        if (c < n_cand && (k > tau64 || (eq && seen + rank < rem64))) pflag[cand_idx[c]] = 1;
        seen += tot;
      }
    }
  } else if (overflow) {  // float32 order, ties to the lower page
    int seen_equal = 0;
    for (int base = 0; base < P; base += QSEL_THREADS) {
      const int pg = base + tid;
      const uint32_t k = pg < P ? keys[pg] : 0u;
      const bool eq = pg < P && k == tau32;
      int tot;
      const int rank = quest_block_scan<QSEL_THREADS>(eq ? 1 : 0, tot, scan_buf);
      if (pg < P) pflag[pg] = (k > tau32 || (eq && seen_equal + rank < rem32)) ? 1 : 0;
      seen_equal += tot;
    }
  }
  __syncthreads();
  // ---- the head's byte per page; its ascending page list where the caller asked for it ----
  unsigned char* hm = p.hmask + ((size_t)b * Hq + head) * p.Prow;
  if (p.pages_out == nullptr && p.cnt_out == nullptr) {
    for (int pg = tid; pg < P; pg += QSEL_THREADS) hm[pg] = pflag[pg];
    return;
  }
  int written = 0;
  int32_t* out = p.pages_out ? p.pages_out + ((size_t)b * Hq + head) * p.Prow : nullptr;
  for (int base = 0; base < P; base += QSEL_THREADS) {
    const int pg = base + tid;
    const bool sel = pg < P && pflag[pg] != 0;
    int tot_sel;
    const int pos = quest_block_scan<QSEL_THREADS>(sel ? 1 : 0, tot_sel, scan_buf);
    if (pg < P) hm[pg] = sel ? 1 : 0;
    if (sel && out) out[written + pos] = pg;
    written += tot_sel;
  }
  if (tid == 0 && p.cnt_out) p.cnt_out[(size_t)b * Hq + head] = written;
}

// The union of the heads' pages of a (sequence, kv-head): the row's token list (every token of a page some head
// keeps, ascending) and a byte per page that says which heads keep it.
__global__ void __launch_bounds__(QS_THREADS) quest_list_kernel(const QuestSelDev p) {
  const int kvh = blockIdx.x, tid = threadIdx.x;
  const int Hkv = p.sh.n_kv_heads, Hq = p.sh.n_q_heads, G = Hq / Hkv, S = p.S;
  __shared__ int scan_buf[QS_THREADS / 32];
  pdl_trigger();
  pdl_wait();
  const int b = p.order[blockIdx.y];  // longest sequences first
  const int bk = b * Hkv + kvh;
  const int T = min(max(p.kv.seq_lens[b], 0), p.kv.max_pages_per_seq * PAGE);
  const int P = (T + S - 1) / S;
  const int32_t* table = p.kv.page_table + (size_t)b * p.kv.max_pages_per_seq;
  const size_t row = (size_t)bk * p.Tmax;
  // the kept pages in ascending order (page and first cache row), then the list entry by entry with full-width
  // stores: every kept page but possibly the sequence's last holds S tokens, so entry n is token n % S of kept
  // page n / S.  (A thread per page writing its S entries one by one took 71 us: each store touched a sector of
  // its own.)
  extern __shared__ __align__(16) unsigned char qlsm2[];
  int* sel_page = reinterpret_cast<int*>(qlsm2);                          // [Prow]
  uint32_t* sel_row0 = reinterpret_cast<uint32_t*>(sel_page + p.Prow);    // [Prow]
  int n_sel = 0;
  bool last_kept = false;  // thread (P - 1) % QS_THREADS: the sequence's last page, the only one that may be short
  if ((p.Prow & 3) == 0) {
    // four pages per thread: the heads' bytes come as 32-bit words, and a quarter of the scans
    for (int base = 0; base < P; base += QS_THREADS * 4) {
      const int pg0 = base + tid * 4;
      uint32_t mm = 0;  // the four pages' head masks, a byte each
      if (pg0 < P) {
        for (int h = 0; h < G; ++h)
          mm |= (*reinterpret_cast<const uint32_t*>(p.hmask + ((size_t)b * Hq + kvh * G + h) * p.Prow + pg0) & 0x01010101u) << h;
        for (int e = 1; e < 4; ++e)
          if (pg0 + e >= P) mm &= ~(0xffu << (8 * e));  // bytes beyond the sequence's pages are stale
        *reinterpret_cast<uint32_t*>(p.page_mask + (size_t)bk * p.Pstride + pg0) = mm;
      }
      const int cnt = ((mm & 0xffu) ? 1 : 0) + ((mm & 0xff00u) ? 1 : 0) + ((mm & 0xff0000u) ? 1 : 0) + ((mm & 0xff000000u) ? 1 : 0);
      int tot_sel;
      int at = n_sel + quest_block_scan(cnt, tot_sel, scan_buf);
      for (int e = 0; e < 4; ++e) {
        if (!((mm >> (8 * e)) & 0xffu)) continue;
        const int pg = pg0 + e;
        if (pg == P - 1) last_kept = true;
        const int tok = pg * S, page = table[tok / PAGE];
        const bool ok = page >= 0 && page < p.kv.num_pages;
        sel_page[at] = pg;
        sel_row0[at] = ok ? (uint32_t)((page * Hkv + kvh) * PAGE + (tok % PAGE)) : 0xffffffffu;
        ++at;
      }
      n_sel += tot_sel;
    }
  } else {
    for (int base = 0; base < P; base += QS_THREADS) {
      const int pg = base + tid;
      unsigned char m = 0;
      if (pg < P)
        for (int h = 0; h < G; ++h) m |= (unsigned char)((p.hmask[((size_t)b * Hq + kvh * G + h) * p.Prow + pg] & 1u) << h);
      if (pg < P) p.page_mask[(size_t)bk * p.Pstride + pg] = m;
      int tot_sel;
      const int pos = quest_block_scan(m ? 1 : 0, tot_sel, scan_buf);
      if (m) {
        if (pg == P - 1) last_kept = true;
        const int tok = pg * S, page = table[tok / PAGE];
        const bool ok = page >= 0 && page < p.kv.num_pages;
        sel_page[n_sel + pos] = pg;
        sel_row0[n_sel + pos] = ok ? (uint32_t)((page * Hkv + kvh) * PAGE + (tok % PAGE)) : 0xffffffffu;
      }
      n_sel += tot_sel;
    }
  }
  // every kept page holds S tokens but the sequence's last, which holds the rest
  const int n_list = min(n_sel * S - (__syncthreads_or(last_kept ? 1 : 0) ? P * S - T : 0), p.Tmax);
  // four entries per store: S is a multiple of four, so they are tokens of one page
  const int sh_s = 31 - __clz(S);  // S is a power of two
  for (int n = tid * 4; n < n_list; n += QS_THREADS * 4) {
    const int i = n >> sh_s, j = n & (S - 1);
    const uint32_t r0 = sel_row0[i];
    const int t0 = sel_page[i] * S + j;
    const bool bad = r0 == 0xffffffffu;
    if (n + 4 <= n_list) {
      *reinterpret_cast<int4*>(p.list_idx + row + n) = make_int4(t0, t0 + 1, t0 + 2, t0 + 3);
      *reinterpret_cast<uint4*>(p.list_row + row + n) = bad ? make_uint4(r0, r0, r0, r0) : make_uint4(r0 + j, r0 + j + 1, r0 + j + 2, r0 + j + 3);
    } else {
      for (int e = 0; n + e < n_list; ++e) {
        p.list_idx[row + n + e] = t0 + e;
        p.list_row[row + n + e] = bad ? r0 : r0 + j + e;
      }
    }
  }
  if (tid == 0) p.kept_cnt[bk] = n_list;
}

void launch_quest_selection(const AttnArgs& a, bool update_meta, cudaStream_t st) {
  const sol_shape_t& sh = a.shape;
  const int Hq = sh.n_q_heads, Hkv = sh.n_kv_heads, hd = sh.head_dim, G = Hq / Hkv, S = sh.quest_page_size;
  const int Tmax = a.kv.max_pages_per_seq * PAGE;

  QuestScoreDev sc;
  sc.sh = sh; sc.kv = a.kv; sc.S = S; sc.Prow = Tmax / S; sc.q_rot = a.q_rot; sc.keys = a.quest_keys; sc.err = a.quest_err;
  sc.status = a.status;
  sc.B = a.B;
  // the tensor-core kernel wants whole operand rows per cache page (S a power of two up to 64 gives that) and at
  // most 8 heads per kv-head, which the shape check has seen to
  sc.qsplit = a.quest_qsplit; sc.l1 = a.quest_l1; sc.order = a.quest_order; sc.update_meta = update_meta ? 1 : 0;
  SOL_LAUNCH("quest_query", quest_query_kernel, dim3(Hkv, a.B), dim3(QQ_THREADS), ((G + 3) / 4) * 16 * 2 * hd * 2, st, sc);
  if (hd == 64) {
    if (G <= 4) launch_quest_score_mma<128, 1>(sc, Hkv, st);
    else launch_quest_score_mma<128, 2>(sc, Hkv, st);
  } else {
    if (G <= 4) launch_quest_score_mma<256, 1>(sc, Hkv, st);
    else launch_quest_score_mma<256, 2>(sc, Hkv, st);
  }

  QuestSelDev d;
  d.keys = a.quest_keys; d.err = a.quest_err; d.order = a.quest_order;
  d.sh = sh; d.kv = a.kv; d.r_permille = a.r_permille; d.Tmax = Tmax; d.S = S;
  d.Pstride = Tmax / 4; d.Prow = Tmax / S;
  d.q_rot = a.q_rot; d.page_mask = a.page_mask; d.list_idx = a.list_idx; d.list_row = a.kept_row;
  d.kept_cnt = a.kept_cnt; d.pages_out = a.quest_pages_out; d.cnt_out = a.quest_cnt_out;
  d.status = a.status;
  d.hmask = a.quest_hmask;
  const int smem = QS_CAND_CAP * (8 + 4 + 1) + d.Prow * (4 + 1) + hd * 4 + 16;
  if (d.Prow <= 4096) {
    ensure_dynamic_smem(reinterpret_cast<const void*>(&quest_select_kernel<128>), smem);
    SOL_LAUNCH("quest_select", quest_select_kernel<128>, dim3(Hq, a.B), dim3(128), smem, st, d);
  } else {
    ensure_dynamic_smem(reinterpret_cast<const void*>(&quest_select_kernel<256>), smem);
    SOL_LAUNCH("quest_select", quest_select_kernel<256>, dim3(Hq, a.B), dim3(256), smem, st, d);
  }
  ensure_dynamic_smem(reinterpret_cast<const void*>(&quest_list_kernel), d.Prow * 8);
  SOL_LAUNCH("quest_list", quest_list_kernel, dim3(Hkv, a.B), dim3(QS_THREADS), d.Prow * 8, st, d);

  // the attention over the lists: launch_quest_attend
}

}  // namespace sol
