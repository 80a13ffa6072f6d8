// Decode attention with a per-sequence keep-rate, as four kernels:
//
//   attn_prep    rotary embedding of q and the new k, append k/v to the paged
//                cache, split q into three bf16 parts (hi + mid + lo == q to
//                2^-24) laid out as tensor-core operand rows
//   attn_score   pass 1: stream every K page once (cp.async.bulk into shared
//                memory), logits of the G heads of the group with m16n8k16
//                MMAs (tokens are the M side, the split query rows the N
//                side), group-summed selection score sigma
//   token_select exact top-k per (sequence, kv-head): radix select on the
//                float32 scores, then every score within a small window of
//                the threshold is re-scored in float64 from the cache rows,
//                so the kept set does not depend on float32 rounding
//   attn_gather  pass 2: only the kept V rows are read; online softmax over
//                the kept logits; split over the kept list + combine
//
// Kept count: ceil(r*T) clamped to [0, T] (appendix "Token sparsity",
// "Budgeted token selection"), raised to the forced set (sinks, window; the
// newest token by default).  Softmax over kept tokens only equals the paper's
// additive -inf mask on dropped keys.
#include <math.h>

#include <type_traits>

#include "sol_common.cuh"
#include "sol_internal.h"
#include "sol_select.cuh"

namespace sol {

// Flat work lists of the attention kernels (AttnArgs::plan): cumulative counts over the sequences of the
// batch, PLAN_STRIDE words each: 64-token pages, 8192-token segments of rows that need a
// selection (histogram), 2048-token segments (scan).  Entry b is the count before sequence b, entry B the total.
enum : int { PLAN_PAGES = 0, PLAN_HSEG = 1, PLAN_SSEG = 2, PLAN_LISTS = 3 };
constexpr int PLAN_STRIDE = 132;
constexpr int PLAN_GROUP_TOKENS = 4 * PAGE;  // tokens of one pass-1 unit (a CTA of attn_score: one page per warp)
constexpr int TH_SEG = 8192;  // tokens per token_hist CTA
constexpr int TS_SEG = 2048;  // tokens per token_scan CTA

// What every selection kernel derives from a row's length and keep-rate.
struct RowPlan {
  int T, n_sink, n_win, nf, k, mode;  // mode 0: keep all; 1: forced only; 2: selection
  __device__ __forceinline__ bool forced(int j) const { return j < n_sink || j >= T - n_win; }
};
__device__ __forceinline__ RowPlan row_plan(const sol_shape_t& sh, const sol_kv_t& kv, const int32_t* r_permille, int b) {
  RowPlan r;
  r.T = min(kv.seq_lens[b], kv.max_pages_per_seq * PAGE);  // never index past the page table
  const int Tp = max(r.T, 0);
  r.n_sink = min(max(sh.n_sink, 0), Tp);
  r.n_win = min(max(sh.n_window, 0), Tp - r.n_sink);
  r.nf = r.n_sink + r.n_win;
  long long bud = ((long long)r_permille[b] * Tp + 999) / 1000;
  if (bud > Tp) bud = Tp;
  r.k = min(Tp, max((int)bud, r.nf));
  r.mode = r.k >= Tp ? 0 : (r.k <= r.nf ? 1 : 2);
  return r;
}

// The sequence that holds flat unit `u` of a cumulative list (cum[b] <= u < cum[b + 1]); n entries + total.
__device__ __forceinline__ int plan_find(const int* cum, int n, int u) {
  int lo = 0, hi = n - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (cum[mid] <= u) lo = mid;
    else hi = mid - 1;
  }
  return lo;
}

// ============================================================================
// attn_prep
// ============================================================================
struct PrepDev {
  sol_shape_t sh;
  sol_kv_t kv;
  const float* qkv;  // [ksplit][B][ldq] partial sums of the QKV projection, or nullptr
  int ldq, ksplit, B;
  const float* qkv_scale;  // [B]
  const uint16_t* q_bf16;  // [B][Hq][hd] or nullptr
  float* q_rot;
  uint16_t* q_split;
  int32_t* work_ctr;  // zeroed here: [0] items emitted, [1] next item, [2 + b*Hkv + kvh] finished items
  uint32_t* row_hist; // zeroed here: [B*Hkv][SEL_BINS] score histogram of rows that span several selection CTAs
  uint32_t* row_ctl;  // zeroed here: [B*Hkv][RC_WORDS]
  uint32_t* seg_pub;  // zeroed here: [B*Hkv][nseg_max]
  int nseg_max;
  int32_t* plan;      // written here by the first CTA: [PLAN_LISTS][PLAN_STRIDE]
  const int32_t* r_permille;
  int split_len, target_items, max_item_chunks;  // for the choice of the pass-2 item length
  int* status;
};

constexpr int PREP_THREADS = 128;
// words of AttnArgs::row_ctl, per (sequence, kv-head): histogram CTAs finished, largest |score|, keep edge,
// drop edge, window (float bits), tickets drawn by the scan CTAs, candidates listed, scan CTAs finished
enum : int { RC_DONE1 = 0, RC_MAX, RC_EDGE, RC_LO, RC_DELTA, RC_TICKET, RC_NCAND, RC_DONE2, RC_WORDS };

// One CTA per (kv-head, sequence): the G query heads of the group, the new k row and the new v row.
__global__ void __launch_bounds__(PREP_THREADS) attn_prep_kernel(const PrepDev p) {
  __shared__ float cs[64], sn[64];  // hd/2 <= 64
  const int kvh = blockIdx.x, b = blockIdx.y;
  const int Hq = p.sh.n_q_heads, Hkv = p.sh.n_kv_heads, hd = p.sh.head_dim, half = hd / 2;
  const int G = Hq / Hkv, HG = (G + 3) / 4;
  const int tid = threadIdx.x;
  const int T = min(p.kv.seq_lens[b], p.kv.max_pages_per_seq * PAGE);  // never index past the page table
  const int pos = T - 1;
  const bool layer = p.qkv != nullptr;
  const bool rope = layer && p.sh.rope_theta > 0.f;
  pdl_trigger();
  pdl_wait();

  // The first CTA lays out the work of the kernels that follow: cumulative page and segment counts over the
  // batch, and the length of the pass-2 work items in chunks of split_len kept tokens: the smallest power of
  // two (up to 1024 tokens) that gives every resident warp of pass 2 at most one item, so that there is no
  // second, partly filled round of items; when even the longest runs leave more items than warps there is
  // work for many rounds, and runs of 1024 tokens (32 batches, enough to amortise filling a warp's ring of
  // row copies), claimed one by one, balance it.
  if (kvh == 0 && b == 0) {
    __shared__ int wsum[PLAN_LISTS][PREP_THREADS / 32];
    __shared__ int n_items[ATTN_ITEM_CHUNKS];
    if (tid < ATTN_ITEM_CHUNKS) n_items[tid] = 0;
    int cnt[PLAN_LISTS] = {0, 0, 0};
    int ch = 0;
    if (tid < p.B) {
      const RowPlan rp = row_plan(p.sh, p.kv, p.r_permille, tid);
      const int Tp = max(rp.T, 0);
      cnt[PLAN_PAGES] = (Tp + PAGE - 1) / PAGE;
      // when no row can be longer than TH_SEG tokens a row is one histogram unit whatever its mode (that CTA
      // does the whole selection of the row); otherwise: histogram units for the rows that need a selection,
      // scan units for all
      const bool local = p.kv.max_pages_per_seq * PAGE <= TH_SEG;
      cnt[PLAN_HSEG] = local ? 1 : (rp.mode == 2 ? (Tp + TH_SEG - 1) / TH_SEG : 0);
      cnt[PLAN_SSEG] = local ? 0 : max(1, (Tp + TS_SEG - 1) / TS_SEG);
      ch = max(1, (rp.k + p.split_len - 1) / p.split_len);
    }
    const int w = tid >> 5, l = tid & 31;
    int incl[PLAN_LISTS];
#pragma unroll
    for (int q = 0; q < PLAN_LISTS; ++q) {
      incl[q] = cnt[q];
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int x = __shfl_up_sync(0xffffffffu, incl[q], o);
        if (l >= o) incl[q] += x;
      }
      if (l == 31) wsum[q][w] = incl[q];
    }
    __syncthreads();
#pragma unroll
    for (int q = 0; q < PLAN_LISTS; ++q) {
      int before = 0;
      for (int x = 0; x < w; ++x) before += wsum[q][x];
      if (tid < p.B) p.plan[q * PLAN_STRIDE + tid + 1] = before + incl[q];
      if (tid == 0) p.plan[q * PLAN_STRIDE] = 0;
    }
    for (int c = 1, q = 0; c <= p.max_item_chunks; c <<= 1, ++q) {
      const int n = __reduce_add_sync(0xffffffffu, tid < p.B ? (ch + c - 1) / c : 0);
      if (l == 0) atomicAdd(&n_items[q], n);
    }
    __syncthreads();
    if (tid == 0) {
      int cpi = p.max_item_chunks;
      for (int c = p.max_item_chunks, q = 31 - __clz(p.max_item_chunks); c >= 1; c >>= 1, --q)
        if ((long long)n_items[q] * Hkv <= p.target_items) cpi = c;
      p.work_ctr[WC_CPI] = cpi;
    }
  }

  // this (sequence, kv-head)'s part of the q/k/v row: G query heads, the k head, the v head.  The K
  // slices of the projection are summed in order (four loads in flight at a time) and scaled.
  __shared__ float rowbuf[(8 + 2) * 128];
  if (layer) {
    const float row_scale = p.qkv_scale ? p.qkv_scale[b] : 1.0f;
    const float* base = p.qkv + (size_t)b * p.ldq;
    const size_t zs = (size_t)p.B * p.ldq;
    for (int i = tid; i < (G + 2) * hd; i += PREP_THREADS) {
      const int col = i < G * hd ? kvh * G * hd + i
                                 : (i < (G + 1) * hd ? Hq * hd + kvh * hd + (i - G * hd)
                                                     : (Hq + Hkv) * hd + kvh * hd + (i - (G + 1) * hd));
      float a = 0.f;
      for (int z0 = 0; z0 < p.ksplit; z0 += 4) {
        float v[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) v[q] = z0 + q < p.ksplit ? base[(size_t)(z0 + q) * zs + col] : 0.f;
#pragma unroll
        for (int q = 0; q < 4; ++q) a += v[q];
      }
      rowbuf[i] = a * row_scale;
    }
  }

  if (tid == 0) {
    p.work_ctr[WC_DONE + b * Hkv + kvh] = 0;
    if (b == 0 && kvh == 0) {
      p.work_ctr[WC_ITEMS] = 0;
      p.work_ctr[WC_NEXT] = 0;
    }
  }
  // scratch of the token selection of this (sequence, kv-head)
  if (tid < RC_WORDS) p.row_ctl[(size_t)(b * Hkv + kvh) * RC_WORDS + tid] = 0u;
  if (tid < p.nseg_max) p.seg_pub[(size_t)(b * Hkv + kvh) * p.nseg_max + tid] = 0u;
  if (T > 8192) {  // rows of one histogram CTA keep their histogram in shared memory
    uint4* hz = reinterpret_cast<uint4*>(p.row_hist + (size_t)(b * Hkv + kvh) * SEL_BINS);
    for (int i = tid; i < SEL_BINS / 4; i += PREP_THREADS) hz[i] = make_uint4(0u, 0u, 0u, 0u);
  }
  if (tid < half) {
    float c = 1.f, s = 0.f;
    if (rope) {
      // angle = pos * theta^(-2i/hd) in float64, reduced to [-pi, pi] before the float32 sine and cosine
      const double inv = exp2(-2.0 * (double)tid / (double)hd * log2((double)p.sh.rope_theta));
      const double a = (double)pos * inv;
      const double k = rint(a * 0.15915494309189535);
      const float r = (float)fma(-k, 6.283185307179586, a);
      sincosf(r, &s, &c);
    }
    cs[tid] = c;
    sn[tid] = s;
  }
  // zero the operand rows of this (sequence, kv-head): pad rows and the unused fourth slot stay zero
  uint16_t* qs = p.q_split + (size_t)(b * Hkv + kvh) * HG * 16 * hd;
  for (int i = tid * 8; i < HG * 16 * hd; i += PREP_THREADS * 8) *reinterpret_cast<uint4*>(qs + i) = make_uint4(0, 0, 0, 0);
  __syncthreads();

  // queries of the group: element pair (f, f + half) of one head per iteration
  for (int i = tid; i < G * half; i += PREP_THREADS) {
    const int gi = i / half, f = i % half, h = kvh * G + gi;
    float q0, q1;
    if (layer) {
      const float x0 = rowbuf[gi * hd + f], x1 = rowbuf[gi * hd + f + half];
      q0 = x0 * cs[f] + (-x1) * sn[f];
      q1 = x1 * cs[f] + x0 * sn[f];
    } else {
      const uint16_t* src = p.q_bf16 + ((size_t)b * Hq + h) * hd;
      q0 = bf2f(src[f]);
      q1 = bf2f(src[f + half]);
    }
    float* qr = p.q_rot + ((size_t)b * Hq + h) * hd;
    qr[f] = q0;
    qr[f + half] = q1;
    const int hg = gi >> 2, t = gi & 3;
    uint16_t* base = qs + (size_t)(hg * 16) * hd;
#pragma unroll
    for (int w = 0; w < 2; ++w) {
      const float q = w ? q1 : q0;
      const int e = w ? f + half : f;
      const uint16_t hi = f2bf(q);
      const float r1 = q - bf2f(hi);
      const uint16_t mid = f2bf(r1);
      const float r2 = r1 - bf2f(mid);
      base[(2 * t) * hd + e] = hi;
      base[(2 * t + 1) * hd + e] = mid;
      base[(8 + 2 * t) * hd + e] = f2bf(r2);
    }
  }

  if (!layer || T <= 0) return;
  // new k (rotated) and v, rounded to bf16, written at position T-1
  const int lp = pos / PAGE, slot = pos % PAGE;
  const int page = lp < p.kv.max_pages_per_seq ? p.kv.page_table[(size_t)b * p.kv.max_pages_per_seq + lp] : -1;
  if (page < 0 || page >= p.kv.num_pages) {
    if (tid == 0) atomicOr(p.status + ST_ERR, ERR_BAD_PAGE);
    return;
  }
  uint16_t* kp = static_cast<uint16_t*>(p.kv.k_pool);
  uint16_t* vp = static_cast<uint16_t*>(p.kv.v_pool);
  const float* kr = rowbuf + G * hd;
  const float* vr = rowbuf + (G + 1) * hd;
  const size_t dst = (((size_t)page * Hkv + kvh) * PAGE + slot) * hd;
  for (int f = tid; f < half; f += PREP_THREADS) {
    const float x0 = kr[f], x1 = kr[f + half];
    kp[dst + f] = f2bf(x0 * cs[f] + (-x1) * sn[f]);
    kp[dst + f + half] = f2bf(x1 * cs[f] + x0 * sn[f]);
    vp[dst + f] = f2bf(vr[f]);
    vp[dst + f + half] = f2bf(vr[f + half]);
  }
}

// ============================================================================
// attn_score (pass 1)
// ============================================================================
struct ScoreDev {
  sol_kv_t kv;
  int Hkv, G, HG, Tmax;
  const uint16_t* q_split;
  float* logits;
  float* sigma;
  int B;
  int* status;
};

constexpr int SC_WARPS = 4;  // pages per CTA
static_assert(SC_WARPS * PAGE == PLAN_GROUP_TOKENS, "a unit of attn_score is one page per warp");
constexpr int SC_MAX_GRID = 32768;  // CTAs launched at most; beyond that a CTA takes several units

template <int HD, int HG, bool FLAT>
__global__ void __launch_bounds__(SC_WARPS * 32) attn_score_kernel(const ScoreDev p) {
  extern __shared__ __align__(128) unsigned char smem[];
  constexpr int PAGE_BYTES = PAGE * HD * 2;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + SC_WARPS * PAGE_BYTES);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  pdl_trigger();
  // Two ways to give the CTAs their unit (sequence, kv-head, group of four pages).  Direct (FLAT = false): a
  // 3-D grid over the longest row the page table allows; CTAs beyond their sequence's length leave at once.
  // That is the cheapest mapping, but an empty CTA costs ~0.5 ns of CTA issue: 70 us for the 131072 CTAs of
  // 128 ragged sequences, four in five of them empty.  Flat (FLAT = true, chosen by the host when the direct
  // grid would exceed SC_MAX_GRID): the units that exist are numbered along the batch; every CTA adds up the
  // sequences' group counts itself from the lengths (an input of the step, so before the wait for the
  // earlier kernels) and takes every gridDim.x-th unit.  The flat mapping costs each CTA two block
  // barriers and a block-wide count, which made uniform batches 6-15 % slower, hence both.
  __shared__ int s_cum[SC_WARPS * 32 + 1], s_len[SC_WARPS * 32], s_wsum[SC_WARPS];
  int my_incl = 0, n_units = 1;
  if (FLAT) {
    const int tid = threadIdx.x;
    int Tt = 0;
    if (tid < p.B) Tt = min(max(p.kv.seq_lens[tid], 0), p.kv.max_pages_per_seq * PAGE);  // never index past the page table
    my_incl = (Tt + PLAN_GROUP_TOKENS - 1) / PLAN_GROUP_TOKENS;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int x = __shfl_up_sync(0xffffffffu, my_incl, o);
      if (lane >= o) my_incl += x;
    }
    if (lane == 31) s_wsum[warp] = my_incl;
    if (tid == 0) s_cum[0] = 0;
    __syncthreads();
    for (int w = 0; w < warp; ++w) my_incl += s_wsum[w];
    s_cum[tid + 1] = my_incl;
    s_len[tid] = Tt;
    __syncthreads();
    n_units = s_cum[p.B] * p.Hkv;
    if ((int)blockIdx.x >= n_units) return;
  } else {
    if (blockIdx.x * SC_WARPS * PAGE >= p.kv.seq_lens[blockIdx.z]) return;
  }
  if (threadIdx.x == 0) {
    for (int i = 0; i < SC_WARPS; ++i) mbar_init(&bars[i], 1);
    fence_mbar_init();
  }
  __syncthreads();
  pdl_wait();
  const int g = lane >> 2, t = lane & 3;
  constexpr int KS = HD / 32;  // pair steps (two MMAs of k=16 each)
  uint32_t phase = 0;
  bool dead = false;  // a wait ran out: no more work, but the block-wide counts below still need this warp
#pragma unroll 1
  for (int u = FLAT ? blockIdx.x : 0; u < n_units; u += gridDim.x) {
    int b, kvh, grp, T;
    if (FLAT) {
      // sequence of unit u: how many cumulative counts lie at or below u / Hkv
      const int key = u / p.Hkv;
      b = __syncthreads_count((int)threadIdx.x < p.B && my_incl <= key);
      const int first = s_cum[b], n_groups = s_cum[b + 1] - first;
      const int rem = u - first * p.Hkv;
      kvh = rem / n_groups;
      grp = rem - kvh * n_groups;
      T = s_len[b];
    } else {
      b = blockIdx.z;
      kvh = blockIdx.y;
      grp = blockIdx.x;
      T = min(p.kv.seq_lens[b], p.kv.max_pages_per_seq * PAGE);  // never index past the page table
    }
    const int lp = grp * SC_WARPS + warp;  // logical page
    if (dead || lp * PAGE >= T || lp >= p.kv.max_pages_per_seq) continue;
    const int page = p.kv.page_table[(size_t)b * p.kv.max_pages_per_seq + lp];
    if (page < 0 || page >= p.kv.num_pages) {
      if (lane == 0) atomicOr(p.status + ST_ERR, ERR_BAD_PAGE);
      continue;
    }
    unsigned char* tile = smem + warp * PAGE_BYTES;
    if (lane == 0) {
      mbar_expect_tx(&bars[warp], PAGE_BYTES);
      bulk_g2s(tile, static_cast<const uint16_t*>(p.kv.k_pool) + ((size_t)page * p.Hkv + kvh) * PAGE * HD, PAGE_BYTES,
               &bars[warp]);
    }

    // query operand fragments: B[k][n] = q_split[n][k]; this lane holds rows g and 8+g, 8 k-values per pair step
    uint4 qf[HG][KS][2];
#pragma unroll
    for (int hg = 0; hg < HG; ++hg) {
      const uint16_t* qb = p.q_split + ((size_t)((b * p.Hkv + kvh) * HG + hg) * 16) * HD;
#pragma unroll
      for (int s = 0; s < KS; ++s) {
        qf[hg][s][0] = *reinterpret_cast<const uint4*>(qb + (size_t)g * HD + s * 32 + t * 8);
        qf[hg][s][1] = *reinterpret_cast<const uint4*>(qb + (size_t)(8 + g) * HD + s * 32 + t * 8);
      }
    }

    if (!mbar_wait(&bars[warp], phase, p.status)) {
      dead = true;
      continue;
    }
    phase ^= 1;

    const uint32_t tb = smem_u32(tile);
    const size_t row0 = ((size_t)b * p.Hkv + kvh) * p.Tmax;
#pragma unroll 1
    for (int mt = 0; mt < PAGE / 16; ++mt) {
      uint4 ka[KS][2];
#pragma unroll
      for (int s = 0; s < KS; ++s) {
        ka[s][0] = lds128(tb + (mt * 16 + g) * (HD * 2) + (s * 32 + t * 8) * 2);
        ka[s][1] = lds128(tb + (mt * 16 + g + 8) * (HD * 2) + (s * 32 + t * 8) * 2);
      }
      float sig0 = 0.f, sig1 = 0.f;  // tokens g and g+8 of this m-tile
      const int tok0 = lp * PAGE + mt * 16 + g, tok1 = tok0 + 8;
#pragma unroll
      for (int hg = 0; hg < HG; ++hg) {
        float d0[4] = {0.f, 0.f, 0.f, 0.f}, d1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int s = 0; s < KS; ++s) {
          mma_bf16(d0, ka[s][0].x, ka[s][1].x, ka[s][0].y, ka[s][1].y, qf[hg][s][0].x, qf[hg][s][0].y);
          mma_bf16(d0, ka[s][0].z, ka[s][1].z, ka[s][0].w, ka[s][1].w, qf[hg][s][0].z, qf[hg][s][0].w);
          mma_bf16(d1, ka[s][0].x, ka[s][1].x, ka[s][0].y, ka[s][1].y, qf[hg][s][1].x, qf[hg][s][1].y);
          mma_bf16(d1, ka[s][0].z, ka[s][1].z, ka[s][0].w, ka[s][1].w, qf[hg][s][1].z, qf[hg][s][1].w);
        }
        // columns 2t, 2t+1 of the first n-tile are head t's hi and mid parts; column 2t of the second its lo part
        const float s0 = d0[0] + (d0[1] + d1[0]);
        const float s1 = d0[2] + (d0[3] + d1[2]);
        const int head = hg * 4 + t;
        if (head < p.G) {
          if (tok0 < T) p.logits[(row0 + tok0) * p.G + head] = s0;
          if (tok1 < T) p.logits[(row0 + tok1) * p.G + head] = s1;
        }
        float q0 = s0, q1 = s1;  // rows of absent heads are zero, so they add nothing
        q0 += __shfl_xor_sync(0xffffffffu, q0, 1);
        q1 += __shfl_xor_sync(0xffffffffu, q1, 1);
        q0 += __shfl_xor_sync(0xffffffffu, q0, 2);
        q1 += __shfl_xor_sync(0xffffffffu, q1, 2);
        sig0 += q0;
        sig1 += q1;
      }
      if (t == 0) {
        if (tok0 < T) p.sigma[row0 + tok0] = sig0 + 0.0f;  // -0 becomes +0: the selection compares floats and keys
        if (tok1 < T) p.sigma[row0 + tok1] = sig1 + 0.0f;
      }
    }
    __syncwarp();  // the tile is rewritten by the next unit's copy
  }
}

// ============================================================================
// token selection: token_hist, token_scan (+ token_list)
// ============================================================================
// Exact top-k of a (sequence, kv-head) row of scores in two kernels, both spread over the row.
//
//   token_hist   one CTA per 8192 tokens: histogram of its scores over 4096 value bins in shared memory,
//                flushed (non-empty bins) to the row's histogram in global memory, and the largest |score|.
//                The CTA that finishes last (rows of one CTA go straight on) finds the bin of the k-th
//                largest score and publishes two values: everything above `edge` (the bin's upper end plus
//                a small window) is kept, everything below `lo` is dropped.
//   token_scan   one CTA per 2048 tokens: kept tokens (above the edge, or forced) go to the row's list at
//                the place given by the counts of the CTAs before it (each CTA publishes its count and
//                adds up those of its predecessors; tickets make sure the predecessors are running);
//                the few tokens between lo and edge are appended to a candidate list.  The CTA that
//                finishes last ranks the candidates in float32, re-scores those within the window of the
//                k-th value in float64 from the cache rows, and appends the kept ones (ascending) to the list.
//   token_list   only when a caller asks for the kept indices: the ascending list, from the patched scores
//                (kept candidates and forced tokens get +inf, so "kept" is the comparison score > edge).
//
// The row's list (token index and page-resolved cache row of every kept token) is what pass 2 reads: segment
// by segment ascending, the settled candidates last; the order is the same on every run.
constexpr int TS_THREADS = 256;
constexpr float TS_FLT_MAX = 3.402823466e+38f;
constexpr uint32_t TS_READY = 0x80000000u;

struct SelectDev {
  sol_shape_t sh;
  sol_kv_t kv;
  const int32_t* r_permille;
  int Tmax, S, split_len, B, nseg_max;
  const int32_t* plan;
  const float* q_rot;
  float* sigma;          // kept candidates and forced tokens are overwritten with +inf (for token_list)
  uint32_t* row_hist;    // [B*Hkv][SEL_BINS], zero on entry
  uint32_t* row_ctl;     // [B*Hkv][RC_WORDS], zero on entry
  uint32_t* seg_pub;     // [B*Hkv][nseg_max] kept count of each 2048-token segment | TS_READY, zero on entry
  int32_t* cand_idx;     // [B*Hkv][SEL_CAND_CAP]
  float* cand_val;       // [B*Hkv][SEL_CAND_CAP]
  int32_t* list_idx;     // [B*Hkv][Tmax] token index of every kept token
  uint32_t* list_row;    // same layout: its cache row (page table applied), 0xffffffff: bad page
  int32_t* kept_cnt;
  int32_t* work_items;
  int32_t* work_ctr;
  int* status;
};

// Exclusive prefix sum of v over the 256 threads (in thread order) and the block total.
__device__ __forceinline__ int ts_block_scan(int v, int& total, int* warp_tot) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int x = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += x;
  }
  __syncthreads();  // earlier readers of warp_tot are done
  if (lane == 31) warp_tot[warp] = incl;
  __syncthreads();
  int before = incl - v;
  total = 0;
#pragma unroll
  for (int w = 0; w < TS_THREADS / 32; ++w) {
    const int x = warp_tot[w];
    if (w < warp) before += x;
    total += x;
  }
  return before;
}

// Shared memory of token_hist: the histogram alone when rows go on to token_scan (more CTAs per SM), the
// whole selection scratch when the CTA takes its row through the selection itself.
struct HistOnly {
  uint32_t hist[SEL_BINS];
};
template <bool LOCAL>
struct HistSmem {
  typename std::conditional<LOCAL, SelectSmem, HistOnly>::type sm;  // its histogram is the one filled here
  double qsum[LOCAL ? 128 : 1];
  int scan_tot[TS_THREADS / 32];
  float fmax_w[TS_THREADS / 32];
  int pick[2];
  int s_flag;
  int cum[PLAN_STRIDE];
};

template <typename Smem>
__device__ __forceinline__ void settle_row(const SelectDev& p, Smem& sm, double* qsum, const RowPlan& rp, int b,
                                           int kvh, int n_list, float edge, float lo, float delta, int ns_all,
                                           bool cands_in_smem);

// One (sequence, kv-head, 8192-token segment) of token_hist.  When the page table allows no row longer than
// 8192 tokens every row is one unit, and its CTA takes the row through the whole selection (edges, list,
// candidates, work items): token_scan and token_settle are then not launched.
template <bool LOCAL>
__device__ __forceinline__ void token_hist_item(const SelectDev& p, HistSmem<LOCAL>& hs, int b, int kvh, int seg) {
  uint32_t* hist = hs.sm.hist;
  int* scan_tot = hs.scan_tot;
  float* fmax_w = hs.fmax_w;
  int* pick = hs.pick;
  int& s_flag = hs.s_flag;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const RowPlan rp = row_plan(p.sh, p.kv, p.r_permille, b);
  const int T = rp.T;
  constexpr bool local = LOCAL;  // no row of this call is longer than one unit
  if (!local && (rp.mode != 2 || seg * TH_SEG >= T)) return;
  const int Hkv = p.sh.n_kv_heads;
  const int bk = b * Hkv + kvh;
  const float* sig = p.sigma + (size_t)bk * p.Tmax;
  uint32_t* ctl = p.row_ctl + (size_t)bk * RC_WORDS;
  uint32_t* gh = p.row_hist + (size_t)bk * SEL_BINS;
  const int nseg = max(1, (T + TH_SEG - 1) / TH_SEG);
  float lo = TS_FLT_MAX, edge = TS_FLT_MAX, delta = 0.f;
  if (rp.mode == 2) {
  for (int i = tid; i < SEL_BINS; i += TS_THREADS) hist[i] = 0;
  __syncthreads();

  // ---- this CTA's scores: 32 per thread, all loads issued before the first use ----
  float mx = 0.f;
  {
    constexpr int VPT = TH_SEG / TS_THREADS / 4;  // float4 loads per thread
    float4 v[VPT];
#pragma unroll
    for (int q = 0; q < VPT; ++q) {
      const int j = seg * TH_SEG + (q * TS_THREADS + tid) * 4;
      v[q] = j < T ? *reinterpret_cast<const float4*>(sig + j) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int q = 0; q < VPT; ++q) {
      const int j0 = seg * TH_SEG + (q * TS_THREADS + tid) * 4;
      const float vv[4] = {v[q].x, v[q].y, v[q].z, v[q].w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int j = j0 + e;
        if (j < T && !rp.forced(j)) {
          atomicAdd(&hist[key_value_bin(float_key(vv[e]))], 1u);
          mx = fmaxf(mx, fabsf(vv[e]));
        }
      }
    }
  }
  mx = warp_max(mx);
  if (lane == 0) fmax_w[warp] = mx;
  __syncthreads();
  mx = 0.f;
#pragma unroll
  for (int w = 0; w < TS_THREADS / 32; ++w) mx = fmaxf(mx, fmax_w[w]);
  if (nseg > 1) {  // only the CTA that arrives last goes on
    for (int i = tid; i < SEL_BINS; i += TS_THREADS) {
      const uint32_t c = hist[i];
      if (c) atomicAdd(gh + i, c);
    }
    if (tid == 0) atomicMax(ctl + RC_MAX, __float_as_uint(mx));
    __threadfence();
    __syncthreads();
    if (tid == 0) s_flag = atomicAdd(ctl + RC_DONE1, 1u) == (uint32_t)(nseg - 1) ? 1 : 0;
    __syncthreads();
    if (!s_flag) return;
    __threadfence();
    for (int i = tid; i < SEL_BINS; i += TS_THREADS) hist[i] = __ldcg(gh + i);
    mx = __uint_as_float(__ldcg(ctl + RC_MAX));
    __syncthreads();
  }

  // ---- the bin that holds the `want`-th largest of the histogrammed scores, and how many lie above it:
  //      thread t owns bins 4095 - 16 t .. 4080 - 16 t
  auto rank_bin = [&](int want) {
    constexpr int BPT = SEL_BINS / TS_THREADS;
    int mine = 0;
#pragma unroll
    for (int q = 0; q < BPT; ++q) mine += (int)hist[SEL_BINS - 1 - tid * BPT - q];
    int total;
    const int before = ts_block_scan(mine, total, scan_tot);
    if (before < want && want <= before + mine) {
      int a = before;
      for (int q = 0; q < BPT; ++q) {
        const int bin = SEL_BINS - 1 - tid * BPT - q;
        const int c = (int)hist[bin];
        if (want <= a + c) {
          pick[0] = bin;
          pick[1] = a;
          break;
        }
        a += c;
      }
    }
    __syncthreads();
  };
  const int need_total = rp.k - rp.nf;
  rank_bin(need_total);
  const int vbin = pick[0], above_bin = pick[1];
  const int pop = (int)hist[vbin];
  uint32_t klo, khi;
  value_bin_key_range(vbin, klo, khi);
  __syncthreads();
  const bool prefix_bin = vbin != 0 && vbin != SEL_BINS / 2 - 1 && vbin != SEL_BINS / 2 && vbin != SEL_BINS - 1;
  if (pop > SEL_CAND_CAP / 2 && prefix_bin) {
    // A crowded bin (many nearly equal scores): histogram the next 12 key bits of the bin's keys (they share
    // their upper 15 bits) and take the sub-bin of the k-th score, so that the candidate list stays short.
    for (int i = tid; i < SEL_BINS; i += TS_THREADS) hist[i] = 0;
    __syncthreads();
#pragma unroll 4
    for (int j = tid; j < T; j += TS_THREADS) {
      if (rp.forced(j)) continue;
      const uint32_t kk = float_key(sig[j]);
      if (kk >= klo && kk <= khi) atomicAdd(&hist[(kk >> 5) & 0xfffu], 1u);
    }
    __syncthreads();
    rank_bin(need_total - above_bin);
    klo = (klo & 0xfffe0000u) | ((uint32_t)pick[0] << 5);
    khi = klo | 31u;
  }
  // window: 2^-16 of the largest score, far above the float32 accumulation error of a head_dim-long dot product
  delta = mx * 1.52587890625e-05f;
  lo = key_to_float(klo) - delta;
  edge = fminf(key_to_float(khi) + delta, TS_FLT_MAX);
  if (tid == 0) {  // for token_scan / token_settle of a long row, and for token_list
    ctl[RC_DELTA] = __float_as_uint(delta);
    ctl[RC_LO] = __float_as_uint(lo);
    ctl[RC_EDGE] = __float_as_uint(edge);
  }
  if (!local) return;
  }  // mode 2

  // ---- a row of one unit: its list and its candidates, 2048 tokens at a time, then the settling ----
  if constexpr (LOCAL) {
  SelectSmem& sm = hs.sm;
  __syncthreads();  // the histogram is not read any more: its space stages the list
  if (tid < 4) sm.counts[tid] = 0;
  __syncthreads();
  const size_t row = (size_t)bk * p.Tmax;
  int32_t* lidx = p.list_idx + row;
  uint32_t* lrow = p.list_row + row;
  const int32_t* table = p.kv.page_table + (size_t)b * p.kv.max_pages_per_seq;
  int32_t* st_idx = reinterpret_cast<int32_t*>(sm.hist);
  uint32_t* st_row = sm.hist + TS_SEG;
  int n_list = 0;
#pragma unroll 1
  for (int base0 = 0; base0 < T; base0 += TS_SEG) {
    const int j0 = base0 + tid * 8;
    uint32_t keep = 0;
    if (j0 < T) {
      if (rp.mode == 0) {
        keep = T - j0 >= 8 ? 0xffu : ((1u << (T - j0)) - 1u);
      } else {
        float vv[8];
        if (rp.mode == 2) {
          const float4 v0 = *reinterpret_cast<const float4*>(sig + j0), v1 = *reinterpret_cast<const float4*>(sig + j0 + 4);
          vv[0] = v0.x; vv[1] = v0.y; vv[2] = v0.z; vv[3] = v0.w; vv[4] = v1.x; vv[5] = v1.y; vv[6] = v1.z; vv[7] = v1.w;
        }
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const int j = j0 + e;
          if (j >= T) continue;
          if (rp.forced(j)) {
            keep |= 1u << e;
          } else if (rp.mode == 2) {
            if (vv[e] > edge) {
              keep |= 1u << e;
            } else if (vv[e] >= lo) {
              const int slot = atomicAdd(&sm.counts[0], 1);
              if (slot < SEL_CAND_CAP) {
                sm.cand_idx[slot] = j;
                sm.f32[slot] = vv[e];
              }
            }
          }
        }
      }
    }
    int total;
    const int before = ts_block_scan(__popc(keep), total, scan_tot);
    if (keep) {
      // eight consecutive tokens share a page
      const int page = table[j0 / PAGE];
      const bool ok = page >= 0 && page < p.kv.num_pages;
      if (!ok) atomicOr(p.status + ST_ERR, ERR_BAD_PAGE);
      const uint32_t r0 = (uint32_t)((page * Hkv + kvh) * PAGE + (j0 % PAGE));
      int pos = before;
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        if ((keep >> e) & 1u) {
          st_idx[pos] = j0 + e;
          st_row[pos] = ok ? r0 + e : 0xffffffffu;
          ++pos;
        }
      }
    }
    __syncthreads();
    for (int i = tid; i < total; i += TS_THREADS) {
      lidx[n_list + i] = st_idx[i];
      lrow[n_list + i] = st_row[i];
    }
    n_list += total;
    __syncthreads();  // the staging space is rewritten by the next 2048 tokens
  }
  const int ns_all = sm.counts[0];
  settle_row(p, sm, hs.qsum, rp, b, kvh, n_list, edge, lo, delta, ns_all, true);
  }  // LOCAL
}

// Persistent CTAs over the flat list of (sequence, kv-head, segment) units of the rows that need a selection.
template <bool LOCAL>
__global__ void __launch_bounds__(TS_THREADS) token_hist_kernel(const SelectDev p) {
  __shared__ HistSmem<LOCAL> hs;
  pdl_trigger();
  pdl_wait();
  for (int i = threadIdx.x; i <= p.B; i += TS_THREADS) hs.cum[i] = p.plan[PLAN_HSEG * PLAN_STRIDE + i];
  __syncthreads();
  const int Hkv = p.sh.n_kv_heads;
  const int n_units = hs.cum[p.B] * Hkv;
  for (int u = blockIdx.x; u < n_units; u += gridDim.x) {
    const int b = plan_find(hs.cum, p.B, u / Hkv);
    const int n = hs.cum[b + 1] - hs.cum[b], rem = u - hs.cum[b] * Hkv;
    token_hist_item<LOCAL>(p, hs, b, rem / n, rem % n);
    __syncthreads();
  }
}

struct ScanSmem {
  SelectSmem sm;
  int s_off;
  int cum[PLAN_STRIDE];
};

// One (sequence, kv-head, 2048-token segment) of token_scan.
__device__ __forceinline__ void token_scan_item(const SelectDev& p, ScanSmem& ss, int b, int kvh, int seg) {
  SelectSmem& sm = ss.sm;
  int& s_off = ss.s_off;
  const int Hkv = p.sh.n_kv_heads;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int bk = b * Hkv + kvh;
  const RowPlan rp = row_plan(p.sh, p.kv, p.r_permille, b);
  const int T = rp.T;
  const size_t row = (size_t)bk * p.Tmax;
  float* sig = p.sigma + row;
  uint32_t* ctl = p.row_ctl + (size_t)bk * RC_WORDS;
  uint32_t* pub = p.seg_pub + (size_t)bk * p.nseg_max;
  int32_t* lidx = p.list_idx + row;
  uint32_t* lrow = p.list_row + row;
  const int32_t* table = p.kv.page_table + (size_t)b * p.kv.max_pages_per_seq;
  const int nseg = max(1, (T + TS_SEG - 1) / TS_SEG);
  const int mode = rp.mode;
  const float edge = mode == 2 ? __uint_as_float(ctl[RC_EDGE]) : TS_FLT_MAX;
  const float lo = mode == 2 ? __uint_as_float(ctl[RC_LO]) : TS_FLT_MAX;

  // ---- classify this CTA's 2048 tokens: 8 consecutive ones per thread ----
  const int j0 = seg * TS_SEG + tid * 8;
  uint32_t keep = 0;
  if (j0 < T) {
    if (mode == 0) {
      keep = T - j0 >= 8 ? 0xffu : ((1u << (T - j0)) - 1u);
    } else {
      float vv[8];
      if (mode == 2) {
        const float4 v0 = *reinterpret_cast<const float4*>(sig + j0), v1 = *reinterpret_cast<const float4*>(sig + j0 + 4);
        vv[0] = v0.x; vv[1] = v0.y; vv[2] = v0.z; vv[3] = v0.w; vv[4] = v1.x; vv[5] = v1.y; vv[6] = v1.z; vv[7] = v1.w;
      }
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const int j = j0 + e;
        if (j >= T) continue;
        if (rp.forced(j)) {
          keep |= 1u << e;
        } else if (mode == 2) {
          if (vv[e] > edge) {
            keep |= 1u << e;
          } else if (vv[e] >= lo) {
            const uint32_t slot = atomicAdd(ctl + RC_NCAND, 1u);
            if (slot < (uint32_t)SEL_CAND_CAP) {
              p.cand_idx[(size_t)bk * SEL_CAND_CAP + slot] = j;
              p.cand_val[(size_t)bk * SEL_CAND_CAP + slot] = vv[e];
            }
          }
        }
      }
    }
  }
  int total;
  const int before = ts_block_scan(__popc(keep), total, sm.scan[0]);

  // ---- this segment's place in the row's list: the kept counts of the segments before it ----
  // The first warp publishes this segment's count and adds up those of the earlier segments, one per lane.
  // The units of a row are taken in ascending order by CTAs that are all resident, so an earlier segment
  // is always being worked on or done.
  if (warp == 0) {
    int off = 0;
    if (lane == 0) {
      __threadfence();
      atomicExch(pub + seg, (uint32_t)total | TS_READY);
    }
    if (nseg > 1) {
      if (lane < seg) {
        uint32_t v = 0, tries = 0;
        while (((v = atomicAdd(pub + lane, 0u)) & TS_READY) == 0u) {
          if (++tries > WAIT_LIMIT) {  // never seen; reported, the row's list is then incomplete
            atomicOr(p.status + ST_ERR, ERR_TIMEOUT);
            break;
          }
        }
        off = (int)(v & ~TS_READY);
      }
      off = __reduce_add_sync(0xffffffffu, off);
    }
    if (lane == 0) s_off = off;
  }
  // staged in shared memory so that the list is written with full-width stores
  int32_t* st_idx = reinterpret_cast<int32_t*>(sm.hist);
  uint32_t* st_row = sm.hist + TS_SEG;
  if (keep) {
    // eight consecutive tokens share a page
    const int page = table[j0 / PAGE];
    const bool ok = page >= 0 && page < p.kv.num_pages;
    if (!ok) atomicOr(p.status + ST_ERR, ERR_BAD_PAGE);
    const uint32_t r0 = (uint32_t)((page * Hkv + kvh) * PAGE + (j0 % PAGE));
    int pos = before;
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      if ((keep >> e) & 1u) {
        st_idx[pos] = j0 + e;
        st_row[pos] = ok ? r0 + e : 0xffffffffu;
        ++pos;
      }
    }
  }
  __syncthreads();
  const int off = s_off;
  for (int i = tid; i < total; i += TS_THREADS) {
    lidx[off + i] = st_idx[i];
    lrow[off + i] = st_row[i];
  }

}

// The end of a row's selection, by one CTA: n_list tokens are already in the row's list (everything above the
// edge, and the forced tokens); ns_all candidates lie between the edges (in shared memory: sm.cand_idx and
// sm.f32, or in the row's global candidate list).  Ranks the candidates in float32, re-scores those within
// the window of the k-th value in float64 from the cache rows, appends the kept ones (ascending) to the
// list, and emits the row's pass-2 work items.
template <typename Smem>
__device__ __forceinline__ void settle_row(const SelectDev& p, Smem& sm, double* qsum, const RowPlan& rp, int b,
                                           int kvh, int n_list, float edge, float lo, float delta, int ns_all,
                                           bool cands_in_smem) {
  const int Hkv = p.sh.n_kv_heads, hd = p.sh.head_dim, G = p.sh.n_q_heads / Hkv;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  constexpr int WARPS = TS_THREADS / 32;
  const int bk = b * Hkv + kvh;
  const int T = rp.T, mode = rp.mode;
  const size_t row = (size_t)bk * p.Tmax;
  float* sig = p.sigma + row;
  int32_t* lidx = p.list_idx + row;
  uint32_t* lrow = p.list_row + row;
  const int32_t* table = p.kv.page_table + (size_t)b * p.kv.max_pages_per_seq;
  __syncthreads();
  if (tid < 4) sm.counts[tid] = 0;
  __syncthreads();
  if (mode == 2) {
    const int need_s = rp.k - n_list;
    if (ns_all > SEL_CAND_CAP || need_s < 0 || need_s > ns_all) {
      // More scores between the edges than the list holds (long runs of equal scores): float32 order with
      // ties to the lower index, by a radix select over the row's keys that lie between the edges.
      if (tid == 0) atomicAdd(p.status + ST_TOK_OVERFLOW, 1);
      auto between = [&](int j, float& v) {
        if (j >= T || rp.forced(j)) return false;
        v = sig[j];
        return v <= edge && v >= lo;
      };
      const int per = (T + TS_THREADS - 1) / TS_THREADS;
      auto key = [&](int i) -> uint32_t {
        float v;
        return between(i * TS_THREADS + tid, v) ? float_key(v) : 0u;
      };
      int tie_need = 0;
      const int want = min(max(need_s, 1), max(ns_all, 1));
      const uint32_t key_thr = select_kth<TS_THREADS, 0, true>(key, want, tie_need, sm, per);
      int ties_taken = 0, at = n_list;
#pragma unroll 1
      for (int base0 = 0; base0 < T && need_s > 0; base0 += TS_SEG) {  // in index order: ties are kept until tie_need runs out
        const int q0 = base0 + tid * 8;
        uint32_t above_mask = 0, tie_mask = 0;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          float v;
          if (between(q0 + e, v)) {
            const uint32_t kk = float_key(v);
            if (kk > key_thr) above_mask |= 1u << e;
            if (kk == key_thr) tie_mask |= 1u << e;
          }
        }
        int tot_ties;
        const int t_before = ties_taken + ts_block_scan(__popc(tie_mask), tot_ties, sm.scan[0]);
        uint32_t take = above_mask;
        int taken = 0;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          if (((tie_mask >> e) & 1u) && t_before + taken < tie_need) {
            take |= 1u << e;
            ++taken;
          }
        }
        int tot_take;
        int pos = at + ts_block_scan(__popc(take), tot_take, sm.scan[1]);
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          if ((take >> e) & 1u) {
            const int j = q0 + e;
            const int page = table[j / PAGE];
            const bool ok = page >= 0 && page < p.kv.num_pages;
            if (!ok) atomicOr(p.status + ST_ERR, ERR_BAD_PAGE);
            lidx[pos] = j;
            lrow[pos] = ok ? (uint32_t)((page * Hkv + kvh) * PAGE + (j % PAGE)) : 0xffffffffu;
            sig[j] = INFINITY;
            ++pos;
          }
        }
        at += tot_take;
        ties_taken += tot_ties;
      }
      n_list = at;
    } else if (need_s > 0) {
      const int ns = ns_all;
      float* sup_val = sm.f32;
      if (!cands_in_smem) {
        for (int c = tid; c < ns; c += TS_THREADS) {
          sm.cand_idx[c] = __ldcg(p.cand_idx + (size_t)bk * SEL_CAND_CAP + c);
          sup_val[c] = __ldcg(p.cand_val + (size_t)bk * SEL_CAND_CAP + c);
        }
      }
      __syncthreads();
      // float32 rank inside the list: the element of rank need_s - 1 carries the k-th value
      for (int c = tid; c < ns; c += TS_THREADS) {
        const float v = sup_val[c];
        const int j = sm.cand_idx[c];
        int rank = 0;
        for (int o = 0; o < ns; ++o) {
          const float vo = sup_val[o];
          rank += (vo > v) || (vo == v && sm.cand_idx[o] < j);
        }
        if (rank == need_s - 1) sm.pick[1] = __float_as_int(v);
      }
      __syncthreads();
      const float thr32 = __int_as_float(sm.pick[1]);
      const float whi = thr32 + delta, wlo = thr32 - delta;
      // classes: above the window (kept, ranks first), inside it (re-scored), below it (dropped)
      int n_above = 0, n_in = 0;
      for (int c = tid; c < ns; c += TS_THREADS) {
        const float v = sup_val[c];
        unsigned char cls = 0;
        if (v > whi) {
          cls = 1;
          ++n_above;
          sm.cand_val[c] = 1.0e300;
        } else if (v >= wlo) {
          cls = 2;
          ++n_in;
          sm.cand_val[c] = (double)v;
        } else {
          sm.cand_val[c] = -1.0e300;
        }
        sm.cand_keep[c] = cls;
      }
      n_above = block_count<TS_THREADS>(n_above, 0, sm);
      n_in = block_count<TS_THREADS>(n_in, 1, sm);
      __syncthreads();
      if (n_above + n_in != need_s) {  // the window holds more than are needed: settle it in float64
        if (tid == 0) atomicAdd(p.status + ST_TOK_REFINED, n_in);
        for (int e = tid; e < hd; e += TS_THREADS) {
          double a = 0.0;
          for (int h = 0; h < G; ++h) a += (double)p.q_rot[((size_t)b * p.sh.n_q_heads + kvh * G + h) * hd + e];
          qsum[e] = a;
        }
        __syncthreads();
        const uint16_t* kp = static_cast<const uint16_t*>(p.kv.k_pool);
        for (int c = warp; c < ns; c += WARPS) {
          if (sm.cand_keep[c] != 2) continue;  // warp-uniform
          const int j = sm.cand_idx[c];
          const int page = table[j / PAGE];
          double a = 0.0;
          if (page >= 0 && page < p.kv.num_pages) {
            const uint16_t* kr = kp + (((size_t)page * Hkv + kvh) * PAGE + (j % PAGE)) * hd;
            for (int e = lane; e < hd; e += 32) a += qsum[e] * (double)bf2f(kr[e]);
          }
          a = warp_sum_d(a);
          if (lane == 0) sm.cand_val[c] = a;
        }
        __syncthreads();
      }
      rank_candidates<TS_THREADS>(ns, need_s, sm);  // cand_keep[c] = 1 for the need_s best of the list
      __syncthreads();
      // the kept candidates join the row's list in ascending index order
      for (int c = tid; c < ns; c += TS_THREADS) {
        if (!sm.cand_keep[c]) continue;
        const int j = sm.cand_idx[c];
        int pos = 0;
        for (int o = 0; o < ns; ++o) pos += sm.cand_keep[o] && sm.cand_idx[o] < j;
        const int page = table[j / PAGE];
        const bool ok = page >= 0 && page < p.kv.num_pages;
        if (!ok) atomicOr(p.status + ST_ERR, ERR_BAD_PAGE);
        lidx[n_list + pos] = j;
        lrow[n_list + pos] = ok ? (uint32_t)((page * Hkv + kvh) * PAGE + (j % PAGE)) : 0xffffffffu;
        sig[j] = INFINITY;
      }
      n_list += need_s;
    }
  }
  // forced tokens read as kept for token_list whatever their score
  if (mode != 0) {
    for (int f = tid; f < rp.nf; f += TS_THREADS) sig[f < rp.n_sink ? f : T - rp.n_win + (f - rp.n_sink)] = INFINITY;
  }
  const int total_kept = T > 0 ? n_list : 0;
  if (tid == 0) p.kept_cnt[bk] = total_kept;

  // Pass-2 work items of this (sequence, kv-head): runs of `cpi` chunks of split_len kept tokens (at least
  // one item, so that the output is always written); cpi was chosen by the first CTA of the score pass.
  const int cpi = p.work_ctr[WC_CPI];
  const int chunks = max(1, (total_kept + p.split_len - 1) / p.split_len);
  const int ns_items = (chunks + cpi - 1) / cpi;
  __syncthreads();
  if (tid == 0) sm.counts[3] = atomicAdd(p.work_ctr + WC_ITEMS, ns_items);
  __syncthreads();
  const int item0 = sm.counts[3];
  for (int i = tid; i < ns_items; i += TS_THREADS) {
    p.work_items[2 * (item0 + i)] = bk * p.S + i * cpi;  // first chunk of the item
    p.work_items[2 * (item0 + i) + 1] = total_kept;
  }
}

// Persistent CTAs over the flat list of (sequence, kv-head, segment) units; a CTA takes its units in
// ascending order, and all CTAs of the grid are resident at once (the launch sizes the grid so).
__global__ void __launch_bounds__(TS_THREADS) token_scan_kernel(const SelectDev p) {
  __shared__ ScanSmem ss;
  pdl_trigger();
  pdl_wait();
  for (int i = threadIdx.x; i <= p.B; i += TS_THREADS) ss.cum[i] = p.plan[PLAN_SSEG * PLAN_STRIDE + i];
  __syncthreads();
  const int Hkv = p.sh.n_kv_heads;
  const int n_units = ss.cum[p.B] * Hkv;
  for (int u = blockIdx.x; u < n_units; u += gridDim.x) {
    const int b = plan_find(ss.cum, p.B, u / Hkv);
    const int n = ss.cum[b + 1] - ss.cum[b], rem = u - ss.cum[b] * Hkv;
    token_scan_item(p, ss, b, rem / n, rem % n);
    __syncthreads();
  }
}

// One CTA per (sequence, kv-head) of the rows that token_scan worked on.
__global__ void __launch_bounds__(TS_THREADS) token_settle_kernel(const SelectDev p) {
  __shared__ SelectSmemOverlay sm;  // candidates from the global list (cands_in_smem = false): never beside the histogram
  __shared__ double qsum[128];
  const int kvh = blockIdx.x, b = blockIdx.y;
  pdl_trigger();
  const RowPlan rp = row_plan(p.sh, p.kv, p.r_permille, b);
  pdl_wait();
  const int bk = b * p.sh.n_kv_heads + kvh;
  const uint32_t* ctl = p.row_ctl + (size_t)bk * RC_WORDS;
  const uint32_t* pub = p.seg_pub + (size_t)bk * p.nseg_max;
  const int nseg = max(1, (rp.T + TS_SEG - 1) / TS_SEG);
  int n_list = 0;  // kept so far: what the segments wrote
  for (int q = 0; q < nseg; ++q) n_list += (int)(pub[q] & ~TS_READY);
  const bool sel = rp.mode == 2;
  settle_row(p, sm, qsum, rp, b, kvh, n_list, sel ? __uint_as_float(ctl[RC_EDGE]) : TS_FLT_MAX,
             sel ? __uint_as_float(ctl[RC_LO]) : TS_FLT_MAX, sel ? __uint_as_float(ctl[RC_DELTA]) : 0.f,
             sel ? (int)ctl[RC_NCAND] : 0, false);
}

struct ListDev {
  sol_shape_t sh;
  sol_kv_t kv;
  const int32_t* r_permille;
  int Tmax;
  const float* sigma;
  const uint32_t* row_ctl;
  int32_t* kept_idx;  // [B*Hkv][Tmax] ascending
};

// One CTA per (sequence, kv-head): the kept token indices in ascending order, for a caller that asks for them.
__global__ void __launch_bounds__(TS_THREADS) token_list_kernel(const ListDev p) {
  __shared__ int warp_tot[TS_THREADS / 32];
  const int kvh = blockIdx.x, b = blockIdx.y, tid = threadIdx.x;
  pdl_trigger();
  const RowPlan rp = row_plan(p.sh, p.kv, p.r_permille, b);
  pdl_wait();
  const int bk = b * p.sh.n_kv_heads + kvh;
  const size_t row = (size_t)bk * p.Tmax;
  const float edge = rp.mode == 2 ? __uint_as_float(p.row_ctl[(size_t)bk * RC_WORDS + RC_EDGE]) : TS_FLT_MAX;
  int at = 0;
#pragma unroll 1
  for (int base0 = 0; base0 < rp.T; base0 += TS_SEG) {
    const int j0 = base0 + tid * 8;
    uint32_t keep = 0;
    if (j0 < rp.T) {
      const float4 v0 = *reinterpret_cast<const float4*>(p.sigma + row + j0);
      const float4 v1 = *reinterpret_cast<const float4*>(p.sigma + row + j0 + 4);
      const float vv[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
#pragma unroll
      for (int e = 0; e < 8; ++e)
        if (j0 + e < rp.T && (rp.mode == 0 || vv[e] > edge)) keep |= 1u << e;
    }
    int total;
    int pos = at + ts_block_scan(__popc(keep), total, warp_tot);
#pragma unroll
    for (int e = 0; e < 8; ++e)
      if ((keep >> e) & 1u) p.kept_idx[row + pos++] = j0 + e;
    at += total;
  }
}

// ============================================================================
// attn_gather (pass 2) with the combine step folded in
// ============================================================================
struct GatherDev {
  sol_kv_t kv;
  int Hq, Hkv, G, Tmax, S;
  const float* logits;
  const int32_t* kept_idx;
  const uint32_t* kept_row;
  const int32_t* work_items;
  int32_t* work_ctr;
  float* part;  // [B][Hkv][S][G][HD + 2]
  float scale_log2;
  float* out_f32;
  uint16_t* out_bf16;
  uint16_t* out_hi;  // packed operand of the output projection (2 out_rows rows: high parts, then low parts)
  int out_rows;
  int* status;
};

constexpr int GA_BATCH = 32;  // kept tokens per warp step: one per lane in the softmax part

__device__ __forceinline__ void cp_async16(uint32_t dst_smem, const void* src, bool valid) {
  const uint32_t n = valid ? 16u : 0u;  // 0: the 16 bytes are filled with zeros and the source is not read
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst_smem), "l"(src), "r"(n) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// Pass 2 is a gather of 128- or 256-byte V rows with G multiply-adds per element: bound by how many row
// fetches are in flight, so the rows travel by asynchronous 16-byte copies into per-warp rings of shared
// memory (about 190 KB per SM, three quarters of it in flight) and the registers only hold accumulators.
//
// The warps of one persistent CTA per SM work through the list of items, each warp on its own: an item is
// (sequence, kv-head, run of kept tokens, at most 1024); a warp's first item is dealt by its index, the
// later ones are claimed from a counter one item ahead.  A warp takes its item in batches of 32 tokens, NST
// batches deep:
//   lane l fetches the list words of token l of a batch (cache row, token index) two steps before the
//   batch's rows are requested and its G logits one step before they are used; when a batch's rows have
//   landed the warp updates its running maximum per head, every lane computes its token's softmax weights,
//   and the weights (as bf16 high and low parts) multiply the rows on the tensor cores.
// A row of one item goes straight to the output; otherwise one partial per item (accumulators, maximum,
// sum) is written and the warp that finishes the last item of a (sequence, kv-head) merges the partials.
template <int HD, int GMAX>
struct GatherCfg {
  static constexpr int WARPS = HD == 64 ? 12 : 8;
  static constexpr int NST = HD == 64 ? 4 : 3;              // batches of rows per warp ring
  static constexpr int STAGE_BYTES = GA_BATCH * HD * 2;      // 4 KB / 8 KB
  static constexpr int THREADS = WARPS * 32;
  static constexpr int RING_BYTES = WARPS * NST * STAGE_BYTES;  // 192 KB
  static constexpr int TAB_BYTES = WARPS * (NST + 1) * GA_BATCH * 8;
  static constexpr int W_BYTES = WARPS * GA_BATCH * GMAX * 4;
  static constexpr int SMEM = RING_BYTES + TAB_BYTES + W_BYTES;
};

template <int HD, int GMAX>
__global__ void __launch_bounds__(GatherCfg<HD, GMAX>::THREADS, 1) attn_gather_kernel(const GatherDev p) {
  using C = GatherCfg<HD, GMAX>;
  constexpr int WARPS = C::WARPS, NST = C::NST;
  constexpr int SPLIT = HD == 64 ? 256 : 128;  // kept tokens per chunk (attn_split_len): the unit of the item list
  constexpr int CPR = HD / 8;                  // 16-byte pieces per row
  constexpr int NT = HD / 8;                   // n-tiles (8 dims each) of the output
  extern __shared__ __align__(128) unsigned char gsm[];
  unsigned char* ring = gsm;
  int2* s_tab = reinterpret_cast<int2*>(gsm + C::RING_BYTES);                 // [WARPS][NST + 1][32] (cache row, token)
  float* s_w = reinterpret_cast<float*>(gsm + C::RING_BYTES + C::TAB_BYTES);  // [WARPS][32][GMAX]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = p.G, Hkv = p.Hkv;
  const uint16_t* vp = static_cast<const uint16_t*>(p.kv.v_pool);
  const int g = lane >> 2, t = lane & 3;  // row group and column pair of the MMA fragments
  unsigned char* my_ring = ring + (size_t)warp * NST * C::STAGE_BYTES;
  int2* my_tab = s_tab + warp * (NST + 1) * GA_BATCH;
  float* my_w = s_w + warp * GA_BATCH * GMAX;
  pdl_trigger();
  pdl_wait();
  const int cpi = p.work_ctr[WC_CPI];
  const int n_items = p.work_ctr[WC_ITEMS];
  const int total_warps = gridDim.x * WARPS;
  // an item's header: (sequence, kv-head) or -1, first token of the run, tokens of the run, kept count of the row
  auto header_of = [&](int item) {
    int4 h = make_int4(-1, 0, 0, 0);
    if (item < n_items) {
      const int2 w = *reinterpret_cast<const int2*>(p.work_items + 2 * item);
      const int n0 = (w.x % p.S) * SPLIT;
      h = make_int4(w.x / p.S, n0, max(0, min(w.y - n0, cpi * SPLIT)), w.y);
    }
    return h;
  };
  int4 cur = header_of(blockIdx.x * WARPS + warp);  // warp-uniform

#pragma unroll 1
  while (cur.x >= 0) {
    // the next item is claimed now and its header fetched while this one is worked on
    int claimed = 0;
    if (lane == 0) claimed = total_warps + atomicAdd(p.work_ctr + WC_NEXT, 1);
    claimed = __shfl_sync(0xffffffffu, claimed, 0);
    const int4 nxt = header_of(claimed);
    const int bk = cur.x, len = cur.z, cnt = cur.w;
    const int b = bk / Hkv, kvh = bk % Hkv;
    const size_t row = (size_t)bk * p.Tmax;
    const uint32_t* krow = p.kept_row + row + cur.y;
    const int32_t* kidx = p.kept_idx + row + cur.y;
    const float* lgrow = p.logits + row * G;
    const int nb = (len + GA_BATCH - 1) / GA_BATCH;  // batches of the item

    // list words of the item's m-th batch: lane l holds token l
    auto load_tab = [&](int m) {
      int2 e = make_int2(-1, 0);
      const int n = m * GA_BATCH + lane;
      if (n < len) e = make_int2((int)krow[n], kidx[n]);
      return e;
    };
    // requests the rows of the m-th batch (its list words are in the table) into ring slot m % NST
    auto request_rows = [&](int m) {
      if (m < nb) {
        const int2* tab = my_tab + (m % (NST + 1)) * GA_BATCH;
        const uint32_t dst0 = smem_u32(my_ring + (m % NST) * C::STAGE_BYTES);
#pragma unroll
        for (int i = 0; i < CPR; ++i) {
          const int c = i * 32 + lane, r = c / CPR, part = c % CPR;
          const int ridx = tab[r].x;
          // piece `part` of row r sits at piece position part ^ (r & 7): the transposing matrix loads below then
          // touch every bank once
          cp_async16(dst0 + r * (HD * 2) + ((part & ~7) | ((part ^ r) & 7)) * 16, vp + (size_t)(ridx < 0 ? 0 : ridx) * HD + part * 8,
                     ridx >= 0);
        }
      }
      cp_async_commit();  // an empty group keeps the count of groups per step fixed
    };
    auto load_logits = [&](int2 e, float (&x)[GMAX]) {
#pragma unroll
      for (int h = 0; h < GMAX; ++h) x[h] = -INFINITY;  // an absent token weighs nothing
      if (e.x < 0) return;
      const float* src = lgrow + (size_t)e.y * G;
      if (GMAX == 4 && G == 4) {
        const float4 v = *reinterpret_cast<const float4*>(src);
        x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
      } else {
#pragma unroll
        for (int h = 0; h < GMAX; ++h)
          if (h < G) x[h] = src[h];
      }
    };

    // Output accumulators of the tensor-core product O[head][dim] += P[head][token] V[token][dim]: the 16 rows of
    // the m16n8k16 tile are the G heads' weights as bf16 high parts (rows 0..7) and low parts (rows 8..15), so
    // that the product is exact to 2^-17 of a weight; d[j] is the tile of dims 8 j .. 8 j + 7.
    float mh[GMAX], ls[GMAX], d[NT][4];
#pragma unroll
    for (int h = 0; h < GMAX; ++h) {
      mh[h] = -INFINITY;
      ls[h] = 0.f;
    }
#pragma unroll
    for (int j = 0; j < NT; ++j)
#pragma unroll
      for (int c = 0; c < 4; ++c) d[j][c] = 0.f;
    // prologue: list words of the first NST batches, rows of the first NST - 1, logits of the first
#pragma unroll
    for (int m = 0; m < NST; ++m) my_tab[(m % (NST + 1)) * GA_BATCH + lane] = load_tab(m);
    __syncwarp();
#pragma unroll
    for (int m = 0; m < NST - 1; ++m) request_rows(m);
    int2 e_far = load_tab(NST);  // held in a register until its table slot is free
    float x_c[GMAX];
    load_logits(my_tab[lane], x_c);

#pragma unroll 1
    for (int m = 0; m < nb; ++m) {
      // the table slot of batch m - 1 is free now: batch m + NST moves in; rows of batch m + NST - 1 are requested
      my_tab[((m + NST) % (NST + 1)) * GA_BATCH + lane] = e_far;
      request_rows(m + NST - 1);
      e_far = load_tab(m + NST + 1);
      float x_n[GMAX];
      load_logits(m + 1 < nb ? my_tab[((m + 1) % (NST + 1)) * GA_BATCH + lane] : make_int2(-1, 0), x_n);

      // ---- softmax weights relative to the running maximum ----
      float scg = 0.f;  // rescaling of this lane's accumulator rows (head g)
#pragma unroll
      for (int h = 0; h < GMAX; ++h) {
        const float x = x_c[h] * p.scale_log2;
        const float nm = fmaxf(mh[h], warp_max(x));
        const float sc = mh[h] == -INFINITY ? 0.f : exp2f(mh[h] - nm);
        const float pw = x == -INFINITY ? 0.f : exp2f(x - nm);
        mh[h] = nm;
        ls[h] = ls[h] * sc + pw;
        if (h == g) scg = sc;
        my_w[lane * GMAX + h] = pw;
      }
#pragma unroll
      for (int j = 0; j < NT; ++j)
#pragma unroll
        for (int c = 0; c < 4; ++c) d[j][c] *= scg;
      cp_async_wait<NST - 1>();  // this lane's pieces of batch m have landed ...
      __syncwarp();              // ... and so have the other lanes'; the weights are in the table

      // ---- weights x rows on the tensor cores ----
      const uint32_t st = smem_u32(my_ring + (m % NST) * C::STAGE_BYTES);
#pragma unroll
      for (int ks = 0; ks < GA_BATCH / 16; ++ks) {
        // A fragment: head g's weights of tokens 2t, 2t+1, 2t+8, 2t+9 of this 16-token step, high and low parts
        float w0 = 0.f, w1 = 0.f, w2 = 0.f, w3 = 0.f;
        if (g < GMAX) {
          const float* wt = my_w + (ks * 16 + 2 * t) * GMAX + g;
          w0 = wt[0];
          w1 = wt[GMAX];
          w2 = wt[8 * GMAX];
          w3 = wt[9 * GMAX];
        }
        const uint16_t h0 = f2bf(w0), h1 = f2bf(w1), h2 = f2bf(w2), h3 = f2bf(w3);
        const uint32_t a0 = (uint32_t)h0 | ((uint32_t)h1 << 16), a2 = (uint32_t)h2 | ((uint32_t)h3 << 16);
        const uint32_t a1 = pack_bf16(w0 - bf2f(h0), w1 - bf2f(h1)), a3 = pack_bf16(w2 - bf2f(h2), w3 - bf2f(h3));
        // B fragments: lanes 0-7 / 8-15 address tokens 0-7 / 8-15 of the step for dims 8 j, lanes 16-31 the same for 8 (j + 1)
        const int tok = ks * 16 + (lane & 15);
        const uint32_t row_addr = st + tok * (HD * 2);
#pragma unroll
        for (int j = 0; j < NT; j += 2) {
          const int piece = j + (lane >> 4);
          uint32_t bfr[4];
          ldsm_x4_trans(bfr, row_addr + ((piece & ~7) | ((piece ^ tok) & 7)) * 16);
          mma_bf16(d[j], a0, a1, a2, a3, bfr[0], bfr[1]);
          mma_bf16(d[j + 1], a0, a1, a2, a3, bfr[2], bfr[3]);
        }
      }
      __syncwarp();  // the weights and the ring slot are rewritten by the next steps
#pragma unroll
      for (int h = 0; h < GMAX; ++h) x_c[h] = x_n[h];
    }
    cp_async_wait<0>();

    // ---- the item's result: this lane holds head g's dims 8 j + 2 t, + 1 (rows g and g + 8 of the tile) ----
#pragma unroll
    for (int h = 0; h < GMAX; ++h) ls[h] = warp_sum(ls[h]);
    float m_g = -INFINITY, l_g = 0.f;
#pragma unroll
    for (int h = 0; h < GMAX; ++h) {
      if (h == g) {
        m_g = mh[h];
        l_g = ls[h];
      }
    }
    const int chunks = max(1, (cnt + SPLIT - 1) / SPLIT);
    const int ns = (chunks + cpi - 1) / cpi;  // items of this (sequence, kv-head)
    auto write_out = [&](int h, int e, float o0, float o1) {
      const size_t idx = ((size_t)b * p.Hq + kvh * G + h) * HD + e;
      if (p.out_f32) *reinterpret_cast<float2*>(p.out_f32 + idx) = make_float2(o0, o1);
      if (p.out_bf16) *reinterpret_cast<uint32_t*>(p.out_bf16 + idx) = pack_bf16(o0, o1);
      if (p.out_hi) {
        const uint16_t h0 = f2bf(o0), h1 = f2bf(o1);
        const int k = (kvh * G + h) * HD + e;  // column of the projection's input; e is even, so k and k + 1 share a piece
        unsigned char* dst = reinterpret_cast<unsigned char*>(p.out_hi) + act_piece_offset(2 * p.out_rows, b, k >> 3) + (k & 7) * 2;
        *reinterpret_cast<uint32_t*>(dst) = (uint32_t)h0 | ((uint32_t)h1 << 16);
        *reinterpret_cast<uint32_t*>(dst + (size_t)p.out_rows * 128) = pack_bf16(o0 - bf2f(h0), o1 - bf2f(h1));
      }
    };
    if (ns == 1) {  // the row is this one item: its output goes out directly
      if (g < G) {
        const float inv = l_g > 0.f ? 1.0f / l_g : 0.f;
#pragma unroll
        for (int j = 0; j < NT; ++j) write_out(g, j * 8 + 2 * t, (d[j][0] + d[j][2]) * inv, (d[j][1] + d[j][3]) * inv);
      }
    } else {
      const int slot_no = (cur.y / SPLIT) / cpi;  // this item's partial
      float* dst = p.part + (((size_t)bk * p.S + slot_no) * G) * (HD + 2);
      if (g < G) {
#pragma unroll
        for (int j = 0; j < NT; ++j)
          *reinterpret_cast<float2*>(dst + g * (HD + 2) + j * 8 + 2 * t) = make_float2(d[j][0] + d[j][2], d[j][1] + d[j][3]);
        if (t == 0) {
          dst[g * (HD + 2) + HD] = m_g;
          dst[g * (HD + 2) + HD + 1] = l_g;
        }
      }
      // ---- the last item of this (sequence, kv-head) merges the partials ----
      __threadfence();
      __syncwarp();
      int last = 0;
      if (lane == 0) last = atomicAdd(p.work_ctr + WC_DONE + bk, 1) == ns - 1 ? 1 : 0;
      last = __shfl_sync(0xffffffffu, last, 0);
      if (last) {
        __threadfence();
        const float* src0 = p.part + ((size_t)bk * p.S * G) * (HD + 2);
        // factors of the partials: f[q][h] = 2^(m_q - M_h) / sum_q l_q 2^(m_q - M_h), in the warp's (idle) ring
        float* fac = reinterpret_cast<float*>(my_ring);
        for (int h = 0; h < G; ++h) {
          float mm = -INFINITY;
          for (int q = lane; q < ns; q += 32) mm = fmaxf(mm, __ldcg(src0 + ((size_t)q * G + h) * (HD + 2) + HD));
          mm = warp_max(mm);
          float l = 0.f;
          for (int q = lane; q < ns; q += 32) {
            const float* src = src0 + ((size_t)q * G + h) * (HD + 2);
            const float m2 = __ldcg(src + HD);
            const float f = m2 == -INFINITY ? 0.f : exp2f(m2 - mm);
            fac[q * GMAX + h] = f;
            l += __ldcg(src + HD + 1) * f;
          }
          l = warp_sum(l);
          const float inv = l > 0.f ? 1.0f / l : 0.f;
          for (int q = lane; q < ns; q += 32) fac[q * GMAX + h] *= inv;
        }
        __syncwarp();
        for (int e0 = lane * 2; e0 < G * HD; e0 += 64) {
          const int h = e0 / HD, e = e0 % HD;
          const float* src = src0 + (size_t)h * (HD + 2) + e;
          float a0 = 0.f, a1 = 0.f;
          int q = 0;
          for (; q + 8 <= ns; q += 8) {  // eight partials' loads in flight
            float2 v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) v[u] = __ldcg(reinterpret_cast<const float2*>(src + (size_t)(q + u) * G * (HD + 2)));
#pragma unroll
            for (int u = 0; u < 8; ++u) {
              const float f = fac[(q + u) * GMAX + h];
              a0 = fmaf(v[u].x, f, a0);
              a1 = fmaf(v[u].y, f, a1);
            }
          }
          for (; q < ns; ++q) {
            const float2 v = __ldcg(reinterpret_cast<const float2*>(src + (size_t)q * G * (HD + 2)));
            const float f = fac[q * GMAX + h];
            a0 = fmaf(v.x, f, a0);
            a1 = fmaf(v.y, f, a1);
          }
          write_out(h, e, a0, a1);
        }
      }
    }
    __syncwarp();
    cur = nxt;
  }
}

// ============================================================================
// host side
// ============================================================================
template <int HD, int HG, bool FLAT>
static void launch_score_as(const ScoreDev& d, dim3 grid, cudaStream_t st) {
  const int smem = SC_WARPS * PAGE * HD * 2 + SC_WARPS * 8 + 32;
  ensure_dynamic_smem(reinterpret_cast<const void*>(&attn_score_kernel<HD, HG, FLAT>), smem);
  SOL_LAUNCH("attn_score", (attn_score_kernel<HD, HG, FLAT>), grid, dim3(SC_WARPS * 32), smem, st, d);
}
// Direct 3-D grid while it stays within SC_MAX_GRID CTAs, else the flat numbering of the units that exist.
template <int HD>
static void launch_score(const ScoreDev& d, int HG, int groups_per_row, cudaStream_t st) {
  const long long direct = (long long)groups_per_row * d.Hkv * d.B;
  if (direct <= SC_MAX_GRID) {
    const dim3 grid(groups_per_row, d.Hkv, d.B);
    if (HG == 1) launch_score_as<HD, 1, false>(d, grid, st);
    else launch_score_as<HD, 2, false>(d, grid, st);
  } else {
    const dim3 grid(SC_MAX_GRID);
    if (HG == 1) launch_score_as<HD, 1, true>(d, grid, st);
    else launch_score_as<HD, 2, true>(d, grid, st);
  }
}

// One CTA per item, at most one per SM (they are persistent).
template <int HD, int GMAX>
static void launch_gather(const GatherDev& d, long long items, cudaStream_t st) {
  using C = GatherCfg<HD, GMAX>;
  ensure_dynamic_smem(reinterpret_cast<const void*>(&attn_gather_kernel<HD, GMAX>), C::SMEM);
  const long long resident = sm_count();
  const int grid = (int)(items < resident ? items : resident);
  SOL_LAUNCH("attn_gather_v", (attn_gather_kernel<HD, GMAX>), dim3(grid), dim3(C::THREADS), C::SMEM, st, d);
}

void launch_attention(const AttnArgs& a, cudaStream_t st) {
  const sol_shape_t& sh = a.shape;
  const int Hq = sh.n_q_heads, Hkv = sh.n_kv_heads, hd = sh.head_dim, G = Hq / Hkv, HG = (G + 3) / 4;
  const int Tmax = a.kv.max_pages_per_seq * PAGE;

  PrepDev pd;
  pd.sh = sh; pd.kv = a.kv; pd.qkv = a.qkv_f32; pd.ldq = a.ldq; pd.ksplit = a.qkv_ksplit; pd.B = a.B;
  pd.qkv_scale = a.qkv_scale;
  pd.q_bf16 = static_cast<const uint16_t*>(a.q_bf16);
  pd.q_rot = a.q_rot; pd.q_split = static_cast<uint16_t*>(a.q_split); pd.work_ctr = a.work_ctr; pd.status = a.status;
  pd.row_hist = a.row_hist; pd.row_ctl = a.row_ctl; pd.seg_pub = a.seg_pub;
  pd.nseg_max = attn_select_segs(a.kv.max_pages_per_seq, PAGE);
  pd.plan = a.plan; pd.r_permille = a.r_permille; pd.split_len = attn_split_len(hd);
  pd.target_items = sm_count() * (hd == 64 ? 12 : 8);  // the pass-2 warps resident at once
  pd.max_item_chunks = 1024 / attn_split_len(hd);
  SOL_LAUNCH("attn_prep_rope_append", attn_prep_kernel, dim3(Hkv, a.B), dim3(PREP_THREADS), 0, st, pd);

  if (a.span_tokens > 0) {  // KV refresh: the rows are spans of one sequence's tokens, every token before a row's own is kept
    launch_span_attention(a, a.span_tokens, st);
    return;
  }
  if (sh.token_select == SOL_SELECT_QUEST_PAGES) {
    // the paper's page selection per query head (sol_quest.cu) instead of pass 1 and the token selection; a
    // layer step has just appended a key, so the extrema of its block are taken again first
    launch_quest_selection(a, a.qkv_f32 != nullptr, st);
    launch_quest_attend(a, st);
    return;
  } else {
    ScoreDev sd;
    sd.kv = a.kv; sd.Hkv = Hkv; sd.G = G; sd.HG = HG; sd.Tmax = Tmax;
    sd.q_split = static_cast<const uint16_t*>(a.q_split);
    sd.logits = a.logits; sd.sigma = a.sigma; sd.status = a.status; sd.B = a.B;
    const int groups_per_row = (a.kv.max_pages_per_seq + SC_WARPS - 1) / SC_WARPS;
    if (hd == 64) launch_score<64>(sd, HG, groups_per_row, st);
    else launch_score<128>(sd, HG, groups_per_row, st);

    SelectDev se;
    se.sh = sh; se.kv = a.kv; se.r_permille = a.r_permille; se.Tmax = Tmax; se.S = a.splits;
    se.split_len = attn_split_len(hd); se.q_rot = a.q_rot; se.B = a.B;
    se.nseg_max = attn_select_segs(a.kv.max_pages_per_seq, PAGE);
    se.sigma = a.sigma; se.row_hist = a.row_hist; se.row_ctl = a.row_ctl; se.seg_pub = a.seg_pub;
    se.cand_idx = a.cand_idx; se.cand_val = a.cand_val; se.list_idx = a.list_idx; se.list_row = a.kept_row;
    se.kept_cnt = a.kept_cnt; se.work_items = a.work_items; se.work_ctr = a.work_ctr; se.status = a.status;
    se.plan = a.plan;
    {
      // persistent grids: never more CTAs than are resident at once, never more than there can be units
      static int hist_per_sm[2] = {0, 0}, scan_per_sm = 0;
      if (scan_per_sm == 0) {
        int n = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, token_hist_kernel<false>, TS_THREADS, 0) != cudaSuccess || n < 1) n = 1;
        hist_per_sm[0] = n;
        n = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, token_hist_kernel<true>, TS_THREADS, 0) != cudaSuccess || n < 1) n = 1;
        hist_per_sm[1] = n;
        n = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, token_scan_kernel, TS_THREADS, 0) != cudaSuccess || n < 1) n = 1;
        scan_per_sm = n;
      }
      const bool local = Tmax <= TH_SEG;
      const long long hist_units = (long long)a.B * Hkv * ((Tmax + TH_SEG - 1) / TH_SEG);
      const long long scan_units = (long long)a.B * Hkv * se.nseg_max;
      const long long hist_res = (long long)sm_count() * hist_per_sm[local ? 1 : 0], scan_res = (long long)sm_count() * scan_per_sm;
      const dim3 hist_grid((unsigned)(hist_units < hist_res ? hist_units : hist_res));
      if (local) SOL_LAUNCH("token_hist", token_hist_kernel<true>, hist_grid, dim3(TS_THREADS), 0, st, se);
      else SOL_LAUNCH("token_hist", token_hist_kernel<false>, hist_grid, dim3(TS_THREADS), 0, st, se);
      if (Tmax > TH_SEG) {  // shorter rows are taken through the whole selection by token_hist
        SOL_LAUNCH("token_scan", token_scan_kernel, dim3((unsigned)(scan_units < scan_res ? scan_units : scan_res)),
                   dim3(TS_THREADS), 0, st, se);
        SOL_LAUNCH("token_settle", token_settle_kernel, dim3(Hkv, a.B), dim3(TS_THREADS), 0, st, se);
      }
    }
    if (a.kept_idx_out != nullptr) {
      ListDev ld;
      ld.sh = sh; ld.kv = a.kv; ld.r_permille = a.r_permille; ld.Tmax = Tmax; ld.sigma = a.sigma; ld.row_ctl = a.row_ctl;
      ld.kept_idx = a.kept_idx_out;
      SOL_LAUNCH("token_list", token_list_kernel, dim3(Hkv, a.B), dim3(TS_THREADS), 0, st, ld);
    }
  }

  GatherDev gd;
  gd.kv = a.kv; gd.Hq = Hq; gd.Hkv = Hkv; gd.G = G; gd.Tmax = Tmax; gd.S = a.splits;
  gd.logits = a.logits; gd.kept_idx = a.list_idx; gd.kept_row = a.kept_row;
  gd.work_items = a.work_items; gd.work_ctr = a.work_ctr; gd.part = a.part;
  gd.scale_log2 = (float)(1.4426950408889634 / sqrt((double)hd));
  gd.out_f32 = a.out_f32;
  gd.out_bf16 = static_cast<uint16_t*>(a.out_bf16);
  gd.out_hi = static_cast<uint16_t*>(a.out_hi); gd.out_rows = a.out_rows;
  gd.status = a.status;
  const long long items = (long long)a.B * Hkv * a.splits;
  if (hd == 64) {
    if (G <= 4) launch_gather<64, 4>(gd, items, st);
    else launch_gather<64, 8>(gd, items, st);
  } else {
    if (G <= 4) launch_gather<128, 4>(gd, items, st);
    else launch_gather<128, 8>(gd, items, st);
  }
}

}  // namespace sol
