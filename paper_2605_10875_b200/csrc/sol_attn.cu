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

#include "sol_common.cuh"
#include "sol_internal.h"
#include "sol_select.cuh"

namespace sol {

constexpr int PAGE = 64;

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
  int* status;
};

constexpr int PREP_THREADS = 128;
// words of AttnArgs::work_ctr
enum : int { WC_ITEMS = 0, WC_NEXT = 1, WC_CPI = 2, WC_DONE = 4 };

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
  // for the choice of the pass-2 item length
  int B, n_sink, n_window, split_len, target_items;
  const int32_t* r_permille;
  int32_t* work_ctr;
  int* status;
};

constexpr int SC_WARPS = 4;  // pages per CTA

template <int HD, int HG>
__global__ void __launch_bounds__(SC_WARPS * 32) attn_score_kernel(const ScoreDev p) {
  extern __shared__ __align__(128) unsigned char smem[];
  constexpr int PAGE_BYTES = PAGE * HD * 2;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + SC_WARPS * PAGE_BYTES);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b = blockIdx.z, kvh = blockIdx.y;
  pdl_trigger();
  // The grid covers the longest row the page table allows; the CTAs beyond this sequence's length leave
  // before anything else (the lengths are an input of the step, not the work of an earlier kernel).  The
  // first CTA stays: it also sizes the pass-2 items.
  if (blockIdx.x * SC_WARPS * PAGE >= p.kv.seq_lens[b] && (blockIdx.x | blockIdx.y | blockIdx.z) != 0) return;
  if (threadIdx.x == 0) {
    for (int i = 0; i < SC_WARPS; ++i) mbar_init(&bars[i], 1);
    fence_mbar_init();
  }
  __syncthreads();
  pdl_wait();

  // Length of the pass-2 work items, in chunks of split_len kept tokens (the first CTA finds it for the batch,
  // from the kept counts the budgets imply): the smallest run length (up to ATTN_ITEM_CHUNKS) that gives
  // every resident CTA of pass 2 at most one item, so that there is no second, partly filled round of
  // items; when even the longest runs leave more items than CTAs there is work for many rounds, and runs
  // of 8 chunks, claimed one by one, balance it.
  if (blockIdx.x == 0 && kvh == 0 && b == 0) {
    __shared__ int n_items[ATTN_ITEM_CHUNKS];
        if (threadIdx.x < ATTN_ITEM_CHUNKS) n_items[threadIdx.x] = 0;
    __syncthreads();
    for (int i0 = warp * 32; i0 < p.B; i0 += SC_WARPS * 32) {  // one sequence per lane
      const int i = i0 + lane;
      int ch = 0;
      if (i < p.B) {
        const int Ti = min(p.kv.seq_lens[i], p.kv.max_pages_per_seq * PAGE);
        ch = 1;
        if (Ti > 0) {
          const int ns_ = min(max(p.n_sink, 0), Ti), nw_ = min(max(p.n_window, 0), Ti - ns_);
          long long bd = ((long long)p.r_permille[i] * Ti + 999) / 1000;
          if (bd > Ti) bd = Ti;
          ch = max(1, (min(Ti, max((int)bd, ns_ + nw_)) + p.split_len - 1) / p.split_len);
        }
      }
#pragma unroll
      for (int c = 1; c <= ATTN_ITEM_CHUNKS; ++c) {
        const int n = __reduce_add_sync(0xffffffffu, (ch + c - 1) / c);
        if (lane == 0) atomicAdd(&n_items[c - 1], n);
      }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      int cpi = 8;
      for (int c = ATTN_ITEM_CHUNKS; c >= 1; --c)
        if ((long long)n_items[c - 1] * p.Hkv <= p.target_items) cpi = c;
      p.work_ctr[WC_CPI] = cpi;
    }
  }

  const int T = min(p.kv.seq_lens[b], p.kv.max_pages_per_seq * PAGE);  // never index past the page table
  const int lp = blockIdx.x * SC_WARPS + warp;  // logical page
  if (lp * PAGE >= T || lp >= p.kv.max_pages_per_seq) return;
  const int page = p.kv.page_table[(size_t)b * p.kv.max_pages_per_seq + lp];
  if (page < 0 || page >= p.kv.num_pages) {
    if (lane == 0) atomicOr(p.status + ST_ERR, ERR_BAD_PAGE);
    return;
  }
  unsigned char* tile = smem + warp * PAGE_BYTES;
  if (lane == 0) {
    mbar_expect_tx(&bars[warp], PAGE_BYTES);
    bulk_g2s(tile, static_cast<const uint16_t*>(p.kv.k_pool) + ((size_t)page * p.Hkv + kvh) * PAGE * HD, PAGE_BYTES,
             &bars[warp]);
  }

  // query operand fragments: B[k][n] = q_split[n][k]; this lane holds rows g and 8+g, 8 k-values per pair step
  const int g = lane >> 2, t = lane & 3;
  constexpr int KS = HD / 32;  // pair steps (two MMAs of k=16 each)
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

  const bool ok = mbar_wait(&bars[warp], 0, p.status);
  if (!ok) return;

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
      if (tok0 < T) p.sigma[row0 + tok0] = sig0;
      if (tok1 < T) p.sigma[row0 + tok1] = sig1;
    }
  }
}

// ============================================================================
// token_select
// ============================================================================
struct SelectDev {
  sol_shape_t sh;
  sol_kv_t kv;
  const int32_t* r_permille;
  int Tmax, S, split_len, B;
  const float* q_rot;
  const float* sigma;
  int32_t* kept_idx;
  int32_t* kept_cnt;
  uint32_t* kept_row;
  int32_t* work_items;
  int32_t* work_ctr;
  int* status;
};

// One CTA per (sequence, kv-head).  Every thread owns `per` consecutive tokens; their scores sit in
// shared memory (as order-preserving keys, slot i of thread t at [i * THREADS + t]) for all passes, and
// every loop over them is a rolled one: the kernel is a long chain of short passes, and unrolled over
// register arrays it spent more time waiting for instructions than for data.  Candidates near the
// threshold are settled in float64.
template <int THREADS>
__global__ void __launch_bounds__(THREADS) token_select_kernel(const SelectDev p) {
  __shared__ SelectSmem sm;
  __shared__ double qsum[128];
  extern __shared__ __align__(16) uint32_t skey[];  // [per][THREADS]

  const int kvh = blockIdx.x, b = blockIdx.y;
  const int Hkv = p.sh.n_kv_heads, hd = p.sh.head_dim, G = p.sh.n_q_heads / Hkv;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  constexpr int WARPS = THREADS / 32;
  constexpr int KPT = 0;  // rolled key loops
  const int bk = b * Hkv + kvh;
  pdl_trigger();
  pdl_wait();
  const int T = min(p.kv.seq_lens[b], p.kv.max_pages_per_seq * PAGE);  // never index past the page table
  const size_t row = (size_t)bk * p.Tmax;
  const float* sig = p.sigma + row;
  // a thread owns `per` consecutive tokens: as few as this sequence needs (a multiple of 4 for the
  // vector loads), so a short context in a long-context batch costs what its own length costs
  const int per = ((max(T, 1) + THREADS - 1) / THREADS + 3) / 4 * 4;
  const int j0 = tid * per;
  auto key = [&](int i) { return skey[i * THREADS + tid]; };  // 0: absent, 0xffffffff: forced

  int total = 0;
  if (T > 0) {
    const int n_sink = min(max(p.sh.n_sink, 0), T);
    const int n_win = min(max(p.sh.n_window, 0), T - n_sink);
    const int nf = n_sink + n_win;
    long long bud = ((long long)p.r_permille[b] * T + 999) / 1000;
    if (bud > T) bud = T;
    const int k = min(T, max((int)bud, nf));
    auto forced = [&](int j) { return j < n_sink || j >= T - n_win; };
    if (tid < 4) sm.counts[tid] = 0;

    // mode 0: keep all; 1: forced only; 2: the key slots hold classes (settled by the window pass and
    // the float64 ranking); 3: key threshold with index-ordered ties (float32 ordering, the candidate
    // list overflowed)
    constexpr uint32_t CLS_DROP = 0u, CLS_KEEP = 2u, CLS_CAND = 3u;
    int mode, tie_need = 0;
    uint32_t key_thr = 0;
    int my_keep = 0, my_ties = 0;  // of this thread's tokens: kept for sure, tied at the threshold

    if (k >= T) {
      mode = 0;
      my_keep = min(max(T - j0, 0), per);
    } else if (k <= nf) {
      mode = 1;
      for (int i = 0; i < per; ++i) my_keep += j0 + i < T && forced(j0 + i);
    } else {
      float mx = 0.f;
#pragma unroll 1
      for (int i = 0; i < per; i += 4) {
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (j0 + i < T) v = *reinterpret_cast<const float4*>(sig + j0 + i);
        const float vv[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int j = j0 + i + e;
          uint32_t kk = 0;
          if (j < T) {
            if (forced(j)) {
              kk = 0xffffffffu;
            } else {
              const float sv = vv[e] + 0.0f;
              kk = float_key(sv);
              mx = fmaxf(mx, fabsf(sv));
            }
          }
          skey[(i + e) * THREADS + tid] = kk;
        }
      }
      mx = block_max<THREADS>(mx, 0, sm);
      key_thr = select_kth<THREADS, KPT, true>(key, k, tie_need, sm, per);

      // ---- window around the threshold, re-scored in float64 ----
      const float thr32 = key_to_float(key_thr);
      // 2^-16 of the largest score: far above the float32 accumulation error of a head_dim-long dot product
      const float delta = mx * 1.52587890625e-05f;
      const float hi = thr32 + delta, lo = thr32 - delta;
      // One pass counts what is clear of the window and lists the candidates inside it.
      int n_in = 0, my_cand = 0;
#pragma unroll 4
      for (int i = 0; i < per; ++i) {
        const uint32_t kk = key(i);
        if (kk == 0xffffffffu) {
          ++my_keep;
        } else if (kk != 0u) {
          const float sv = key_to_float(kk);
          if (sv > hi) {
            ++n_in;
          } else if (sv >= lo) {
            ++my_cand;
            const int slot = atomicAdd(&sm.counts[0], 1);
            if (slot < SEL_CAND_CAP) sm.cand_idx[slot] = j0 + i;
          }
        }
      }
      my_keep += n_in;
      n_in = block_count<THREADS>(n_in, 0, sm);
      const int n_cand = sm.counts[0];
      const int need = k - nf - n_in;
      if (n_cand > SEL_CAND_CAP) {
        if (tid == 0) atomicAdd(p.status + ST_TOK_OVERFLOW, 1);
        mode = 3;
        my_keep = 0;
#pragma unroll 1
        for (int i = 0; i < per; ++i) {
          const uint32_t kk = key(i);
          my_keep += kk > key_thr && kk != 0u;
          my_ties += kk == key_thr;
        }
      } else {
        if (n_cand != need) {
          if (tid == 0) atomicAdd(p.status + ST_TOK_REFINED, n_cand);
          for (int e = tid; e < hd; e += THREADS) {
            double a = 0.0;
            for (int h = 0; h < G; ++h) a += (double)p.q_rot[((size_t)b * p.sh.n_q_heads + kvh * G + h) * hd + e];
            qsum[e] = a;
          }
          __syncthreads();
          const uint16_t* kp = static_cast<const uint16_t*>(p.kv.k_pool);
          for (int c = warp; c < n_cand; c += WARPS) {
            const int j = sm.cand_idx[c];
            const int page = p.kv.page_table[(size_t)b * p.kv.max_pages_per_seq + j / PAGE];
            double a = 0.0;
            if (page >= 0 && page < p.kv.num_pages) {
              const uint16_t* kr = kp + (((size_t)page * Hkv + kvh) * PAGE + (j % PAGE)) * hd;
              for (int e = lane; e < hd; e += 32) a += qsum[e] * (double)bf2f(kr[e]);
            }
            a = warp_sum_d(a);
            if (lane == 0) sm.cand_val[c] = a;
          }
          __syncthreads();
          rank_candidates<THREADS>(n_cand, need, sm);
        } else {
          for (int c = tid; c < n_cand; c += THREADS) sm.cand_keep[c] = 1;
        }
        mode = 2;
        __syncthreads();
        // the key slot of every candidate takes its class: a kept one sorts above every key, a dropped
        // one below (token j is slot j % per of thread j / per), so that one comparison with the window
        // classifies any slot from here on
        for (int c = tid; c < n_cand; c += THREADS) {
          const int j = sm.cand_idx[c];
          skey[(j % per) * THREADS + j / per] = sm.cand_keep[c] ? 0xffffffffu : 0u;
        }
        __syncthreads();
        if (my_cand > 0) {  // few threads own candidates: they count their kept ones
#pragma unroll 1
          for (int i = 0; i < per; ++i) {
            const uint32_t kk = key(i);
            // a forced token or a kept candidate now; the forced ones were counted above
            my_keep += kk == 0xffffffffu && !(j0 + i < T && forced(j0 + i));
          }
        }
        key_thr = float_key(hi);  // kept: keys above the window (candidates inside it are settled)
      }
    }

    // class of this thread's i-th token: 2 kept, 1 tie, 0 dropped
    auto klass = [&](int i) -> int {
      const int j = j0 + i;
      if (j >= T) return 0;
      if (mode == 0) return 2;
      if (mode == 1) return forced(j) ? 2 : 0;
      const uint32_t kk = key(i);
      if (mode == 2) return kk > key_thr ? 2 : 0;
      return kk > key_thr ? 2 : (kk == key_thr ? 1 : 0);
    };
    // beside the index list, the cache row of every kept token (page table applied), so that pass 2
    // goes from the list straight to the V rows
    const int32_t* table = p.kv.page_table + (size_t)b * p.kv.max_pages_per_seq;
    auto emit = [&](int i, bool keep, int pos) {
      if (!keep) return;
      const int j = j0 + i;
      const int page = table[j / PAGE];
      uint32_t ridx = 0xffffffffu;
      if (page >= 0 && page < p.kv.num_pages) ridx = (uint32_t)((page * Hkv + kvh) * PAGE + (j % PAGE));
      else atomicOr(p.status + ST_ERR, ERR_BAD_PAGE);
      p.kept_row[row + pos] = ridx;
    };
    total = compact_counted<THREADS, KPT>(my_keep, my_ties, klass, emit, mode == 3 ? tie_need : 0, p.kept_idx + row,
                                          sm, per);
  }
  if (tid == 0) p.kept_cnt[bk] = total;

  // Pass-2 work items of this (sequence, kv-head): runs of `cpi` chunks of split_len kept tokens (at least
  // one item, so that the output is always written); cpi was chosen by the query preparation kernel.
  const int cpi = p.work_ctr[WC_CPI];
  const int chunks = max(1, (total + p.split_len - 1) / p.split_len);
  const int ns = (chunks + cpi - 1) / cpi;
  if (tid == 0) sm.counts[3] = atomicAdd(p.work_ctr + WC_ITEMS, ns);
  __syncthreads();
  const int base = sm.counts[3];
  for (int i = tid; i < ns; i += THREADS) {
    p.work_items[2 * (base + i)] = bk * p.S + i * cpi;  // first chunk of the item
    p.work_items[2 * (base + i) + 1] = total;
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
  uint16_t* out_hi;
  uint16_t* out_lo;
  int* status;
};

constexpr int GA_WARPS = 8;
constexpr int GA_THREADS = GA_WARPS * 32;
constexpr int GA_BATCH = 32;  // kept tokens per warp step: one per lane in the softmax part
constexpr int GA_ROWS_IN_FLIGHT = 8;  // row loads a lane issues before it consumes the first

// Pass 2 is a gather of 128- or 256-byte V rows with G multiply-adds per element: bound by memory
// latency, not by arithmetic, so it runs on the FMA pipes with many warps per SM and no shared-memory
// staging of the rows.
//
// Persistent CTAs work through the list of items: (sequence, kv-head, run of at most 1024 kept tokens);
// a CTA's first item is dealt by its index, the later ones are claimed from a counter one item ahead.
// The 8 warps of a CTA take the item's tokens in batches of 32, each warp on its own:
//   lane l of the warp fetches the index words and the G logits of token l of the batch (the next
//   batch's while the current one is processed), the warp updates its running maximum per head and
//   every lane computes its token's softmax weights; cache rows and weights go to a small
//   shared-memory table; then the warp walks over the batch's rows: a row is read by HD/4 lanes (8
//   bytes each, 8 rows in flight per lane) and multiplied into the lane's float32 accumulators
//   (G heads x 4 columns).
// Per item one partial (accumulators, maximum, sum; merged over the warps) is written; the CTA that
// finishes the last item of a (sequence, kv-head) merges its partials.
template <int HD, int GMAX>
__global__ void __launch_bounds__(GA_THREADS, GMAX == 4 ? 4 : 2) attn_gather_kernel(const GatherDev p) {
  constexpr int SPLIT = HD == 64 ? 256 : 128;  // kept tokens per chunk (attn_split_len): the unit of the item list
  constexpr int LPT = HD / 4;                  // lanes per row
  constexpr int TPS = 32 / LPT;                // rows per warp-wide load
  constexpr int U = GA_ROWS_IN_FLIGHT;
  static_assert(GA_BATCH % (U * TPS) == 0, "a batch is a whole number of load groups");
  __shared__ uint32_t s_row[GA_WARPS][GA_BATCH];
  __shared__ __align__(16) float s_w[GA_WARPS][GA_BATCH][GMAX];
  __shared__ __align__(16) float sc_acc[GA_WARPS][GMAX][HD];
  __shared__ float sc_ml[GA_WARPS][GMAX][2];
  __shared__ __align__(16) int hdr[2][4];  // (sequence, kv-head) or -1, first token, tokens, kept count
  __shared__ int flag;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = p.G, Hkv = p.Hkv;
  const uint16_t* vp = static_cast<const uint16_t*>(p.kv.v_pool);
  const int sub = lane / LPT, col = (lane % LPT) * 4;  // which row of a load step, which four columns
  pdl_trigger();
  pdl_wait();
  const int cpi = p.work_ctr[WC_CPI];
  const int n_items = p.work_ctr[WC_ITEMS];
  auto header_of = [&](int2 w) {
    const int bk = w.x / p.S, n0 = (w.x % p.S) * SPLIT;
    return make_int4(bk, n0, max(0, min(w.y - n0, cpi * SPLIT)), w.y);
  };
  if (tid == 0) {
    int4 h = make_int4(-1, 0, 0, 0);
    if ((int)blockIdx.x < n_items) h = header_of(*reinterpret_cast<const int2*>(p.work_items + 2 * blockIdx.x));
    *reinterpret_cast<int4*>(hdr[0]) = h;
  }
  __syncthreads();

#pragma unroll 1
  for (int it = 0;; ++it) {
    const int4 cur = *reinterpret_cast<const int4*>(hdr[it & 1]);
    if (cur.x < 0) break;
    int claimed = 0;
    if (tid == 0) claimed = (int)gridDim.x + atomicAdd(p.work_ctr + WC_NEXT, 1);
    const int bk = cur.x, len = cur.z, cnt = cur.w;
    const int b = bk / Hkv, kvh = bk % Hkv;
    const size_t row = (size_t)bk * p.Tmax;
    const uint32_t* krow = p.kept_row + row + cur.y;
    const int32_t* kidx = p.kept_idx + row + cur.y;
    const float* lgrow = p.logits + row * G;
    const int nb = (len + GA_BATCH - 1) / GA_BATCH;

    auto load_idx = [&](int q, uint32_t& r, int& j) {
      const int n = q * GA_BATCH + lane;
      r = 0xffffffffu;
      j = 0;
      if (q < nb && n < len) {
        r = krow[n];
        j = kidx[n];
      }
    };
    auto load_logits = [&](uint32_t r, int j, float (&x)[GMAX]) {
#pragma unroll
      for (int h = 0; h < GMAX; ++h) x[h] = -INFINITY;  // an absent token weighs nothing
      if (r == 0xffffffffu) return;
      const float* src = lgrow + (size_t)j * G;
      if (GMAX == 4 && G == 4) {
        const float4 v = *reinterpret_cast<const float4*>(src);
        x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
      } else {
#pragma unroll
        for (int h = 0; h < GMAX; ++h)
          if (h < G) x[h] = src[h];
      }
    };

    float mh[GMAX], ls[GMAX], acc[GMAX][4];
#pragma unroll
    for (int h = 0; h < GMAX; ++h) {
      mh[h] = -INFINITY;
      ls[h] = 0.f;
#pragma unroll
      for (int c = 0; c < 4; ++c) acc[h][c] = 0.f;
    }
    uint32_t r_c, r_n;
    int j_c, j_n;
    float x_c[GMAX];
    load_idx(warp, r_c, j_c);
    load_idx(warp + GA_WARPS, r_n, j_n);
    load_logits(r_c, j_c, x_c);

#pragma unroll 1
    for (int q = warp; q < nb; q += GA_WARPS) {
      // the next batch's logits and the index words of the batch after it start now
      float x_n[GMAX];
      load_logits(r_n, j_n, x_n);
      uint32_t r_nn;
      int j_nn;
      load_idx(q + 2 * GA_WARPS, r_nn, j_nn);

      // ---- softmax weights relative to the running maximum ----
#pragma unroll
      for (int h = 0; h < GMAX; ++h) {
        const float x = x_c[h] * p.scale_log2;
        const float nm = fmaxf(mh[h], warp_max(x));
        const float sc = mh[h] == -INFINITY ? 0.f : exp2f(mh[h] - nm);
        const float pw = x == -INFINITY ? 0.f : exp2f(x - nm);
        mh[h] = nm;
        ls[h] = ls[h] * sc + pw;
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[h][c] *= sc;
        s_w[warp][lane][h] = pw;
      }
      s_row[warp][lane] = r_c;
      __syncwarp();

      // ---- weights x rows ----
      const int nt = min(GA_BATCH, len - q * GA_BATCH);
#pragma unroll 1
      for (int k0 = 0; k0 < nt; k0 += U * TPS) {
        uint2 v[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
          const uint32_t r = s_row[warp][k0 + u * TPS + sub];
          v[u] = make_uint2(0u, 0u);
          if (r != 0xffffffffu) v[u] = __ldcs(reinterpret_cast<const uint2*>(vp + (size_t)r * HD + col));
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
          const float* w = s_w[warp][k0 + u * TPS + sub];
          const float f0 = __uint_as_float(v[u].x << 16), f1 = __uint_as_float(v[u].x & 0xffff0000u);
          const float f2 = __uint_as_float(v[u].y << 16), f3 = __uint_as_float(v[u].y & 0xffff0000u);
#pragma unroll
          for (int h4 = 0; h4 < GMAX; h4 += 4) {
            const float4 w4 = *reinterpret_cast<const float4*>(w + h4);
            const float ww[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              acc[h4 + e][0] = fmaf(ww[e], f0, acc[h4 + e][0]);
              acc[h4 + e][1] = fmaf(ww[e], f1, acc[h4 + e][1]);
              acc[h4 + e][2] = fmaf(ww[e], f2, acc[h4 + e][2]);
              acc[h4 + e][3] = fmaf(ww[e], f3, acc[h4 + e][3]);
            }
          }
        }
      }
      __syncwarp();  // the tables are rewritten for the next batch
      r_c = r_n;
      j_c = j_n;
#pragma unroll
      for (int h = 0; h < GMAX; ++h) x_c[h] = x_n[h];
      r_n = r_nn;
      j_n = j_nn;
    }

    // ---- one partial per item: merge the warps ----
    if (TPS == 2) {  // two rows per load step: the half-warps hold partial sums of the same columns
#pragma unroll
      for (int h = 0; h < GMAX; ++h)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[h][c] += __shfl_xor_sync(0xffffffffu, acc[h][c], 16);
    }
#pragma unroll
    for (int h = 0; h < GMAX; ++h) ls[h] = warp_sum(ls[h]);
    if (sub == 0) {
#pragma unroll
      for (int h = 0; h < GMAX; ++h)
        *reinterpret_cast<float4*>(&sc_acc[warp][h][col]) = make_float4(acc[h][0], acc[h][1], acc[h][2], acc[h][3]);
    }
    if (lane == 0) {
#pragma unroll
      for (int h = 0; h < GMAX; ++h) {
        sc_ml[warp][h][0] = mh[h];
        sc_ml[warp][h][1] = ls[h];
      }
    }
    // the header of the claimed item is fetched while the partial is put together
    int2 claimed_words = make_int2(0, 0);
    if (tid == 0 && claimed < n_items) claimed_words = *reinterpret_cast<const int2*>(p.work_items + 2 * claimed);
    __syncthreads();
    const int slot_no = (cur.y / SPLIT) / cpi;  // this item's partial
    float* dst = p.part + (((size_t)bk * p.S + slot_no) * G) * (HD + 2);
    for (int e0 = tid; e0 < G * HD; e0 += GA_THREADS) {
      const int h = e0 / HD, e = e0 % HD;
      float M = -INFINITY;
#pragma unroll
      for (int w = 0; w < GA_WARPS; ++w) M = fmaxf(M, sc_ml[w][h][0]);
      float a = 0.f, l = 0.f;
#pragma unroll
      for (int w = 0; w < GA_WARPS; ++w) {
        const float mw = sc_ml[w][h][0];
        const float f = mw == -INFINITY ? 0.f : exp2f(mw - M);
        a += sc_acc[w][h][e] * f;
        l += sc_ml[w][h][1] * f;
      }
      dst[h * (HD + 2) + e] = a;
      if (e == 0) {
        dst[h * (HD + 2) + HD] = M;
        dst[h * (HD + 2) + HD + 1] = l;
      }
    }

    // ---- the last item of this (sequence, kv-head) merges the partials ----
    const int chunks = max(1, (cnt + SPLIT - 1) / SPLIT);
    const int ns = (chunks + cpi - 1) / cpi;
    __threadfence();
    __syncthreads();
    if (tid == 0) {
      flag = atomicAdd(p.work_ctr + WC_DONE + bk, 1) == ns - 1 ? 1 : 0;
      int4 h = make_int4(-1, 0, 0, 0);
      if (claimed < n_items) h = header_of(claimed_words);
      *reinterpret_cast<int4*>(hdr[(it + 1) & 1]) = h;
    }
    __syncthreads();
    if (flag) {
      __threadfence();
      const float* src0 = p.part + ((size_t)bk * p.S * G) * (HD + 2);
      for (int e0 = tid; e0 < G * HD; e0 += GA_THREADS) {
        const int h = e0 / HD, e = e0 % HD;
        float m = -INFINITY, l = 0.f, a = 0.f;
        for (int q = 0; q < ns; ++q) {
          const float* src = src0 + ((size_t)q * G + h) * (HD + 2);
          const float m2 = __ldcg(src + HD), l2 = __ldcg(src + HD + 1), a2 = __ldcg(src + e);
          const float mn = fmaxf(m, m2);
          const float e1 = (m == -INFINITY) ? 0.f : exp2f(m - mn);
          const float e2 = (m2 == -INFINITY) ? 0.f : exp2f(m2 - mn);
          l = l * e1 + l2 * e2;
          a = a * e1 + a2 * e2;
          m = mn;
        }
        const float o = l > 0.f ? a / l : 0.f;
        const size_t idx = ((size_t)b * p.Hq + kvh * G + h) * HD + e;
        if (p.out_f32) p.out_f32[idx] = o;
        if (p.out_bf16) p.out_bf16[idx] = f2bf(o);
        if (p.out_hi) {
          const uint16_t hi = f2bf(o);
          p.out_hi[idx] = hi;
          p.out_lo[idx] = f2bf(o - bf2f(hi));
        }
      }
    }
    __syncthreads();  // the merge scratch, the flag and the headers are reused by the next item
  }
}

// ============================================================================
// host side
// ============================================================================
template <int HD>
static void launch_score(const ScoreDev& d, int HG, dim3 grid, cudaStream_t st) {
  const int smem = SC_WARPS * PAGE * HD * 2 + SC_WARPS * 8 + 32;
  if (HG == 1) {
    ensure_dynamic_smem(reinterpret_cast<const void*>(&attn_score_kernel<HD, 1>), smem);
    SOL_LAUNCH("attn_score", (attn_score_kernel<HD, 1>), grid, dim3(SC_WARPS * 32), smem, st, d);
  } else {
    ensure_dynamic_smem(reinterpret_cast<const void*>(&attn_score_kernel<HD, 2>), smem);
    SOL_LAUNCH("attn_score", (attn_score_kernel<HD, 2>), grid, dim3(SC_WARPS * 32), smem, st, d);
  }
}

// One CTA per item, at most as many CTAs as are resident at once (they are persistent).
template <int HD, int GMAX>
static void launch_gather(const GatherDev& d, long long items, cudaStream_t st) {
  static int per_sm = 0;  // the same on every device this library supports
  if (per_sm == 0) {
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, attn_gather_kernel<HD, GMAX>, GA_THREADS, 0) != cudaSuccess || n < 1)
      n = 1;
    per_sm = n;
  }
  const long long resident = (long long)sm_count() * per_sm;
  const int grid = (int)(items < resident ? items : resident);
  SOL_LAUNCH("attn_gather_v", (attn_gather_kernel<HD, GMAX>), dim3(grid), dim3(GA_THREADS), 0, st, d);
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
  SOL_LAUNCH("attn_prep_rope_append", attn_prep_kernel, dim3(Hkv, a.B), dim3(PREP_THREADS), 0, st, pd);

  ScoreDev sd;
  sd.kv = a.kv; sd.Hkv = Hkv; sd.G = G; sd.HG = HG; sd.Tmax = Tmax;
  sd.q_split = static_cast<const uint16_t*>(a.q_split);
  sd.logits = a.logits; sd.sigma = a.sigma; sd.status = a.status;
  sd.B = a.B; sd.n_sink = sh.n_sink; sd.n_window = sh.n_window; sd.split_len = attn_split_len(hd);
  sd.target_items = sm_count() * (G <= 4 ? 4 : 2);  // the pass-2 CTAs resident at once
  sd.r_permille = a.r_permille; sd.work_ctr = a.work_ctr;
  dim3 sgrid((a.kv.max_pages_per_seq + SC_WARPS - 1) / SC_WARPS, Hkv, a.B);
  if (hd == 64) launch_score<64>(sd, HG, sgrid, st);
  else launch_score<128>(sd, HG, sgrid, st);

  SelectDev se;
  se.sh = sh; se.kv = a.kv; se.r_permille = a.r_permille; se.Tmax = Tmax; se.S = a.splits;
  se.split_len = attn_split_len(hd); se.q_rot = a.q_rot; se.B = a.B;
  se.sigma = a.sigma; se.kept_idx = a.kept_idx; se.kept_cnt = a.kept_cnt; se.kept_row = a.kept_row;
  se.work_items = a.work_items; se.work_ctr = a.work_ctr; se.status = a.status;
  {
    // keys of the longest row in shared memory: 4 bytes per token, rounded up to four per thread; rows up
    // to 1024 tokens take 256 threads, longer ones 1024
    const dim3 grid(Hkv, a.B);
    if (Tmax <= 1024) {
      const int smem = ((Tmax + 256 - 1) / 256 + 3) / 4 * 4 * 256 * 4;
      ensure_dynamic_smem(reinterpret_cast<const void*>(&token_select_kernel<256>), smem);
      SOL_LAUNCH("token_select", token_select_kernel<256>, grid, dim3(256), smem, st, se);
    } else {
      const int smem = ((Tmax + 1024 - 1) / 1024 + 3) / 4 * 4 * 1024 * 4;
      ensure_dynamic_smem(reinterpret_cast<const void*>(&token_select_kernel<1024>), smem);
      SOL_LAUNCH("token_select", token_select_kernel<1024>, grid, dim3(1024), smem, st, se);
    }
  }

  GatherDev gd;
  gd.kv = a.kv; gd.Hq = Hq; gd.Hkv = Hkv; gd.G = G; gd.Tmax = Tmax; gd.S = a.splits;
  gd.logits = a.logits; gd.kept_idx = a.kept_idx; gd.kept_row = a.kept_row;
  gd.work_items = a.work_items; gd.work_ctr = a.work_ctr; gd.part = a.part;
  gd.scale_log2 = (float)(1.4426950408889634 / sqrt((double)hd));
  gd.out_f32 = a.out_f32;
  gd.out_bf16 = static_cast<uint16_t*>(a.out_bf16);
  gd.out_hi = static_cast<uint16_t*>(a.out_hi); gd.out_lo = static_cast<uint16_t*>(a.out_lo);
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
