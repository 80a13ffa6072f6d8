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
  const float* qkv;  // [B][ldq] or nullptr
  int ldq;
  const uint16_t* q_bf16;  // [B][Hq][hd] or nullptr
  float* q_rot;
  uint16_t* q_split;
  int* status;
};

__global__ void __launch_bounds__(256) attn_prep_kernel(const PrepDev p) {
  __shared__ float cs[64], sn[64];  // hd/2 <= 64
  const int b = blockIdx.x;
  const int Hq = p.sh.n_q_heads, Hkv = p.sh.n_kv_heads, hd = p.sh.head_dim, half = hd / 2;
  const int G = Hq / Hkv, HG = (G + 3) / 4;
  const int T = min(p.kv.seq_lens[b], p.kv.max_pages_per_seq * PAGE);  // never index past the page table
  const int pos = T - 1;
  const bool layer = p.qkv != nullptr;
  const bool rope = layer && p.sh.rope_theta > 0.f;
  if (threadIdx.x < half) {
    float c = 1.f, s = 0.f;
    if (rope) {
      const double inv = pow((double)p.sh.rope_theta, -2.0 * (double)threadIdx.x / (double)hd);
      double sd, cd;
      sincos((double)pos * inv, &sd, &cd);
      c = (float)cd;
      s = (float)sd;
    }
    cs[threadIdx.x] = c;
    sn[threadIdx.x] = s;
  }
  __syncthreads();

  // zero the operand rows that carry no head (pad rows and the unused fourth slot)
  uint16_t* qs = p.q_split + (size_t)b * Hkv * HG * 16 * hd;
  for (int i = threadIdx.x; i < Hkv * HG * 16 * hd; i += blockDim.x) qs[i] = 0;
  __syncthreads();

  // queries
  for (int i = threadIdx.x; i < Hq * hd; i += blockDim.x) {
    const int h = i / hd, e = i % hd;
    float q;
    if (layer) {
      const float* src = p.qkv + (size_t)b * p.ldq + h * hd;
      const int f = e < half ? e : e - half;
      const float other = e < half ? -src[e + half] : src[e - half];
      q = src[e] * cs[f] + other * sn[f];
    } else {
      q = bf2f(p.q_bf16[((size_t)b * Hq + h) * hd + e]);
    }
    p.q_rot[((size_t)b * Hq + h) * hd + e] = q;
    const uint16_t hi = f2bf(q);
    const float r1 = q - bf2f(hi);
    const uint16_t mid = f2bf(r1);
    const float r2 = r1 - bf2f(mid);
    const uint16_t lo = f2bf(r2);
    const int kvh = h / G, gi = h % G, hg = gi >> 2, t = gi & 3;
    uint16_t* base = qs + ((size_t)(kvh * HG + hg) * 16) * hd + e;
    base[(2 * t) * hd] = hi;
    base[(2 * t + 1) * hd] = mid;
    base[(8 + 2 * t) * hd] = lo;
  }

  if (!layer) return;
  // new k (rotated) and v, rounded to bf16, written at position T-1
  if (T <= 0) return;
  const int lp = pos / PAGE, slot = pos % PAGE;
  const int page = lp < p.kv.max_pages_per_seq ? p.kv.page_table[(size_t)b * p.kv.max_pages_per_seq + lp] : -1;
  if (page < 0 || page >= p.kv.num_pages) {
    if (threadIdx.x == 0) atomicOr(p.status + ST_ERR, ERR_BAD_PAGE);
    return;
  }
  uint16_t* kp = static_cast<uint16_t*>(p.kv.k_pool);
  uint16_t* vp = static_cast<uint16_t*>(p.kv.v_pool);
  for (int i = threadIdx.x; i < Hkv * hd; i += blockDim.x) {
    const int h = i / hd, e = i % hd;
    const float* ks = p.qkv + (size_t)b * p.ldq + (Hq + h) * hd;
    const float* vs = p.qkv + (size_t)b * p.ldq + (Hq + Hkv + h) * hd;
    const int f = e < half ? e : e - half;
    const float other = e < half ? -ks[e + half] : ks[e - half];
    const float k = ks[e] * cs[f] + other * sn[f];
    const size_t dst = (((size_t)page * Hkv + h) * PAGE + slot) * hd + e;
    kp[dst] = f2bf(k);
    vp[dst] = f2bf(vs[e]);
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
  if (threadIdx.x == 0) {
    for (int i = 0; i < SC_WARPS; ++i) mbar_init(&bars[i], 1);
    fence_mbar_init();
  }
  __syncthreads();

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
  int Tmax;
  const float* q_rot;
  float* sigma;  // candidates are overwritten with +-inf once decided
  int32_t* kept_idx;
  int32_t* kept_cnt;
  int* status;
};

__global__ void __launch_bounds__(SEL_THREADS) token_select_kernel(const SelectDev p) {
  __shared__ SelectSmem sm;
  __shared__ double qsum[128];

  const int kvh = blockIdx.x, b = blockIdx.y;
  const int Hkv = p.sh.n_kv_heads, hd = p.sh.head_dim, G = p.sh.n_q_heads / Hkv;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int T = min(p.kv.seq_lens[b], p.kv.max_pages_per_seq * PAGE);  // never index past the page table
  const size_t row = ((size_t)b * Hkv + kvh) * p.Tmax;
  float* sig = p.sigma + row;
  if (T <= 0) {
    if (tid == 0) p.kept_cnt[b * Hkv + kvh] = 0;
    return;
  }
  const int n_sink = min(max(p.sh.n_sink, 0), T);
  const int n_win = min(max(p.sh.n_window, 0), T - n_sink);
  const int nf = n_sink + n_win;
  long long bud = ((long long)p.r_permille[b] * T + 999) / 1000;
  if (bud > T) bud = T;
  const int k = min(T, max((int)bud, nf));
  auto forced = [&](int j) { return j < n_sink || j >= T - n_win; };

  // mode 0: keep all; 1: forced only; 2: kept iff sigma > thr (candidates already decided and
  // overwritten with +-inf); 3: key threshold with index-ordered ties (float32 ordering)
  float thr = 0.f;
  uint32_t key_thr = 0;
  int tie_need = 0;
  int mode;

  if (k >= T) {
    mode = 0;
  } else if (k <= nf) {
    mode = 1;
  } else {
    key_thr = radix_select_kth(
        [&](int j) { return forced(j) ? 0xffffffffu : float_key(sig[j] + 0.0f); }, T, k, tie_need, sm);
    mode = 3;

    // ---- window around the threshold, re-scored in float64 ----
    const float thr32 = key_to_float(key_thr);
    float mx = 0.f;
    for (int j = tid; j < T; j += SEL_THREADS)
      if (!forced(j)) mx = fmaxf(mx, fabsf(sig[j]));
    mx = warp_max(mx);
    if (lane == 0) sm.f[warp] = mx;
    if (tid < 4) sm.counts[tid] = 0;
    __syncthreads();
    mx = sm.f[0];
    for (int i = 1; i < SEL_WARPS; ++i) mx = fmaxf(mx, sm.f[i]);
    // 2^-16 of the largest score: far above the float32 accumulation error of a head_dim-long dot product
    const float delta = mx * 1.52587890625e-05f;
    const float hi = thr32 + delta, lo = thr32 - delta;
    int n_in = 0;
    for (int j = tid; j < T; j += SEL_THREADS) {
      if (forced(j)) continue;
      const float s = sig[j] + 0.0f;
      if (s > hi) {
        ++n_in;
      } else if (s >= lo) {
        const int slot = atomicAdd(&sm.counts[0], 1);
        if (slot < SEL_CAND_CAP) sm.cand_idx[slot] = j;
      }
    }
    if (n_in) atomicAdd(&sm.counts[1], n_in);
    __syncthreads();
    const int n_cand = sm.counts[0];
    const int need = k - nf - sm.counts[1];
    if (n_cand > SEL_CAND_CAP) {
      if (tid == 0) atomicAdd(p.status + ST_TOK_OVERFLOW, 1);
    } else {
      if (n_cand != need) {
        if (tid == 0) atomicAdd(p.status + ST_TOK_REFINED, n_cand);
        for (int e = tid; e < hd; e += SEL_THREADS) {
          double a = 0.0;
          for (int h = 0; h < G; ++h) a += (double)p.q_rot[((size_t)b * p.sh.n_q_heads + kvh * G + h) * hd + e];
          qsum[e] = a;
        }
        __syncthreads();
        const uint16_t* kp = static_cast<const uint16_t*>(p.kv.k_pool);
        for (int c = warp; c < n_cand; c += SEL_WARPS) {
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
        rank_candidates(n_cand, need, sm, [&](int c, bool keep) { sig[sm.cand_idx[c]] = keep ? INFINITY : -INFINITY; });
      } else {
        for (int c = tid; c < n_cand; c += SEL_THREADS) sig[sm.cand_idx[c]] = INFINITY;
      }
      thr = hi;
      mode = 2;
      __syncthreads();
    }
  }

  auto klass = [&](int j) -> int {
    if (mode == 0) return 2;
    if (forced(j)) return 2;
    if (mode == 1) return 0;
    const float s = sig[j] + 0.0f;
    if (mode == 2) return s > thr ? 2 : 0;
    const uint32_t key = float_key(s);
    return key > key_thr ? 2 : (key == key_thr ? 1 : 0);
  };
  ordered_compact(klass, [](int, bool) {}, T, mode == 3 ? tie_need : 0, p.kept_idx + row,
                  p.kept_cnt + (b * Hkv + kvh), sm);
}

// ============================================================================
// attn_gather (pass 2) and combine
// ============================================================================
struct GatherDev {
  sol_kv_t kv;
  int Hkv, G, Tmax, S;
  const float* logits;
  const int32_t* kept_idx;
  const int32_t* kept_cnt;
  float* part;  // [B][Hkv][S][G][HD + 2]
  float scale_log2;
  int* status;
};

__device__ __forceinline__ void softmax_merge(float& m, float& l, float* acc, int n, float m2, float l2,
                                              const float* acc2) {
  const float mn = fmaxf(m, m2);
  const float e1 = (m == -INFINITY) ? 0.f : exp2f(m - mn);
  const float e2 = (m2 == -INFINITY) ? 0.f : exp2f(m2 - mn);
  l = l * e1 + l2 * e2;
  for (int i = 0; i < n; ++i) acc[i] = acc[i] * e1 + acc2[i] * e2;
  m = mn;
}

constexpr int GA_WARPS = 4;

template <int HD, int GMAX>
__global__ void __launch_bounds__(GA_WARPS * 32) attn_gather_kernel(const GatherDev p) {
  constexpr int LPT = HD / 8;       // lanes per token row (16 bytes each)
  constexpr int TPW = 32 / LPT;     // tokens per warp iteration
  __shared__ float sh_acc[GA_WARPS][GMAX][HD];
  __shared__ float sh_ml[GA_WARPS][GMAX][2];
  const int s = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int cnt = p.kept_cnt[b * p.Hkv + kvh];
  const int n0 = s * ATTN_SPLIT_LEN, n1 = min(cnt, n0 + ATTN_SPLIT_LEN);
  if (n0 >= n1) return;
  const size_t row = ((size_t)b * p.Hkv + kvh) * p.Tmax;
  const int grp = lane / LPT, sub = lane % LPT;
  const uint16_t* vp = static_cast<const uint16_t*>(p.kv.v_pool);
  const int G = p.G;

  float m[GMAX], l[GMAX], acc[GMAX][8];
#pragma unroll
  for (int h = 0; h < GMAX; ++h) {
    m[h] = -INFINITY;
    l[h] = 0.f;
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[h][e] = 0.f;
  }

  for (int n = n0 + warp * TPW + grp; n < n1; n += GA_WARPS * TPW) {
    const int j = p.kept_idx[row + n];
    const int page = p.kv.page_table[(size_t)b * p.kv.max_pages_per_seq + j / PAGE];
    if (page < 0 || page >= p.kv.num_pages) {
      atomicOr(p.status + ST_ERR, ERR_BAD_PAGE);
      continue;
    }
    const uint4 vw = *reinterpret_cast<const uint4*>(vp + (((size_t)page * p.Hkv + kvh) * PAGE + (j % PAGE)) * HD + sub * 8);
    const float v[8] = {bf16_lo(vw.x), bf16_hi(vw.x), bf16_lo(vw.y), bf16_hi(vw.y),
                        bf16_lo(vw.z), bf16_hi(vw.z), bf16_lo(vw.w), bf16_hi(vw.w)};
    const float* lg = p.logits + (row + j) * G;
#pragma unroll
    for (int h = 0; h < GMAX; ++h) {
      if (h < G) {
        const float x = lg[h] * p.scale_log2;
        const float mn = fmaxf(m[h], x);
        const float corr = exp2f(m[h] - mn);  // m = -inf gives 0
        const float pw = exp2f(x - mn);
        l[h] = l[h] * corr + pw;
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[h][e] = acc[h][e] * corr + pw * v[e];
        m[h] = mn;
      }
    }
  }

  // merge the token groups of the warp (lanes with equal `sub` hold the same dims)
#pragma unroll
  for (int o = LPT; o < 32; o <<= 1) {
#pragma unroll
    for (int h = 0; h < GMAX; ++h) {
      if (h < G) {
        const float m2 = __shfl_xor_sync(0xffffffffu, m[h], o);
        const float l2 = __shfl_xor_sync(0xffffffffu, l[h], o);
        float a2[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) a2[e] = __shfl_xor_sync(0xffffffffu, acc[h][e], o);
        softmax_merge(m[h], l[h], acc[h], 8, m2, l2, a2);
      }
    }
  }
  if (grp == 0) {
#pragma unroll
    for (int h = 0; h < GMAX; ++h) {
      if (h < G) {
#pragma unroll
        for (int e = 0; e < 8; ++e) sh_acc[warp][h][sub * 8 + e] = acc[h][e];
        if (sub == 0) {
          sh_ml[warp][h][0] = m[h];
          sh_ml[warp][h][1] = l[h];
        }
      }
    }
  }
  __syncthreads();
  // merge the warps and write the partial of this split
  float* dst = p.part + (((size_t)(b * p.Hkv + kvh) * p.S + s) * G) * (HD + 2);
  for (int i = threadIdx.x; i < G * HD; i += GA_WARPS * 32) {
    const int h = i / HD, e = i % HD;
    float mm = sh_ml[0][h][0], ll = sh_ml[0][h][1], a = sh_acc[0][h][e];
    for (int w = 1; w < GA_WARPS; ++w) {
      const float a2 = sh_acc[w][h][e];
      softmax_merge(mm, ll, &a, 1, sh_ml[w][h][0], sh_ml[w][h][1], &a2);
    }
    dst[h * (HD + 2) + e] = a;
    if (e == 0) {
      dst[h * (HD + 2) + HD] = mm;
      dst[h * (HD + 2) + HD + 1] = ll;
    }
  }
}

struct CombineDev {
  int Hq, Hkv, G, hd, S;
  const int32_t* kept_cnt;
  const float* part;
  float* out_f32;
  uint16_t* out_bf16;
  uint16_t* out_hi;
  uint16_t* out_lo;
};

__global__ void attn_combine_kernel(const CombineDev p) {
  const int b = blockIdx.y, h = blockIdx.x;
  const int kvh = h / p.G, gi = h % p.G;
  const int cnt = p.kept_cnt[b * p.Hkv + kvh];
  const int ns = (cnt + ATTN_SPLIT_LEN - 1) / ATTN_SPLIT_LEN;
  const int e = threadIdx.x;
  if (e >= p.hd) return;
  float m = -INFINITY, l = 0.f, a = 0.f;
  for (int s = 0; s < ns; ++s) {
    const float* src = p.part + ((((size_t)(b * p.Hkv + kvh) * p.S + s) * p.G) + gi) * (p.hd + 2);
    const float a2 = src[e];
    softmax_merge(m, l, &a, 1, src[p.hd], src[p.hd + 1], &a2);
  }
  const float o = l > 0.f ? a / l : 0.f;
  const size_t idx = ((size_t)b * p.Hq + h) * p.hd + e;
  if (p.out_f32) p.out_f32[idx] = o;
  if (p.out_bf16) p.out_bf16[idx] = f2bf(o);
  if (p.out_hi) {
    const uint16_t hi = f2bf(o);
    p.out_hi[idx] = hi;
    p.out_lo[idx] = f2bf(o - bf2f(hi));
  }
}

// ============================================================================
// host side
// ============================================================================
template <int HD>
static void launch_score(const ScoreDev& d, int HG, dim3 grid, cudaStream_t st) {
  const int smem = SC_WARPS * PAGE * HD * 2 + SC_WARPS * 8 + 32;
  if (HG == 1) {
    cudaFuncSetAttribute(attn_score_kernel<HD, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    SOL_LAUNCH("attn_score", (attn_score_kernel<HD, 1>), grid, dim3(SC_WARPS * 32), smem, st, d);
  } else {
    cudaFuncSetAttribute(attn_score_kernel<HD, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    SOL_LAUNCH("attn_score", (attn_score_kernel<HD, 2>), grid, dim3(SC_WARPS * 32), smem, st, d);
  }
}

void launch_attention(const AttnArgs& a, cudaStream_t st) {
  const sol_shape_t& sh = a.shape;
  const int Hq = sh.n_q_heads, Hkv = sh.n_kv_heads, hd = sh.head_dim, G = Hq / Hkv, HG = (G + 3) / 4;
  const int Tmax = a.kv.max_pages_per_seq * PAGE;

  PrepDev pd;
  pd.sh = sh; pd.kv = a.kv; pd.qkv = a.qkv_f32; pd.ldq = a.ldq;
  pd.q_bf16 = static_cast<const uint16_t*>(a.q_bf16);
  pd.q_rot = a.q_rot; pd.q_split = static_cast<uint16_t*>(a.q_split); pd.status = a.status;
  SOL_LAUNCH("attn_prep_rope_append", attn_prep_kernel, dim3(a.B), dim3(256), 0, st, pd);

  ScoreDev sd;
  sd.kv = a.kv; sd.Hkv = Hkv; sd.G = G; sd.HG = HG; sd.Tmax = Tmax;
  sd.q_split = static_cast<const uint16_t*>(a.q_split);
  sd.logits = a.logits; sd.sigma = a.sigma; sd.status = a.status;
  dim3 sgrid((a.kv.max_pages_per_seq + SC_WARPS - 1) / SC_WARPS, Hkv, a.B);
  if (hd == 64) launch_score<64>(sd, HG, sgrid, st);
  else launch_score<128>(sd, HG, sgrid, st);

  SelectDev se;
  se.sh = sh; se.kv = a.kv; se.r_permille = a.r_permille; se.Tmax = Tmax; se.q_rot = a.q_rot;
  se.sigma = a.sigma; se.kept_idx = a.kept_idx; se.kept_cnt = a.kept_cnt; se.status = a.status;
  SOL_LAUNCH("token_select", token_select_kernel, dim3(Hkv, a.B), dim3(SEL_THREADS), 0, st, se);

  GatherDev gd;
  gd.kv = a.kv; gd.Hkv = Hkv; gd.G = G; gd.Tmax = Tmax; gd.S = a.splits;
  gd.logits = a.logits; gd.kept_idx = a.kept_idx; gd.kept_cnt = a.kept_cnt; gd.part = a.part;
  gd.scale_log2 = (float)(1.4426950408889634 / sqrt((double)hd));
  gd.status = a.status;
  dim3 ggrid(a.splits, Hkv, a.B);
  if (hd == 64) {
    if (G <= 4) SOL_LAUNCH("attn_gather_v", (attn_gather_kernel<64, 4>), ggrid, dim3(GA_WARPS * 32), 0, st, gd);
    else SOL_LAUNCH("attn_gather_v", (attn_gather_kernel<64, 8>), ggrid, dim3(GA_WARPS * 32), 0, st, gd);
  } else {
    if (G <= 4) SOL_LAUNCH("attn_gather_v", (attn_gather_kernel<128, 4>), ggrid, dim3(GA_WARPS * 32), 0, st, gd);
    else SOL_LAUNCH("attn_gather_v", (attn_gather_kernel<128, 8>), ggrid, dim3(GA_WARPS * 32), 0, st, gd);
  }

  CombineDev cd;
  cd.Hq = Hq; cd.Hkv = Hkv; cd.G = G; cd.hd = hd; cd.S = a.splits;
  cd.kept_cnt = a.kept_cnt; cd.part = a.part; cd.out_f32 = a.out_f32;
  cd.out_bf16 = static_cast<uint16_t*>(a.out_bf16);
  cd.out_hi = static_cast<uint16_t*>(a.out_hi); cd.out_lo = static_cast<uint16_t*>(a.out_lo);
  SOL_LAUNCH("attn_combine", attn_combine_kernel, dim3(Hq, a.B), dim3(hd), 0, st, cd);
}

}  // namespace sol
