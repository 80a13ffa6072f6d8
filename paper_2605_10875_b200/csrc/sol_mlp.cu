// Per-token top-k over the intermediate channels of the SwiGLU MLP.
//
// For token i keep the m = ceil((1 - p_i) * ff) channels with the largest
// |t_j| = |silu(g_j) * u_j| (the count mirrors the paper's m = ceil(rho * d),
// "Per-token channel selection", with rho = 1 - p; ties: lower index).
//
// The gate/up projection leaves, per token, a 4096-bin histogram of |t| and
// the largest |g|, |u|.  channel_select_multi spreads every token over
// ff/1024 CTAs: each finds the histogram bin that holds the m-th largest |t|,
// keeps what lies above that bin (by more than the float32 error bound of t),
// drops what lies below, and recomputes the few channels in between exactly
// from the weight rows; the last CTA of a token ranks those candidates and
// patches the kept ones in.  Outputs: the masked activations as two bf16
// parts (hi + lo) for the tensor-core down projection, a keep mask, and the
// "granule is live" flags that let the down projection skip weight rows
// nobody keeps.  A token with more candidates than the list holds (massive
// ties) is redone by the single-CTA kernel channel_select, which is exact for
// any input; channel_list turns the mask into the ascending index list when a
// caller asks for it.
#include <math.h>

#include "sol_common.cuh"
#include "sol_internal.h"
#include "sol_select.cuh"

namespace sol {

struct ChanDev {
  int d, ff;
  const int32_t* p_permille;
  const float* g;
  const float* u;
  const float* t;
  const unsigned char* a_op;  // packed operand, Mpad rows
  const float* scale;
  const unsigned char* w_gu;  // packed gate/up weights: rows alternate gate_c, up_c
  int R, chunks, Mpad;        // rows per tile and 64-wide chunks of the packed weights; rows of the operand blocks
  uint32_t* sel;
  double* cand_val;
  int32_t* cand_idx;
  unsigned char* keep;
  int32_t* kept_ch;
  int32_t* scratch_idx;  // [B][ff] list written by the single-CTA kernel (not an output)
  int32_t* kept_cnt;
  unsigned char* t_op;  // packed operand of the down projection: 2 Mpad rows (high parts, then low parts)
  int32_t* live;
  int* status;
};

// Running sum held as an unevaluated pair of floats (hi + lo): adds x with the rounding error of
// hi + x captured exactly (two-sum) and gathered in lo.  With terms that are exact float32 numbers the
// pair follows the exact sum to about 2^-45, on the float32 pipes instead of the scarce float64 ones.
__device__ __forceinline__ void pair_add(float& hi, float& lo, float x) {
  const float s = __fadd_rn(hi, x);
  const float bb = __fsub_rn(s, hi);
  const float e = __fadd_rn(__fsub_rn(hi, __fsub_rn(s, bb)), __fsub_rn(x, bb));
  hi = s;
  lo = __fadd_rn(lo, e);
}

template <int THREADS, int KPT>
__global__ void __launch_bounds__(THREADS) channel_select_kernel(const ChanDev p) {
  __shared__ SelectSmem sm;
  static_assert(KPT % 8 == 0 && KPT <= 64, "a thread owns whole 16-byte groups of bf16 outputs");
  const int b = blockIdx.x;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  constexpr int WARPS = THREADS / 32;
  const int ff = p.ff, d = p.d;
  pdl_trigger();
  pdl_wait();
  if (p.sel[(size_t)b * CH_SEL_WORDS + CH_FALLBACK] == 0u) return;  // the multi-CTA kernel settled this token
  const float* tt = p.t + (size_t)b * ff;
  const int m = (int)(((long long)(1000 - p.p_permille[b]) * ff + 999) / 1000);
  const int j0 = tid * KPT;
  if (tid < 4) sm.counts[tid] = 0;

  // one pass over global memory: |t| as keys (0: absent) and signs in registers, and (when a selection
  // is needed) the largest |g|, |u| for the error window
  const bool select = m < ff && m > 0;
  uint32_t key[KPT];
  uint64_t neg = 0;
  float gmax = 0.f, umax = 0.f;
  {
    const float* gg = p.g + (size_t)b * ff;
    const float* uu = p.u + (size_t)b * ff;
#pragma unroll
    for (int i = 0; i < KPT; i += 4) {
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      const bool in = j0 + i < ff;  // ff is a multiple of 4, so a group is present or absent as a whole
      if (in) v = *reinterpret_cast<const float4*>(tt + j0 + i);
      const float vv[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        key[i + e] = in ? float_key(fabsf(vv[e])) : 0u;
        if (vv[e] < 0.f) neg |= 1ull << (i + e);
      }
      if (select && in) {
        const float4 g4 = *reinterpret_cast<const float4*>(gg + j0 + i), u4 = *reinterpret_cast<const float4*>(uu + j0 + i);
        gmax = fmaxf(fmaxf(gmax, fmaxf(fabsf(g4.x), fabsf(g4.y))), fmaxf(fabsf(g4.z), fabsf(g4.w)));
        umax = fmaxf(fmaxf(umax, fmaxf(fabsf(u4.x), fabsf(u4.y))), fmaxf(fabsf(u4.z), fabsf(u4.w)));
      }
    }
  }

  // mode 0: keep all; 1: keep none; 2: kept iff |t| above the window or a candidate decided in float64;
  // 3: float32 order with index-ordered ties (candidate list overflowed)
  int mode, tie_need = 0, n_cand = 0;
  uint32_t key_thr = 0;
  float hi = 0.f, lo = 0.f;

  if (m >= ff) {
    mode = 0;
  } else if (m <= 0) {
    mode = 1;
  } else {
    gmax = block_max<THREADS>(gmax, 0, sm);
    umax = block_max<THREADS>(umax, 1, sm);
    key_thr = select_kth<THREADS, KPT>([&](int i) { return key[i]; }, m, tie_need, sm, KPT);
    mode = 3;
    const float thr32 = key_to_float(key_thr);
    // error taken for g_j, u_j: the tensor cores add each 16-long slice of the dot product to the running
    // float32 sum with truncation, so the error grows with the d/16 steps: (d/16) * 2^-24 of the largest
    // magnitude, and never less than 2^-18 of it
    const float eps = fmaxf(3.814697265625e-06f, (float)(d / 16) * 5.9604644775390625e-08f) * fmaxf(gmax, umax);
    const float delta = 2.0f * eps * (1.1f * umax + gmax) + 1e-6f * thr32;  // |silu'| <= 1.1, |silu(g)| <= |g|
    hi = thr32 + delta;
    lo = thr32 - delta;
    int n_in = 0;
#pragma unroll
    for (int i = 0; i < KPT; ++i) {
      if (key[i] == 0u) continue;
      const float sv = key_to_float(key[i]);
      if (sv > hi) {
        ++n_in;
      } else if (sv >= lo) {
        const int slot = atomicAdd(&sm.counts[0], 1);
        if (slot < SEL_CAND_CAP) sm.cand_idx[slot] = j0 + i;
      }
    }
    n_in = block_count<THREADS>(n_in, 0, sm);
    n_cand = sm.counts[0];
    const int need = m - n_in;
    if (n_cand > SEL_CAND_CAP) {
      if (tid == 0) atomicAdd(p.status + ST_CH_OVERFLOW, 1);
      n_cand = 0;
    } else {
      if (n_cand != need) {
        if (tid == 0) atomicAdd(p.status + ST_CH_REFINED, n_cand);
        // g_j = scale * sum_e x_e w_je with x the quantizer codes (or the bf16 row): every product of two
        // bf16 numbers is an exact float32, so the sums are gathered exactly in float pairs
        const double sc = (double)p.scale[b];
        for (int c = warp; c < n_cand; c += WARPS) {
          const int j = sm.cand_idx[c];
          float gh = 0.f, gl = 0.f, uh = 0.f, ul = 0.f;
          // RB 256-wide slices per round, all loads of a round issued before the first use
          constexpr int RB = THREADS >= 1024 ? 2 : 4;  // 64 registers per thread at 1024 threads
          for (int e0 = lane * 8; e0 < d; e0 += RB * 256) {
            uint4 xv[RB], gv[RB], uv[RB];
#pragma unroll
            for (int r = 0; r < RB; ++r) {
              const int e = e0 + r * 256;
              if (e < d) {  // the piece of elements e .. e + 7 of the operand row and of the channel's two weight rows
                xv[r] = *reinterpret_cast<const uint4*>(p.a_op + act_piece_offset(p.Mpad, b, e >> 3));
                gv[r] = *reinterpret_cast<const uint4*>(p.w_gu + nk_piece_offset(p.R, p.chunks, 2 * j, e >> 6, (e >> 3) & 7));
                uv[r] = *reinterpret_cast<const uint4*>(p.w_gu + nk_piece_offset(p.R, p.chunks, 2 * j + 1, e >> 6, (e >> 3) & 7));
              }
            }
#pragma unroll
            for (int r = 0; r < RB; ++r) {
              if (e0 + r * 256 >= d) break;
              const uint32_t xa[4] = {xv[r].x, xv[r].y, xv[r].z, xv[r].w}, ga[4] = {gv[r].x, gv[r].y, gv[r].z, gv[r].w},
                             ua[4] = {uv[r].x, uv[r].y, uv[r].z, uv[r].w};
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                const float x0 = bf16_lo(xa[q]), x1 = bf16_hi(xa[q]);
                pair_add(gh, gl, __fmul_rn(x0, bf16_lo(ga[q])));
                pair_add(gh, gl, __fmul_rn(x1, bf16_hi(ga[q])));
                pair_add(uh, ul, __fmul_rn(x0, bf16_lo(ua[q])));
                pair_add(uh, ul, __fmul_rn(x1, bf16_hi(ua[q])));
              }
            }
          }
          const double ag = warp_sum_d((double)gh + (double)gl) * sc;
          const double au = warp_sum_d((double)uh + (double)ul) * sc;
          if (lane == 0) sm.cand_val[c] = fabs(ag / (1.0 + exp(-ag)) * au);
        }
        __syncthreads();
        rank_candidates<THREADS>(n_cand, need, sm);
      } else {
        for (int c = tid; c < n_cand; c += THREADS) sm.cand_keep[c] = 1;
      }
      mode = 2;
      __syncthreads();
    }
  }

  auto klass = [&](int i) -> int {
    const int j = j0 + i;
    if (j >= ff || mode == 1) return 0;
    if (mode == 0) return 2;
    if (mode == 2) {
      const float sv = key_to_float(key[i]);
      if (sv > hi) return 2;
      if (sv >= lo) {  // within the window: look the channel up in the decided list
        for (int q = 0; q < n_cand; ++q)
          if (sm.cand_idx[q] == j) return sm.cand_keep[q] ? 2 : 0;
      }
      return 0;
    }
    return key[i] > key_thr ? 2 : (key[i] == key_thr ? 1 : 0);
  };
  // masked activations as bf16 high + low parts, 8 channels (16 bytes) at a time, and the live flags
  uint32_t hw[4], lw[4];
  bool any = false;
  auto emit = [&](int i, bool keep, int) {
    uint16_t hv = 0, lv = 0;
    if (keep) {
      const float a = key_to_float(key[i]);
      const float v = ((neg >> i) & 1ull) ? -a : a;
      hv = f2bf(v);
      lv = f2bf(v - bf2f(hv));
      any = true;
    }
    const int e = i & 7;
    if ((e & 1) == 0) {
      hw[e >> 1] = hv;
      lw[e >> 1] = lv;
    } else {
      hw[e >> 1] |= (uint32_t)hv << 16;
      lw[e >> 1] |= (uint32_t)lv << 16;
    }
    if (j0 + i < ff) p.keep[(size_t)b * ff + j0 + i] = keep ? 1 : 0;
    if (e == 7 && j0 + i < ff) {  // channels j0 + i - 7 .. j0 + i are one piece of the packed operand
      unsigned char* dst = p.t_op + act_piece_offset(2 * p.Mpad, b, (j0 + i) >> 3);
      *reinterpret_cast<uint4*>(dst) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
      *reinterpret_cast<uint4*>(dst + (size_t)p.Mpad * 128) = make_uint4(lw[0], lw[1], lw[2], lw[3]);
    }
    if (((j0 + i) & 31) == 31 || i == KPT - 1) {  // end of a 32-channel granule or of this thread's range
      if (any && j0 + i < ff) p.live[(j0 + i) >> 5] = 1;
      any = false;
    }
  };
  // the index list itself is written by channel_list from the mask; here it goes to the candidate scratch
  const int total =
      compact_indices<THREADS, KPT>(klass, emit, mode == 3 ? tie_need : 0, p.scratch_idx + (size_t)b * ff, sm, KPT);
  if (tid == 0) p.kept_cnt[b] = total;
}

// ============================================================================
// channel_select_multi
// ============================================================================
constexpr int CM_THREADS = 256;
constexpr int CM_MAX_GROUPS = 2;  // groups of four channels per thread at most (template parameter of the kernel)

struct ChanMultiSmem {
  int scan[CM_THREADS / 32];
  int pick[2];
  int n_local;
  int flag;
  int local_idx[CM_THREADS * 4 * CM_MAX_GROUPS];
  __align__(16) uint16_t x[8192];  // the token's operand row (d_model <= 8192)
  double val[CH_CAND_CAP];
  int idx[CH_CAND_CAP];
};

// CM_GROUPS: groups of four channels per thread, so CM_THREADS * 4 * CM_GROUPS channels per CTA: the launch takes
// two groups when one group per thread would need more CTAs than are resident at once (a second, partly filled
// wave of these latency-bound CTAs cost 15 % at batch 128; four groups were slower again: 37 against 34 us).
template <int CM_GROUPS>
__global__ void __launch_bounds__(CM_THREADS, 3) channel_select_multi_kernel(const ChanDev p) {
  constexpr int CM_SLICE = CM_THREADS * 4 * CM_GROUPS;
  __shared__ ChanMultiSmem sm;
  const int slice = blockIdx.x, b = blockIdx.y, S = gridDim.x;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  constexpr int WARPS = CM_THREADS / 32;
  const int ff = p.ff, d = p.d;
  pdl_trigger();
  pdl_wait();
  uint32_t* sel = p.sel + (size_t)b * CH_SEL_WORDS;
  const int m = (int)(((long long)(1000 - p.p_permille[b]) * ff + 999) / 1000);
  if (tid == 0) sm.n_local = 0;
  // What the later steps read is requested now, so that it arrives while the histogram is scanned: this CTA's
  // channels of t (and of g, u when there is a selection to make) and the token's operand row for the exact
  // re-scoring (into shared memory; a selection almost always leaves a few channels to re-score).
  const bool selecting = m > 0 && m < ff;
  float4 v[CM_GROUPS], gq[CM_GROUPS], uq[CM_GROUPS];
#pragma unroll
  for (int gi = 0; gi < CM_GROUPS; ++gi) {
    const int j0 = slice * CM_SLICE + (gi * CM_THREADS + tid) * 4;
    v[gi] = gq[gi] = uq[gi] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (j0 < ff) {  // ff is a multiple of 4: a thread's group is present or absent as a whole
      v[gi] = *reinterpret_cast<const float4*>(p.t + (size_t)b * ff + j0);
      if (selecting) {
        gq[gi] = *reinterpret_cast<const float4*>(p.g + (size_t)b * ff + j0);
        uq[gi] = *reinterpret_cast<const float4*>(p.u + (size_t)b * ff + j0);
      }
    }
  }
  if (selecting)
    for (int e = tid * 8; e < d; e += CM_THREADS * 8)
      *reinterpret_cast<uint4*>(sm.x + e) = *reinterpret_cast<const uint4*>(p.a_op + act_piece_offset(p.Mpad, b, e >> 3));

  // ---- the histogram bin of the m-th largest |t| (every CTA of the token finds the same one) ----
  // keep at or above hi_edge + e_j, drop below lo_edge - e_j, exact in between; e_j = eps * (1.1 |u_j| + |g_j|)
  // bounds the error of this channel's own float32 |t|
  float hi_edge = 0.f, lo_edge = 0.f, eps = 0.f;
  if (m >= ff) {
    hi_edge = 0.f;  // everything is kept
    lo_edge = 0.f;
  } else if (m <= 0) {
    hi_edge = INFINITY;
    lo_edge = INFINITY;
  } else {
    constexpr int BPT = CH_BINS / CM_THREADS;  // bins per thread, descending
    int mine = 0;
#pragma unroll
    for (int q = 0; q < BPT; ++q) mine += (int)sel[CH_BINS - 1 - tid * BPT - q];
    int incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    if (lane == 31) sm.scan[warp] = incl;
    __syncthreads();
    int before = incl - mine;
    for (int w = 0; w < warp; ++w) before += sm.scan[w];
    if (before < m && m <= before + mine) {
      int a = before;
      for (int q = 0; q < BPT; ++q) {
        const int bin = CH_BINS - 1 - tid * BPT - q;
        const int c = (int)sel[bin];
        if (m <= a + c) {
          sm.pick[0] = bin;
          break;
        }
        a += c;
      }
    }
    __syncthreads();
    const int tb = sm.pick[0];
    const float gmax = __uint_as_float(sel[CH_GMAX]), umax = __uint_as_float(sel[CH_UMAX]);
    const float bin_lo = chan_bin_lo(tb), bin_hi = tb >= CH_BINS - 1 ? INFINITY : chan_bin_lo(tb + 1);
    // error taken for g_j, u_j: the tensor cores add each 16-long slice of the dot product to the running
    // float32 sum with truncation, so the error grows with the d/16 steps: (d/16) * 2^-24 of the largest
    // magnitude, and never less than 2^-18 of it; carried into t through |silu'| <= 1.1, |silu(g)| <= |g|
    eps = fmaxf(3.814697265625e-06f, (float)(d / 16) * 5.9604644775390625e-08f) * fmaxf(gmax, umax);
    // the m-th largest exact |t| lies within the largest error any channel can carry of the bin; a channel is
    // settled when its own error cannot carry it across that
    const float delta = eps * (1.1f * umax + gmax) + 1e-6f * (tb >= CH_BINS - 1 ? bin_lo : bin_hi);
    lo_edge = bin_lo - delta;
    hi_edge = bin_hi + delta;
  }

  // ---- classify this CTA's channels: CM_GROUPS groups of four per thread ----
  int n_above = 0;
#pragma unroll
  for (int gi = 0; gi < CM_GROUPS; ++gi) {
    const int j0 = slice * CM_SLICE + (gi * CM_THREADS + tid) * 4;
    const bool in = j0 < ff;
    const float vv[4] = {v[gi].x, v[gi].y, v[gi].z, v[gi].w}, gg[4] = {gq[gi].x, gq[gi].y, gq[gi].z, gq[gi].w},
                uu[4] = {uq[gi].x, uq[gi].y, uq[gi].z, uq[gi].w};
    uint32_t hw[2] = {0, 0}, lw[2] = {0, 0}, kw = 0;
    bool any = false;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float a = fabsf(vv[e]);
      if (!in) continue;
      const float ej = eps * (1.1f * fabsf(uu[e]) + fabsf(gg[e]));
      if (a >= hi_edge + ej) {
        const uint16_t hv = f2bf(vv[e]);
        const uint16_t lv = f2bf(vv[e] - bf2f(hv));
        hw[e >> 1] |= (uint32_t)hv << (16 * (e & 1));
        lw[e >> 1] |= (uint32_t)lv << (16 * (e & 1));
        kw |= 1u << (8 * e);
        ++n_above;
        any = true;
      } else if (a >= lo_edge - ej) {
        sm.local_idx[atomicAdd(&sm.n_local, 1)] = j0 + e;
      }
    }
    if (in) {  // four channels: half a piece of the packed operand
      unsigned char* dst = p.t_op + act_piece_offset(2 * p.Mpad, b, j0 >> 3) + (j0 & 7) * 2;
      *reinterpret_cast<uint2*>(dst) = make_uint2(hw[0], hw[1]);
      *reinterpret_cast<uint2*>(dst + (size_t)p.Mpad * 128) = make_uint2(lw[0], lw[1]);
      *reinterpret_cast<uint32_t*>(p.keep + (size_t)b * ff + j0) = kw;
      if (any) p.live[j0 >> 5] = 1;
    }
  }
  n_above = __reduce_add_sync(0xffffffffu, n_above);
  if (lane == 0 && n_above) atomicAdd(sel + CH_N_ABOVE, (uint32_t)n_above);
  __syncthreads();

  // ---- exact |t| of the channels in between, from the weight rows ----
  // g_j = scale * sum_e x_e w_je with x the quantizer codes (or the bf16 row): every product of two bf16
  // numbers is an exact float32, so the sums are gathered exactly in float pairs
  const int n_local = sm.n_local;
  if (n_local > 0) {
    const double sc = (double)p.scale[b];
    // the token's operand row (requested at the start) is in shared memory: the barrier above has passed
    for (int c = warp; c < n_local; c += WARPS) {
      const int j = sm.local_idx[c];
      float gh = 0.f, gl = 0.f, uh = 0.f, ul = 0.f;
      for (int e0 = lane * 8; e0 < d; e0 += 2048) {  // eight 256-wide slices of both rows per round, loads before uses
        uint4 gv[8], uv[8];
#pragma unroll
        for (int r = 0; r < 8; ++r) {
          const int e = e0 + r * 256;
          if (e < d) {  // the piece of elements e .. e + 7 of the channel's gate row and of its up row
            gv[r] = *reinterpret_cast<const uint4*>(p.w_gu + nk_piece_offset(p.R, p.chunks, 2 * j, e >> 6, (e >> 3) & 7));
            uv[r] = *reinterpret_cast<const uint4*>(p.w_gu + nk_piece_offset(p.R, p.chunks, 2 * j + 1, e >> 6, (e >> 3) & 7));
          }
        }
#pragma unroll
        for (int r = 0; r < 8; ++r) {
          const int e = e0 + r * 256;
          if (e >= d) break;
          const uint4 xv = *reinterpret_cast<const uint4*>(sm.x + e);
          const uint32_t xa[4] = {xv.x, xv.y, xv.z, xv.w}, ga[4] = {gv[r].x, gv[r].y, gv[r].z, gv[r].w},
                         ua[4] = {uv[r].x, uv[r].y, uv[r].z, uv[r].w};
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const float x0 = bf16_lo(xa[q]), x1 = bf16_hi(xa[q]);
            pair_add(gh, gl, __fmul_rn(x0, bf16_lo(ga[q])));
            pair_add(gh, gl, __fmul_rn(x1, bf16_hi(ga[q])));
            pair_add(uh, ul, __fmul_rn(x0, bf16_lo(ua[q])));
            pair_add(uh, ul, __fmul_rn(x1, bf16_hi(ua[q])));
          }
        }
      }
      const double ag = warp_sum_d((double)gh + (double)gl) * sc;
      const double au = warp_sum_d((double)uh + (double)ul) * sc;
      if (lane == 0) {
        const uint32_t slot = atomicAdd(sel + CH_N_CAND, 1u);
        if (slot < (uint32_t)CH_CAND_CAP) {
          p.cand_val[(size_t)b * CH_CAND_CAP + slot] = fabs(ag / (1.0 + exp(-ag)) * au);
          p.cand_idx[(size_t)b * CH_CAND_CAP + slot] = j;
        }
      }
    }
  }

  // ---- the last CTA of the token ranks the candidates and patches the kept ones in ----
  __threadfence();
  __syncthreads();
  if (tid == 0) sm.flag = atomicAdd(sel + CH_DONE, 1u) == (uint32_t)(S - 1) ? 1 : 0;
  __syncthreads();
  if (!sm.flag) return;
  __threadfence();
  const int n_cand = (int)__ldcg(sel + CH_N_CAND);
  const int need = m - (int)__ldcg(sel + CH_N_ABOVE);
  if (m >= ff || m <= 0) {
    if (tid == 0) p.kept_cnt[b] = m >= ff ? ff : 0;
    return;
  }
  if (n_cand > CH_CAND_CAP || need < 0 || need > n_cand) {  // more candidates than the list holds: redo the token
    if (tid == 0) {
      sel[CH_FALLBACK] = 1u;
      atomicAdd(p.status + ST_CH_OVERFLOW, 1);
    }
    return;
  }
  for (int c = tid; c < n_cand; c += CM_THREADS) {
    sm.val[c] = __ldcg(p.cand_val + (size_t)b * CH_CAND_CAP + c);
    sm.idx[c] = __ldcg(p.cand_idx + (size_t)b * CH_CAND_CAP + c);
  }
  __syncthreads();
  for (int c = tid; c < n_cand; c += CM_THREADS) {
    const double vc = sm.val[c];
    const int j = sm.idx[c];
    int rank = 0;
    for (int o = 0; o < n_cand; ++o) {
      const double vo = sm.val[o];
      rank += (vo > vc) || (vo == vc && sm.idx[o] < j);
    }
    if (rank < need) {
      const float tv = p.t[(size_t)b * ff + j];
      const uint16_t hv = f2bf(tv);
      uint16_t* dst = reinterpret_cast<uint16_t*>(p.t_op + act_piece_offset(2 * p.Mpad, b, j >> 3) + (j & 7) * 2);
      dst[0] = hv;
      dst[(size_t)p.Mpad * 64] = f2bf(tv - bf2f(hv));
      p.keep[(size_t)b * ff + j] = 1;
      p.live[j >> 5] = 1;
    }
  }
  if (tid == 0) {
    p.kept_cnt[b] = m;
    atomicAdd(p.status + ST_CH_REFINED, n_cand);
  }
}

// ============================================================================
// channel_list: keep mask -> ascending index list (only when a caller asks for the list)
// ============================================================================
template <int THREADS, int KPT>
__global__ void __launch_bounds__(THREADS) channel_list_kernel(const unsigned char* __restrict__ keep, int ff,
                                                               int32_t* __restrict__ kept_ch) {
  __shared__ SelectSmem sm;
  pdl_trigger();
  pdl_wait();
  const int b = blockIdx.x, j0 = threadIdx.x * KPT;
  const unsigned char* k = keep + (size_t)b * ff;
  auto klass = [&](int i) -> int { return (j0 + i < ff && k[j0 + i]) ? 2 : 0; };
  compact_indices<THREADS, KPT>(klass, [](int, bool, int) {}, 0, kept_ch + (size_t)b * ff, sm, KPT);
}

void launch_channel_select(const ChannelSelectArgs& a, cudaStream_t st) {
  ChanDev c;
  c.d = a.d; c.ff = a.ff; c.p_permille = a.p_permille; c.g = a.g; c.u = a.u; c.t = a.t;
  c.a_op = static_cast<const unsigned char*>(a.a_op); c.scale = a.scale;
  c.w_gu = static_cast<const unsigned char*>(a.w_gate_up);
  const NKGeom geo = nk_geom_gate_up(a.ff, a.d, sm_count());
  c.R = geo.R; c.chunks = geo.chunks; c.Mpad = pad_rows(a.B);
  c.sel = a.sel; c.cand_val = a.cand_val; c.cand_idx = a.cand_idx; c.keep = a.keep;
  c.kept_ch = a.kept_ch; c.scratch_idx = a.scratch_idx; c.kept_cnt = a.kept_cnt;
  c.t_op = static_cast<unsigned char*>(a.t_op);
  c.live = a.live; c.status = a.status;
  const long long resident = 3LL * sm_count();
  const int groups = (long long)((a.ff + CM_THREADS * 4 - 1) / (CM_THREADS * 4)) * a.B > resident ? 2 : 1;
  const dim3 mgrid((a.ff + CM_THREADS * 4 * groups - 1) / (CM_THREADS * 4 * groups), a.B);
  if (groups == 1) SOL_LAUNCH("channel_select", channel_select_multi_kernel<1>, mgrid, dim3(CM_THREADS), 0, st, c);
  else SOL_LAUNCH("channel_select", channel_select_multi_kernel<2>, mgrid, dim3(CM_THREADS), 0, st, c);
  const dim3 grid(a.B);
  // tokens the multi-CTA kernel handed over (it sets their flag); every other CTA leaves at once
  if (a.ff <= 2048) SOL_LAUNCH("channel_select_exact", (channel_select_kernel<256, 8>), grid, dim3(256), 0, st, c);
  else if (a.ff <= 8192) SOL_LAUNCH("channel_select_exact", (channel_select_kernel<512, 16>), grid, dim3(512), 0, st, c);
  else if (a.ff <= 16384) SOL_LAUNCH("channel_select_exact", (channel_select_kernel<1024, 16>), grid, dim3(1024), 0, st, c);
  else if (a.ff <= 32768) SOL_LAUNCH("channel_select_exact", (channel_select_kernel<1024, 32>), grid, dim3(1024), 0, st, c);
  else SOL_LAUNCH("channel_select_exact", (channel_select_kernel<1024, 48>), grid, dim3(1024), 0, st, c);
  if (a.kept_ch != nullptr) {
    if (a.ff <= 4096) SOL_LAUNCH("channel_list", (channel_list_kernel<256, 16>), grid, dim3(256), 0, st, a.keep, a.ff, a.kept_ch);
    else if (a.ff <= 16384) SOL_LAUNCH("channel_list", (channel_list_kernel<1024, 16>), grid, dim3(1024), 0, st, a.keep, a.ff, a.kept_ch);
    else SOL_LAUNCH("channel_list", (channel_list_kernel<1024, 48>), grid, dim3(1024), 0, st, a.keep, a.ff, a.kept_ch);
  }
}

}  // namespace sol
