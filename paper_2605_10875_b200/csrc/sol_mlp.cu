// Per-token top-k over the intermediate channels of the SwiGLU MLP.
//
// For token i keep the m = ceil((1 - p_i) * ff) channels with the largest
// |t_j| = |silu(g_j) * u_j| (the count mirrors the paper's m = ceil(rho * d),
// "Per-token channel selection", with rho = 1 - p).  One CTA per token: exact
// k-th largest of the float32 |t| held in registers, then every channel within
// a small window of the threshold has g_j and u_j recomputed exactly from the
// weight rows, so the kept set does not depend on float32 rounding.  Emits
// the ascending kept-channel list, the masked activations as two bf16 parts
// (hi + lo) for the tensor-core down projection, and the "granule is live"
// flags that let the down projection skip weight rows nobody keeps.
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
  const uint16_t* a_op;
  const float* scale;
  const uint16_t* w_gate;
  const uint16_t* w_up;
  int32_t* kept_ch;
  int32_t* kept_cnt;
  uint16_t* t_hi;
  uint16_t* t_lo;
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
    key_thr = select_kth<THREADS, KPT>(key, m, tie_need, sm);
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
        const uint16_t* x = p.a_op + (size_t)b * d;
        for (int c = warp; c < n_cand; c += WARPS) {
          const int j = sm.cand_idx[c];
          const uint16_t* wg = p.w_gate + (size_t)j * d;
          const uint16_t* wu = p.w_up + (size_t)j * d;
          float gh = 0.f, gl = 0.f, uh = 0.f, ul = 0.f;
          // RB 256-wide slices per round, all loads of a round issued before the first use
          constexpr int RB = THREADS >= 1024 ? 2 : 4;  // 64 registers per thread at 1024 threads
          for (int e0 = lane * 8; e0 < d; e0 += RB * 256) {
            uint4 xv[RB], gv[RB], uv[RB];
#pragma unroll
            for (int r = 0; r < RB; ++r) {
              const int e = e0 + r * 256;
              if (e < d) {
                xv[r] = *reinterpret_cast<const uint4*>(x + e);
                gv[r] = *reinterpret_cast<const uint4*>(wg + e);
                uv[r] = *reinterpret_cast<const uint4*>(wu + e);
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
  uint16_t* th = p.t_hi + (size_t)b * ff;
  uint16_t* tl = p.t_lo + (size_t)b * ff;
  uint32_t hw[4], lw[4];
  bool any = false;
  auto emit = [&](int i, bool keep) {
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
    if (e == 7 && j0 + i < ff) {
      *reinterpret_cast<uint4*>(th + j0 + i - 7) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
      *reinterpret_cast<uint4*>(tl + j0 + i - 7) = make_uint4(lw[0], lw[1], lw[2], lw[3]);
    }
    if (((j0 + i) & 31) == 31 || i == KPT - 1) {  // end of a 32-channel granule or of this thread's range
      if (any && j0 + i < ff) p.live[(j0 + i) >> 5] = 1;
      any = false;
    }
  };
  const int total = compact_indices<THREADS, KPT>(klass, emit, mode == 3 ? tie_need : 0, p.kept_ch + (size_t)b * ff, sm);
  if (tid == 0) p.kept_cnt[b] = total;
}

void launch_channel_select(const ChannelSelectArgs& a, cudaStream_t st) {
  ChanDev c;
  c.d = a.d; c.ff = a.ff; c.p_permille = a.p_permille; c.g = a.g; c.u = a.u; c.t = a.t;
  c.a_op = static_cast<const uint16_t*>(a.a_op); c.scale = a.scale;
  c.w_gate = static_cast<const uint16_t*>(a.w_gate); c.w_up = static_cast<const uint16_t*>(a.w_up);
  c.kept_ch = a.kept_ch; c.kept_cnt = a.kept_cnt;
  c.t_hi = static_cast<uint16_t*>(a.t_hi); c.t_lo = static_cast<uint16_t*>(a.t_lo);
  c.live = a.live; c.status = a.status;
  const dim3 grid(a.B);
  if (a.ff <= 2048) SOL_LAUNCH("channel_select", (channel_select_kernel<256, 8>), grid, dim3(256), 0, st, c);
  else if (a.ff <= 8192) SOL_LAUNCH("channel_select", (channel_select_kernel<512, 16>), grid, dim3(512), 0, st, c);
  else if (a.ff <= 16384) SOL_LAUNCH("channel_select", (channel_select_kernel<1024, 16>), grid, dim3(1024), 0, st, c);
  else if (a.ff <= 32768) SOL_LAUNCH("channel_select", (channel_select_kernel<1024, 32>), grid, dim3(1024), 0, st, c);
  else SOL_LAUNCH("channel_select", (channel_select_kernel<1024, 48>), grid, dim3(1024), 0, st, c);
}

}  // namespace sol
