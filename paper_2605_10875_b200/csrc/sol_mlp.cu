// Per-token top-k over the intermediate channels of the SwiGLU MLP.
//
// For token i keep the m = ceil((1 - p_i) * ff) channels with the largest
// |t_j| = |silu(g_j) * u_j| (the count mirrors the paper's m = ceil(rho * d),
// "Per-token channel selection", with rho = 1 - p).  One 1024-thread CTA per
// token: radix select on the float32 |t|, then every channel within a small
// window of the threshold has g_j and u_j recomputed in float64 from the
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

__global__ void __launch_bounds__(SEL_THREADS) channel_select_kernel(const ChanDev p) {
  extern __shared__ __align__(16) float tv[];  // [ff] silu(g)*u of this token
  __shared__ SelectSmem sm;
  const int b = blockIdx.x;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int ff = p.ff, d = p.d;
  const float* tt = p.t + (size_t)b * ff;
  const int m = (int)(((long long)(1000 - p.p_permille[b]) * ff + 999) / 1000);

  // mode 0: keep all; 1: keep none; 2: kept iff |t| > thr or decided candidate; 3: float32 order with ties
  int mode, tie_need = 0;
  uint32_t key_thr = 0;
  float thr = 0.f, thr_lo = 0.f;
  // decided candidates are recorded in the list itself: cand_idx[c] = j or ~j (dropped)
  int n_cand = 0;

  // one pass over global memory: t into shared memory, and (when a selection is needed) the largest |g|, |u|
  const bool select = m < ff && m > 0;
  float gmax = 0.f, umax = 0.f;
  {
    const float* gg = p.g + (size_t)b * ff;
    const float* uu = p.u + (size_t)b * ff;
    for (int j = tid * 4; j < ff; j += SEL_THREADS * 4) {
      *reinterpret_cast<float4*>(tv + j) = *reinterpret_cast<const float4*>(tt + j);
      if (select) {
        const float4 g4 = *reinterpret_cast<const float4*>(gg + j), u4 = *reinterpret_cast<const float4*>(uu + j);
        gmax = fmaxf(fmaxf(gmax, fmaxf(fabsf(g4.x), fabsf(g4.y))), fmaxf(fabsf(g4.z), fabsf(g4.w)));
        umax = fmaxf(fmaxf(umax, fmaxf(fabsf(u4.x), fabsf(u4.y))), fmaxf(fabsf(u4.z), fabsf(u4.w)));
      }
    }
  }
  __syncthreads();

  if (m >= ff) {
    mode = 0;
  } else if (m <= 0) {
    mode = 1;
  } else {
    key_thr = radix_select_kth([&](int j) { return float_key(fabsf(tv[j])); }, ff, m, tie_need, sm);
    mode = 3;
    const float thr32 = key_to_float(key_thr);
    gmax = warp_max(gmax);
    umax = warp_max(umax);
    if (lane == 0) {
      sm.f[warp] = gmax;
      sm.i[warp] = __float_as_int(umax);
    }
    if (tid < 4) sm.counts[tid] = 0;
    __syncthreads();
    gmax = sm.f[0];
    umax = __int_as_float(sm.i[0]);
    for (int i = 1; i < SEL_WARPS; ++i) {
      gmax = fmaxf(gmax, sm.f[i]);
      umax = fmaxf(umax, __int_as_float(sm.i[i]));
    }
    // error taken for g_j, u_j: the tensor cores add each 16-long slice of the dot product to the running
    // float32 sum with truncation, so the error grows with the d/16 steps: (d/16) * 2^-24 of the largest
    // magnitude, and never less than 2^-18 of it
    const float eps = fmaxf(3.814697265625e-06f, (float)(d / 16) * 5.9604644775390625e-08f) * fmaxf(gmax, umax);
    const float delta = 2.0f * eps * (1.1f * umax + gmax) + 1e-6f * thr32;  // |silu'| <= 1.1, |silu(g)| <= |g|
    const float hi = thr32 + delta, lo = thr32 - delta;
    int n_in = 0;
    for (int j = tid; j < ff; j += SEL_THREADS) {
      const float s = fabsf(tv[j]);
      if (s > hi) {
        ++n_in;
      } else if (s >= lo) {
        const int slot = atomicAdd(&sm.counts[0], 1);
        if (slot < SEL_CAND_CAP) sm.cand_idx[slot] = j;
      }
    }
    if (n_in) atomicAdd(&sm.counts[1], n_in);
    __syncthreads();
    n_cand = sm.counts[0];
    const int need = m - sm.counts[1];
    if (n_cand > SEL_CAND_CAP) {
      if (tid == 0) atomicAdd(p.status + ST_CH_OVERFLOW, 1);
      n_cand = 0;
    } else {
      if (n_cand != need) {
        if (tid == 0) atomicAdd(p.status + ST_CH_REFINED, n_cand);
        const double sc = (double)p.scale[b];
        const uint16_t* x = p.a_op + (size_t)b * d;
        for (int c = warp; c < n_cand; c += SEL_WARPS) {
          const int j = sm.cand_idx[c];
          const uint16_t* wg = p.w_gate + (size_t)j * d;
          const uint16_t* wu = p.w_up + (size_t)j * d;
          double ag = 0.0, au = 0.0;
          for (int e = lane * 8; e < d; e += 256) {
            const uint4 xv = *reinterpret_cast<const uint4*>(x + e);
            const uint4 gv = *reinterpret_cast<const uint4*>(wg + e);
            const uint4 uv = *reinterpret_cast<const uint4*>(wu + e);
            const uint32_t xa[4] = {xv.x, xv.y, xv.z, xv.w}, ga[4] = {gv.x, gv.y, gv.z, gv.w},
                           ua[4] = {uv.x, uv.y, uv.z, uv.w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const double x0 = (double)bf16_lo(xa[q]) * sc, x1 = (double)bf16_hi(xa[q]) * sc;
              ag += x0 * (double)bf16_lo(ga[q]);
              ag += x1 * (double)bf16_hi(ga[q]);
              au += x0 * (double)bf16_lo(ua[q]);
              au += x1 * (double)bf16_hi(ua[q]);
            }
          }
          ag = warp_sum_d(ag);
          au = warp_sum_d(au);
          if (lane == 0) sm.cand_val[c] = fabs(ag / (1.0 + exp(-ag)) * au);
        }
        __syncthreads();
        rank_candidates(n_cand, need, sm, [&](int c, bool keep) {
          // safe to rewrite in place: every thread reads idx[o] only for the `<` tie-break of equal values,
          // so defer the rewrite until all ranks are known
          sm.hist[c] = keep ? 1u : 0u;
        });
        __syncthreads();
        for (int c = tid; c < n_cand; c += SEL_THREADS)
          if (!sm.hist[c]) sm.cand_idx[c] = ~sm.cand_idx[c];
      }
      thr = hi;
      thr_lo = lo;
      mode = 2;
      __syncthreads();
    }
  }

  auto klass = [&](int j) -> int {
    if (mode == 0) return 2;
    if (mode == 1) return 0;
    const float s = fabsf(tv[j]);
    if (mode == 2) {
      if (s > thr) return 2;
      if (s >= thr_lo) {  // within the window: look the channel up in the decided list
        for (int c = 0; c < n_cand; ++c)
          if (sm.cand_idx[c] == j) return 2;
      }
      return 0;
    }
    const uint32_t key = float_key(s);
    return key > key_thr ? 2 : (key == key_thr ? 1 : 0);
  };
  uint16_t* th = p.t_hi + (size_t)b * ff;
  uint16_t* tl = p.t_lo + (size_t)b * ff;
  auto emit = [&](int j, bool keep) {
    uint16_t hi = 0, lo = 0;
    if (keep) {
      const float v = tv[j];
      hi = f2bf(v);
      lo = f2bf(v - bf2f(hi));
      p.live[j >> 5] = 1;
    }
    th[j] = hi;
    tl[j] = lo;
  };
  ordered_compact(klass, emit, ff, mode == 3 ? tie_need : 0, p.kept_ch + (size_t)b * ff, p.kept_cnt + b, sm);
}

void launch_channel_select(const ChannelSelectArgs& a, cudaStream_t st) {
  ChanDev c;
  c.d = a.d; c.ff = a.ff; c.p_permille = a.p_permille; c.g = a.g; c.u = a.u; c.t = a.t;
  c.a_op = static_cast<const uint16_t*>(a.a_op); c.scale = a.scale;
  c.w_gate = static_cast<const uint16_t*>(a.w_gate); c.w_up = static_cast<const uint16_t*>(a.w_up);
  c.kept_ch = a.kept_ch; c.kept_cnt = a.kept_cnt;
  c.t_hi = static_cast<uint16_t*>(a.t_hi); c.t_lo = static_cast<uint16_t*>(a.t_lo);
  c.live = a.live; c.status = a.status;
  cudaMemsetAsync(a.live, 0, sizeof(int32_t) * (a.ff / 32), st);
  const int smem = a.ff * 4;
  ensure_dynamic_smem(reinterpret_cast<const void*>(&channel_select_kernel), smem);
  SOL_LAUNCH("channel_select", channel_select_kernel, dim3(a.B), dim3(SEL_THREADS), smem, st, c);
}

}  // namespace sol
