// Block-wide exact top-k building blocks shared by the token and the channel
// selection kernels (one 1024-thread CTA per selection problem):
//
//   radix_select_kth   the k-th largest 32-bit key among n, 8 bits per pass,
//                      plus how many keys equal to it are still needed
//   ordered_compact    writes the kept indices in ascending order; class 2 is
//                      kept, class 1 ("tie") is kept in ascending index order
//                      until tie_need runs out, class 0 is dropped
//   rank_candidates    ranks a short candidate list by (value descending,
//                      index ascending)
#pragma once
#include "sol_common.cuh"

namespace sol {

constexpr int SEL_THREADS = 1024;
constexpr int SEL_WARPS = SEL_THREADS / 32;
constexpr int SEL_HGROUPS = 8;
constexpr int SEL_CAND_CAP = 1024;

struct SelectSmem {
  uint32_t hist[SEL_HGROUPS * 256];
  int pick[2];
  float f[SEL_WARPS];
  int i[SEL_WARPS * 2];
  int cand_idx[SEL_CAND_CAP];
  double cand_val[SEL_CAND_CAP];
  int counts[4];
};

// Warp 0 finds the digit that holds the `remaining`-th largest key and the
// number of keys in higher digits.
__device__ __forceinline__ void pick_digit(const uint32_t* hist, int remaining, int* out2) {
  if (threadIdx.x < 32) {
    const int lane = threadIdx.x;
    int cnt[8];
    int tot = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      int c = 0;
      for (int gI = 0; gI < SEL_HGROUPS; ++gI) c += hist[gI * 256 + lane * 8 + i];
      cnt[i] = c;
      tot += c;
    }
    int run = tot;  // becomes the inclusive suffix sum over lanes >= lane
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_down_sync(0xffffffffu, run, o);
      if (lane + o < 32) run += v;
    }
    const int above = run - tot;
    if (above < remaining && remaining <= above + tot) {
      int a = above;
      for (int i = 7; i >= 0; --i) {
        if (remaining <= a + cnt[i]) {
          out2[0] = lane * 8 + i;
          out2[1] = a;
          break;
        }
        a += cnt[i];
      }
    }
  }
}

// key(j) -> uint32 for j in [0, n).  Requires 1 <= k <= n.  All threads call.
template <typename KeyFn>
__device__ __forceinline__ uint32_t radix_select_kth(KeyFn key, int n, int k, int& tie_need, SelectSmem& sm) {
  const int tid = threadIdx.x, warp = tid >> 5;
  uint32_t prefix = 0, mask = 0;
  int remaining = k;
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    for (int i = tid; i < SEL_HGROUPS * 256; i += SEL_THREADS) sm.hist[i] = 0;
    __syncthreads();
    uint32_t* myh = sm.hist + (warp & (SEL_HGROUPS - 1)) * 256;
    for (int j = tid; j < n; j += SEL_THREADS) {
      const uint32_t kk = key(j);
      if ((kk & mask) == prefix) atomicAdd(&myh[(kk >> shift) & 255u], 1u);
    }
    __syncthreads();
    pick_digit(sm.hist, remaining, sm.pick);
    __syncthreads();
    prefix |= ((uint32_t)sm.pick[0]) << shift;
    mask |= 255u << shift;
    remaining -= sm.pick[1];
    __syncthreads();
  }
  tie_need = remaining;
  return prefix;
}

// Inverse of float_key.
__device__ __forceinline__ float key_to_float(uint32_t key) {
  return __uint_as_float((key & 0x80000000u) ? (key & 0x7fffffffu) : ~key);
}

// Ranks the first n_cand candidates; decide(c, keep) is called once per
// candidate with keep = (rank < need).
template <typename DecideFn>
__device__ __forceinline__ void rank_candidates(int n_cand, int need, SelectSmem& sm, DecideFn decide) {
  for (int c = threadIdx.x; c < n_cand; c += SEL_THREADS) {
    const double v = sm.cand_val[c];
    const int j = sm.cand_idx[c];
    int rank = 0;
    for (int o = 0; o < n_cand; ++o) {
      const double vo = sm.cand_val[o];
      rank += (vo > v) || (vo == v && sm.cand_idx[o] < j);
    }
    decide(c, rank < need);
  }
}

// klass(j) in {0,1,2}; emit(j, keep) is called for every j in [0, n) (may be a
// no-op); kept indices go to out[] ascending; returns nothing, thread 0
// writes the kept count to *out_cnt.  All threads call.
template <typename ClassFn, typename EmitFn>
__device__ __forceinline__ void ordered_compact(ClassFn klass, EmitFn emit, int n, int tie_need, int32_t* out,
                                                int32_t* out_cnt, SelectSmem& sm) {
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int per_warp = ((n + SEL_WARPS - 1) / SEL_WARPS + 31) / 32 * 32;
  const int w0 = warp * per_warp, w1 = min(n, w0 + per_warp);
  int c2 = 0, c1 = 0;
  for (int j = w0 + lane; j < w0 + per_warp; j += 32) {
    const int c = j < w1 ? klass(j) : 0;
    c2 += __popc(__ballot_sync(0xffffffffu, c == 2));
    c1 += __popc(__ballot_sync(0xffffffffu, c == 1));
  }
  __syncthreads();
  if (lane == 0) {
    sm.i[warp] = c2;
    sm.i[SEL_WARPS + warp] = c1;
  }
  __syncthreads();
  int tie_before = 0, kept_before = 0, total = 0;
  {
    int tb = 0;
    for (int w = 0; w < SEL_WARPS; ++w) {
      const int t1 = sm.i[SEL_WARPS + w];
      const int kept_w = sm.i[w] + min(max(tie_need - tb, 0), t1);
      if (w < warp) {
        kept_before += kept_w;
        tie_before = tb + t1;
      }
      total += kept_w;
      tb += t1;
    }
  }
  if (tid == 0) *out_cnt = total;
  int pos = kept_before, ties = tie_before;
  for (int j = w0 + lane; j < w0 + per_warp; j += 32) {
    const int c = j < w1 ? klass(j) : 0;
    const unsigned m1 = __ballot_sync(0xffffffffu, c == 1);
    const int my_tie_rank = ties + __popc(m1 & ((1u << lane) - 1));
    const bool keep = c == 2 || (c == 1 && my_tie_rank < tie_need);
    const unsigned mk = __ballot_sync(0xffffffffu, keep);
    if (keep) out[pos + __popc(mk & ((1u << lane) - 1))] = j;
    if (j < w1) emit(j, keep);
    pos += __popc(mk);
    ties += __popc(m1);
  }
}

}  // namespace sol
