// Block-wide exact top-k building blocks shared by the token and the channel
// selection kernels (one CTA per selection problem).
//
// Every thread owns a run of consecutive elements whose 32-bit keys (key order
// = value order, see float_key) are read through an accessor key(i): a
// register array walked by fully unrolled loops (KPT > 0), or shared memory
// walked by rolled loops (KPT == 0: small code, any run length); nothing is
// re-read from global memory between passes.
//
//   select_kth        the k-th largest key of the block (histogram of the top
//                     key bits, then exact ranking inside the threshold bin),
//                     plus how many keys equal to it are still needed
//   block_count/max   reductions over the block
//   rank_candidates   ranks a short candidate list by (value descending,
//                     index ascending)
//   compact_indices   writes the kept indices in ascending order
#pragma once
#include "sol_common.cuh"

namespace sol {

constexpr int SEL_CAND_CAP = 1024;
constexpr int SEL_RANK_CAP = 128;  // a threshold bin this small is ranked exactly instead of split further
constexpr int SEL_BINS = 4096;
constexpr int SEL_MAX_WARPS = 32;

struct SelectSmem {
  uint32_t hist[SEL_BINS];
  uint32_t rank_key[SEL_RANK_CAP];
  int pick[3];
  int scan[2][SEL_MAX_WARPS];  // per-warp totals of block_count / compact_indices / select_kth
  float f[2][SEL_MAX_WARPS];
  int cand_idx[SEL_CAND_CAP];
  double cand_val[SEL_CAND_CAP];
  unsigned char cand_keep[SEL_CAND_CAP];
  float f32[SEL_CAND_CAP];
  int counts[4];
};

// The same members for a kernel that never needs the histogram and the candidate arrays at the same time (the
// settling kernel: a row either fits the candidate list or is redone by the radix select, which alone uses the
// histogram): they share their space, 19 KB instead of 35 KB, so that one more CTA fits on an SM.
struct SelectSmemOverlay {
  union {
    uint32_t hist[SEL_BINS];
    struct {
      int cand_idx[SEL_CAND_CAP];
      double cand_val[SEL_CAND_CAP];
      float f32[SEL_CAND_CAP];
    };
  };
  unsigned char cand_keep[SEL_CAND_CAP];
  uint32_t rank_key[SEL_RANK_CAP];
  int pick[3];
  int scan[2][SEL_MAX_WARPS];
  float f[2][SEL_MAX_WARPS];
  int counts[4];
};

// f(i) for the first `per` elements of a thread: unrolled over KPT register slots, or (KPT == 0) a
// rolled loop.
template <int KPT, typename F>
__device__ __forceinline__ void for_keys(int per, F f) {
  if constexpr (KPT > 0) {
#pragma unroll
    for (int i = 0; i < KPT; ++i) {
      if (i >= per) break;
      f(i);
    }
  } else {  // four at a time: the loads of a group are independent, the loop overhead is shared
    int i = 0;
#pragma unroll 1
    for (; i + 4 <= per; i += 4) {
      f(i);
      f(i + 1);
      f(i + 2);
      f(i + 3);
    }
#pragma unroll 1
    for (; i < per; ++i) f(i);
  }
}

// Inverse of float_key.
__device__ __forceinline__ float key_to_float(uint32_t key) {
  return __uint_as_float((key & 0x80000000u) ? (key & 0x7fffffffu) : ~key);
}

// Order-preserving bin (0..4095) of a key by the value it stands for: the sign, then 32 binades of
// magnitude (2^-18 .. 2^14, clamped at both ends) with 64 steps each.  Keys of one sign, binade and
// step share their upper 15 bits, so a bin that is not a clamped one is a key prefix.  Scores spread
// over hundreds of these bins where the upper 12 key bits (3 mantissa bits) put most of them into a
// dozen, which serialises the shared-memory atomics of the histogram.
constexpr int VB_EXP0 = 109;  // biased exponent of the smallest resolved binade
__device__ __forceinline__ int key_value_bin(uint32_t key) {
  const uint32_t u = (key & 0x80000000u) ? (key & 0x7fffffffu) : ~key;  // the float's bits
  int m = (int)((u & 0x7fffffffu) >> 17) - (VB_EXP0 << 6);
  m = min(max(m, 0), SEL_BINS / 2 - 1);
  return (u >> 31) ? SEL_BINS / 2 - 1 - m : SEL_BINS / 2 + m;
}

// Smallest and largest key of a value bin: key_value_bin(key) == bin exactly for klo <= key <= khi (keys of
// NaNs aside: the clamped end bins stop at the keys of -inf and +inf).
__device__ __forceinline__ void value_bin_key_range(int bin, uint32_t& klo, uint32_t& khi) {
  const bool pos = bin >= SEL_BINS / 2;
  const int m = pos ? bin - SEL_BINS / 2 : SEL_BINS / 2 - 1 - bin;
  // magnitudes of the bin as float bit patterns without the sign
  const uint32_t mlo = m == 0 ? 0u : (uint32_t)(m + (VB_EXP0 << 6)) << 17;
  const uint32_t mhi = m == SEL_BINS / 2 - 1 ? 0x7f800000u : (((uint32_t)(m + (VB_EXP0 << 6)) + 1u) << 17) - 1u;
  if (pos) {
    klo = mlo | 0x80000000u;
    khi = mhi | 0x80000000u;
  } else {
    klo = 0x7fffffffu - mhi;
    khi = 0x7fffffffu - mlo;
  }
}

// The k-th largest of the block's keys (1 <= k <= number of keys); key(i), i < per_thread, are a
// thread's keys.  Absent elements carry key 0 and count like any other key, so k must not
// exceed the number of present elements.  tie_need = how many
// keys equal to the result belong to the top k.  All threads call.
//
// A histogram pass (shared-memory atomics) finds the bin that holds the k-th key; if that bin is small
// its keys are listed and ranked exactly, otherwise the next key bits are histogrammed within it.
// Plain schedule: 12 + 12 + 8 key bits.  VALUE_BINS: the first pass uses key_value_bin (15 key bits
// unless the bin is a clamped one, then the plain schedule starts over), then 12 + 5 bits.
template <int THREADS, int KPT, bool VALUE_BINS = false, typename KeyFn, typename Smem>
__device__ __forceinline__ uint32_t select_kth(KeyFn key, int k, int& tie_need, Smem& sm, int per_thread) {
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  uint32_t prefix = 0, mask = 0;
  int remaining = k, pop = 0;
  // One pass: histogram of digit(key) (negative: the key does not take part) over nb bins, then the bin
  // that holds rank `remaining` (bins in descending order).  Leaves bin, keys above it, its size in sm.pick.
  auto run_level = [&](int nb, auto digit) {
    for (int i = tid; i < nb; i += THREADS) sm.hist[i] = 0;
    __syncthreads();
    for_keys<KPT>(per_thread, [&](int i) {
      const int d = digit(key(i));
      if (d >= 0) atomicAdd(&sm.hist[d], 1u);
    });
    __syncthreads();
    // thread t owns bins nb-1-t*bpt .. nb-bpt-t*bpt (those that exist)
    const int bpt = (nb + THREADS - 1) / THREADS;
    const bool active = tid * bpt < nb;
    int mine = 0;
    if (active)
      for (int q = 0; q < bpt && nb - 1 - tid * bpt - q >= 0; ++q) mine += (int)sm.hist[nb - 1 - tid * bpt - q];
    int incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    if (lane == 31) sm.scan[0][warp] = incl;
    __syncthreads();
    int before = incl - mine;
    for (int w = 0; w < warp; ++w) before += sm.scan[0][w];
    if (active && before < remaining && remaining <= before + mine) {
      int a = before;
      for (int q = 0; q < bpt; ++q) {
        const int bin = nb - 1 - tid * bpt - q;
        if (bin < 0) break;
        const int c = (int)sm.hist[bin];
        if (remaining <= a + c) {
          sm.pick[0] = bin;
          sm.pick[1] = a;
          sm.pick[2] = c;
          break;
        }
        a += c;
      }
    }
    __syncthreads();
  };
  auto radix_level = [&](int bits, int shift) {
    const uint32_t dm = (1u << bits) - 1u;
    run_level(1 << bits, [&](uint32_t kk) { return (kk & mask) == prefix ? (int)((kk >> shift) & dm) : -1; });
    prefix |= (uint32_t)sm.pick[0] << shift;
    mask |= dm << shift;
    remaining -= sm.pick[1];
    pop = sm.pick[2];
  };

  bool done = false;
  if (VALUE_BINS) {
    run_level(SEL_BINS, [&](uint32_t kk) { return key_value_bin(kk); });
    const int bin = sm.pick[0];
    const int m = bin >= SEL_BINS / 2 ? bin - SEL_BINS / 2 : SEL_BINS / 2 - 1 - bin;
    if (m >= 1 && m < SEL_BINS / 2 - 1) {  // not a clamped bin: its keys share their upper 15 bits
      const uint32_t u = (uint32_t)(m + (VB_EXP0 << 6)) << 17;
      prefix = bin >= SEL_BINS / 2 ? (u | 0x80000000u) : (~(u | 0x80000000u) & 0xfffe0000u);
      mask = 0xfffe0000u;
      remaining -= sm.pick[1];
      pop = sm.pick[2];
      if (pop > SEL_RANK_CAP) radix_level(12, 5);
      if (pop > SEL_RANK_CAP) radix_level(5, 0);
      done = true;
    }
    __syncthreads();  // sm.pick is rewritten by the passes below
  }
  if (!done) {
    radix_level(12, 20);
    if (pop > SEL_RANK_CAP) radix_level(12, 8);
    if (pop > SEL_RANK_CAP) radix_level(8, 0);
  }
  if (mask == 0xffffffffu) {  // every bit decided: the keys left are all equal to the result
    tie_need = remaining;
    return prefix;
  }
  // list the keys under the prefix and rank them exactly
  if (tid == 0) sm.counts[2] = 0;
  __syncthreads();
  for_keys<KPT>(per_thread, [&](int i) {
    const uint32_t kk = key(i);
    if ((kk & mask) == prefix) sm.rank_key[atomicAdd(&sm.counts[2], 1)] = kk;
  });
  __syncthreads();
  for (int c = tid; c < pop; c += THREADS) {
    const uint32_t kc = sm.rank_key[c];
    int gt = 0, ge = 0;
    for (int o = 0; o < pop; ++o) {
      const uint32_t ko = sm.rank_key[o];
      gt += ko > kc;
      ge += ko >= kc;
    }
    if (gt < remaining && remaining <= ge) {  // equal keys all write the same pair
      sm.pick[0] = (int)kc;
      sm.pick[1] = remaining - gt;
    }
  }
  __syncthreads();
  tie_need = sm.pick[1];
  return (uint32_t)sm.pick[0];
}

// Sum of v over the block, returned to every thread.  `slot` (0 or 1) picks the scratch row so that
// two calls in a row need no barrier between them.
template <int THREADS, typename Smem>
__device__ __forceinline__ int block_count(int v, int slot, Smem& sm) {
  constexpr int WARPS = THREADS / 32;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  v = __reduce_add_sync(0xffffffffu, v);
  if (lane == 0) sm.scan[slot][warp] = v;
  __syncthreads();
  return __reduce_add_sync(0xffffffffu, lane < WARPS ? sm.scan[slot][lane] : 0);
}

template <int THREADS, typename Smem>
__device__ __forceinline__ float block_max(float v, int slot, Smem& sm) {
  constexpr int WARPS = THREADS / 32;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  v = warp_max(v);
  if (lane == 0) sm.f[slot][warp] = v;
  __syncthreads();
  return warp_max(lane < WARPS ? sm.f[slot][lane] : 0.f);
}

// Ranks the first n_cand candidates (cand_val, cand_idx) and sets cand_keep[c] = (rank < need).
// A barrier must separate the writes of cand_val from this call and this call from the readers.
template <int THREADS, typename Smem>
__device__ __forceinline__ void rank_candidates(int n_cand, int need, Smem& sm) {
  for (int c = threadIdx.x; c < n_cand; c += THREADS) {
    const double v = sm.cand_val[c];
    const int j = sm.cand_idx[c];
    int rank = 0;
    for (int o = 0; o < n_cand; ++o) {
      const double vo = sm.cand_val[o];
      rank += (vo > v) || (vo == v && sm.cand_idx[o] < j);
    }
    sm.cand_keep[c] = rank < need ? 1 : 0;
  }
}

// klass(i) in {0 dropped, 1 tie, 2 kept} for element j = first + tid*per_thread + i, i < per_thread (called
// twice per element).  Ties
// are kept in ascending index order until tie_need runs out.  Kept indices go to out[] ascending;
// emit(i, keep, pos) reports the final decision of every element and, for a kept one, its place in out[].  Returns the kept total to every thread.
// All threads call; uses sm.scan.
template <int THREADS, int KPT, typename ClassFn, typename EmitFn, typename Smem>
__device__ __forceinline__ int compact_counted(int c2, int c1, ClassFn klass, EmitFn emit, int tie_need, int32_t* out,
                                               Smem& sm, int per_thread, int first = 0);

template <int THREADS, int KPT, typename ClassFn, typename EmitFn, typename Smem>
__device__ __forceinline__ int compact_indices(ClassFn klass, EmitFn emit, int tie_need, int32_t* out, Smem& sm,
                                               int per_thread, int first = 0) {
  int c2 = 0, c1 = 0;
  for_keys<KPT>(per_thread, [&](int i) {
    const int c = klass(i);
    c2 += c == 2;
    c1 += c == 1;
  });
  return compact_counted<THREADS, KPT>(c2, c1, klass, emit, tie_need, out, sm, per_thread, first);
}

// The same when the caller already knows how many of its elements are of class 2 (c2) and 1 (c1).
template <int THREADS, int KPT, typename ClassFn, typename EmitFn, typename Smem>
__device__ __forceinline__ int compact_counted(int c2, int c1, ClassFn klass, EmitFn emit, int tie_need, int32_t* out,
                                               Smem& sm, int per_thread, int first) {
  constexpr int WARPS = THREADS / 32;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // exclusive prefix of ties over the block (threads in index order), then of kept elements
  int t_incl = c1;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int v = __shfl_up_sync(0xffffffffu, t_incl, o);
    if (lane >= o) t_incl += v;
  }
  __syncthreads();  // earlier readers of sm.scan are done
  if (lane == 31) sm.scan[0][warp] = t_incl;
  __syncthreads();
  int t_before = t_incl - c1;
  for (int w = 0; w < warp; ++w) t_before += sm.scan[0][w];
  const int my_ties = min(max(tie_need - t_before, 0), c1);
  const int mine = c2 + my_ties;
  int k_incl = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int v = __shfl_up_sync(0xffffffffu, k_incl, o);
    if (lane >= o) k_incl += v;
  }
  if (lane == 31) sm.scan[1][warp] = k_incl;
  __syncthreads();
  int pos = k_incl - mine, total = 0;
  for (int w = 0; w < WARPS; ++w) {
    const int v = sm.scan[1][w];
    if (w < warp) pos += v;
    total += v;
  }
  int ties_left = my_ties;
  const int j0 = first + threadIdx.x * per_thread;
  for_keys<KPT>(per_thread, [&](int i) {
    const int c = klass(i);
    bool kp = c == 2;
    if (c == 1 && ties_left > 0) {
      kp = true;
      --ties_left;
    }
    if (kp) out[pos] = j0 + i;
    emit(i, kp, pos);
    if (kp) ++pos;
  });
  __syncthreads();  // sm.scan may be reused by the caller
  return total;
}

}  // namespace sol
