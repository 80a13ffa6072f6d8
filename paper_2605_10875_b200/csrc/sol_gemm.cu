// Weight-streaming skinny GEMMs on the Blackwell tensor cores.
//
// The batch (16..128 rows after padding) is the small side, so every weight
// byte is read from HBM exactly once and the kernels are bound by HBM
// bandwidth.  Weights are packed once at load time (sol_pack_weights) into the
// order the tensor cores read them from shared memory, and the activation
// operands are written in that order by the kernels that produce them, so:
//
//   * a pipeline stage is two large contiguous bulk copies (cp.async.bulk,
//     8..32 KB each) into a ring of shared-memory stages guarded by mbarriers
//     (bounded waits): one for the weight tile, one for the activation tile;
//   * one thread issues tcgen05.mma (bf16 x bf16 -> float32) with the WEIGHT
//     tile as the 128-row M side and the batch as the N side, accumulating in
//     tensor memory; tcgen05.commit releases each stage when its MMAs finish;
//   * sixteen warps read the accumulators back with tcgen05.ld and apply the
//     epilogue, writing out[m][n] with the weight row n along the lanes.
//
//   umma_nk   : Y[M][N] = A[M][K] . W[N][K]^T   (QKV, output and gate/up projections).  A CTA owns one tile
//               of R weight rows; QKV / output: R = 128 and a slice of K (raw partial sums per slice, summed by
//               the consumer); gate/up: the whole of K, rows alternating gate_c, up_c, so that a channel's two
//               sums sit in neighbouring accumulator lanes and SwiGLU is a lane exchange.  The MMA always
//               spans 128 rows; rows beyond the tile read whatever follows in shared memory and land in
//               accumulator lanes that are never stored.
//   umma_down : Y[M][d] = T[M][ff] . W[ff][d]   (down projection).  W rows are intermediate channels, so the
//               weight tile is the MN-major operand.  CTA = (128 output columns, range of 64-channel
//               blocks); blocks in which no token keeps a channel are neither copied nor multiplied;
//               partial sums per range are reduced by reduce_out.
#include <cstring>

#include "sol_internal.h"
#include "sol_umma.cuh"

namespace sol {

constexpr int UM_EPI_WARPS = 16;     // epilogue warps: four per 32 accumulator lanes (a warp reaches the lanes 32 (w % 4) ..)
constexpr int UM_THREADS = (UM_EPI_WARPS + 2) * 32;  // then warp 16: producer, warp 17: MMA issuer + TMEM owner
constexpr int UM_PRODUCER = UM_EPI_WARPS, UM_MMA = UM_EPI_WARPS + 1;
constexpr int UM_EPI_SETS = UM_EPI_WARPS / 4;  // warps that share a quarter of the lanes take alternate groups of tokens
constexpr int UM_MAX_STAGES = 8;
constexpr int UM_TILE_SPAN = 16384;  // bytes one 128-row operand read spans from the start of a chunk tile
constexpr int UM_SMEM_BUDGET = 204 * 1024;
constexpr int UM_LIVE_CAP = 512;     // 64-channel blocks per CTA of the down projection whose live flags are staged in shared memory

struct UmBarriers {
  uint64_t full[UM_MAX_STAGES];
  uint64_t empty[UM_MAX_STAGES];
  uint64_t accum;
  uint32_t tmem_base;
  int n_issued;
  uint32_t gmax[4][128], umax[4][128];  // SwiGLU epilogue: per token and accumulator quarter, the largest |g| and |u| (float bits)
  alignas(16) float scale[128];   // SwiGLU epilogue: the tokens' quantizer scales
  unsigned char need_hist[128];   // SwiGLU epilogue: the token's channel selection is a real one (0 < kept < ff)
  unsigned char live[UM_LIVE_CAP];  // down projection: which of this CTA's 64-channel blocks hold a kept channel
};

__device__ __forceinline__ unsigned char* align_1024(unsigned char* p) {
  const uint32_t a = smem_u32(p);
  return p + (((a + 1023u) & ~1023u) - a);
}

// ============================================================================
// umma_nk
// ============================================================================
struct NKDev {
  int M, Mpad, K, N;  // N: outputs per token (EPI_SWIGLU: channels, with a gate and an up row each)
  int R;              // packed weight rows per tile
  int chunks;         // K / 64
  int ksplit;         // K slices (blockIdx.y); EPI_PARTIAL writes one partial per slice
  int cps, stages;    // 64-wide k chunks per stage, ring depth
  int n_b;            // 1, or 2: the activation rows are a high-part block followed by a low-part block of
                      // Mpad rows each; one MMA of N = 2 Mpad multiplies both, the epilogue adds the halves
  uint32_t tmem_cols;
  const unsigned char* w;  // packed weights
  const unsigned char* x;  // packed activations
  const float* row_scale;
  float* out0;
  float* out1;
  float* out2;
  uint32_t* sel;
  const int32_t* sel_p;  // [M] prune rates or nullptr
  int* status;
};

template <int EPI>
__global__ void __launch_bounds__(UM_THREADS, 1) umma_nk_kernel(const NKDev p) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* stages = align_1024(smem_raw);
  const int nb_rows = p.n_b * p.Mpad;                      // N of the MMA
  const int w_tile = p.R * 128, x_tile = nb_rows * 128;    // bytes per 64-wide k chunk
  const int stage_bytes = p.cps * (w_tile + x_tile);
  UmBarriers* bars = reinterpret_cast<UmBarriers*>(stages + (size_t)p.stages * stage_bytes + UM_TILE_SPAN);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  pdl_trigger();
  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(&bars->full[s], 1);
      mbar_init(&bars->empty[s], 1);
    }
    mbar_init(&bars->accum, 1);
    fence_mbar_init();
  }
  if (EPI == EPI_SWIGLU)
    for (int i = threadIdx.x; i < 4 * 128; i += UM_THREADS) (&bars->gmax[0][0])[i] = (&bars->umax[0][0])[i] = 0u;
  if (warp == UM_MMA) tmem_alloc(&bars->tmem_base, p.tmem_cols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(&bars->tmem_base);

  const int tile = blockIdx.x;
  // this CTA's K slice, in 64-wide chunks (cps == 1 whenever K is split)
  const int ch0 = (int)(((long long)p.chunks * blockIdx.y) / p.ksplit);
  const int ch1 = (int)(((long long)p.chunks * (blockIdx.y + 1)) / p.ksplit);
  const int n_iter = (ch1 - ch0) / p.cps;
  const unsigned char* w_src = p.w + ((size_t)tile * p.chunks + ch0) * w_tile;  // this tile's chunks are contiguous
  const unsigned char* x_src = p.x + (size_t)ch0 * x_tile;                     // and so are the activation chunks

  if (warp == UM_PRODUCER) {
    // -------------------------------- producer -------------------------------
    // Weights do not depend on earlier kernels: the first ring of weight tiles is requested before
    // pdl_wait(), the activation tiles of those stages after it.
    if (lane == 0) {
      const int pre = min(n_iter, p.stages);
      for (int it = 0; it < pre; ++it) {
        unsigned char* st = stages + (size_t)it * stage_bytes;
        mbar_expect_tx(&bars->full[it], stage_bytes);
        bulk_g2s(st, w_src + (size_t)it * p.cps * w_tile, p.cps * w_tile, &bars->full[it]);
      }
      pdl_wait();
      for (int it = 0; it < pre; ++it) {
        unsigned char* xs = stages + (size_t)it * stage_bytes + p.cps * w_tile;
        bulk_g2s(xs, x_src + (size_t)it * p.cps * x_tile, p.cps * x_tile, &bars->full[it]);
      }
      // ring position and phase are counted along: a division per stage costs the lone issuing thread ~0.1 us
      int s = 0;
      uint32_t ph = 1;
      for (int it = pre; it < n_iter; ++it) {
        if (!mbar_wait(&bars->empty[s], ph ^ 1, p.status)) break;
        unsigned char* st = stages + (size_t)s * stage_bytes;
        mbar_expect_tx(&bars->full[s], stage_bytes);
        bulk_g2s(st, w_src + (size_t)it * p.cps * w_tile, p.cps * w_tile, &bars->full[s]);
        bulk_g2s(st + p.cps * w_tile, x_src + (size_t)it * p.cps * x_tile, p.cps * x_tile, &bars->full[s]);
        if (++s == p.stages) {
          s = 0;
          ph ^= 1;
        }
      }
    }
  } else if (warp == UM_MMA) {
    // ------------------------------- MMA issuer ------------------------------
    // The mbarrier wait orders the copies before the MMA reads; no tcgen05 fence is needed per stage.
    const uint32_t idesc = umma_idesc_bf16_m128(nb_rows, 0, 0);
    bool acc = false, ok = true;
    // the first stage fills only after the producer's own pdl_wait(): without this wait the bounded poll
    // below would start counting while earlier kernels of the stream are still running
    pdl_wait();
    int s = 0;
    uint32_t ph = 0;
    for (int it = 0; it < n_iter; ++it) {
      ok = __all_sync(0xffffffffu, mbar_wait(&bars->full[s], ph, p.status));
      if (!ok) break;
      const uint32_t st = smem_u32(stages + (size_t)s * stage_bytes);
      const uint32_t xs = st + p.cps * w_tile;
      const uint64_t a_base = umma_smem_desc(st, 16, 1024), b_base = umma_smem_desc(xs, 16, 1024);
      for (int c = 0; c < p.cps; ++c) {
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
          // descriptors advance in units of 16 bytes: a chunk tile per c, 32 bytes per 16-wide k step
          const uint64_t a0 = a_base + (uint64_t)((c * w_tile + ks * 32) >> 4);
          const uint64_t b0 = b_base + (uint64_t)((c * x_tile + ks * 32) >> 4);
          if (elect_one()) umma_bf16(tmem, a0, b0, idesc, acc);
          acc = true;
        }
      }
      if (elect_one()) umma_commit(&bars->empty[s]);  // the stage is free again once these MMAs have read it
      __syncwarp();
      if (++s == p.stages) {
        s = 0;
        ph ^= 1;
      }
    }
    if (ok && elect_one()) umma_commit(&bars->accum);
  } else {
    // -------------------------------- epilogue -------------------------------
    pdl_wait();  // the epilogue reads scales and overwrites buffers earlier kernels used
    if (EPI == EPI_SWIGLU) {
      // the scales come to shared memory while the weights stream: a global load per token inside the loop
      // below would put its latency between every two tokens
      if ((int)threadIdx.x < p.Mpad) bars->scale[threadIdx.x] = (p.row_scale && (int)threadIdx.x < p.M) ? p.row_scale[threadIdx.x] : 1.0f;
      if ((int)threadIdx.x < p.Mpad) {
        bool need = (int)threadIdx.x < p.M;
        if (need && p.sel_p != nullptr) {  // the kept count as the selection kernel computes it
          const int m = (int)(((long long)(1000 - p.sel_p[threadIdx.x]) * p.N + 999) / 1000);
          need = m > 0 && m < p.N;
        }
        bars->need_hist[threadIdx.x] = need ? 1 : 0;
      }
      asm volatile("bar.sync 1, %0;" ::"n"(UM_EPI_WARPS * 32) : "memory");  // the epilogue warps
    }
    // warps w, w + 4, w + 8, w + 12 share the accumulator lanes 32 (w % 4) .. and take alternate groups of tokens
    const int quarter = warp & 3, half = warp >> 2;
    if (quarter * 32 < p.R) {
      const bool ok = mbar_wait(&bars->accum, 0, p.status);
      tc_fence_after();
      const int r = quarter * 32 + lane;  // row of the tile = accumulator lane
      const uint32_t tl = tmem + ((uint32_t)(quarter * 32) << 16);
      if (EPI == EPI_SWIGLU) {
        // Even lanes hold a channel's gate sums, their odd neighbours its up sums.  Every CTA runs this code
        // once, so it is fetched cold: a short loop body (eight tokens, not unrolled further) that is fetched once
        // and then runs from the instruction cache beats straight-line code for all tokens, which ran at ~14
        // cycles per instruction.  The tokens are taken in pairs: the even lane gives away its gate sum of the
        // second token and gets the up sum of the first, so each lane of a pair computes SwiGLU for one of the
        // two tokens and no lane repeats its neighbour's work.  The chains of the four pairs are independent and
        // branch-free (fast exponential and division: relative errors of about 2^-21 |g| and 2^-22, far inside
        // the error the channel selection already allows for g itself).
        const int ch = (tile * p.R + r) >> 1;
        const bool valid = r < p.R && ch < p.N;
        const bool even = (lane & 1) == 0;
        float* const dst = even ? p.out0 : p.out1;
#pragma unroll 1
        for (int c0 = half * 8; c0 < p.M && ok; c0 += 8 * UM_EPI_SETS) {
          uint32_t ra[8], rb[8];
          tmem_ld8_issue(tl + c0, ra);
          tmem_ld8_issue(tl + (p.n_b == 2 ? p.Mpad : 0) + c0, rb);  // high-part and low-part products
          const float4 s0 = *reinterpret_cast<const float4*>(&bars->scale[c0]);
          const float4 s1 = *reinterpret_cast<const float4*>(&bars->scale[c0 + 4]);
          const float sc[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
          tmem_ld_wait8(ra, rb);
          float v[8], tv[4];
#pragma unroll
          for (int i = 0; i < 8; ++i) v[i] = (__uint_as_float(ra[i]) + (p.n_b == 2 ? __uint_as_float(rb[i]) : 0.f)) * sc[i];
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const float got = __shfl_xor_sync(0xffffffffu, even ? v[2 * j + 1] : v[2 * j], 1);
            const float g = even ? v[2 * j] : got, u = even ? got : v[2 * j + 1];
            tv[j] = __fdividef(g, 1.0f + __expf(-g)) * u;
          }
#pragma unroll
          for (int i = 0; i < 8; ++i)
            if (c0 + i < p.M && valid) dst[(size_t)(c0 + i) * p.N + ch] = v[i];
          const int mine = c0 + (even ? 0 : 1);  // the token of pair 0 whose t this lane holds
#pragma unroll
          for (int j = 0; j < 4; ++j)
            if (mine + 2 * j < p.M && valid) p.out2[(size_t)(mine + 2 * j) * p.N + ch] = tv[j];
          if (p.sel != nullptr) {
            // what the channel selection needs from all of a token's channels: a histogram of |t| and the largest
            // |g|, |u| (non-negative floats order like their bit patterns).  The maxima of this warp's 16 channels
            // go to the warp's own words in shared memory (no atomics); the CTA merges them at the end.
#pragma unroll
            for (int j = 0; j < 4; ++j)
              if (mine + 2 * j < p.M && valid && bars->need_hist[mine + 2 * j])
                atomicAdd(p.sel + (size_t)(mine + 2 * j) * CH_SEL_WORDS + chan_bin(fabsf(tv[j])), 1u);
            uint32_t gs = 0u, us = 0u;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const uint32_t a = valid ? __float_as_uint(fabsf(v[i])) : 0u;
              const uint32_t gm = __reduce_max_sync(0xffffffffu, even ? a : 0u);
              const uint32_t um = __reduce_max_sync(0xffffffffu, even ? 0u : a);
              gs = lane == i ? gm : gs;
              us = lane == i ? um : us;
            }
            if (lane < 8) {
              bars->gmax[quarter][c0 + lane] = gs;
              bars->umax[quarter][c0 + lane] = us;
            }
          }
        }
      } else {
        const int n = tile * p.R + r;
        const bool valid = r < p.R && n < p.N;
        for (int c0 = half * 16; c0 < p.Mpad && ok; c0 += 16 * UM_EPI_SETS) {
          float v[16];
          tmem_ld16(tl + c0, v);
          if (p.n_b == 2) {  // high-part and low-part products
            float w2[16];
            tmem_ld16(tl + p.Mpad + c0, w2);
#pragma unroll
            for (int i = 0; i < 16; ++i) v[i] += w2[i];
          }
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const int m = c0 + i;
            if (m < p.M && valid) p.out0[((size_t)blockIdx.y * p.M + m) * p.N + n] = v[i];
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == UM_MMA) tmem_dealloc(tmem, p.tmem_cols);
  if (EPI == EPI_SWIGLU && p.sel != nullptr && (int)threadIdx.x < p.M) {
    const int m = threadIdx.x;
    uint32_t* sel = p.sel + (size_t)m * CH_SEL_WORDS;
    atomicMax(sel + CH_GMAX, max(max(bars->gmax[0][m], bars->gmax[1][m]), max(bars->gmax[2][m], bars->gmax[3][m])));
    atomicMax(sel + CH_UMAX, max(max(bars->umax[0][m], bars->umax[1][m]), max(bars->umax[2][m], bars->umax[3][m])));
  }
}

// ============================================================================
// umma_down
// ============================================================================
struct DownDev {
  int M, Mpad, ff, d;
  int chunks, stages;
  uint32_t tmem_cols;
  const unsigned char* w;  // packed W_down_t: [slab][64-channel block][16 KB]
  const unsigned char* t;  // packed masked activations: [64-channel chunk][2 Mpad rows][128 B]
  const int32_t* live;     // [ff/32]
  float* partial;          // [chunks][Mpad][d]
  int* status;
};

__device__ __forceinline__ bool block_live(const int32_t* live, int jb, int granules) {
  return live[2 * jb] != 0 || (2 * jb + 1 < granules && live[2 * jb + 1] != 0);
}

__global__ void __launch_bounds__(UM_THREADS, 1) umma_down_kernel(const DownDev p) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* stages = align_1024(smem_raw);
  const int t_tile = 2 * p.Mpad * 128;
  const int stage_bytes = UM_TILE_SPAN + t_tile;
  UmBarriers* bars = reinterpret_cast<UmBarriers*>(stages + (size_t)p.stages * stage_bytes);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  pdl_trigger();
  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(&bars->full[s], 1);
      mbar_init(&bars->empty[s], 1);
    }
    mbar_init(&bars->accum, 1);
    bars->n_issued = 0;
    fence_mbar_init();
  }
  if (warp == UM_MMA) tmem_alloc(&bars->tmem_base, p.tmem_cols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  pdl_wait();  // which channel blocks are live is decided by the selection kernel
  const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(&bars->tmem_base);

  const int slab = blockIdx.x, chunk = blockIdx.y;
  const int granules = p.ff / 32, jblocks = (p.ff + 63) / 64;
  const int jb0 = (int)(((long long)jblocks * chunk) / p.chunks);
  const int jb1 = (int)(((long long)jblocks * (chunk + 1)) / p.chunks);
  // the flags of this CTA's blocks, read by all threads at once: the producer and the MMA issuer walk the
  // same list, and a global load per block would put its latency between every two copies
  const bool staged = jb1 - jb0 <= UM_LIVE_CAP;
  if (staged) {
    for (int i = threadIdx.x; i < jb1 - jb0; i += UM_THREADS) bars->live[i] = block_live(p.live, jb0 + i, granules) ? 1 : 0;
    __syncthreads();
  }

  if (warp == UM_PRODUCER) {
    if (lane == 0) {
      int s = 0;
      uint32_t ph = 0;
      for (int jb = jb0; jb < jb1; ++jb) {
        if (!(staged ? bars->live[jb - jb0] != 0 : block_live(p.live, jb, granules))) continue;
        if (!mbar_wait(&bars->empty[s], ph ^ 1, p.status)) break;
        unsigned char* st = stages + (size_t)s * stage_bytes;
        mbar_expect_tx(&bars->full[s], stage_bytes);
        bulk_g2s(st, p.w + ((size_t)slab * jblocks + jb) * UM_TILE_SPAN, UM_TILE_SPAN, &bars->full[s]);
        bulk_g2s(st + UM_TILE_SPAN, p.t + (size_t)jb * t_tile, t_tile, &bars->full[s]);  // high rows then low rows
        if (++s == p.stages) {
          s = 0;
          ph ^= 1;
        }
      }
    }
  } else if (warp == UM_MMA) {
    const uint32_t idesc = umma_idesc_bf16_m128(2 * p.Mpad, 1, 0);
    bool acc = false, ok = true;
    int s = 0;
    uint32_t ph = 0;
    for (int jb = jb0; jb < jb1; ++jb) {
      if (!(staged ? bars->live[jb - jb0] != 0 : block_live(p.live, jb, granules))) continue;
      ok = __all_sync(0xffffffffu, mbar_wait(&bars->full[s], ph, p.status));
      if (!ok) break;
      const uint32_t st = smem_u32(stages + (size_t)s * stage_bytes);
      // weight tile: two 64-column blocks of [64 channels][128 bytes]; 16 channels = two 8-row groups
      const uint64_t a_base = umma_smem_desc(st, 8192, 1024);
      const uint64_t t_base = umma_smem_desc(st + UM_TILE_SPAN, 16, 1024);  // [2 Mpad rows][64 channels]
#pragma unroll
      for (int ks = 0; ks < 4; ++ks) {
        if (elect_one())
          umma_bf16(tmem, a_base + (uint64_t)((ks * 2048) >> 4), t_base + (uint64_t)((ks * 32) >> 4), idesc, acc);
        acc = true;
      }
      if (elect_one()) umma_commit(&bars->empty[s]);
      __syncwarp();
      if (++s == p.stages) {
        s = 0;
        ph ^= 1;
      }
    }
    if (lane == 0) {
      *reinterpret_cast<volatile int*>(&bars->n_issued) = acc ? 1 : 0;
      __threadfence_block();
    }
    __syncwarp();
    if (ok && elect_one()) umma_commit(&bars->accum);
  } else {
    const bool ok = mbar_wait(&bars->accum, 0, p.status);
    tc_fence_after();
    const bool any = *reinterpret_cast<volatile int*>(&bars->n_issued) > 0;
    const int quarter = warp & 3, half = warp >> 2;  // as in umma_nk: four warps per 32 accumulator lanes
    const int n = slab * 128 + quarter * 32 + lane;
    const uint32_t tl = tmem + ((uint32_t)(quarter * 32) << 16);
    float* out = p.partial + (size_t)chunk * p.Mpad * p.d;
    for (int c0 = half * 16; c0 < p.Mpad && ok; c0 += 16 * UM_EPI_SETS) {
      float v[16];
      if (any) {
        float w2[16];
        tmem_ld16(tl + c0, v);
        tmem_ld16(tl + p.Mpad + c0, w2);
#pragma unroll
        for (int i = 0; i < 16; ++i) v[i] += w2[i];
      } else {
#pragma unroll
        for (int i = 0; i < 16; ++i) v[i] = 0.f;
      }
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const int m = c0 + i;
        if (m < p.M) out[(size_t)m * p.d + n] = v[i];
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == UM_MMA) tmem_dealloc(tmem, p.tmem_cols);
}

// ============================================================================
// down_rows: the down projection of a small batch, row by row
// ============================================================================
// At batch <= 8 the union of the channels that some token keeps is well below d_ff when tokens are pruned, and a
// 64-channel block is almost never dead as a whole: this kernel reads W_down channel by channel and skips
// every channel that no token keeps, so the bytes follow the union of kept rows.  CTA = (128 output columns,
// range of channels) as in umma_down; a warp takes groups of 32 channels of the range, finds the kept ones with
// one ballot, reads each kept channel's 256 bytes of the slab (two 128-byte pieces of the packed layout, one per
// column half) and multiplies them into float32 accumulators (<= 8 tokens x 4 columns per lane) on the FMA
// pipes; the warps are merged through shared memory.
constexpr int DR_WARPS = 8;
constexpr int DR_MAXB = 8;

struct DownRowsDev {
  int M, Mpad, ff, d, chunks;
  const unsigned char* w;     // packed W_down_t
  const float* t;             // [M][ff] silu(g) u before masking
  const unsigned char* keep;  // [M][ff] 1 = kept
  float* partial;             // [chunks][Mpad][d]
};

__global__ void __launch_bounds__(DR_WARPS * 32) down_rows_kernel(const DownRowsDev p) {
  __shared__ float red[DR_WARPS][DR_MAXB][128];
  const int slab = blockIdx.x, chunk = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int jblocks = (p.ff + 63) / 64;
  const int j0 = (int)(((long long)p.ff * chunk) / p.chunks), j1 = (int)(((long long)p.ff * (chunk + 1)) / p.chunks);
  pdl_trigger();
  pdl_wait();
  float acc[DR_MAXB][4];
#pragma unroll
  for (int m = 0; m < DR_MAXB; ++m)
#pragma unroll
    for (int c = 0; c < 4; ++c) acc[m][c] = 0.f;
  // A warp takes groups of 32 consecutive channels of the CTA's range.  Lane l first looks channel l of the group
  // up in the tokens' keep masks and fetches the tokens' t for it (one round trip, all loads independent); the
  // channels that some token keeps are then taken eight at a time: their weight pieces are requested together
  // (256 bytes per channel, coalesced), the tokens' t come from the owning lane by a shuffle.  Looking one
  // channel up after the other put three dependent round trips in front of every four channels (66 us for
  // the whole matrix at batch 1).
#pragma unroll 1
  for (int g0 = j0 + warp * 32; g0 < j1; g0 += DR_WARPS * 32) {
    const int jl = g0 + lane;
    float tl[DR_MAXB];
    bool mine = false;
#pragma unroll
    for (int m = 0; m < DR_MAXB; ++m) {
      tl[m] = 0.f;
      if (jl < j1 && m < p.M) {
        const bool k = p.keep[(size_t)m * p.ff + jl] != 0;
        const float v = p.t[(size_t)m * p.ff + jl];
        tl[m] = k ? v : 0.f;
        mine = mine || k;
      }
    }
    unsigned todo = __ballot_sync(0xffffffffu, mine);
    while (todo) {  // warp-uniform
      int ch[8];
      uint32_t wv[8][2];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        ch[u] = -1;
        wv[u][0] = wv[u][1] = 0u;
        if (todo) {
          ch[u] = __ffs(todo) - 1;
          todo &= todo - 1;
          // channel j of the slab: block j / 64, row c = j % 64; lane l holds columns 2 l, 2 l + 1 of each 64-column half
          const int j = g0 + ch[u], c = j & 63;
          const unsigned char* base = p.w + ((size_t)slab * jblocks + (j >> 6)) * UM_TILE_SPAN + c * 128 +
                                      (((lane >> 2) ^ (c & 7)) * 16) + (lane & 3) * 4;
          wv[u][0] = *reinterpret_cast<const uint32_t*>(base);
          wv[u][1] = *reinterpret_cast<const uint32_t*>(base + 8192);
        }
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        if (ch[u] < 0) continue;  // warp-uniform
        const float w0 = bf16_lo(wv[u][0]), w1 = bf16_hi(wv[u][0]), w2 = bf16_lo(wv[u][1]), w3 = bf16_hi(wv[u][1]);
#pragma unroll
        for (int m = 0; m < DR_MAXB; ++m) {
          const float tv = __shfl_sync(0xffffffffu, tl[m], ch[u]);
          acc[m][0] = fmaf(tv, w0, acc[m][0]);
          acc[m][1] = fmaf(tv, w1, acc[m][1]);
          acc[m][2] = fmaf(tv, w2, acc[m][2]);
          acc[m][3] = fmaf(tv, w3, acc[m][3]);
        }
      }
    }
  }
  // columns of the slab held by lane l: 2 l, 2 l + 1 (first half), 64 + 2 l, 64 + 2 l + 1 (second half)
#pragma unroll
  for (int m = 0; m < DR_MAXB; ++m) {
    red[warp][m][2 * lane] = acc[m][0];
    red[warp][m][2 * lane + 1] = acc[m][1];
    red[warp][m][64 + 2 * lane] = acc[m][2];
    red[warp][m][64 + 2 * lane + 1] = acc[m][3];
  }
  __syncthreads();
  for (int i = threadIdx.x; i < p.M * 128; i += DR_WARPS * 32) {
    const int m = i >> 7, c = i & 127;
    float a = 0.f;
#pragma unroll
    for (int w = 0; w < DR_WARPS; ++w) a += red[w][m][c];
    p.partial[((size_t)chunk * p.Mpad + m) * p.d + slab * 128 + c] = a;
  }
}

// ============================================================================
// one-time packing of the weights
// ============================================================================
// One thread per 16-byte piece of the packed matrix.
__global__ void pack_nk_kernel(const uint4* __restrict__ src0, const uint4* __restrict__ src1, uint4* __restrict__ dst,
                               int n_src_rows, int K, int R, int tiles, int chunks, int interleaved) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const size_t total = (size_t)tiles * chunks * R * 8;
  if (i >= total) return;
  const int q_dst = (int)(i & 7);
  const size_t row_lin = i >> 3;  // ((tile * chunks + chunk) * R + r)
  const int r = (int)(row_lin % R);
  const int chunk = (int)((row_lin / R) % chunks);
  const int tile = (int)(row_lin / ((size_t)R * chunks));
  const int q = q_dst ^ (r & 7);  // the source piece that lives at this position
  const int n = tile * R + r;     // packed row
  uint4 v = make_uint4(0u, 0u, 0u, 0u);
  const int src_row = interleaved ? n >> 1 : n;
  if (src_row < n_src_rows) {
    const uint4* src = (interleaved && (n & 1)) ? src1 : src0;
    v = src[((size_t)src_row * K + (size_t)chunk * 64 + q * 8) / 8];
  }
  dst[i] = v;
}

__global__ void pack_down_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst, int ff, int d) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int jblocks = (ff + 63) / 64;
  const size_t total = (size_t)(d / 128) * jblocks * 1024;  // pieces
  if (i >= total) return;
  const int q_dst = (int)(i & 7);
  const int c = (int)((i >> 3) & 63);         // channel within the block
  const int cb = (int)((i >> 9) & 1);         // 64-column half of the slab
  const int jb = (int)((i >> 10) % jblocks);
  const int slab = (int)((i >> 10) / jblocks);
  const int q = q_dst ^ (c & 7);
  const int j = jb * 64 + c;
  uint4 v = make_uint4(0u, 0u, 0u, 0u);
  if (j < ff) v = src[((size_t)j * d + slab * 128 + cb * 64 + q * 8) / 8];
  dst[i] = v;
}

void launch_pack_weights(const sol_shape_t& s, int kind, const void* src0, const void* src1, void* dst, cudaStream_t st) {
  const int d = s.d_model, qo = s.n_q_heads * s.head_dim, nqkv = (s.n_q_heads + 2 * s.n_kv_heads) * s.head_dim;
  if (kind == SOL_W_DOWN) {
    const size_t pieces = down_packed_bytes(s.d_ff, d) / 16;
    pack_down_kernel<<<(unsigned)((pieces + 255) / 256), 256, 0, st>>>(static_cast<const uint4*>(src0), static_cast<uint4*>(dst),
                                                                      s.d_ff, d);
  } else {
    NKGeom g;
    int rows;
    if (kind == SOL_W_QKV) { g = nk_geom_plain(nqkv, d); rows = nqkv; }
    else if (kind == SOL_W_O) { g = nk_geom_plain(d, qo); rows = d; }
    else { g = nk_geom_gate_up(s.d_ff, d, sm_count()); rows = s.d_ff; }
    const size_t pieces = nk_packed_bytes(g) / 16;
    pack_nk_kernel<<<(unsigned)((pieces + 255) / 256), 256, 0, st>>>(static_cast<const uint4*>(src0), static_cast<const uint4*>(src1),
                                                                    static_cast<uint4*>(dst), rows, g.K, g.R, g.tiles,
                                                                    g.chunks, kind == SOL_W_GATE_UP ? 1 : 0);
  }
  record_cuda_error(cudaGetLastError(), "weight packing");
}

// ============================================================================
// launchers
// ============================================================================
namespace {

uint32_t pow2_cols(int n) {
  uint32_t c = 32;
  while ((int)c < n) c <<= 1;
  return c;
}

}  // namespace

int pad_rows(int B) {
  const int mt = (B + 15) / 16;
  return 16 * (mt <= 1 ? 1 : (mt <= 2 ? 2 : (mt <= 4 ? 4 : 8)));
}

// Split-K of the EPI_PARTIAL projections: as many K slices as it takes to give every SM a CTA.
int nk_ksplit(int N, int K) {
  const NKGeom g = nk_geom_plain(N, K);
  int z = sm_count() / g.tiles;
  if (z > g.chunks) z = g.chunks;
  if (z > NK_MAX_KSPLIT) z = NK_MAX_KSPLIT;
  if (z < 1) z = 1;
  return z;
}

void launch_gemm_nk(const GemmNK& g, GemmEpilogue epi, cudaStream_t st) {
  NKDev d;
  memset(&d, 0, sizeof(d));
  d.M = g.M; d.Mpad = pad_rows(g.M); d.K = g.K; d.N = g.N;
  d.n_b = g.n_b;
  const NKGeom geo = epi == EPI_SWIGLU ? nk_geom_gate_up(g.N, g.K, sm_count()) : nk_geom_plain(g.N, g.K);
  d.R = geo.R;
  d.chunks = geo.chunks;
  d.ksplit = epi == EPI_PARTIAL ? nk_ksplit(g.N, g.K) : 1;
  const int chunk_bytes = 128 * (d.R + d.n_b * d.Mpad);
  int cps = d.ksplit > 1 ? 1 : 4;
  while (cps > 1 && (cps * chunk_bytes > 64 * 1024 || d.chunks % cps)) cps >>= 1;  // few, large stages: every stage costs a commit
  d.cps = cps;
  const int stage_bytes = cps * chunk_bytes;
  const int iters = (d.chunks / d.ksplit + (d.chunks % d.ksplit ? 1 : 0)) / cps;  // of the longest slice
  int stages = UM_SMEM_BUDGET / stage_bytes;
  if (stages > UM_MAX_STAGES) stages = UM_MAX_STAGES;
  if (stages > iters) stages = iters;
  if (stages < 1) stages = 1;
  d.stages = stages;
  d.tmem_cols = pow2_cols(d.n_b * d.Mpad);
  d.w = static_cast<const unsigned char*>(g.w);
  d.x = static_cast<const unsigned char*>(g.a);
  d.row_scale = g.row_scale;
  d.out0 = g.out0; d.out1 = g.out1; d.out2 = g.out2; d.sel = g.sel; d.sel_p = g.sel_p_permille; d.status = g.status;
  const int smem = 1024 + stages * stage_bytes + UM_TILE_SPAN + (int)sizeof(UmBarriers);
  const dim3 grid(geo.tiles, d.ksplit);
  if (epi == EPI_SWIGLU) {
    ensure_dynamic_smem(reinterpret_cast<const void*>(&umma_nk_kernel<EPI_SWIGLU>), smem);
    SOL_LAUNCH("gemm_gate_up_swiglu", umma_nk_kernel<EPI_SWIGLU>, grid, dim3(UM_THREADS), smem, st, d);
  } else {
    ensure_dynamic_smem(reinterpret_cast<const void*>(&umma_nk_kernel<EPI_PARTIAL>), smem);
    SOL_LAUNCH(g.name ? g.name : "gemm_partial", umma_nk_kernel<EPI_PARTIAL>, grid, dim3(UM_THREADS), smem, st, d);
  }
}

int down_chunks(int ff, int d) {
  const int slabs = d / 128;
  const int jblocks = (ff + 63) / 64;
  int c = sm_count() / (slabs > 0 ? slabs : 1);
  if (c < 1) c = 1;
  if (c > jblocks) c = jblocks;
  return c;
}

void launch_gemm_down(const GemmDown& g, cudaStream_t st) {
  if (g.M <= DR_MAXB && g.t_f32 != nullptr && g.keep != nullptr) {  // small batch: channel by channel, only kept rows
    DownRowsDev r;
    r.M = g.M; r.Mpad = pad_rows(g.M); r.ff = g.ff; r.d = g.d; r.chunks = g.chunks;
    r.w = static_cast<const unsigned char*>(g.w); r.t = g.t_f32; r.keep = g.keep; r.partial = g.partial;
    SOL_LAUNCH("gemm_down_gathered", down_rows_kernel, dim3(g.d / 128, g.chunks), dim3(DR_WARPS * 32), 0, st, r);
    return;
  }
  DownDev d;
  memset(&d, 0, sizeof(d));
  d.M = g.M; d.Mpad = pad_rows(g.M); d.ff = g.ff; d.d = g.d;
  d.chunks = g.chunks;
  const int stage_bytes = UM_TILE_SPAN + 2 * d.Mpad * 128;
  int stages = UM_SMEM_BUDGET / stage_bytes;
  if (stages > UM_MAX_STAGES) stages = UM_MAX_STAGES;
  d.stages = stages;
  d.tmem_cols = pow2_cols(2 * d.Mpad);
  d.w = static_cast<const unsigned char*>(g.w);
  d.t = static_cast<const unsigned char*>(g.t);
  d.live = g.live; d.partial = g.partial; d.status = g.status;
  const int smem = 1024 + stages * stage_bytes + (int)sizeof(UmBarriers);
  ensure_dynamic_smem(reinterpret_cast<const void*>(&umma_down_kernel), smem);
  SOL_LAUNCH("gemm_down_gathered", umma_down_kernel, dim3(g.d / 128, g.chunks), dim3(UM_THREADS), smem, st, d);
}

// ============================================================================
// reduce the down-projection partials, add the residual, emit bf16 / fp32
// ============================================================================
__global__ void reduce_out_kernel(const float* __restrict__ partial, int chunks, int M, int Mpad, int d,
                                  const void* __restrict__ resid, int resid_f32, uint16_t* __restrict__ out_bf16,
                                  float* __restrict__ out_f32, float* __restrict__ out_f32_b, int32_t* __restrict__ live,
                                  int n_live) {
  pdl_trigger();
  pdl_wait();
  const int gi = blockIdx.x * blockDim.x + threadIdx.x;
  if (gi < n_live) live[gi] = 0;  // the down projection has read the flags; the next selection starts from zero
  const int i = gi * 4;
  if (i >= M * d) return;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int c0 = 0; c0 < chunks; c0 += 4) {  // four partials' loads in flight, added in order
    float4 v[4];
#pragma unroll
    for (int q = 0; q < 4; ++q)
      v[q] = c0 + q < chunks ? *reinterpret_cast<const float4*>(partial + (size_t)(c0 + q) * Mpad * d + i)
                             : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      acc.x += v[q].x; acc.y += v[q].y; acc.z += v[q].z; acc.w += v[q].w;
    }
  }
  if (resid != nullptr) {
    if (resid_f32) {
      const float4 r = *reinterpret_cast<const float4*>(static_cast<const float*>(resid) + i);
      acc.x += r.x; acc.y += r.y; acc.z += r.z; acc.w += r.w;
    } else {
      const uint2 r = *reinterpret_cast<const uint2*>(static_cast<const uint16_t*>(resid) + i);
      acc.x += bf16_lo(r.x); acc.y += bf16_hi(r.x); acc.z += bf16_lo(r.y); acc.w += bf16_hi(r.y);
    }
  }
  if (out_bf16) {
    uint2 o;
    o.x = pack_bf16(acc.x, acc.y);
    o.y = pack_bf16(acc.z, acc.w);
    *reinterpret_cast<uint2*>(out_bf16 + i) = o;
  }
  if (out_f32) *reinterpret_cast<float4*>(out_f32 + i) = acc;
  if (out_f32_b) *reinterpret_cast<float4*>(out_f32_b + i) = acc;
}

void launch_reduce_out(const float* partial, int chunks, int M, int Mpad, int d, const void* resid, int resid_f32,
                       void* out_bf16, float* out_f32, float* out_f32_b, int32_t* live, int n_live, cudaStream_t st) {
  int n4 = M * d / 4;
  if (n4 < n_live) n4 = n_live;
  SOL_LAUNCH("down_reduce_residual", reduce_out_kernel, dim3((n4 + 255) / 256), dim3(256), 0, st, partial, chunks, M,
             Mpad, d, resid, resid_f32, static_cast<uint16_t*>(out_bf16), out_f32, out_f32_b, live, n_live);
}

}  // namespace sol
