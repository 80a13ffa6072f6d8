// Weight-streaming skinny GEMMs on the Blackwell tensor cores.
//
// The batch (16..128 rows after padding) is the small side, so every weight
// byte is read from HBM exactly once and the kernels are bound by HBM
// bandwidth.  They are built so that one thread keeps large TMA copies in
// flight and nobody touches the data with ordinary instructions:
//
//   * weights and activations arrive by TMA tiled loads through tensor maps
//     (128-byte swizzle, several 64-wide k chunks per copy) into a ring of
//     shared-memory stages guarded by mbarriers (bounded waits);
//   * one thread issues tcgen05.mma (bf16 x bf16 -> float32) with the WEIGHT
//     tile as the 128-row M side and the batch as the N side, accumulating in
//     tensor memory; tcgen05.commit releases each stage when its MMAs finish;
//   * four warps read the accumulators back with tcgen05.ld and apply the
//     epilogue (quantizer scale / residual / SwiGLU), writing out[m][n] with
//     the weight row n along the lanes (coalesced).
//
//   umma_nk   : Y[M][N] = A[M][K] . W[N][K]^T   (QKV, output and gate/up projections).  Each CTA owns
//               a contiguous range of `rows` weight rows (a multiple of 8 chosen so that one wave of
//               CTAs covers all SMs) over the whole of K.  The MMA always spans 128 rows; rows beyond
//               the CTA's range read whatever follows in shared memory and land in accumulator lanes
//               that are never stored (an output row depends only on its own weight row).
//   umma_down : Y[M][d] = T[M][ff] . W[ff][d]   (down projection).  W rows are intermediate channels,
//               so the weight tile is the MN-major operand.  CTA = (128 output columns, range of 64-
//               channel blocks); blocks in which no token keeps a channel are neither copied nor
//               multiplied; partial sums per range are reduced by reduce_out.
#include <cstring>
#include <mutex>
#include <unordered_map>

#include <cudaTypedefs.h>

#include "sol_internal.h"
#include "sol_umma.cuh"

namespace sol {

constexpr int UM_THREADS = 192;      // warps 0-3: epilogue, warp 4: TMA producer, warp 5: MMA issuer + TMEM owner
constexpr int UM_MAX_STAGES = 8;
constexpr int UM_TILE_SPAN = 16384;  // bytes one 128-row operand read spans from the start of a chunk tile
constexpr int UM_SMEM_BUDGET = 204 * 1024;

struct UmBarriers {
  uint64_t full[UM_MAX_STAGES];
  uint64_t empty[UM_MAX_STAGES];
  uint64_t accum;
  uint32_t tmem_base;
  int n_issued;
};

__device__ __forceinline__ unsigned char* align_1024(unsigned char* p) {
  const uint32_t a = smem_u32(p);
  return p + (((a + 1023u) & ~1023u) - a);
}

// ============================================================================
// umma_nk
// ============================================================================
struct NKDev {
  int M, Mpad, K, N;  // N: weight rows (EPI_SWIGLU: channels, with a gate and an up row each)
  int rows;           // weight rows per CTA
  int ksplit;         // K slices (blockIdx.y); EPI_PARTIAL writes one partial per slice
  int cps, stages;    // 64-wide k chunks per stage, ring depth
  int n_b;            // 1, or 2: the activation rows are a high-part block followed by a low-part block of
                      // Mpad rows each; one MMA of N = 2 Mpad multiplies both, the epilogue adds the halves
  uint32_t tmem_cols;
  const float* row_scale;
  float* out0;
  float* out1;
  float* out2;
  uint32_t* sel;
  int* status;
};

template <int EPI>
__global__ void __launch_bounds__(UM_THREADS, 1)
umma_nk_kernel(const __grid_constant__ CUtensorMap tm_w0, const __grid_constant__ CUtensorMap tm_w1,
               const __grid_constant__ CUtensorMap tm_x0, const NKDev p) {
  extern __shared__ unsigned char smem_raw[];
  constexpr int NW = EPI == EPI_SWIGLU ? 2 : 1;
  unsigned char* stages = align_1024(smem_raw);
  const int nb_rows = p.n_b * p.Mpad;                      // N of the MMA
  const int w_tile = p.rows * 128, x_tile = nb_rows * 128;  // bytes per 64-wide k chunk
  const int stage_bytes = p.cps * (NW * w_tile + x_tile);
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
  if (warp == 5) tmem_alloc(&bars->tmem_base, p.tmem_cols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(&bars->tmem_base);

  const int row0 = blockIdx.x * p.rows;
  // this CTA's K slice, in 64-wide chunks (cps == 1 whenever K is split)
  const int chunks = p.K / 64;
  const int ch0 = (int)(((long long)chunks * blockIdx.y) / p.ksplit);
  const int ch1 = (int)(((long long)chunks * (blockIdx.y + 1)) / p.ksplit);
  const int n_iter = (ch1 - ch0) / p.cps;

  if (warp == 4) {
    // ------------------------------ TMA producer -----------------------------
    // Weights do not depend on earlier kernels: the first ring of weight tiles is requested before
    // pdl_wait(), the activation tiles of those stages after it.
    if (lane == 0) {
      tma_prefetch_map(&tm_w0);
      tma_prefetch_map(&tm_x0);
      const int pre = min(n_iter, p.stages);
      for (int it = 0; it < pre; ++it) {
        unsigned char* st = stages + (size_t)it * stage_bytes;
        mbar_expect_tx(&bars->full[it], stage_bytes);
        tma_load_3d(st, &tm_w0, 0, row0, ch0 + it * p.cps, &bars->full[it]);
        if (NW == 2) tma_load_3d(st + p.cps * w_tile, &tm_w1, 0, row0, ch0 + it * p.cps, &bars->full[it]);
      }
      pdl_wait();
      for (int it = 0; it < pre; ++it) {
        unsigned char* xs = stages + (size_t)it * stage_bytes + NW * p.cps * w_tile;
        tma_load_3d(xs, &tm_x0, 0, 0, ch0 + it * p.cps, &bars->full[it]);
      }
      for (int it = pre; it < n_iter; ++it) {
        const int s = it % p.stages;
        const uint32_t ph = (it / p.stages) & 1;
        if (!mbar_wait(&bars->empty[s], ph ^ 1, p.status)) break;
        unsigned char* st = stages + (size_t)s * stage_bytes;
        mbar_expect_tx(&bars->full[s], stage_bytes);
        tma_load_3d(st, &tm_w0, 0, row0, ch0 + it * p.cps, &bars->full[s]);
        if (NW == 2) tma_load_3d(st + p.cps * w_tile, &tm_w1, 0, row0, ch0 + it * p.cps, &bars->full[s]);
        unsigned char* xs = st + NW * p.cps * w_tile;
        tma_load_3d(xs, &tm_x0, 0, 0, ch0 + it * p.cps, &bars->full[s]);
      }
    }
  } else if (warp == 5) {
    // ------------------------------- MMA issuer ------------------------------
    // The mbarrier wait orders the TMA writes before the MMA reads; no tcgen05 fence is needed per stage.
    const uint32_t idesc = umma_idesc_bf16_m128(nb_rows, 0, 0);
    bool acc = false, ok = true;
    // the first stage fills only after the producer's own pdl_wait(): without this wait the bounded poll
    // below would start counting while earlier kernels of the stream are still running
    pdl_wait();
    for (int it = 0; it < n_iter; ++it) {
      const int s = it % p.stages;
      const uint32_t ph = (it / p.stages) & 1;
      ok = __all_sync(0xffffffffu, mbar_wait(&bars->full[s], ph, p.status));
      if (!ok) break;
      const uint32_t st = smem_u32(stages + (size_t)s * stage_bytes);
      const uint32_t xs = st + NW * p.cps * w_tile;
      const uint64_t a_base = umma_smem_desc(st, 16, 1024), b_base = umma_smem_desc(xs, 16, 1024);
      for (int c = 0; c < p.cps; ++c) {
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
          // descriptors advance in units of 16 bytes: a chunk tile per c, 32 bytes per 16-wide k step
          const uint64_t a0 = a_base + (uint64_t)((c * w_tile + ks * 32) >> 4);
          const uint64_t a1 = a_base + (uint64_t)(((p.cps + c) * w_tile + ks * 32) >> 4);
          const uint64_t b0 = b_base + (uint64_t)((c * x_tile + ks * 32) >> 4);
          if (elect_one()) {
            umma_bf16(tmem, a0, b0, idesc, acc);
            if (NW == 2) umma_bf16(tmem + nb_rows, a1, b0, idesc, acc);
          }
          acc = true;
        }
      }
      if (elect_one()) umma_commit(&bars->empty[s]);  // the stage is free again once these MMAs have read it
      __syncwarp();
    }
    if (ok && elect_one()) umma_commit(&bars->accum);
  } else {
    // -------------------------------- epilogue -------------------------------
    pdl_wait();  // the epilogue reads scales / the residual and overwrites buffers earlier kernels used
    if (warp * 32 < p.rows) {
      const bool ok = mbar_wait(&bars->accum, 0, p.status);
      tc_fence_after();
      const int r = warp * 32 + lane, n = row0 + r;
      const bool valid = r < p.rows && n < p.N;
      const uint32_t tl = tmem + ((uint32_t)(warp * 32) << 16);
      for (int c0 = 0; c0 < p.Mpad && ok; c0 += 16) {
        float v[16], u[16];
        tmem_ld16(tl + c0, v);
        if (NW == 2) tmem_ld16(tl + nb_rows + c0, u);
        if (p.n_b == 2) {  // high-part and low-part products
          float w2[16];
          tmem_ld16(tl + p.Mpad + c0, w2);
#pragma unroll
          for (int i = 0; i < 16; ++i) v[i] += w2[i];
        }
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const int m = c0 + i;
          if (m < p.M) {  // warp-uniform
            const size_t o = (size_t)m * p.N + n;
            if (EPI == EPI_SWIGLU) {
              const float sc = p.row_scale ? p.row_scale[m] : 1.0f;
              const float gg = v[i] * sc, uu = u[i] * sc;
              const float tv = (gg / (1.0f + expf(-gg))) * uu;
              if (valid) {
                p.out0[o] = gg;
                p.out1[o] = uu;
                p.out2[o] = tv;
              }
              if (p.sel != nullptr) {
                // what the channel selection needs from all of a token's channels: a histogram of |t|
                // and the largest |g|, |u| (non-negative floats order like their bit patterns)
                uint32_t* sel = p.sel + (size_t)m * CH_SEL_WORDS;
                if (valid) atomicAdd(sel + chan_bin(fabsf(tv)), 1u);
                const uint32_t gm = __reduce_max_sync(0xffffffffu, valid ? __float_as_uint(fabsf(gg)) : 0u);
                const uint32_t um = __reduce_max_sync(0xffffffffu, valid ? __float_as_uint(fabsf(uu)) : 0u);
                if (lane == 0) {
                  atomicMax(sel + CH_GMAX, gm);
                  atomicMax(sel + CH_UMAX, um);
                }
              }
            } else if (valid) {
              p.out0[(size_t)blockIdx.y * p.M * p.N + o] = v[i];
            }
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 5) tmem_dealloc(tmem, p.tmem_cols);
}

// ============================================================================
// umma_down
// ============================================================================
struct DownDev {
  int M, Mpad, ff, d;
  int chunks, stages;
  uint32_t tmem_cols;
  const int32_t* live;  // [ff/32]
  float* partial;       // [chunks][Mpad][d]
  int* status;
};

__device__ __forceinline__ bool block_live(const int32_t* live, int jb, int granules) {
  return live[2 * jb] != 0 || (2 * jb + 1 < granules && live[2 * jb + 1] != 0);
}

__global__ void __launch_bounds__(UM_THREADS, 1)
umma_down_kernel(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_t, const DownDev p) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* stages = align_1024(smem_raw);
  const int t_tile = p.Mpad * 128;
  const int stage_bytes = UM_TILE_SPAN + 2 * t_tile;
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
  if (warp == 5) tmem_alloc(&bars->tmem_base, p.tmem_cols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  pdl_wait();  // which channel blocks are live is decided by the selection kernel
  const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(&bars->tmem_base);

  const int slab = blockIdx.x, chunk = blockIdx.y;
  const int granules = p.ff / 32, jblocks = (p.ff + 63) / 64;
  const int jb0 = (int)(((long long)jblocks * chunk) / p.chunks);
  const int jb1 = (int)(((long long)jblocks * (chunk + 1)) / p.chunks);

  if (warp == 4) {
    if (lane == 0) {
      tma_prefetch_map(&tm_w);
      int it = 0;
      for (int jb = jb0; jb < jb1; ++jb) {
        if (!block_live(p.live, jb, granules)) continue;
        const int s = it % p.stages;
        const uint32_t ph = (it / p.stages) & 1;
        ++it;
        if (!mbar_wait(&bars->empty[s], ph ^ 1, p.status)) break;
        unsigned char* st = stages + (size_t)s * stage_bytes;
        mbar_expect_tx(&bars->full[s], stage_bytes);
        tma_load_3d(st, &tm_w, 0, jb * 64, slab * 2, &bars->full[s]);
        tma_load_2d(st + UM_TILE_SPAN, &tm_t, jb * 64, 0, &bars->full[s]);  // high rows then low rows
      }
    }
  } else if (warp == 5) {
    const uint32_t idesc = umma_idesc_bf16_m128(2 * p.Mpad, 1, 0);
    bool acc = false, ok = true;
    int it = 0;
    for (int jb = jb0; jb < jb1; ++jb) {
      if (!block_live(p.live, jb, granules)) continue;
      const int s = it % p.stages;
      const uint32_t ph = (it / p.stages) & 1;
      ++it;
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
    const int n = slab * 128 + warp * 32 + lane;
    const uint32_t tl = tmem + ((uint32_t)(warp * 32) << 16);
    float* out = p.partial + (size_t)chunk * p.Mpad * p.d;
    for (int c0 = 0; c0 < p.Mpad && ok; c0 += 16) {
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
  if (warp == 5) tmem_dealloc(tmem, p.tmem_cols);
}

// ============================================================================
// tensor maps (host)
// ============================================================================
namespace {

struct MapKey {
  uintptr_t ptr;
  uint64_t dim[3];
  uint64_t stride[2];
  uint32_t box[3];
  uint32_t rank;
  bool operator==(const MapKey& o) const {
    return ptr == o.ptr && rank == o.rank && dim[0] == o.dim[0] && dim[1] == o.dim[1] && dim[2] == o.dim[2] &&
           stride[0] == o.stride[0] && stride[1] == o.stride[1] && box[0] == o.box[0] && box[1] == o.box[1] &&
           box[2] == o.box[2];
  }
};
struct MapKeyHash {
  size_t operator()(const MapKey& k) const {
    uint64_t h = k.ptr * 0x9e3779b97f4a7c15ull;
    auto mix = [&](uint64_t v) { h = (h ^ v) * 0x100000001b3ull + (h >> 29); };
    mix(k.dim[0]); mix(k.dim[1]); mix(k.dim[2]); mix(k.stride[0]); mix(k.stride[1]);
    mix(k.box[0]); mix(k.box[1]); mix(k.box[2]); mix(k.rank);
    return (size_t)h;
  }
};

PFN_cuTensorMapEncodeTiled encode_fn() {
  static PFN_cuTensorMapEncodeTiled fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      p = nullptr;
    return reinterpret_cast<PFN_cuTensorMapEncodeTiled>(p);
  }();
  return fn;
}

// bf16 tensor map with 128-byte swizzle; encoded maps are remembered (the encoding is a pure function
// of the key, and the same weight matrices come back every step).
bool tensor_map(CUtensorMap* out, const void* ptr, uint32_t rank, const uint64_t* dim, const uint64_t* stride,
                const uint32_t* box) {
  static std::mutex mu;
  static std::unordered_map<MapKey, CUtensorMap, MapKeyHash> cache;
  MapKey k;
  memset(&k, 0, sizeof(k));
  k.ptr = reinterpret_cast<uintptr_t>(ptr);
  k.rank = rank;
  for (uint32_t i = 0; i < rank; ++i) {
    k.dim[i] = dim[i];
    k.box[i] = box[i];
    if (i + 1 < rank) k.stride[i] = stride[i];
  }
  std::lock_guard<std::mutex> lock(mu);
  auto it = cache.find(k);
  if (it != cache.end()) {
    *out = it->second;
    return true;
  }
  PFN_cuTensorMapEncodeTiled fn = encode_fn();
  if (!fn) {
    record_cuda_error(cudaErrorNotSupported, "cuTensorMapEncodeTiled entry point");
    return false;
  }
  const cuuint32_t ones[3] = {1, 1, 1};
  CUtensorMap m;
  const CUresult r = fn(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, rank, const_cast<void*>(ptr), dim, stride, box, ones,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    record_cuda_error(cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
    return false;
  }
  if (cache.size() > (1u << 16)) cache.clear();
  cache.emplace(k, m);
  *out = m;
  return true;
}

// [rows][K] row-major bf16 viewed as (64 k, rows, K/64 chunks): a box of (64, box_rows, cps) lands in
// shared memory as cps consecutive [box_rows][64] tiles, each in the 128-byte-swizzled K-major layout.
bool kmajor_map(CUtensorMap* out, const void* ptr, int rows, int K, int box_rows, int cps) {
  const uint64_t dim[3] = {64, (uint64_t)rows, (uint64_t)(K / 64)};
  const uint64_t stride[2] = {(uint64_t)K * 2, 128};
  const uint32_t box[3] = {64, (uint32_t)box_rows, (uint32_t)cps};
  return tensor_map(out, ptr, 3, dim, stride, box);
}

uint32_t pow2_cols(int n) {
  uint32_t c = 32;
  while ((int)c < n) c <<= 1;
  return c;
}

int round_mpad(int M) {
  const int mt = (M + 15) / 16;
  return 16 * (mt <= 1 ? 1 : (mt <= 2 ? 2 : (mt <= 4 ? 4 : 8)));
}

}  // namespace

// ============================================================================
// launchers
// ============================================================================
// Split-K geometry of the EPI_PARTIAL projections: full 128-row weight tiles (so that one TMA box and
// one MMA cover as many weight bytes as possible) and as many K slices as it takes to give every SM a CTA.
static void nk_partial_geometry(int N, int K, int* rows, int* tiles, int* ksplit) {
  int r = (N + 7) / 8 * 8;
  if (r > 128) r = 128;
  const int t = (N + r - 1) / r;
  const int chunks = K / 64;
  int z = sm_count() / t;
  if (z > chunks) z = chunks;
  if (z > NK_MAX_KSPLIT) z = NK_MAX_KSPLIT;
  if (z < 1) z = 1;
  *rows = r;
  *tiles = t;
  *ksplit = z;
}

int nk_ksplit(int N, int K) {
  int rows, tiles, z;
  nk_partial_geometry(N, K, &rows, &tiles, &z);
  return z;
}

void launch_gemm_nk(const GemmNK& g, GemmEpilogue epi, cudaStream_t st) {
  const int nw = epi == EPI_SWIGLU ? 2 : 1;
  NKDev d;
  memset(&d, 0, sizeof(d));
  d.M = g.M; d.Mpad = round_mpad(g.M); d.K = g.K; d.N = g.N;
  d.n_b = g.a_lo ? 2 : 1;
  if (g.a_lo && static_cast<const char*>(g.a_lo) != static_cast<const char*>(g.a_hi) + (size_t)d.Mpad * g.K * 2) {
    record_cuda_error(cudaErrorInvalidValue, "split activation operand must be contiguous (high rows, then low rows)");
    return;
  }
  const int chunks = g.K / 64;
  int rows, tiles, ksplit = 1;
  if (epi == EPI_PARTIAL) {
    nk_partial_geometry(g.N, g.K, &rows, &tiles, &ksplit);
  } else {
    // whole K per CTA, one wave of CTAs: `rows` channels (a gate and an up row each) per CTA
    const int sms = sm_count();
    rows = ((g.N + sms - 1) / sms + 7) / 8 * 8;
    if (rows > 128) rows = 128;
    tiles = (g.N + rows - 1) / rows;
  }
  d.rows = rows;
  d.ksplit = ksplit;
  const int chunk_bytes = 128 * (nw * rows + d.n_b * d.Mpad);
  int cps = ksplit > 1 ? 1 : 4;
  while (cps > 1 && (cps * chunk_bytes > 36 * 1024 || chunks % cps)) cps >>= 1;
  d.cps = cps;
  const int stage_bytes = cps * chunk_bytes;
  const int iters = (chunks / ksplit + (chunks % ksplit ? 1 : 0)) / cps;  // of the longest slice
  int stages = UM_SMEM_BUDGET / stage_bytes;
  if (stages > UM_MAX_STAGES) stages = UM_MAX_STAGES;
  if (stages > iters) stages = iters;
  if (stages < 1) stages = 1;
  d.stages = stages;
  d.tmem_cols = pow2_cols(nw * d.n_b * d.Mpad);
  d.row_scale = g.row_scale;
  d.out0 = g.out0; d.out1 = g.out1; d.out2 = g.out2; d.sel = g.sel; d.status = g.status;

  CUtensorMap w0, w1, x0;
  bool ok = kmajor_map(&w0, g.w0, g.N, g.K, rows, cps);
  ok = ok && kmajor_map(&w1, nw == 2 ? g.w1 : g.w0, g.N, g.K, rows, cps);
  ok = ok && kmajor_map(&x0, g.a_hi, d.n_b * d.Mpad, g.K, d.n_b * d.Mpad, cps);
  if (!ok) return;
  const int smem = 1024 + stages * stage_bytes + UM_TILE_SPAN + (int)sizeof(UmBarriers);
  const dim3 grid(tiles, ksplit);
  if (epi == EPI_SWIGLU) {
    ensure_dynamic_smem(reinterpret_cast<const void*>(&umma_nk_kernel<EPI_SWIGLU>), smem);
    SOL_LAUNCH("gemm_gate_up_swiglu", umma_nk_kernel<EPI_SWIGLU>, grid, dim3(UM_THREADS), smem, st, w0, w1, x0, d);
  } else {
    ensure_dynamic_smem(reinterpret_cast<const void*>(&umma_nk_kernel<EPI_PARTIAL>), smem);
    SOL_LAUNCH(g.name ? g.name : "gemm_partial", umma_nk_kernel<EPI_PARTIAL>, grid, dim3(UM_THREADS), smem, st, w0, w1, x0, d);
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
  DownDev d;
  memset(&d, 0, sizeof(d));
  d.M = g.M; d.Mpad = round_mpad(g.M); d.ff = g.ff; d.d = g.d;
  d.chunks = g.chunks;
  const int stage_bytes = UM_TILE_SPAN + 2 * d.Mpad * 128;
  int stages = UM_SMEM_BUDGET / stage_bytes;
  if (stages > UM_MAX_STAGES) stages = UM_MAX_STAGES;
  d.stages = stages;
  d.tmem_cols = pow2_cols(2 * d.Mpad);
  d.live = g.live; d.partial = g.partial; d.status = g.status;

  if (static_cast<const char*>(g.t_lo) != static_cast<const char*>(g.t_hi) + (size_t)d.Mpad * g.ff * 2) {
    record_cuda_error(cudaErrorInvalidValue, "split activation operand must be contiguous (high rows, then low rows)");
    return;
  }
  CUtensorMap w, tm;
  // W[ff][d] viewed as (64 columns, ff channels, d/64 column blocks): a box of (64, 64, 2) lands as two
  // [64 channels][64 columns] blocks, the MN-major operand layout for 128 output columns
  const uint64_t wdim[3] = {64, (uint64_t)g.ff, (uint64_t)(g.d / 64)};
  const uint64_t wstride[2] = {(uint64_t)g.d * 2, 128};
  const uint32_t wbox[3] = {64, 64, 2};
  bool ok = tensor_map(&w, g.w, 3, wdim, wstride, wbox);
  // activations [2 Mpad][ff] (high rows, then low rows): (ff, 2 Mpad) with a box of (64 channels, all rows); channels past ff read as zero
  const uint64_t tdim[2] = {(uint64_t)g.ff, (uint64_t)(2 * d.Mpad)};
  const uint64_t tstride[1] = {(uint64_t)g.ff * 2};
  const uint32_t tbox[2] = {64, (uint32_t)(2 * d.Mpad)};
  ok = ok && tensor_map(&tm, g.t_hi, 2, tdim, tstride, tbox);
  if (!ok) return;
  const int smem = 1024 + stages * stage_bytes + (int)sizeof(UmBarriers);
  ensure_dynamic_smem(reinterpret_cast<const void*>(&umma_down_kernel), smem);
  SOL_LAUNCH("gemm_down_gathered", umma_down_kernel, dim3(g.d / 128, g.chunks), dim3(UM_THREADS), smem, st, w, tm, d);
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
