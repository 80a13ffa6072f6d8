// Weight-streaming skinny GEMMs.  The batch (16..128 rows) is the small side;
// each weight byte is read from HBM exactly once, so these kernels are bound
// by HBM bandwidth and are built around keeping many bulk copies in flight:
// a producer warp streams weight tiles into a shared-memory ring with
// cp.async.bulk (the 1-D TMA path, completion on mbarriers), eight consumer
// warps feed them to bf16 tensor-core MMAs with fp32 accumulation.
//
//   gemm_nk   : Y[M][N] = A[M][K] . W[N][K]^T   (QKV, output and gate/up projections)
//   gemm_down : Y[M][d] = T[M][ff] . W[ff][d]   (down projection; rows of W whose
//               32-channel granule no token keeps are neither copied nor multiplied)
#include "sol_common.cuh"
#include "sol_internal.h"

namespace sol {

// ============================================================================
// gemm_nk
// ============================================================================
constexpr int NK_CONSUMERS = 8;                 // consumer warps
constexpr int NK_THREADS = (NK_CONSUMERS + 1) * 32;
constexpr int NK_KC = 256;                      // k columns per stage
constexpr int NK_ROWS = 32;                     // weight rows per stage (4 n-tiles)
constexpr int NK_ROW_BYTES = NK_KC * 2;         // 512
constexpr int NK_ROW_STRIDE = NK_ROW_BYTES + 64;  // +64: conflict-free 128-bit fragment loads
constexpr int NK_STAGE_BYTES = NK_ROWS * NK_ROW_STRIDE;  // 18432
constexpr int NK_STAGES = 8;
constexpr int NK_RED_BYTES = NK_CONSUMERS * 4 * 128 * 4;  // 16 KB cross-warp reduction buffer
constexpr int NK_SMEM = NK_STAGES * NK_STAGE_BYTES + NK_RED_BYTES + 2 * NK_STAGES * 8 + 64;

__device__ __forceinline__ void consumer_bar() { asm volatile("bar.sync 1, %0;" ::"n"(NK_CONSUMERS * 32)); }

struct NKDev {
  const uint16_t* a_hi;
  const uint16_t* a_lo;
  const uint16_t* w0;
  const uint16_t* w1;
  int M, K, N, MT;
  const float* row_scale;
  const void* resid;
  int resid_f32;
  float* out0;
  float* out1;
  float* out2;
  int* status;
  int n_tiles;  // virtual n-tiles of 8 rows (EPI_SWIGLU: 2 per 8 channels, gate then up)
};

template <int EPI, int MT>
__global__ void __launch_bounds__(NK_THREADS, 1) gemm_nk_kernel(const NKDev p) {
  extern __shared__ __align__(128) unsigned char smem[];
  unsigned char* stages = smem;
  float* red = reinterpret_cast<float*>(smem + NK_STAGES * NK_STAGE_BYTES);
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + NK_STAGES * NK_STAGE_BYTES + NK_RED_BYTES);
  uint64_t* empty = full + NK_STAGES;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < NK_STAGES; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], NK_CONSUMERS);
    }
    fence_mbar_init();
  }
  __syncthreads();

  // this CTA's range of n-tiles, in units of 2 so gate/up pairs stay together
  const int pairs = p.n_tiles / 2;
  const int pr0 = (int)(((long long)pairs * blockIdx.x) / gridDim.x);
  const int pr1 = (int)(((long long)pairs * (blockIdx.x + 1)) / gridDim.x);
  const int vt0 = 2 * pr0, vt1 = 2 * pr1;
  const int kchunks = p.K / NK_KC;

  // row r of virtual n-tile vt -> weight row pointer
  auto w_row = [&](int vt, int r) -> const uint16_t* {
    if (EPI == EPI_SWIGLU) {
      const uint16_t* base = (vt & 1) ? p.w1 : p.w0;
      return base + (size_t)((vt >> 1) * 8 + r) * p.K;
    }
    return p.w0 + (size_t)(vt * 8 + r) * p.K;
  };

  if (warp == NK_CONSUMERS) {
    // ------------------------------ producer -------------------------------
    bool ok = true;
    uint32_t it = 0;
    for (int vb = vt0; vb < vt1; vb += 4) {
      const int nt = min(4, vt1 - vb);
      for (int kc = 0; kc < kchunks; ++kc, ++it) {
        const int s = it % NK_STAGES;
        const uint32_t ph = (it / NK_STAGES) & 1;
        if (ok) ok = mbar_wait(&empty[s], ph ^ 1, p.status);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) continue;
        if (lane == 0) mbar_expect_tx(&full[s], nt * 8 * NK_ROW_BYTES);
        __syncwarp();
        if (lane < nt * 8) {
          const uint16_t* src = w_row(vb + (lane >> 3), lane & 7) + (size_t)kc * NK_KC;
          bulk_g2s(stages + (size_t)s * NK_STAGE_BYTES + lane * NK_ROW_STRIDE, src, NK_ROW_BYTES, &full[s]);
        }
      }
    }
    return;
  }

  // -------------------------------- consumers --------------------------------
  const int g = lane >> 2, t = lane & 3;
  bool ok = true;
  uint32_t it = 0;
  for (int vb = vt0; vb < vt1; vb += 4) {
    const int nt = min(4, vt1 - vb);
    float acc[MT][4][4];
#pragma unroll
    for (int m = 0; m < MT; ++m)
#pragma unroll
      for (int j = 0; j < 4; ++j)
#pragma unroll
        for (int r = 0; r < 4; ++r) acc[m][j][r] = 0.f;

    for (int kc = 0; kc < kchunks; ++kc, ++it) {
      const int s = it % NK_STAGES;
      const uint32_t ph = (it / NK_STAGES) & 1;
      const size_t kofs = (size_t)kc * NK_KC + warp * 32 + t * 8;
      // activation fragments come from global memory (L1/L2 resident); with a single m-tile they are
      // fetched before the wait so their latency overlaps it
      auto load_a = [&](int m, uint4 (&ah)[2], uint4 (&al)[2]) {
        ah[0] = *reinterpret_cast<const uint4*>(p.a_hi + (size_t)(m * 16 + g) * p.K + kofs);
        ah[1] = *reinterpret_cast<const uint4*>(p.a_hi + (size_t)(m * 16 + g + 8) * p.K + kofs);
        if (p.a_lo != nullptr) {
          al[0] = *reinterpret_cast<const uint4*>(p.a_lo + (size_t)(m * 16 + g) * p.K + kofs);
          al[1] = *reinterpret_cast<const uint4*>(p.a_lo + (size_t)(m * 16 + g + 8) * p.K + kofs);
        }
      };
      uint4 ah[2], al[2];
      if (MT == 1) load_a(0, ah, al);
      if (ok) ok = mbar_wait(&full[s], ph, p.status);
      if (ok) {
        const uint32_t base = smem_u32(stages + (size_t)s * NK_STAGE_BYTES) + g * NK_ROW_STRIDE + (warp * 32 + t * 8) * 2;
        uint4 w[4];
#pragma unroll
        for (int j = 0; j < 4; ++j)
          if (j < nt) w[j] = lds128(base + j * 8 * NK_ROW_STRIDE);
#pragma unroll
        for (int m = 0; m < MT; ++m) {
          if (MT > 1) load_a(m, ah, al);
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            if (j < nt) {
              mma_bf16(acc[m][j], ah[0].x, ah[1].x, ah[0].y, ah[1].y, w[j].x, w[j].y);
              mma_bf16(acc[m][j], ah[0].z, ah[1].z, ah[0].w, ah[1].w, w[j].z, w[j].w);
              if (p.a_lo != nullptr) {
                mma_bf16(acc[m][j], al[0].x, al[1].x, al[0].y, al[1].y, w[j].x, w[j].y);
                mma_bf16(acc[m][j], al[0].z, al[1].z, al[0].w, al[1].w, w[j].z, w[j].w);
              }
            }
          }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty[s]);
    }

    // cross-warp reduction (each warp holds a K sub-slice) and epilogue, one m-tile at a time
#pragma unroll
    for (int m = 0; m < MT; ++m) {
      consumer_bar();  // previous round's readers are done with `red`
#pragma unroll
      for (int j = 0; j < 4; ++j)
        *reinterpret_cast<float4*>(red + ((warp * 4 + j) * 128 + lane * 4)) =
            make_float4(acc[m][j][0], acc[m][j][1], acc[m][j][2], acc[m][j][3]);
      consumer_bar();
      // thread -> (tile pair pr, lane l, register r); tiles 2pr and 2pr+1
      const int pr = threadIdx.x >> 7, idx = threadIdx.x & 127;
      const int l = idx >> 2, r = idx & 3;
      float v0 = 0.f, v1 = 0.f;
#pragma unroll
      for (int w = 0; w < NK_CONSUMERS; ++w) {
        v0 += red[(w * 4 + 2 * pr) * 128 + idx];
        v1 += red[(w * 4 + 2 * pr + 1) * 128 + idx];
      }
      const int row = m * 16 + (l >> 2) + ((r & 2) ? 8 : 0);
      const int col = (l & 3) * 2 + (r & 1);
      if (row < p.M) {
        const float sc = p.row_scale ? p.row_scale[row] : 1.0f;
        v0 *= sc;
        v1 *= sc;
        if (EPI == EPI_SWIGLU) {
          if (2 * pr < nt) {
            const int ch = ((vb >> 1) + pr) * 8 + col;
            const size_t o = (size_t)row * p.N + ch;
            const float gg = v0, uu = v1;
            p.out0[o] = gg;
            p.out1[o] = uu;
            p.out2[o] = (gg / (1.0f + expf(-gg))) * uu;
          }
        } else {
#pragma unroll
          for (int q = 0; q < 2; ++q) {
            const int j = 2 * pr + q;
            if (j < nt) {
              const int n = (vb + j) * 8 + col;
              const size_t o = (size_t)row * p.N + n;
              float v = q ? v1 : v0;
              if (EPI == EPI_RESIDUAL) {
                v += p.resid_f32 ? static_cast<const float*>(p.resid)[o]
                                 : bf2f(static_cast<const uint16_t*>(p.resid)[o]);
              }
              p.out0[o] = v;
            }
          }
        }
      }
    }
  }
}

template <int EPI>
static void launch_nk_mt(const NKDev& d, int grid, cudaStream_t st) {
  const char* name = EPI == EPI_SWIGLU ? "gemm_gate_up_swiglu" : (EPI == EPI_RESIDUAL ? "gemm_out_proj" : "gemm_qkv");
#define SOL_NK_CASE(MTV)                                                                                      \
  case MTV: {                                                                                                 \
    ensure_dynamic_smem(reinterpret_cast<const void*>(&gemm_nk_kernel<EPI, MTV>), NK_SMEM);                   \
    SOL_LAUNCH(name, (gemm_nk_kernel<EPI, MTV>), dim3(grid), dim3(NK_THREADS), NK_SMEM, st, d);               \
  } break;
  switch (d.MT) {
    SOL_NK_CASE(1)
    SOL_NK_CASE(2)
    SOL_NK_CASE(4)
    SOL_NK_CASE(8)
    default: break;
  }
#undef SOL_NK_CASE
}

static int round_mt(int M) {
  int mt = (M + 15) / 16;
  return mt <= 1 ? 1 : (mt <= 2 ? 2 : (mt <= 4 ? 4 : 8));
}

void launch_gemm_nk(const GemmNK& p, GemmEpilogue epi, cudaStream_t st) {
  NKDev d;
  d.a_hi = static_cast<const uint16_t*>(p.a_hi);
  d.a_lo = static_cast<const uint16_t*>(p.a_lo);
  d.w0 = static_cast<const uint16_t*>(p.w0);
  d.w1 = static_cast<const uint16_t*>(p.w1);
  d.M = p.M; d.K = p.K; d.N = p.N; d.MT = round_mt(p.M);
  d.row_scale = p.row_scale; d.resid = p.resid; d.resid_f32 = p.resid_f32;
  d.out0 = p.out0; d.out1 = p.out1; d.out2 = p.out2; d.status = p.status;
  d.n_tiles = (epi == EPI_SWIGLU) ? 2 * (p.N / 8) : p.N / 8;
  const int grid = min(sm_count(), max(1, d.n_tiles / 2));
  if (epi == EPI_SWIGLU) launch_nk_mt<EPI_SWIGLU>(d, grid, st);
  else if (epi == EPI_RESIDUAL) launch_nk_mt<EPI_RESIDUAL>(d, grid, st);
  else launch_nk_mt<EPI_SCALE>(d, grid, st);
}

// ============================================================================
// gemm_down
// ============================================================================
constexpr int DN_CONSUMERS = 8;
constexpr int DN_THREADS = (DN_CONSUMERS + 1) * 32;
constexpr int DN_KG = 32;                        // channels per stage (one granule)
constexpr int DN_NS = 256;                       // output columns per CTA
constexpr int DN_W_STRIDE = DN_NS * 2 + 16;      // 528: conflict-free ldmatrix rows
constexpr int DN_W_BYTES = DN_KG * DN_W_STRIDE;  // 16896
constexpr int DN_A_STRIDE = DN_KG * 2 + 16;      // 80
constexpr int DN_SMEM_BUDGET = 200 * 1024;

struct DownDev {
  const uint16_t* t_hi;
  const uint16_t* t_lo;
  const uint16_t* w;
  const int32_t* live;
  int M, Mpad, ff, d;
  float* partial;
  int chunks, stages, stage_bytes;
  int* status;
};

template <int MT>
__global__ void __launch_bounds__(DN_THREADS, 1) gemm_down_kernel(const DownDev p) {
  extern __shared__ __align__(128) unsigned char smem[];
  const int NST = p.stages;
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + (size_t)NST * p.stage_bytes);
  uint64_t* empty = full + NST;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < NST; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], DN_CONSUMERS);
    }
    fence_mbar_init();
  }
  __syncthreads();

  const int slab = blockIdx.x;   // 256 output columns
  const int chunk = blockIdx.y;  // range of granules
  const int granules = p.ff / DN_KG;
  const int g0 = (int)(((long long)granules * chunk) / p.chunks);
  const int g1 = (int)(((long long)granules * (chunk + 1)) / p.chunks);
  const int a_bytes = MT * 16 * DN_A_STRIDE;

  if (warp == DN_CONSUMERS) {
    bool ok = true;
    uint32_t it = 0;
    for (int gi = g0; gi < g1; ++gi) {
      if (p.live[gi] == 0) continue;
      const int s = it % NST;
      const uint32_t ph = (it / NST) & 1;
      ++it;
      if (ok) ok = mbar_wait(&empty[s], ph ^ 1, p.status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) continue;
      unsigned char* st = smem + (size_t)s * p.stage_bytes;
      if (lane == 0) mbar_expect_tx(&full[s], DN_KG * DN_NS * 2 + 2 * MT * 16 * DN_KG * 2);
      __syncwarp();
      // weight rows: one 512-byte copy per channel
      bulk_g2s(st + lane * DN_W_STRIDE, p.w + (size_t)(gi * DN_KG + lane) * p.d + slab * DN_NS, DN_NS * 2, &full[s]);
      // activation tiles: 64 bytes per batch row, high and low parts
      for (int r = lane; r < MT * 16; r += 32) {
        const size_t src = (size_t)r * p.ff + (size_t)gi * DN_KG;
        bulk_g2s(st + DN_W_BYTES + r * DN_A_STRIDE, p.t_hi + src, DN_KG * 2, &full[s]);
        bulk_g2s(st + DN_W_BYTES + a_bytes + r * DN_A_STRIDE, p.t_lo + src, DN_KG * 2, &full[s]);
      }
    }
    return;
  }

  float acc[MT][4][4];
#pragma unroll
  for (int m = 0; m < MT; ++m)
#pragma unroll
    for (int j = 0; j < 4; ++j)
#pragma unroll
      for (int r = 0; r < 4; ++r) acc[m][j][r] = 0.f;

  bool ok = true;
  uint32_t it = 0;
  const int mi = lane >> 3, mr = lane & 7;  // ldmatrix: this lane addresses row mr of matrix mi
  for (int gi = g0; gi < g1; ++gi) {
    if (p.live[gi] == 0) continue;
    const int s = it % NST;
    const uint32_t ph = (it / NST) & 1;
    ++it;
    if (ok) ok = mbar_wait(&full[s], ph, p.status);
    if (ok) {
      const uint32_t st = smem_u32(smem + (size_t)s * p.stage_bytes);
#pragma unroll
      for (int ks = 0; ks < 2; ++ks) {
        uint32_t bfr[2][4];  // [pair of n-tiles][b0,b1 of tile a, b0,b1 of tile a+1]
#pragma unroll
        for (int pr = 0; pr < 2; ++pr) {
          const int krow = ks * 16 + (mi & 1) * 8 + mr;
          const int ncol = warp * 32 + (2 * pr + (mi >> 1)) * 8;
          ldsm_x4_trans(bfr[pr], st + krow * DN_W_STRIDE + ncol * 2);
        }
#pragma unroll
        for (int m = 0; m < MT; ++m) {
          uint32_t ah[4], al[4];
          const int mrow = m * 16 + (mi & 1) * 8 + mr;
          const int kcol = ks * 16 + (mi >> 1) * 8;
          ldsm_x4(ah, st + DN_W_BYTES + mrow * DN_A_STRIDE + kcol * 2);
          ldsm_x4(al, st + DN_W_BYTES + a_bytes + mrow * DN_A_STRIDE + kcol * 2);
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const uint32_t b0 = bfr[j >> 1][(j & 1) * 2], b1 = bfr[j >> 1][(j & 1) * 2 + 1];
            mma_bf16(acc[m][j], ah[0], ah[1], ah[2], ah[3], b0, b1);
            mma_bf16(acc[m][j], al[0], al[1], al[2], al[3], b0, b1);
          }
        }
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&empty[s]);
  }

  // partial sums of this chunk
  const int g = lane >> 2, t = lane & 3;
  float* out = p.partial + (size_t)chunk * p.Mpad * p.d;
#pragma unroll
  for (int m = 0; m < MT; ++m)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int col = slab * DN_NS + warp * 32 + j * 8 + t * 2;
      const int r0 = m * 16 + g, r1 = r0 + 8;
      if (r0 < p.M) *reinterpret_cast<float2*>(out + (size_t)r0 * p.d + col) = make_float2(acc[m][j][0], acc[m][j][1]);
      if (r1 < p.M) *reinterpret_cast<float2*>(out + (size_t)r1 * p.d + col) = make_float2(acc[m][j][2], acc[m][j][3]);
    }
}

int down_chunks(int ff, int d) {
  const int slabs = d / DN_NS;
  const int granules = ff / DN_KG;
  int c = sm_count() / (slabs > 0 ? slabs : 1);
  if (c < 1) c = 1;
  if (c > granules) c = granules;
  return c;
}

void launch_gemm_down(const GemmDown& p, cudaStream_t st) {
  DownDev d;
  d.t_hi = static_cast<const uint16_t*>(p.t_hi);
  d.t_lo = static_cast<const uint16_t*>(p.t_lo);
  d.w = static_cast<const uint16_t*>(p.w);
  d.live = p.live;
  d.M = p.M; d.ff = p.ff; d.d = p.d;
  const int mt = round_mt(p.M);
  d.Mpad = mt * 16;
  d.partial = p.partial; d.chunks = p.chunks; d.status = p.status;
  d.stage_bytes = DN_W_BYTES + 2 * mt * 16 * DN_A_STRIDE;
  d.stage_bytes = (d.stage_bytes + 127) / 128 * 128;
  d.stages = DN_SMEM_BUDGET / d.stage_bytes;
  if (d.stages > 8) d.stages = 8;
  const int smem = d.stages * d.stage_bytes + 2 * d.stages * 8 + 64;
  dim3 grid(p.d / DN_NS, p.chunks);
#define SOL_DN_CASE(MTV)                                                                                  \
  case MTV: {                                                                                             \
    ensure_dynamic_smem(reinterpret_cast<const void*>(&gemm_down_kernel<MTV>), smem);                     \
    SOL_LAUNCH("gemm_down_gathered", gemm_down_kernel<MTV>, grid, dim3(DN_THREADS), smem, st, d);         \
  } break;
  switch (mt) {
    SOL_DN_CASE(1)
    SOL_DN_CASE(2)
    SOL_DN_CASE(4)
    SOL_DN_CASE(8)
    default: break;
  }
#undef SOL_DN_CASE
}

// ============================================================================
// reduce the down-projection partials, add the residual, emit bf16 / fp32
// ============================================================================
__global__ void reduce_out_kernel(const float* __restrict__ partial, int chunks, int M, int Mpad, int d,
                                  const void* __restrict__ resid, int resid_f32, uint16_t* __restrict__ out_bf16,
                                  float* __restrict__ out_f32, float* __restrict__ out_f32_b) {
  const int i = (blockIdx.x * blockDim.x + threadIdx.x) * 4;
  if (i >= M * d) return;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int c = 0; c < chunks; ++c) {
    const float4 v = *reinterpret_cast<const float4*>(partial + (size_t)c * Mpad * d + i);
    acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
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
                       void* out_bf16, float* out_f32, float* out_f32_b, cudaStream_t st) {
  const int n4 = M * d / 4;
  SOL_LAUNCH("down_reduce_residual", reduce_out_kernel, dim3((n4 + 255) / 256), dim3(256), 0, st, partial, chunks, M,
             Mpad, d, resid, resid_f32, static_cast<uint16_t*>(out_bf16), out_f32, out_f32_b);
}

}  // namespace sol
