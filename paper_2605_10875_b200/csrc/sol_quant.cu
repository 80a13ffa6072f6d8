// RMSNorm + per-token symmetric activation quantizer.  One token per CTA; the
// token's row is a few KB, so the kernel is latency-bound: 128-bit loads, the
// row held in registers, two block reductions (sum of squares, absmax).
//
// Quantizer (appendix "Activation quantization", "Quantizer"):
//   q_max = 2^(b-1) - 1, a = max|x|, s = a / q_max, code = clip(rne(x / s)).
// Both divisions are IEEE float32 (__fdiv_rn) so the codes are reproducible
// bit for bit.
#include <type_traits>

#include "sol_common.cuh"
#include "sol_internal.h"
#include "sol_select.cuh"

namespace sol {

constexpr int NQ_THREADS = 256;
constexpr int NQ_VEC = 8;                       // elements per 128-bit bf16 load
constexpr int NQ_MAX_PER_THREAD = 4;            // vectors per thread -> d <= 8192

__device__ __forceinline__ float block_reduce(float v, bool is_max, float* sh) {
  v = is_max ? warp_max(v) : warp_sum(v);
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  __syncthreads();  // protect sh from the previous use
  if (l == 0) sh[w] = v;
  __syncthreads();
  float r = sh[0];
  for (int i = 1; i < NQ_THREADS / 32; ++i) r = is_max ? fmaxf(r, sh[i]) : r + sh[i];
  return r;
}

// What the input-channel gating of the MLP block needs beside the row (GATE variant only).
struct GateArgs {
  const int32_t* p_permille;  // [B] prune rate: ceil((1 - p) d) channels of largest |x| survive
  float* xm;                  // optional tap: [B][d] the masked normalised row
};
struct NoSmem {
  int unused;
};

template <bool IN_F32, bool GATE>
__global__ void __launch_bounds__(NQ_THREADS)
norm_quant_kernel(const void* __restrict__ in, const float* __restrict__ part, int ksplit, size_t part_stride,
                  float* __restrict__ sum_out, const uint16_t* __restrict__ gamma, float eps,
                  const int32_t* __restrict__ bits, int d, uint16_t* __restrict__ a_op, int a_op_rows,
                  float* __restrict__ scale,
                  float* __restrict__ xn, int8_t* __restrict__ codes, int16_t* __restrict__ codes16, int* __restrict__ status,
                  uint32_t* __restrict__ clear, int clear_words, int32_t* __restrict__ zero_flags, int n_zero_flags,
                  const GateArgs gate) {
  __shared__ float sh[NQ_THREADS / 32];
  __shared__ typename std::conditional<GATE, SelectSmem, NoSmem>::type gsm;
  pdl_trigger();
  pdl_wait();
  const int row = blockIdx.x;
  if (zero_flags != nullptr)
    for (int i = blockIdx.x * NQ_THREADS + threadIdx.x; i < n_zero_flags; i += gridDim.x * NQ_THREADS) zero_flags[i] = 0;
  if (clear != nullptr)  // this token's scratch of the kernels that follow
    for (int i = threadIdx.x; i < clear_words; i += NQ_THREADS) clear[(size_t)row * clear_words + i] = 0u;
  const int nvec = d / NQ_VEC;
  float x[NQ_MAX_PER_THREAD][NQ_VEC];

  // load the row (zero-fill vectors beyond d)
  float ss = 0.f;
#pragma unroll
  for (int i = 0; i < NQ_MAX_PER_THREAD; ++i) {
    const int v = threadIdx.x + i * NQ_THREADS;
#pragma unroll
    for (int e = 0; e < NQ_VEC; ++e) x[i][e] = 0.f;
    if (v < nvec) {
      if (IN_F32) {
        const float4* p = reinterpret_cast<const float4*>(static_cast<const float*>(in) + (size_t)row * d) + 2 * v;
        float4 a = p[0], b = p[1];
        x[i][0] = a.x; x[i][1] = a.y; x[i][2] = a.z; x[i][3] = a.w;
        x[i][4] = b.x; x[i][5] = b.y; x[i][6] = b.z; x[i][7] = b.w;
      } else {
        uint4 w = reinterpret_cast<const uint4*>(static_cast<const uint16_t*>(in) + (size_t)row * d)[v];
        x[i][0] = bf16_lo(w.x); x[i][1] = bf16_hi(w.x); x[i][2] = bf16_lo(w.y); x[i][3] = bf16_hi(w.y);
        x[i][4] = bf16_lo(w.z); x[i][5] = bf16_hi(w.z); x[i][6] = bf16_lo(w.w); x[i][7] = bf16_hi(w.w);
      }
      if (part != nullptr) {  // partial sums of the projection that produced this row, in slice order
        for (int z0 = 0; z0 < ksplit; z0 += 4) {  // four slices' loads in flight, added in slice order
          float4 a[4], b[4];
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            a[q] = b[q] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (z0 + q < ksplit) {
              const float4* src =
                  reinterpret_cast<const float4*>(part + (size_t)(z0 + q) * part_stride + (size_t)row * d) + 2 * v;
              a[q] = src[0];
              b[q] = src[1];
            }
          }
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            x[i][0] += a[q].x; x[i][1] += a[q].y; x[i][2] += a[q].z; x[i][3] += a[q].w;
            x[i][4] += b[q].x; x[i][5] += b[q].y; x[i][6] += b[q].z; x[i][7] += b[q].w;
          }
        }
      }
      if (sum_out != nullptr) {
        float4* o = reinterpret_cast<float4*>(sum_out + (size_t)row * d) + 2 * v;
        o[0] = make_float4(x[i][0], x[i][1], x[i][2], x[i][3]);
        o[1] = make_float4(x[i][4], x[i][5], x[i][6], x[i][7]);
      }
#pragma unroll
      for (int e = 0; e < NQ_VEC; ++e) ss += x[i][e] * x[i][e];
    }
  }

  if (gamma != nullptr) {
    const float tot = block_reduce(ss, false, sh);
    const float inv = 1.0f / sqrtf(tot / (float)d + eps);
#pragma unroll
    for (int i = 0; i < NQ_MAX_PER_THREAD; ++i) {
      const int v = threadIdx.x + i * NQ_THREADS;
      if (v < nvec) {
        uint4 w = reinterpret_cast<const uint4*>(gamma)[v];
        float gm[NQ_VEC] = {bf16_lo(w.x), bf16_hi(w.x), bf16_lo(w.y), bf16_hi(w.y),
                            bf16_lo(w.z), bf16_hi(w.z), bf16_lo(w.w), bf16_hi(w.w)};
#pragma unroll
        for (int e = 0; e < NQ_VEC; ++e) x[i][e] = (x[i][e] * gm[e]) * inv;
      }
    }
  }

  if (xn != nullptr) {
#pragma unroll
    for (int i = 0; i < NQ_MAX_PER_THREAD; ++i) {
      const int v = threadIdx.x + i * NQ_THREADS;
      if (v < nvec) {
        float4* p = reinterpret_cast<float4*>(xn + (size_t)row * d) + 2 * v;
        p[0] = make_float4(x[i][0], x[i][1], x[i][2], x[i][3]);
        p[1] = make_float4(x[i][4], x[i][5], x[i][6], x[i][7]);
      }
    }
  }

  if constexpr (GATE) {
    // The paper's structured MLP pruning (appendix "Structured MLP activation pruning"): keep the
    // m = ceil((1 - p) d) channels of largest |x|, ties to the lower index, zero the rest.  |x| orders like its
    // bit pattern; element j = 8 v + e of the row is slot i * 8 + e of thread v - 256 i.
    const int m = (int)(((long long)(1000 - gate.p_permille[row]) * d + 999) / 1000);
    if (m < d) {
      auto key = [&](int q) -> uint32_t {
        const int v = threadIdx.x + (q >> 3) * NQ_THREADS;
        return v < nvec ? __float_as_uint(fabsf(x[q >> 3][q & 7])) : 0u;
      };
      int tie_need = 0;
      uint32_t thr = 0xffffffffu;
      if (m > 0) thr = select_kth<NQ_THREADS, NQ_MAX_PER_THREAD * NQ_VEC>(key, m, tie_need, gsm, NQ_MAX_PER_THREAD * NQ_VEC);
      // ties at the threshold are kept in index order until tie_need runs out: index order is (i, thread, e)
      int taken = 0;  // ties granted to earlier rounds (block-uniform)
#pragma unroll
      for (int i = 0; i < NQ_MAX_PER_THREAD; ++i) {
        const int v = threadIdx.x + i * NQ_THREADS;
        uint32_t tie_mask = 0;
#pragma unroll
        for (int e = 0; e < NQ_VEC; ++e)
          if (m > 0 && v < nvec && __float_as_uint(fabsf(x[i][e])) == thr) tie_mask |= 1u << e;
        // exclusive prefix of the tie counts over the threads of this round
        const int mine = __popc(tie_mask);
        int incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int y = __shfl_up_sync(0xffffffffu, incl, o);
          if ((threadIdx.x & 31) >= o) incl += y;
        }
        __syncthreads();
        if ((threadIdx.x & 31) == 31) gsm.scan[0][threadIdx.x >> 5] = incl;
        __syncthreads();
        int before = taken + incl - mine, total = 0;
        for (int wq = 0; wq < NQ_THREADS / 32; ++wq) {
          const int y = gsm.scan[0][wq];
          if (wq < (int)(threadIdx.x >> 5)) before += y;
          total += y;
        }
        taken += total;
#pragma unroll
        for (int e = 0; e < NQ_VEC; ++e) {
          const uint32_t kk = __float_as_uint(fabsf(x[i][e]));
          bool keep = m > 0 && kk > thr;
          if ((tie_mask >> e) & 1u) {
            keep = before < tie_need;
            ++before;
          }
          if (!keep) x[i][e] = 0.f;
        }
      }
    }
    if (gate.xm != nullptr) {
#pragma unroll
      for (int i = 0; i < NQ_MAX_PER_THREAD; ++i) {
        const int v = threadIdx.x + i * NQ_THREADS;
        if (v < nvec) {
          float4* p = reinterpret_cast<float4*>(gate.xm + (size_t)row * d) + 2 * v;
          p[0] = make_float4(x[i][0], x[i][1], x[i][2], x[i][3]);
          p[1] = make_float4(x[i][4], x[i][5], x[i][6], x[i][7]);
        }
      }
    }
  }

  int b = bits ? bits[row] : 16;
  // widths of 9..15 bits need int16 codes, and their codes are no exact bf16 numbers: they are served only where
  // no tensor-core operand is produced (the stand-alone wide quantizer call)
  const int b_max = (codes16 != nullptr && a_op == nullptr) ? 15 : 8;
  if (b != 16 && (b < 2 || b > b_max)) {  // no kernel for this width: pass through and flag it
    if (threadIdx.x == 0 && status != nullptr) atomicOr(status + ST_ERR, ERR_BAD_ACTION);
    b = 16;
  }
  float s = 1.0f;
  float q_max = 0.f;
  if (b != 16) {
    float a = 0.f;
#pragma unroll
    for (int i = 0; i < NQ_MAX_PER_THREAD; ++i)
#pragma unroll
      for (int e = 0; e < NQ_VEC; ++e) a = fmaxf(a, fabsf(x[i][e]));
    a = block_reduce(a, true, sh);
    q_max = (float)((1 << (b - 1)) - 1);
    s = __fdiv_rn(a, q_max);
  }
  if (threadIdx.x == 0 && scale != nullptr) scale[row] = s;

#pragma unroll
  for (int i = 0; i < NQ_MAX_PER_THREAD; ++i) {
    const int v = threadIdx.x + i * NQ_THREADS;
    if (v >= nvec) continue;
    float c[NQ_VEC];
    if (b == 16) {
#pragma unroll
      for (int e = 0; e < NQ_VEC; ++e) c[e] = x[i][e];
    } else {
#pragma unroll
      for (int e = 0; e < NQ_VEC; ++e) {
        float r = (s == 0.f) ? 0.f : rintf(__fdiv_rn(x[i][e], s));
        c[e] = fminf(fmaxf(r, -q_max), q_max) + 0.0f;  // +0.0f turns a rounded -0 into +0
      }
    }
    if (a_op != nullptr) {
      uint4 w;
      w.x = pack_bf16(c[0], c[1]); w.y = pack_bf16(c[2], c[3]);
      w.z = pack_bf16(c[4], c[5]); w.w = pack_bf16(c[6], c[7]);
      // vector v is the 16-byte piece of elements 8 v .. 8 v + 7: its place in the packed operand layout, or in the plain row
      if (a_op_rows > 0) *reinterpret_cast<uint4*>(reinterpret_cast<unsigned char*>(a_op) + act_piece_offset(a_op_rows, row, v)) = w;
      else reinterpret_cast<uint4*>(a_op + (size_t)row * d)[v] = w;
    }
    if (codes16 != nullptr) {
      int q[NQ_VEC];
#pragma unroll
      for (int e = 0; e < NQ_VEC; ++e) q[e] = (b == 16) ? 0 : (int)c[e];
      uint4 w;
      w.x = (q[0] & 0xffff) | ((uint32_t)(q[1] & 0xffff) << 16);
      w.y = (q[2] & 0xffff) | ((uint32_t)(q[3] & 0xffff) << 16);
      w.z = (q[4] & 0xffff) | ((uint32_t)(q[5] & 0xffff) << 16);
      w.w = (q[6] & 0xffff) | ((uint32_t)(q[7] & 0xffff) << 16);
      reinterpret_cast<uint4*>(codes16 + (size_t)row * d)[v] = w;
    }
    if (codes != nullptr) {
      int q[NQ_VEC];
#pragma unroll
      for (int e = 0; e < NQ_VEC; ++e) q[e] = (b == 16) ? 0 : (int)c[e];
      uint2 w;
      w.x = (q[0] & 0xff) | ((q[1] & 0xff) << 8) | ((q[2] & 0xff) << 16) | ((uint32_t)(q[3] & 0xff) << 24);
      w.y = (q[4] & 0xff) | ((q[5] & 0xff) << 8) | ((q[6] & 0xff) << 16) | ((uint32_t)(q[7] & 0xff) << 24);
      reinterpret_cast<uint2*>(codes + (size_t)row * d)[v] = w;
    }
  }
}

void launch_norm_quant(const NormQuantArgs& a, cudaStream_t st) {
  const size_t stride = a.part_stride ? a.part_stride : (size_t)a.B * a.d;
  GateArgs g;
  g.p_permille = a.gate_p_permille;
  g.xm = a.xm;
#define SOL_NQ_LAUNCH(F32, GATE)                                                                                       \
  SOL_LAUNCH("norm_quant", (norm_quant_kernel<F32, GATE>), dim3(a.B), dim3(NQ_THREADS), 0, st, a.in, a.part, a.ksplit,  \
             stride, a.sum_out, static_cast<const uint16_t*>(a.gamma_bf16), a.eps, a.bits, a.d,                        \
             static_cast<uint16_t*>(a.a_op), a.a_op_rows, a.scale, a.xn, a.codes, a.codes16, a.status, a.clear,         \
             a.clear_words, a.zero_flags, a.n_zero_flags, g)
  if (a.gate_p_permille != nullptr) {
    if (a.in_f32) SOL_NQ_LAUNCH(true, true);
    else SOL_NQ_LAUNCH(false, true);
  } else {
    if (a.in_f32) SOL_NQ_LAUNCH(true, false);
    else SOL_NQ_LAUNCH(false, false);
  }
#undef SOL_NQ_LAUNCH
}

// ============================================================================
// fake-quantization of the MLP output (the paper's placement of the quantizer)
// ============================================================================
// One token per CTA: z = sum of the down projection's partial sums; per-token symmetric quantizer at
// bits[row] on z (appendix "Activation quantization": a = max|z|, s = a / q_max, code = clip(rne(z / s))),
// z_hat = code * s, from 16 bits on z_hat = z; out = resid + z_hat.
__global__ void __launch_bounds__(NQ_THREADS)
quant_out_kernel(const float* __restrict__ partial, int chunks, size_t chunk_stride, int d, const void* __restrict__ resid,
                 int resid_f32, const int32_t* __restrict__ bits, uint16_t* __restrict__ out_bf16, float* __restrict__ out_f32,
                 float* __restrict__ out_f32_b, float* __restrict__ z_tap, int16_t* __restrict__ z_codes,
                 float* __restrict__ z_scale, int32_t* __restrict__ live, int n_live, int* __restrict__ status) {
  __shared__ float sh[NQ_THREADS / 32];
  pdl_trigger();
  pdl_wait();
  const int row = blockIdx.x;
  // the down projection has read the "granule is live" flags; the next selection starts from zero
  for (int i = blockIdx.x * NQ_THREADS + threadIdx.x; i < n_live; i += gridDim.x * NQ_THREADS) live[i] = 0;
  const int nvec = d / 4;
  constexpr int VPT = 8;  // float4 vectors per thread: d <= 8192
  float4 z[VPT];
  float a = 0.f;
#pragma unroll
  for (int i = 0; i < VPT; ++i) {
    const int v = threadIdx.x + i * NQ_THREADS;
    z[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (v < nvec) {
      for (int c0 = 0; c0 < chunks; c0 += 4) {  // four partials' loads in flight, added in order
        float4 t[4];
#pragma unroll
        for (int q = 0; q < 4; ++q)
          t[q] = c0 + q < chunks ? reinterpret_cast<const float4*>(partial + (size_t)(c0 + q) * chunk_stride + (size_t)row * d)[v]
                                 : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          z[i].x += t[q].x; z[i].y += t[q].y; z[i].z += t[q].z; z[i].w += t[q].w;
        }
      }
      if (z_tap) reinterpret_cast<float4*>(z_tap + (size_t)row * d)[v] = z[i];
      a = fmaxf(a, fmaxf(fmaxf(fabsf(z[i].x), fabsf(z[i].y)), fmaxf(fabsf(z[i].z), fabsf(z[i].w))));
    }
  }
  int b = bits[row];
  if (b < 2) {
    if (threadIdx.x == 0 && status != nullptr) atomicOr(status + ST_ERR, ERR_BAD_ACTION);
    b = 16;
  }
  float s = 1.0f, q_max = 0.f;
  if (b < 16) {
    a = block_reduce(a, true, sh);
    q_max = (float)((1 << (b - 1)) - 1);
    s = __fdiv_rn(a, q_max);
  }
  if (threadIdx.x == 0 && z_scale) z_scale[row] = s;
#pragma unroll
  for (int i = 0; i < VPT; ++i) {
    const int v = threadIdx.x + i * NQ_THREADS;
    if (v >= nvec) continue;
    float zz[4] = {z[i].x, z[i].y, z[i].z, z[i].w};
    int cc[4] = {0, 0, 0, 0};
    if (b < 16) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float r = (s == 0.f) ? 0.f : rintf(__fdiv_rn(zz[e], s));
        const float c = fminf(fmaxf(r, -q_max), q_max) + 0.0f;
        cc[e] = (int)c;
        zz[e] = __fmul_rn(c, s);
      }
    }
    if (z_codes) {
      uint2 w;
      w.x = (cc[0] & 0xffff) | ((uint32_t)(cc[1] & 0xffff) << 16);
      w.y = (cc[2] & 0xffff) | ((uint32_t)(cc[3] & 0xffff) << 16);
      reinterpret_cast<uint2*>(z_codes + (size_t)row * d)[v] = w;
    }
    float4 acc = make_float4(zz[0], zz[1], zz[2], zz[3]);
    if (resid != nullptr) {
      if (resid_f32) {
        const float4 r = reinterpret_cast<const float4*>(static_cast<const float*>(resid) + (size_t)row * d)[v];
        acc.x += r.x; acc.y += r.y; acc.z += r.z; acc.w += r.w;
      } else {
        const uint2 r = reinterpret_cast<const uint2*>(static_cast<const uint16_t*>(resid) + (size_t)row * d)[v];
        acc.x += bf16_lo(r.x); acc.y += bf16_hi(r.x); acc.z += bf16_lo(r.y); acc.w += bf16_hi(r.y);
      }
    }
    if (out_bf16) {
      uint2 o;
      o.x = pack_bf16(acc.x, acc.y);
      o.y = pack_bf16(acc.z, acc.w);
      reinterpret_cast<uint2*>(out_bf16 + (size_t)row * d)[v] = o;
    }
    if (out_f32) reinterpret_cast<float4*>(out_f32 + (size_t)row * d)[v] = acc;
    if (out_f32_b) reinterpret_cast<float4*>(out_f32_b + (size_t)row * d)[v] = acc;
  }
}

void launch_quant_out(const QuantOutArgs& a, cudaStream_t st) {
  SOL_LAUNCH("mlp_out_quant_residual", quant_out_kernel, dim3(a.M), dim3(NQ_THREADS), 0, st, a.partial, a.chunks,
             (size_t)a.Mpad * a.d, a.d, a.resid, a.resid_f32, a.bits, static_cast<uint16_t*>(a.out_bf16), a.out_f32, a.out_f32_b,
             a.z_tap, a.z_codes, a.z_scale, a.live, a.n_live, a.status);
}

}  // namespace sol
