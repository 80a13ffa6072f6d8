// Shared device helpers for the sm_100a kernels: bf16 packing, mbarrier and
// bulk-copy (TMA 1-D) wrappers with bounded waits, warp MMA wrappers.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace sol {

// ---- device status words (first 256 bytes of every workspace) -------------
enum : int {
  ST_ERR = 0,            // bit mask: 1 = bounded wait gave up, 2 = bad page id skipped, 4 = unsupported bit-width
  ST_TOK_OVERFLOW = 1,   // token selections that fell back to float32 ordering
  ST_CH_OVERFLOW = 2,    // channel selections that fell back
  ST_TOK_REFINED = 3,    // token candidates re-scored in float64
  ST_CH_REFINED = 4,     // channel candidates re-scored in float64
  ST_WORDS = 8
};
constexpr int ERR_TIMEOUT = 1;
constexpr int ERR_BAD_PAGE = 2;
constexpr int ERR_BAD_ACTION = 4;

// ---- bf16 helpers ----------------------------------------------------------
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
__device__ __forceinline__ uint16_t f2bf(float x) { return __bfloat16_as_ushort(__float2bfloat16_rn(x)); }
__device__ __forceinline__ float bf2f(uint16_t u) { return __uint_as_float(((uint32_t)u) << 16); }
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  return (uint32_t)f2bf(lo) | ((uint32_t)f2bf(hi) << 16);
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}

// ---- mbarrier + bulk async copy --------------------------------------------
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_mbar_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: gives up after `limit` polls, raises ERR_TIMEOUT in the status
// words and returns false; the caller then skips its work and leaves.
constexpr uint32_t WAIT_LIMIT = 1u << 20;
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, int* status, uint32_t limit = WAIT_LIMIT) {
  for (uint32_t i = 0; i < limit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
  }
  atomicOr(status + ST_ERR, ERR_TIMEOUT);
  return false;
}
// 1-D bulk copy global -> shared, completion counted in bytes on `bar`.
// Both addresses 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_g2s(void* dst_smem, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(dst_smem)),
               "l"(src), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}

// ---- warp-level tensor-core MMA (bf16 x bf16 -> fp32, m16n8k16) -----------
__device__ __forceinline__ void mma_bf16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}

// ---- histogram of |t| shared by the gate/up epilogue (which fills it) and the channel selection ----
// 4096 bins: 32 octaves from 2^-24 to 2^8 with 128 steps each (the top mantissa bits); smaller values
// share bin 0, larger ones bin 4095.  Bin order is value order.
constexpr int CH_BINS = 4096;
__device__ __forceinline__ int chan_bin(float a) {  // a >= 0
  const int b = (int)(__float_as_uint(a) >> 16) - (103 << 7);
  return min(max(b, 0), CH_BINS - 1);
}
__device__ __forceinline__ float chan_bin_lo(int b) {  // smallest value of bin b (0 for bin 0)
  return b <= 0 ? 0.f : __uint_as_float((uint32_t)(b + (103 << 7)) << 16);
}
// Per-token scratch words of the channel selection, cleared by the RMSNorm kernel before the projection:
// the histogram, then these.
enum : int { CH_GMAX = CH_BINS, CH_UMAX, CH_N_ABOVE, CH_N_CAND, CH_DONE, CH_FALLBACK, CH_SEL_WORDS = CH_BINS + 8 };
constexpr int CH_CAND_CAP = 1024;  // exactly re-scored candidates per token before the single-CTA path takes over

// ---- programmatic dependent launch ---------------------------------------------
// pdl_trigger: the next kernel in the stream may be scheduled from now on (it still waits in
// pdl_wait for this grid to finish).  pdl_wait: returns once every earlier kernel has completed and
// its writes are visible; until then only constants (weights, shapes) may be read.
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// ---- small reductions ---------------------------------------------------------
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ double warp_sum_d(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Order-preserving map float -> uint32 (larger float -> larger key).
__device__ __forceinline__ uint32_t float_key(float f) {
  uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

}  // namespace sol
