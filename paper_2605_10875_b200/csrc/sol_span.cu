// Dense causal attention of a span of consecutive query tokens per sequence: the attention step of the periodic
// KV-cache refresh (Background, paragraph "Episodes and control horizon": a fully dense pass over the last T
// already-known tokens rebuilds their cache entries).
//
// The rows of the batch are n_seq sequences times n_tok tokens; row s * n_tok + i is token i of the span of
// sequence s, its context ends at its own position (length T_s - n_tok + 1 + i).  The decode step's attention
// would read the sequence's keys and values once per row; here the n_tok query tokens of a head are the 16 rows
// of one MMA tile, so a (sequence, kv-head) streams its cache once for all of them:
//
//   span_attn_kernel     grid (split, kv-head, sequence), a warp per query head of the group.  The CTA walks its
//                        share of the sequence's cache pages; a page's keys and values (64 tokens) come by
//                        cp.async into swizzled shared-memory tiles, two stages, one barrier per page.  Per page and warp:
//                        S = Q K^T on mma.sync m16n8k16 with Q as bf16 high + low parts (the oracle does not
//                        round q), causal mask, online softmax in the base-2 domain, O += P V with P as bf16
//                        high + low parts (V through ldmatrix.trans).  Leaves (O, m, l) per row, head and split.
//   span_combine_kernel  merges the splits and writes the row's output in the forms the output projection and
//                        the callers read.
//
// No selection happens: every token up to the row's own is kept (keep-rate 1).
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "sol_common.cuh"
#include "sol_internal.h"

namespace sol {

struct SpanDev {
  sol_kv_t kv;  // page_table, seq_lens: one entry per ROW (the rows of a sequence share the table)
  int Hq, Hkv, G, n_tok, n_seq;
  int nsplit;  // splits of the longest context the table allows: the stride of `part`; a sequence uses the first ceil(pages / pps)
  int pps;     // cache pages per split
  float scale_log2;     // log2(e) / sqrt(head_dim)
  const float* q_rot;   // [rows][Hq][hd]
  float* part;          // [rows][Hq][nsplit][hd + 2]: O, m (base-2 domain), l
  float* out_f32;       // each optional
  uint16_t* out_bf16;
  uint16_t* out_hi;     // packed operand of the output projection (2 out_rows rows: high parts, then low parts)
  int out_rows;
  int* status;
};

__device__ __forceinline__ void span_cp16(uint32_t dst_smem, const void* src, bool valid) {
  const int n = valid ? 16 : 0;  // 0: the 16 bytes are filled with zeros
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst_smem), "l"(src), "r"(n) : "memory");
}
__device__ __forceinline__ void span_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void span_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

constexpr int SPAN_ROWS = 16;      // query tokens per sequence at most (the rows of one MMA tile)
constexpr int SPAN_PAGES = 8;      // cache pages per CTA

template <int HD>
__global__ void __launch_bounds__(256, HD == 64 ? 2 : 1) span_attn_kernel(const SpanDev p) {
  constexpr int PPR = HD / 8;             // 16-byte pieces per row
  constexpr int TILE = PAGE * HD * 2;     // bytes of a page's keys (or values) of one kv-head
  constexpr int QT = SPAN_ROWS * HD * 2;  // bytes of a head's query tile (one part)
  constexpr int ND = HD / 8;              // n-tiles of the output
  extern __shared__ __align__(128) unsigned char ssm[];
  unsigned char* kt = ssm;                 // [2][TILE]
  unsigned char* vt = ssm + 2 * TILE;      // [2][TILE]
  unsigned char* qs = ssm + 4 * TILE;      // [G][2][QT]: high parts, low parts
  const int split = blockIdx.x, kvh = blockIdx.y, s = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nthr = blockDim.x;
  const int g = lane >> 2, t = lane & 3;
  const int n = p.n_tok, head = kvh * p.G + warp, row0 = s * n;
  pdl_trigger();
  pdl_wait();  // the rotated queries and the appended keys and values come from the kernel before
  const int T = min(max(p.kv.seq_lens[row0 + n - 1], 0), p.kv.max_pages_per_seq * PAGE);  // the last row sees it all
  const int NP = (T + PAGE - 1) / PAGE;
  const int pg0 = split * p.pps, pg1 = min(NP, pg0 + p.pps);
  if (pg0 >= pg1) return;  // the sequence ends before this split (the combine step knows how many it has)
  const int32_t* table = p.kv.page_table + (size_t)row0 * p.kv.max_pages_per_seq;

  // a page's keys and values into stage st: piece c of token r sits at piece c ^ (r & 7) of its row
  auto request = [&](int pg, int st) {
    int page = table[pg];
    if (page < 0 || page >= p.kv.num_pages) {
      if (threadIdx.x == 0) atomicOr(p.status + ST_ERR, ERR_BAD_PAGE);
      page = 0;
    }
    const size_t base = ((size_t)page * p.Hkv + kvh) * PAGE * HD;
    const uint16_t* ksrc = static_cast<const uint16_t*>(p.kv.k_pool) + base;
    const uint16_t* vsrc = static_cast<const uint16_t*>(p.kv.v_pool) + base;
    const uint32_t kd = smem_u32(kt + st * TILE), vd = smem_u32(vt + st * TILE);
    for (int i = threadIdx.x; i < PAGE * PPR; i += nthr) {
      const int r = i / PPR, c = i - r * PPR;
      const bool valid = pg * PAGE + r < T;  // slots beyond the sequence hold whatever was there: zeros instead
      const uint32_t off = (uint32_t)(r * PPR + (c ^ (r & 7))) * 16;
      span_cp16(kd + off, ksrc + (size_t)r * HD + c * 8, valid);
      span_cp16(vd + off, vsrc + (size_t)r * HD + c * 8, valid);
    }
  };
  request(pg0, 0);
  span_commit();

  // ---- this warp's queries as bf16 high and low parts, rows beyond the span zero ----
  unsigned char* qh = qs + (size_t)warp * 2 * QT;
  unsigned char* ql = qh + QT;
  for (int i = lane; i < SPAN_ROWS * PPR; i += 32) {
    const int r = i / PPR, c = i - r * PPR;
    uint4 hi = make_uint4(0u, 0u, 0u, 0u), lo = hi;
    if (r < n) {
      const float* q = p.q_rot + ((size_t)(row0 + r) * p.Hq + head) * HD + c * 8;
      const float4 a = *reinterpret_cast<const float4*>(q), b = *reinterpret_cast<const float4*>(q + 4);
      const float v[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
      uint32_t h[4], l[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const uint16_t h0 = f2bf(v[2 * e]), h1 = f2bf(v[2 * e + 1]);
        h[e] = (uint32_t)h0 | ((uint32_t)h1 << 16);
        l[e] = pack_bf16(v[2 * e] - bf2f(h0), v[2 * e + 1] - bf2f(h1));
      }
      hi = make_uint4(h[0], h[1], h[2], h[3]);
      lo = make_uint4(l[0], l[1], l[2], l[3]);
    }
    const uint32_t off = (uint32_t)(r * PPR + (c ^ (r & 7))) * 16;
    *reinterpret_cast<uint4*>(qh + off) = hi;
    *reinterpret_cast<uint4*>(ql + off) = lo;
  }
  __syncwarp();

  // rows g and g + 8 of the tile: how many tokens each sees
  const int len0 = g < n ? T - n + 1 + g : 0, len1 = g + 8 < n ? T - n + 1 + g + 8 : 0;
  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;  // running maxima (base-2 domain), this lane's share of the sums
  float o[ND][4];
#pragma unroll
  for (int j = 0; j < ND; ++j) o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f;

  const uint32_t qh_u = smem_u32(qh), ql_u = smem_u32(ql);
  const int a_row = (lane & 7) + ((lane >> 3) & 1) * 8, a_half = lane >> 4;  // ldmatrix addresses of an A tile
#pragma unroll 1
  for (int pg = pg0; pg < pg1; ++pg) {
    const int st = (pg - pg0) & 1;
    span_wait<0>();   // this thread's pieces of the page have landed ...
    __syncthreads();  // ... and everybody's; and every warp is done with the other stage (the page before)
    if (pg + 1 < pg1) {
      request(pg + 1, st ^ 1);  // travels while this page is worked on
      span_commit();
    }
    const uint32_t kb = smem_u32(kt + st * TILE), vb = smem_u32(vt + st * TILE);

    // ---- S = Q K^T for 64 tokens: 8 n-tiles, two k-steps (32 dims) per pass ----
    float sc[8][4];
#pragma unroll
    for (int j = 0; j < 8; ++j) sc[j][0] = sc[j][1] = sc[j][2] = sc[j][3] = 0.f;
#pragma unroll
    for (int k2 = 0; k2 < HD / 32; ++k2) {
      uint32_t ah[2][4], al[2][4];
#pragma unroll
      for (int x = 0; x < 2; ++x) {
        const int c = (k2 * 2 + x) * 2 + a_half;
        const uint32_t off = (uint32_t)(a_row * PPR + (c ^ (a_row & 7))) * 16;
        ldsm_x4(ah[x], qh_u + off);
        ldsm_x4(al[x], ql_u + off);
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int r = j * 8 + (lane & 7), c = k2 * 4 + (lane >> 3);
        uint32_t b[4];
        ldsm_x4(b, kb + (uint32_t)(r * PPR + (c ^ (r & 7))) * 16);
        mma_bf16(sc[j], ah[0][0], ah[0][1], ah[0][2], ah[0][3], b[0], b[1]);
        mma_bf16(sc[j], al[0][0], al[0][1], al[0][2], al[0][3], b[0], b[1]);
        mma_bf16(sc[j], ah[1][0], ah[1][1], ah[1][2], ah[1][3], b[2], b[3]);
        mma_bf16(sc[j], al[1][0], al[1][1], al[1][2], al[1][3], b[2], b[3]);
      }
    }
    // ---- scale, causal mask, online softmax ----
    float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int tok = pg * PAGE + j * 8 + 2 * t;
      sc[j][0] = tok < len0 ? sc[j][0] * p.scale_log2 : -INFINITY;
      sc[j][1] = tok + 1 < len0 ? sc[j][1] * p.scale_log2 : -INFINITY;
      sc[j][2] = tok < len1 ? sc[j][2] * p.scale_log2 : -INFINITY;
      sc[j][3] = tok + 1 < len1 ? sc[j][3] * p.scale_log2 : -INFINITY;
      mx0 = fmaxf(mx0, fmaxf(sc[j][0], sc[j][1]));
      mx1 = fmaxf(mx1, fmaxf(sc[j][2], sc[j][3]));
    }
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
    const float n0 = fmaxf(m0, mx0), n1 = fmaxf(m1, mx1);
    const float u0 = n0 == -INFINITY ? 0.f : n0, u1 = n1 == -INFINITY ? 0.f : n1;  // a row that has seen nothing yet
    const float al0 = exp2f(m0 - u0), al1 = exp2f(m1 - u1);                         // exp2f(-inf) = 0
    m0 = n0;
    m1 = n1;
    l0 *= al0;
    l1 *= al1;
#pragma unroll
    for (int j = 0; j < ND; ++j) {
      o[j][0] *= al0;
      o[j][1] *= al0;
      o[j][2] *= al1;
      o[j][3] *= al1;
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      sc[j][0] = exp2f(sc[j][0] - u0);
      sc[j][1] = exp2f(sc[j][1] - u0);
      sc[j][2] = exp2f(sc[j][2] - u1);
      sc[j][3] = exp2f(sc[j][3] - u1);
      l0 += sc[j][0] + sc[j][1];
      l1 += sc[j][2] + sc[j][3];
    }
    // ---- O += P V: P as high + low parts, 16 tokens per k-step ----
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {
      uint32_t ph[4], pl[4];
#pragma unroll
      for (int x = 0; x < 4; ++x) {  // x: (n-tile 2 kk + (x >> 1)), row half (x & 1)
        const float v0 = sc[2 * kk + (x >> 1)][(x & 1) * 2], v1 = sc[2 * kk + (x >> 1)][(x & 1) * 2 + 1];
        const uint16_t h0 = f2bf(v0), h1 = f2bf(v1);
        ph[x] = (uint32_t)h0 | ((uint32_t)h1 << 16);
        pl[x] = pack_bf16(v0 - bf2f(h0), v1 - bf2f(h1));
      }
#pragma unroll
      for (int j2 = 0; j2 < ND / 2; ++j2) {
        const int r = kk * 16 + ((lane >> 3) & 1) * 8 + (lane & 7), c = j2 * 2 + (lane >> 4);
        uint32_t b[4];
        ldsm_x4_trans(b, vb + (uint32_t)(r * PPR + (c ^ (r & 7))) * 16);
        mma_bf16(o[2 * j2], ph[0], ph[1], ph[2], ph[3], b[0], b[1]);
        mma_bf16(o[2 * j2], pl[0], pl[1], pl[2], pl[3], b[0], b[1]);
        mma_bf16(o[2 * j2 + 1], ph[0], ph[1], ph[2], ph[3], b[2], b[3]);
        mma_bf16(o[2 * j2 + 1], pl[0], pl[1], pl[2], pl[3], b[2], b[3]);
      }
    }
  }
  l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
  l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
  // ---- this split's share of rows g and g + 8 ----
#pragma unroll
  for (int half = 0; half < 2; ++half) {
    const int i = g + half * 8;
    if (i >= n) continue;
    float* dst = p.part + (((size_t)(row0 + i) * p.Hq + head) * p.nsplit + split) * (HD + 2);
#pragma unroll
    for (int j = 0; j < ND; ++j)
      *reinterpret_cast<float2*>(dst + j * 8 + 2 * t) = make_float2(o[j][half * 2], o[j][half * 2 + 1]);
    if (t == 0) {
      dst[HD] = half ? m1 : m0;
      dst[HD + 1] = half ? l1 : l0;
    }
  }
}

// One (row, query head) per CTA of 128 threads: the splits' maxima and sums are read side by side (a thread per
// split), then 128 / (HD / 2) groups of threads each add up every n-th split's share of the output (one thread
// walking up to 64 splits with dependent reads took twice as long).
constexpr int SC_THREADS = 128;
constexpr int SC_MAX_SPLITS = MAX_PAGES_PER_SEQ / SPAN_PAGES;

template <int HD>
__global__ void __launch_bounds__(SC_THREADS) span_combine_kernel(const SpanDev p) {
  constexpr int PAIRS = HD / 2, GROUPS = SC_THREADS / PAIRS;
  __shared__ float s_w[SC_MAX_SPLITS];
  __shared__ float s_red[SC_THREADS / 32], s_red2[SC_THREADS / 32];
  __shared__ float2 s_o[GROUPS][PAIRS];
  const int head = blockIdx.x, row = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  pdl_trigger();
  pdl_wait();
  const float* src = p.part + ((size_t)row * p.Hq + head) * p.nsplit * (HD + 2);
  const int s_last = (row / p.n_tok) * p.n_tok + p.n_tok - 1;  // the sequence's last row sees all of its context
  const int T = min(max(p.kv.seq_lens[s_last], 0), p.kv.max_pages_per_seq * PAGE);
  const int ns = min(min(p.nsplit, SC_MAX_SPLITS), ((T + PAGE - 1) / PAGE + p.pps - 1) / p.pps);  // the splits that wrote a share
  float m = -INFINITY;
  for (int sidx = tid; sidx < ns; sidx += SC_THREADS) {
    const float ms = src[sidx * (HD + 2) + HD];
    s_w[sidx] = ms;
    m = fmaxf(m, ms);
  }
  m = warp_max(m);
  if (lane == 0) s_red[warp] = m;
  __syncthreads();
  m = fmaxf(fmaxf(s_red[0], s_red[1]), fmaxf(s_red[2], s_red[3]));
  float l = 0.f;
  for (int sidx = tid; sidx < ns; sidx += SC_THREADS) {
    const float ms = s_w[sidx];
    const float w = ms == -INFINITY ? 0.f : exp2f(ms - m);  // -inf: a split that saw no token of this row
    s_w[sidx] = w;
    l += w * src[sidx * (HD + 2) + HD + 1];
  }
  l = warp_sum(l);
  if (lane == 0) s_red2[warp] = l;
  __syncthreads();
  l = (s_red2[0] + s_red2[1]) + (s_red2[2] + s_red2[3]);
  const int gq = tid / PAIRS, e = (tid - gq * PAIRS) * 2;
  float o0 = 0.f, o1 = 0.f;
  for (int sidx = gq; sidx < ns; sidx += GROUPS) {
    const float w = s_w[sidx];
    const float2 v = *reinterpret_cast<const float2*>(src + sidx * (HD + 2) + e);
    o0 += w * v.x;
    o1 += w * v.y;
  }
  s_o[gq][tid - gq * PAIRS] = make_float2(o0, o1);
  __syncthreads();
  if (gq != 0) return;
#pragma unroll
  for (int x = 1; x < GROUPS; ++x) {
    o0 += s_o[x][tid].x;
    o1 += s_o[x][tid].y;
  }
  const float inv = l > 0.f ? 1.0f / l : 0.f;
  o0 *= inv;
  o1 *= inv;
  const size_t idx = ((size_t)row * p.Hq + head) * HD + e;
  if (p.out_f32) *reinterpret_cast<float2*>(p.out_f32 + idx) = make_float2(o0, o1);
  if (p.out_bf16) *reinterpret_cast<uint32_t*>(p.out_bf16 + idx) = pack_bf16(o0, o1);
  if (p.out_hi) {
    const uint16_t h0 = f2bf(o0), h1 = f2bf(o1);
    const int k = head * HD + e;  // column of the projection's input; e is even, so k and k + 1 share a piece
    unsigned char* dst = reinterpret_cast<unsigned char*>(p.out_hi) + act_piece_offset(2 * p.out_rows, row, k >> 3) + (k & 7) * 2;
    *reinterpret_cast<uint32_t*>(dst) = (uint32_t)h0 | ((uint32_t)h1 << 16);
    *reinterpret_cast<uint32_t*>(dst + (size_t)p.out_rows * 128) = pack_bf16(o0 - bf2f(h0), o1 - bf2f(h1));
  }
}

template <int HD>
static void launch_span(const SpanDev& d, cudaStream_t st) {
  const int smem = 4 * PAGE * HD * 2 + d.G * 2 * SPAN_ROWS * HD * 2;
  ensure_dynamic_smem(reinterpret_cast<const void*>(&span_attn_kernel<HD>), smem);
  SOL_LAUNCH("span_attn", span_attn_kernel<HD>, dim3(d.nsplit, d.Hkv, d.n_seq), dim3(d.G * 32), smem, st, d);
  SOL_LAUNCH("span_combine", span_combine_kernel<HD>, dim3(d.Hq, d.n_seq * d.n_tok), dim3(SC_THREADS), 0, st, d);
}

// After the query preparation of a batch whose rows are n_seq spans of n_tok tokens (1 <= n_tok <= 16).
void launch_span_attention(const AttnArgs& a, int n_tok, cudaStream_t st) {
  const sol_shape_t& sh = a.shape;
  SpanDev d;
  d.kv = a.kv;
  d.Hq = sh.n_q_heads; d.Hkv = sh.n_kv_heads; d.G = d.Hq / d.Hkv; d.n_tok = n_tok; d.n_seq = a.B / n_tok;
  // A CTA takes SPAN_PAGES cache pages of a (sequence, kv-head): contexts of very different lengths then give CTAs
  // of the same length (a fixed number of splits per sequence left the longest sequence's CTAs running alone:
  // 100 us per launch where this takes a third).  The shares go to the decode path's array of partial results
  // ([B][Hkv][splits][G][hd + 2]), which bounds the number of splits.
  d.pps = SPAN_PAGES;
  while ((a.kv.max_pages_per_seq + d.pps - 1) / d.pps > a.splits) d.pps *= 2;
  d.nsplit = (a.kv.max_pages_per_seq + d.pps - 1) / d.pps;
  d.scale_log2 = 1.4426950408889634f / sqrtf((float)sh.head_dim);
  d.q_rot = a.q_rot; d.part = a.part;
  d.out_f32 = a.out_f32; d.out_bf16 = static_cast<uint16_t*>(a.out_bf16); d.out_hi = static_cast<uint16_t*>(a.out_hi);
  d.out_rows = a.out_rows; d.status = a.status;
  if (sh.head_dim == 64) launch_span<64>(d, st);
  else launch_span<128>(d, st);
}

}  // namespace sol
