// Attention over the kept pages of the Quest selection in one pass (appendix "Token sparsity via Quest",
// "Sparse attention"): for every listed token of a (sequence, kv-head) its key and its value are read once, the
// logits of the G query heads, the additive mask of the heads that did not keep the token's page, the softmax
// and the weighted sum of the values all happen on the tile in shared memory.  (The token selection's two passes
// need every token's logits before they can select; here the selection comes from the page bounds, so nothing
// forces the logits through memory: as two kernels, logits then pass 2, this took 119 + 162 us per layer on the
// ragged batch.)
//
//   quest_attend_kernel   a warp takes split_len consecutive list entries of a row, 32 (head_dim 64) or 16 at a time: their cache
//                         rows of K and V come by cp.async into swizzled tiles (two stages per warp).  The 16
//                         rows of the m16n8k16 tiles are the G heads' queries as bf16 high parts (rows 0..7)
//                         and low parts (rows 8..15): S = Q K^T, then per head mask, online softmax (base 2),
//                         and O += P V with the weights again as high and low parts.  Leaves (O, m, l) per
//                         (row, split, head) in the array of partial results of pass 2.
//   quest_combine_kernel  merges a row's splits and writes the output in the forms the callers read.
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "sol_common.cuh"
#include "sol_internal.h"

namespace sol {

struct QuestAttendDev {
  sol_kv_t kv;
  int B, Hq, Hkv, G, Tmax, S, Pstride, splits, split_len;
  float scale_log2;  // log2(e) / sqrt(head_dim)
  const float* q_rot;             // [B][Hq][hd]
  const int32_t* list_idx;        // [B][Hkv][Tmax] token index of every listed token
  const uint32_t* list_row;       // ... its cache row (page table applied), 0xffffffff: bad page
  const int32_t* kept_cnt;        // [B][Hkv]
  const unsigned char* page_mask; // [B][Hkv][Pstride]: per Quest page, bit h = head h of the group keeps it
  float* part;                    // [B][Hkv][splits][G][hd + 2]: O, m (base-2 domain), l
  float* out_f32;                 // each optional
  uint16_t* out_bf16;
  uint16_t* out_hi;
  int out_rows;
  uint32_t n_rows;
  int* status;
};

__device__ __forceinline__ void qa_cp16(uint32_t dst_smem, const void* src, bool valid) {
  const int n = valid ? 16 : 0;  // 0: the 16 bytes are filled with zeros
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst_smem), "l"(src), "r"(n) : "memory");
}
__device__ __forceinline__ void qa_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void qa_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

constexpr int QA_WARPS = 4;

template <int HD>
struct QaCfg {
  static constexpr int PPR = HD / 8;                    // 16-byte pieces per row
  static constexpr int TILE = HD == 64 ? 32 : 16;       // list entries per tile: 4 KB of keys either way
  static constexpr int TILE_BYTES = TILE * HD * 2;      // keys (or values) of a tile
  static constexpr int WARP_BYTES = 4 * TILE_BYTES + 2 * TILE * 8;  // K, V x two stages; (row, mask) per entry x two stages
  static constexpr int SMEM = QA_WARPS * WARP_BYTES;
};

template <int HD>
__global__ void __launch_bounds__(QA_WARPS * 32) quest_attend_kernel(const QuestAttendDev p) {
  using C = QaCfg<HD>;
  constexpr int PPR = C::PPR, ND = HD / 8, KS = HD / 16, QA_TILE = C::TILE, NTL = QA_TILE / 8;
  extern __shared__ __align__(128) unsigned char qasm[];
  __shared__ int s_cum[QA_WARPS * 32 + 1], s_wsum[QA_WARPS];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, tid = threadIdx.x;
  const int g = lane >> 2, t = lane & 3;
  unsigned char* mine = qasm + (size_t)warp * C::WARP_BYTES;
  unsigned char* kt = mine;                                  // [2][TILE_BYTES]
  unsigned char* vt = mine + 2 * C::TILE_BYTES;              // [2][TILE_BYTES]
  int2* tab = reinterpret_cast<int2*>(mine + 4 * C::TILE_BYTES);  // [2][QA_TILE]: (cache row or -1, head mask)
  const int unit_len = QA_WARPS * p.split_len;  // list entries per CTA unit
  pdl_trigger();
  if (tid == 0) s_cum[0] = 0;
  pdl_wait();  // the lists and their lengths come from the selection
  int my_incl = 0;
  if (tid < p.B) {
    int mx = 0;
    for (int h = 0; h < p.Hkv; ++h) mx = max(mx, min(p.kept_cnt[tid * p.Hkv + h], p.Tmax));
    my_incl = max(1, (mx + unit_len - 1) / unit_len);  // units of the sequence's longest list (one at least: the output is always written)
  }
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int x = __shfl_up_sync(0xffffffffu, my_incl, o);
    if (lane >= o) my_incl += x;
  }
  if (lane == 31) s_wsum[warp] = my_incl;
  __syncthreads();
  for (int w = 0; w < warp; ++w) my_incl += s_wsum[w];
  s_cum[tid + 1] = my_incl;
  __syncthreads();
  const int n_units = s_cum[p.B] * p.Hkv;
  const uint16_t* kp = static_cast<const uint16_t*>(p.kv.k_pool);
  const uint16_t* vp = static_cast<const uint16_t*>(p.kv.v_pool);
#pragma unroll 1
  for (int u = blockIdx.x; u < n_units; u += gridDim.x) {
    const int key = u / p.Hkv;
    const int b = __syncthreads_count(tid < p.B && my_incl <= key);
    const int first = s_cum[b], n_groups = s_cum[b + 1] - first;
    const int rem = u - first * p.Hkv;
    const int kvh = rem / n_groups, grp = rem - kvh * n_groups;
    const int bk = b * p.Hkv + kvh;
    const int cnt = min(p.kept_cnt[bk], p.Tmax);
    const int split = grp * QA_WARPS + warp;
    const int n0 = split * p.split_len;  // this warp's run of list entries
    if (n0 >= cnt || split >= p.splits) continue;
    const int len = min(p.split_len, cnt - n0);
    const int nt = (len + QA_TILE - 1) / QA_TILE;
    const size_t row = (size_t)bk * p.Tmax;

    // ---- the group's queries as A fragments: rows 0..7 high parts, rows 8..15 low parts of head g ----
    uint32_t qa[KS][4];
    {
      const float* q = p.q_rot + ((size_t)b * p.Hq + kvh * p.G + g) * HD;
#pragma unroll
      for (int kk = 0; kk < KS; ++kk) {
        float2 x0 = make_float2(0.f, 0.f), x1 = x0;
        if (g < p.G) {
          x0 = *reinterpret_cast<const float2*>(q + kk * 16 + 2 * t);
          x1 = *reinterpret_cast<const float2*>(q + kk * 16 + 8 + 2 * t);
        }
        const uint16_t h0 = f2bf(x0.x), h1 = f2bf(x0.y), h2 = f2bf(x1.x), h3 = f2bf(x1.y);
        qa[kk][0] = (uint32_t)h0 | ((uint32_t)h1 << 16);
        qa[kk][1] = pack_bf16(x0.x - bf2f(h0), x0.y - bf2f(h1));
        qa[kk][2] = (uint32_t)h2 | ((uint32_t)h3 << 16);
        qa[kk][3] = pack_bf16(x1.x - bf2f(h2), x1.y - bf2f(h3));
      }
    }
    // list words of tile i: lane l holds entry l (cache row checked, not trusted)
    auto load_entry = [&](int i) {
      int2 e = make_int2(-1, 0);
      const int n = i * QA_TILE + lane;
      if (lane < QA_TILE && i < nt && n < len) {
        const uint32_t r = p.list_row[row + n0 + n];
        const int j = p.list_idx[row + n0 + n];
        if (r != 0xffffffffu && r < p.n_rows && j >= 0 && j < p.Tmax) {
          e = make_int2((int)r, (int)p.page_mask[(size_t)bk * p.Pstride + j / p.S]);
        } else if (r != 0xffffffffu) {
          atomicMax(p.status + 5, 3);
        }
      }
      return e;
    };
    // rows of tile i (its entries are in the table) into stage i & 1
    auto request = [&](int i) {
      if (i < nt) {
        const int2* tb = tab + (i & 1) * QA_TILE;
        const uint32_t kd = smem_u32(kt + (i & 1) * C::TILE_BYTES), vd = smem_u32(vt + (i & 1) * C::TILE_BYTES);
#pragma unroll
        for (int x = 0; x < QA_TILE * PPR / 32; ++x) {
          const int c = x * 32 + lane, r = c / PPR, part = c % PPR;
          const int ridx = tb[r].x;
          const uint32_t off = (uint32_t)(r * PPR + ((part & ~7) | ((part ^ r) & 7))) * 16;
          const size_t src = (size_t)(ridx < 0 ? 0 : ridx) * HD + part * 8;
          qa_cp16(kd + off, kp + src, ridx >= 0);
          qa_cp16(vd + off, vp + src, ridx >= 0);
        }
      }
      qa_commit();  // an empty group keeps the count of groups per step fixed
    };

    float m = -INFINITY, l = 0.f;  // head g: running maximum (base 2), this lane's share of the sum
    float o[ND][4];
#pragma unroll
    for (int j = 0; j < ND; ++j) o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f;

    __syncwarp();  // the table and the tiles of the unit before are not read any more
    if (lane < QA_TILE) tab[lane] = load_entry(0);
    __syncwarp();
    request(0);
    int2 e_next = load_entry(1);
#pragma unroll 1
    for (int i = 0; i < nt; ++i) {
      const int st = i & 1;
      if (lane < QA_TILE) tab[(st ^ 1) * QA_TILE + lane] = e_next;  // the other stage was worked on in the step before
      __syncwarp();
      request(i + 1);
      e_next = load_entry(i + 2);
      qa_wait<1>();  // this lane's pieces of tile i have landed ...
      __syncwarp();  // ... and so have the other lanes'
      const uint32_t kb = smem_u32(kt + st * C::TILE_BYTES), vb = smem_u32(vt + st * C::TILE_BYTES);
      const int2* tb = tab + st * QA_TILE;

      // ---- S = Q K^T: n-tiles of 8 entries ----
      float sc[NTL][4];
#pragma unroll
      for (int j = 0; j < NTL; ++j) sc[j][0] = sc[j][1] = sc[j][2] = sc[j][3] = 0.f;
#pragma unroll
      for (int k2 = 0; k2 < KS / 2; ++k2) {
#pragma unroll
        for (int j = 0; j < NTL; ++j) {
          const int r = j * 8 + (lane & 7), c = k2 * 4 + (lane >> 3);
          uint32_t bq[4];
          ldsm_x4(bq, kb + (uint32_t)(r * PPR + ((c & ~7) | ((c ^ r) & 7))) * 16);
          mma_bf16(sc[j], qa[2 * k2][0], qa[2 * k2][1], qa[2 * k2][2], qa[2 * k2][3], bq[0], bq[1]);
          mma_bf16(sc[j], qa[2 * k2 + 1][0], qa[2 * k2 + 1][1], qa[2 * k2 + 1][2], qa[2 * k2 + 1][3], bq[2], bq[3]);
        }
      }
      // ---- head g: high + low parts, scale, mask (absent entries; pages this head did not keep), softmax ----
      float pw[NTL][2];
      float mx = -INFINITY;
#pragma unroll
      for (int j = 0; j < NTL; ++j) {
        const int2 e0 = tb[j * 8 + 2 * t], e1 = tb[j * 8 + 2 * t + 1];
        const bool on0 = e0.x >= 0 && ((e0.y >> g) & 1), on1 = e1.x >= 0 && ((e1.y >> g) & 1);
        pw[j][0] = on0 ? (sc[j][0] + sc[j][2]) * p.scale_log2 : -INFINITY;
        pw[j][1] = on1 ? (sc[j][1] + sc[j][3]) * p.scale_log2 : -INFINITY;
        mx = fmaxf(mx, fmaxf(pw[j][0], pw[j][1]));
      }
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      const float nm = fmaxf(m, mx);
      const float ref = nm == -INFINITY ? 0.f : nm;  // a head that has seen nothing yet
      const float al = exp2f(m - ref);               // exp2f(-inf) = 0
      m = nm;
      l *= al;
#pragma unroll
      for (int j = 0; j < ND; ++j) {
        o[j][0] *= al;
        o[j][1] *= al;
        o[j][2] *= al;
        o[j][3] *= al;
      }
#pragma unroll
      for (int j = 0; j < NTL; ++j) {
        pw[j][0] = exp2f(pw[j][0] - ref);
        pw[j][1] = exp2f(pw[j][1] - ref);
        l += pw[j][0] + pw[j][1];
      }
      // ---- O += P V: k-steps of 16 entries; rows 0..7 the weights' high parts, rows 8..15 their low parts ----
#pragma unroll
      for (int kk = 0; kk < NTL / 2; ++kk) {
        const uint16_t h0 = f2bf(pw[2 * kk][0]), h1 = f2bf(pw[2 * kk][1]);
        const uint16_t h2 = f2bf(pw[2 * kk + 1][0]), h3 = f2bf(pw[2 * kk + 1][1]);
        const uint32_t a0 = (uint32_t)h0 | ((uint32_t)h1 << 16), a2 = (uint32_t)h2 | ((uint32_t)h3 << 16);
        const uint32_t a1 = pack_bf16(pw[2 * kk][0] - bf2f(h0), pw[2 * kk][1] - bf2f(h1));
        const uint32_t a3 = pack_bf16(pw[2 * kk + 1][0] - bf2f(h2), pw[2 * kk + 1][1] - bf2f(h3));
#pragma unroll
        for (int j2 = 0; j2 < ND / 2; ++j2) {
          const int r = kk * 16 + ((lane >> 3) & 1) * 8 + (lane & 7), c = j2 * 2 + (lane >> 4);
          uint32_t bv[4];
          ldsm_x4_trans(bv, vb + (uint32_t)(r * PPR + ((c & ~7) | ((c ^ r) & 7))) * 16);
          mma_bf16(o[2 * j2], a0, a1, a2, a3, bv[0], bv[1]);
          mma_bf16(o[2 * j2 + 1], a0, a1, a2, a3, bv[2], bv[3]);
        }
      }
      __syncwarp();  // the stage and its table are rewritten by the next steps
    }
    qa_wait<0>();
    l += __shfl_xor_sync(0xffffffffu, l, 1);
    l += __shfl_xor_sync(0xffffffffu, l, 2);
    if (g < p.G) {
      float* dst = p.part + (((size_t)bk * p.splits + split) * p.G + g) * (HD + 2);
#pragma unroll
      for (int j = 0; j < ND; ++j)
        *reinterpret_cast<float2*>(dst + j * 8 + 2 * t) = make_float2(o[j][0] + o[j][2], o[j][1] + o[j][3]);
      if (t == 0) {
        dst[HD] = m;
        dst[HD + 1] = l;
      }
    }
  }
}

// One (sequence, query head) per CTA of 128 threads.  A long row has hundreds of splits: their maxima and sums
// are read side by side (a thread per split), and the threads form 128 / (HD / 2) groups that each add up every
// n-th split's share of the output (one thread walking all splits with dependent reads took 41 us per layer).
constexpr int QC_THREADS = 128;
constexpr int QC_MAX_SPLITS = MAX_PAGES_PER_SEQ * PAGE / 128;

template <int HD>
__global__ void __launch_bounds__(QC_THREADS) quest_combine_kernel(const QuestAttendDev p) {
  constexpr int PAIRS = HD / 2, GROUPS = QC_THREADS / PAIRS;
  __shared__ float s_w[QC_MAX_SPLITS];
  __shared__ float s_red[QC_THREADS / 32], s_red2[QC_THREADS / 32];
  __shared__ float2 s_o[GROUPS][PAIRS];
  const int head = blockIdx.x, b = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  pdl_trigger();
  pdl_wait();
  const int kvh = head / p.G, gi = head - kvh * p.G, bk = b * p.Hkv + kvh;
  const int cnt = min(p.kept_cnt[bk], p.Tmax);
  const int ns = min(min(p.splits, QC_MAX_SPLITS), (cnt + p.split_len - 1) / p.split_len);
  const float* src = p.part + ((size_t)bk * p.splits * p.G + gi) * (HD + 2);
  const size_t stride = (size_t)p.G * (HD + 2);
  // ---- the row's maximum ----
  float m = -INFINITY;
  for (int s = tid; s < ns; s += QC_THREADS) {
    const float ms = src[s * stride + HD];
    s_w[s] = ms;
    m = fmaxf(m, ms);
  }
  m = warp_max(m);
  if (lane == 0) s_red[warp] = m;
  __syncthreads();
  m = fmaxf(fmaxf(s_red[0], s_red[1]), fmaxf(s_red[2], s_red[3]));
  // ---- the splits' weights and the sum ----
  float l = 0.f;
  for (int s = tid; s < ns; s += QC_THREADS) {
    const float ms = s_w[s];
    const float w = ms == -INFINITY ? 0.f : exp2f(ms - m);  // -inf: a split without a token of this head's pages
    s_w[s] = w;
    l += w * src[s * stride + HD + 1];
  }
  l = warp_sum(l);
  if (lane == 0) s_red2[warp] = l;
  __syncthreads();
  l = (s_red2[0] + s_red2[1]) + (s_red2[2] + s_red2[3]);
  // ---- the output: group gq adds the shares of splits gq, gq + GROUPS, ... ----
  const int gq = tid / PAIRS, e = (tid - gq * PAIRS) * 2;
  float o0 = 0.f, o1 = 0.f;
  for (int s = gq; s < ns; s += GROUPS) {
    const float w = s_w[s];
    const float2 v = *reinterpret_cast<const float2*>(src + s * stride + e);
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
  const size_t idx = ((size_t)b * p.Hq + head) * HD + e;
  if (p.out_f32) *reinterpret_cast<float2*>(p.out_f32 + idx) = make_float2(o0, o1);
  if (p.out_bf16) *reinterpret_cast<uint32_t*>(p.out_bf16 + idx) = pack_bf16(o0, o1);
  if (p.out_hi) {
    const uint16_t h0 = f2bf(o0), h1 = f2bf(o1);
    const int k = head * HD + e;  // column of the projection's input; e is even, so k and k + 1 share a piece
    unsigned char* dst = reinterpret_cast<unsigned char*>(p.out_hi) + act_piece_offset(2 * p.out_rows, b, k >> 3) + (k & 7) * 2;
    *reinterpret_cast<uint32_t*>(dst) = (uint32_t)h0 | ((uint32_t)h1 << 16);
    *reinterpret_cast<uint32_t*>(dst + (size_t)p.out_rows * 128) = pack_bf16(o0 - bf2f(h0), o1 - bf2f(h1));
  }
}

template <int HD>
static void launch_qa(const QuestAttendDev& d, cudaStream_t st) {
  using C = QaCfg<HD>;
  const int unit_len = QA_WARPS * d.split_len;
  const long long upper = (long long)((d.Tmax + unit_len - 1) / unit_len) * d.Hkv * d.B;
  const long long cap = (long long)sm_count() * (227 * 1024 / (C::SMEM + 2048)) * 4;  // four rounds of the resident CTAs
  ensure_dynamic_smem(reinterpret_cast<const void*>(&quest_attend_kernel<HD>), C::SMEM);
  SOL_LAUNCH("quest_attend", quest_attend_kernel<HD>, dim3((unsigned)(upper < cap ? upper : cap)), dim3(QA_WARPS * 32), C::SMEM, st, d);
  SOL_LAUNCH("quest_combine", quest_combine_kernel<HD>, dim3(d.Hq, d.B), dim3(QC_THREADS), 0, st, d);
}

// After launch_quest_selection (token lists, head masks per page): the attention itself.
void launch_quest_attend(const AttnArgs& a, cudaStream_t st) {
  const sol_shape_t& sh = a.shape;
  QuestAttendDev d;
  d.kv = a.kv; d.B = a.B; d.Hq = sh.n_q_heads; d.Hkv = sh.n_kv_heads; d.G = d.Hq / d.Hkv;
  d.Tmax = a.kv.max_pages_per_seq * PAGE; d.S = sh.quest_page_size; d.Pstride = d.Tmax / 4;
  d.splits = a.splits; d.split_len = attn_split_len(sh.head_dim);
  d.scale_log2 = (float)(1.4426950408889634 / sqrt((double)sh.head_dim));
  d.q_rot = a.q_rot; d.list_idx = a.list_idx; d.list_row = a.kept_row; d.kept_cnt = a.kept_cnt;
  d.page_mask = a.page_mask; d.part = a.part;
  d.out_f32 = a.out_f32; d.out_bf16 = static_cast<uint16_t*>(a.out_bf16); d.out_hi = static_cast<uint16_t*>(a.out_hi);
  d.out_rows = a.out_rows; d.n_rows = (uint32_t)a.kv.num_pages * d.Hkv * PAGE; d.status = a.status;
  if (sh.head_dim == 64) launch_qa<64>(d, st);
  else launch_qa<128>(d, st);
}

}  // namespace sol
