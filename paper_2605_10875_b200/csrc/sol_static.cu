// sol_sparse_decode_attn_static: the decode attention for callers that cannot
// hand the library a workspace.
//
// Some hosts of this library never get to call cudaMalloc on the decode path:
// a serving process whose memory pool was carved up at start-up and has
// nothing left to lend, a plugin running inside another runtime that owns
// the allocator, a latency-critical loop where an allocation (or the implicit
// synchronisation a free can bring) is not allowed.  For them the scratch of
// the attention call (split queries, logits, selection scores, kept lists,
// split partials, status words) lives in one fixed array that is part of the
// library image: SOL_STATIC_SCRATCH_BYTES of device memory on every GPU that
// loads the library, held until the process exits.
//
// The array's name in host code is only a handle for the runtime, not a device
// address, so the address is looked up once per device with
// cudaGetSymbolAddress (with that device current) and that pointer is what
// the kernels receive.
#include <mutex>

#include "sol_common.cuh"
#include "sol_internal.h"

namespace {

constexpr size_t kScratchBytes = SOL_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
unsigned char* g_scratch_ptr[kMaxDevices] = {nullptr};

// Device address of the array on the current device; resolved on the first call per device.
sol_status_t scratch_of_current_device(unsigned char** out) {
  int dev = 0;
  if (sol::record_cuda_error(cudaGetDevice(&dev), "cudaGetDevice")) return SOL_ERR_CUDA;
  if (dev < 0 || dev >= kMaxDevices) return SOL_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_mu);
  if (g_scratch_ptr[dev] == nullptr) {
    void* p = nullptr;
    if (sol::record_cuda_error(cudaGetSymbolAddress(&p, g_static_scratch), "cudaGetSymbolAddress")) return SOL_ERR_CUDA;
    if (p == nullptr) return SOL_ERR_CUDA;
    g_scratch_ptr[dev] = static_cast<unsigned char*>(p);
  }
  *out = g_scratch_ptr[dev];
  return SOL_OK;
}

// status words first, then the attention scratch
constexpr size_t kStatusBytes = 256;

bool attention_shape_ok(const sol_shape_t* s) {
  if (!s) return false;
  if (s->head_dim != 64 && s->head_dim != 128) return false;
  if (s->page_size != 64) return false;
  if (s->n_kv_heads <= 0 || s->n_q_heads <= 0 || s->n_q_heads % s->n_kv_heads) return false;
  if (s->n_q_heads / s->n_kv_heads > 8) return false;
  return s->n_sink >= 0 && s->n_window >= 0 && s->token_select == SOL_SELECT_TOKENS;
}

}  // namespace

extern "C" sol_status_t sol_sparse_decode_attn_static(const sol_shape_t* shape, const void* q_bf16,
                                                      const sol_kv_t* kv, int32_t B, const int32_t* r_permille,
                                                      void* out_bf16, int32_t* kept_idx, int32_t* kept_cnt,
                                                      int32_t* status_out, sol_stream_t stream) {
  if (!shape || !q_bf16 || !kv || !kv->k_pool || !kv->v_pool || !kv->page_table || !kv->seq_lens ||
      kv->max_pages_per_seq <= 0 || kv->num_pages <= 0 || !r_permille || !out_bf16 || B < 0)
    return SOL_ERR_INVALID_ARG;
  if (!attention_shape_ok(shape) || B > 128 || kv->max_pages_per_seq > sol::MAX_PAGES_PER_SEQ) return SOL_ERR_UNSUPPORTED;
  if (B == 0) return SOL_OK;
  const sol::AttnScratch L = sol::attn_scratch_layout(*shape, B, kv->max_pages_per_seq, kStatusBytes);
  if (L.end > kScratchBytes) return SOL_ERR_WORKSPACE_TOO_SMALL;  // the fixed scratch cannot hold this problem

  unsigned char* base = nullptr;
  const sol_status_t s = scratch_of_current_device(&base);
  if (s != SOL_OK) {
    sol::take_cuda_failure();  // reported here; the mark must not leak into this thread's next call
    return s;
  }
  cudaStream_t st = (cudaStream_t)stream;
  // the array keeps whatever the previous call left; only the status words must start at zero
  if (sol::record_cuda_error(cudaMemsetAsync(base, 0, kStatusBytes, st), "status memset")) {
    sol::take_cuda_failure();
    return SOL_ERR_CUDA;
  }

  sol::AttnArgs a;
  a.shape = *shape;
  a.kv = *kv;
  a.B = B;
  a.span_tokens = 0;
  a.r_permille = r_permille;
  a.qkv_f32 = nullptr;
  a.ldq = 0;
  a.qkv_ksplit = 0;
  a.qkv_scale = nullptr;
  a.q_bf16 = q_bf16;
  sol::attn_scratch_bind(a, base, L, kept_idx, kept_cnt);
  a.out_f32 = nullptr;
  a.out_bf16 = out_bf16;
  a.out_hi = nullptr;
  a.out_lo = nullptr;
  a.out_rows = 0;
  a.page_mask = nullptr;
  a.quest_keys = nullptr;
  a.quest_err = nullptr;
  a.quest_hmask = nullptr;
  a.quest_qsplit = nullptr;
  a.quest_l1 = nullptr;
  a.quest_order = nullptr;
  a.quest_pages_out = nullptr;
  a.quest_cnt_out = nullptr;
  a.status = reinterpret_cast<int*>(base);
  sol::launch_attention(a, st);
  if (status_out != nullptr)
    sol::record_cuda_error(cudaMemcpyAsync(status_out, base, sizeof(int32_t) * sol::ST_WORDS, cudaMemcpyDeviceToDevice, st),
                           "status copy");
  return sol::take_cuda_failure() ? SOL_ERR_CUDA : SOL_OK;
}
