// swiftkv_tail_attention_noalloc: the split-KV single-query attention for callers that cannot allocate device
// memory or lend a scratch buffer.  The per-split partial results go to a fixed array that is part of this
// library's device image (one copy per GPU that loads the library, held until the process exits).
#include <mutex>

#include "common.cuh"

namespace {

// Scratch of the no-allocation entry point.  In host code this name is only a handle for the runtime, not a device
// address: the address is looked up once per device with cudaGetSymbolAddress below and that pointer is what the
// kernels receive.
static __device__ __align__(256) float g_noalloc_scratch[SWIFTKV_NOALLOC_SCRATCH_BYTES / sizeof(float)];

constexpr int MAX_DEVICES = 64;
std::mutex g_mu;
float *g_scratch_ptr[MAX_DEVICES] = {};

// Device address of the array on the current device (looked up on the first call per device).
int32_t scratch_for_current_device(float **out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return skv::report_error(SWIFTKV_ERR_CUDA, cudaGetErrorString(e));
  if (dev < 0 || dev >= MAX_DEVICES) return skv::report_error(SWIFTKV_ERR_UNSUPPORTED, "device ordinal out of range");
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_scratch_ptr[dev]) {
    float *p = nullptr;
    e = cudaGetSymbolAddress(reinterpret_cast<void **>(&p), g_noalloc_scratch);
    if (e != cudaSuccess || !p) return skv::report_error(SWIFTKV_ERR_CUDA, cudaGetErrorString(e));
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return SWIFTKV_OK;
}

}  // namespace

extern "C" int32_t swiftkv_tail_attention_noalloc(const float *q, const void *k_cache, const void *v_cache, float *out,
                                                  const int32_t *cu_seqlens, int32_t n_seqs, int32_t max_seq_len,
                                                  int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim, int32_t dtype,
                                                  void *cuda_stream) {
  using namespace skv;
  if (!q || !k_cache || !v_cache || !out || !cu_seqlens) return report_error(SWIFTKV_ERR_INVALID_ARG, "null argument");
  if (n_seqs < 1 || n_seqs > MAX_TAIL_ROWS || max_seq_len < 1 || n_q_heads < 1 || n_kv_heads < 1 || n_q_heads % n_kv_heads ||
      head_dim < 2 || head_dim > 256)
    return report_error(SWIFTKV_ERR_INVALID_ARG, "bad shape (n_seqs must be in [1, 8], head_dim in [2, 256], n_q_heads a multiple of n_kv_heads)");
  if (dtype != SWIFTKV_DTYPE_BF16 && dtype != SWIFTKV_DTYPE_F32) return report_error(SWIFTKV_ERR_INVALID_ARG, "unknown dtype");
  const size_t need = tail_attention_scratch_bytes(n_seqs, n_q_heads, head_dim, max_seq_len);
  if (need > SWIFTKV_NOALLOC_SCRATCH_BYTES)
    return report_error(SWIFTKV_ERR_WORKSPACE_SMALL,
                        "this problem needs more split-KV scratch than the built-in 9 MiB array: use swiftkv_tail_attention");
  float *scratch = nullptr;
  int32_t rc = scratch_for_current_device(&scratch);
  if (rc) return rc;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  // every (prompt, head, split) entry that the merge pass reads is written by the partial pass of this same call,
  // so stale contents from an earlier call are never observed
  if (dtype == SWIFTKV_DTYPE_BF16)
    launch_tail_attention<bf16>(q, (const bf16 *)k_cache, (const bf16 *)v_cache, nullptr, nullptr, out, cu_seqlens, nullptr, nullptr, 0, n_seqs, max_seq_len, n_q_heads,
                                n_kv_heads, head_dim, scratch, st);
  else
    launch_tail_attention<float>(q, (const float *)k_cache, (const float *)v_cache, nullptr, nullptr, out, cu_seqlens, nullptr, nullptr, 0, n_seqs, max_seq_len,
                                 n_q_heads, n_kv_heads, head_dim, scratch, st);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return report_error(SWIFTKV_ERR_CUDA, cudaGetErrorString(e));
  return SWIFTKV_OK;
}
