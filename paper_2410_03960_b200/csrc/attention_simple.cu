// Shape-generic causal varlen grouped-query attention with fp32 arithmetic (Sec. 3.1).
// One warp per (query token, query head).  Keys are visited 32 at a time: each lane scores one key
// (full head_dim dot product), the warp takes the running max / sum (online softmax), then the 32
// probabilities are broadcast one by one while the lanes accumulate their slice of the output row.
// This is the fp32 model's attention and the bf16 model's path for head dims the tensor-core kernel
// does not cover.
#include "common.cuh"

namespace skv {

template <typename TQ, typename T, int MAX_E>   // MAX_E = ceil(hd / 32) output elements per lane
__global__ void __launch_bounds__(128) attention_simple_kernel(const TQ *__restrict__ q, const T *__restrict__ k,
                                                               const T *__restrict__ v, TQ *__restrict__ out,
                                                               const int32_t *__restrict__ cu, int n_seqs,
                                                               const int32_t *__restrict__ k_row0,
                                                               const int32_t *__restrict__ kv_len,
                                                               const int32_t *__restrict__ blk, int blk_stride, int n_tokens,
                                                               int n_q, int n_kv, int hd, float scale) {
  extern __shared__ float q_sm[];   // [4 warps][hd]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long item = (long long)blockIdx.x * 4 + warp;
  if (item >= (long long)n_tokens * n_q) return;
  const int t = (int)(item / n_q), h = (int)(item % n_q);
  const int kvh = h / (n_q / n_kv);
  int lo = 0, hi = n_seqs;   // the sequence of query t from the offsets of the new tokens
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (cu[mid] <= t) lo = mid; else hi = mid;
  }
  const int n_new = cu[lo + 1] - cu[lo];
  const int past = kv_len ? kv_len[lo] - n_new : 0;
  const int p = past + (t - cu[lo]);                    // position of this query: it sees keys 0..p
  const int first = k_row0 ? k_row0[lo] : cu[lo];       // K / V row of the sequence's first token
  float *qs = q_sm + warp * hd;
  const TQ *qr = q + ((size_t)t * n_q + h) * hd;
  for (int i = lane; i < hd; i += 32) qs[i] = to_f(qr[i]) * scale;
  __syncwarp();

  float m = -INFINITY, l = 0.f;
  float acc[MAX_E];
#pragma unroll
  for (int e = 0; e < MAX_E; ++e) acc[e] = 0.f;

  for (int c0 = 0; c0 <= p; c0 += 32) {
    const int key = c0 + lane;
    float s = -INFINITY;
    if (key <= p) {
      const T *kr = k + (kv_row_of(blk, blk_stride, lo, first, key) * n_kv + kvh) * hd;
      float dot = 0.f;
      for (int i = 0; i < hd; ++i) dot = fmaf(qs[i], to_f(kr[i]), dot);
      s = dot;
    }
    const float m_new = fmaxf(m, warp_max(s));
    const float pe = (key <= p) ? __expf(s - m_new) : 0.f;
    const float corr = __expf(m - m_new);   // m = -inf on the first chunk gives 0
    l = l * corr + warp_sum(pe);
#pragma unroll
    for (int e = 0; e < MAX_E; ++e) acc[e] *= corr;
    m = m_new;
    const int n_here = min(32, p - c0 + 1);
    for (int i = 0; i < n_here; ++i) {
      const float pi = __shfl_sync(0xffffffffu, pe, i);
      const T *vr = v + (kv_row_of(blk, blk_stride, lo, first, c0 + i) * n_kv + kvh) * hd;
#pragma unroll
      for (int e = 0; e < MAX_E; ++e) {
        const int dd = lane + 32 * e;
        if (dd < hd) acc[e] = fmaf(pi, to_f(vr[dd]), acc[e]);
      }
    }
  }
  TQ *orow = out + ((size_t)t * n_q + h) * hd;
  const float inv = 1.f / l;
#pragma unroll
  for (int e = 0; e < MAX_E; ++e) {
    const int dd = lane + 32 * e;
    if (dd < hd) orow[dd] = from_f<TQ>(acc[e] * inv);
  }
}

template <typename TQ, typename T>
void launch_attention_simple(const TQ *q, const T *k, const T *v, TQ *out, const int32_t *cu_seqlens, int n_seqs,
                             const int32_t *k_row0, const int32_t *kv_len, const int32_t *blk, int blk_stride,
                             int n_tokens, int n_q, int n_kv, int hd, cudaStream_t st) {
  if (n_tokens <= 0) return;
  const long long items = (long long)n_tokens * n_q;
  const unsigned blocks = (unsigned)((items + 3) / 4);
  const float scale = 1.0f / sqrtf((float)hd);
  const size_t smem = 4 * hd * sizeof(float);
  if (hd <= 32) attention_simple_kernel<TQ, T, 1><<<blocks, 128, smem, st>>>(q, k, v, out, cu_seqlens, n_seqs, k_row0, kv_len, blk, blk_stride, n_tokens, n_q, n_kv, hd, scale);
  else if (hd <= 64) attention_simple_kernel<TQ, T, 2><<<blocks, 128, smem, st>>>(q, k, v, out, cu_seqlens, n_seqs, k_row0, kv_len, blk, blk_stride, n_tokens, n_q, n_kv, hd, scale);
  else if (hd <= 128) attention_simple_kernel<TQ, T, 4><<<blocks, 128, smem, st>>>(q, k, v, out, cu_seqlens, n_seqs, k_row0, kv_len, blk, blk_stride, n_tokens, n_q, n_kv, hd, scale);
  else attention_simple_kernel<TQ, T, 8><<<blocks, 128, smem, st>>>(q, k, v, out, cu_seqlens, n_seqs, k_row0, kv_len, blk, blk_stride, n_tokens, n_q, n_kv, hd, scale);
}
template void launch_attention_simple<float, float>(const float *, const float *, const float *, float *, const int32_t *, int,
                                                    const int32_t *, const int32_t *, const int32_t *, int, int, int, int, int, cudaStream_t);
template void launch_attention_simple<bf16, bf16>(const bf16 *, const bf16 *, const bf16 *, bf16 *, const int32_t *, int,
                                                  const int32_t *, const int32_t *, const int32_t *, int, int, int, int, int, cudaStream_t);
template void launch_attention_simple<__half, bf16>(const __half *, const bf16 *, const bf16 *, __half *, const int32_t *, int,
                                                    const int32_t *, const int32_t *, const int32_t *, int, int, int, int, int, cudaStream_t);

}  // namespace skv
