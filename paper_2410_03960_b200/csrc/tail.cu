// The last-token path of SwiftKV prefill: only the last token of each prompt runs layers l+1..L (footnote of
// Sec. 3.2; Sec. 3.5), so every projection here has at most a handful of rows and is bound by streaming the
// weights from HBM exactly once, and attention is one query per (prompt, head) over the cache that the
// SingleInputKV projection filled.
#include "common.cuh"

namespace skv {

// ---------------------------------------------------------------------------------------------------------
// skinny GEMM: out[b, n] = sum_k act[b, k] * W[n, k] for b < n_rows <= 8.  One warp per output feature:
// the lanes stream W's row with 128-bit loads (each byte of W is read once), the few activation rows come
// from L1/L2, fp32 accumulation, warp-shuffle reduction.
// ---------------------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) skinny_gemm_kernel(const T *__restrict__ act, const T *__restrict__ W,
                                                          int n_rows, int N, int K, OutDesc out) {
  constexpr int V = 16 / sizeof(T);
  const int lane = threadIdx.x & 31;
  const int warps_total = gridDim.x * (blockDim.x >> 5);
  const bool vec = (K % V) == 0;
  for (int n = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); n < N; n += warps_total) {
    float acc[MAX_TAIL_ROWS];
#pragma unroll
    for (int r = 0; r < MAX_TAIL_ROWS; ++r) acc[r] = 0.f;
    const T *wr = W + (size_t)n * K;
    if (vec) {
      for (int k = lane * V; k < K; k += 32 * V) {
        const uint4 wraw = __ldcs(reinterpret_cast<const uint4 *>(wr + k));   // streamed once: evict first
        const T *we = reinterpret_cast<const T *>(&wraw);
        float wf[V];
#pragma unroll
        for (int i = 0; i < V; ++i) wf[i] = to_f(we[i]);
#pragma unroll
        for (int r = 0; r < MAX_TAIL_ROWS; ++r) {
          if (r < n_rows) {
            const uint4 araw = *reinterpret_cast<const uint4 *>(act + (size_t)r * K + k);
            const T *ae = reinterpret_cast<const T *>(&araw);
#pragma unroll
            for (int i = 0; i < V; ++i) acc[r] = fmaf(wf[i], to_f(ae[i]), acc[r]);
          }
        }
      }
    } else {
      for (int k = lane; k < K; k += 32) {
        const float w = to_f(wr[k]);
#pragma unroll
        for (int r = 0; r < MAX_TAIL_ROWS; ++r)
          if (r < n_rows) acc[r] = fmaf(w, to_f(act[(size_t)r * K + k]), acc[r]);
      }
    }
#pragma unroll
    for (int r = 0; r < MAX_TAIL_ROWS; ++r) {
      if (r < n_rows) {
        const float s = warp_sum(acc[r]);
        if (lane == 0) store_out<T>(out, r, n, s);
      }
    }
  }
}

template <typename T>
void launch_skinny_gemm(const T *act, const T *W, int n_rows, int N, int K, OutDesc out, cudaStream_t st) {
  if (n_rows <= 0 || N <= 0) return;
  int blocks = (N + 7) / 8;
  if (blocks > 148 * 8) blocks = 148 * 8;
  skinny_gemm_kernel<T><<<blocks, 256, 0, st>>>(act, W, n_rows, N, K, out);
}
template void launch_skinny_gemm<float>(const float *, const float *, int, int, int, OutDesc, cudaStream_t);
template void launch_skinny_gemm<bf16>(const bf16 *, const bf16 *, int, int, int, OutDesc, cudaStream_t);

// ---------------------------------------------------------------------------------------------------------
// single-query attention over the cache, split along the keys.
//   pass 1: block (split, head, prompt) scans its key range with 4 warps (online softmax as in the
//           prefill kernel), merges the warps in shared memory and writes (max, sum, acc[hd]) to scratch;
//   pass 2: block (head, prompt) merges the splits and writes the normalised output row.
// ---------------------------------------------------------------------------------------------------------
constexpr int TAIL_WARPS = 4;

__host__ __device__ inline int tail_chunk(int max_seq_len) {
  int c = (max_seq_len + 63) / 64;          // at most 64 splits
  c = (c + 31) / 32 * 32;
  return c < 256 ? 256 : c;
}

template <typename T, int MAX_E>
__global__ void __launch_bounds__(TAIL_WARPS * 32) tail_attention_partial_kernel(
    const T *__restrict__ q, const T *__restrict__ kc, const T *__restrict__ vc, const int32_t *__restrict__ cu,
    int n_q, int n_kv, int hd, int chunk, int n_splits, float scale, float *__restrict__ scratch) {
  extern __shared__ float sm[];   // q[hd] | per-warp (m, l) [2*TAIL_WARPS] | per-warp acc [TAIL_WARPS*hd]
  float *qs = sm;
  float *ml = sm + hd;
  float *accs = ml + 2 * TAIL_WARPS;
  const int split = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int first = cu[b], n = cu[b + 1] - cu[b];
  const int kvh = h / (n_q / n_kv);
  const int k_begin = split * chunk, k_end = min(n, k_begin + chunk);
  const T *qr = q + ((size_t)b * n_q + h) * hd;
  for (int i = threadIdx.x; i < hd; i += blockDim.x) qs[i] = to_f(qr[i]) * scale;
  __syncthreads();

  float m = -INFINITY, l = 0.f;
  float acc[MAX_E];
#pragma unroll
  for (int e = 0; e < MAX_E; ++e) acc[e] = 0.f;
  for (int c0 = k_begin + warp * 32; c0 < k_end; c0 += TAIL_WARPS * 32) {
    const int key = c0 + lane;
    float s = -INFINITY;
    if (key < k_end) {
      const T *kr = kc + ((size_t)(first + key) * n_kv + kvh) * hd;
      float dot = 0.f;
      for (int i = 0; i < hd; ++i) dot = fmaf(qs[i], to_f(kr[i]), dot);
      s = dot;
    }
    const float m_new = fmaxf(m, warp_max(s));
    const float pe = (key < k_end) ? __expf(s - m_new) : 0.f;
    const float corr = __expf(m - m_new);
    l = l * corr + warp_sum(pe);
#pragma unroll
    for (int e = 0; e < MAX_E; ++e) acc[e] *= corr;
    m = m_new;
    const int n_here = min(32, k_end - c0);
    for (int i = 0; i < n_here; ++i) {
      const float pi = __shfl_sync(0xffffffffu, pe, i);
      const T *vr = vc + ((size_t)(first + c0 + i) * n_kv + kvh) * hd;
#pragma unroll
      for (int e = 0; e < MAX_E; ++e) {
        const int dd = lane + 32 * e;
        if (dd < hd) acc[e] = fmaf(pi, to_f(vr[dd]), acc[e]);
      }
    }
  }
  if (lane == 0) { ml[2 * warp] = m; ml[2 * warp + 1] = l; }
#pragma unroll
  for (int e = 0; e < MAX_E; ++e) {
    const int dd = lane + 32 * e;
    if (dd < hd) accs[warp * hd + dd] = acc[e];
  }
  __syncthreads();
  float M = -INFINITY;
#pragma unroll
  for (int w = 0; w < TAIL_WARPS; ++w) M = fmaxf(M, ml[2 * w]);
  float *dst = scratch + (((size_t)b * n_q + h) * n_splits + split) * (hd + 2);
  float Lsum = 0.f;
#pragma unroll
  for (int w = 0; w < TAIL_WARPS; ++w) Lsum += (ml[2 * w] == -INFINITY) ? 0.f : ml[2 * w + 1] * __expf(ml[2 * w] - M);
  if (threadIdx.x == 0) { dst[0] = M; dst[1] = Lsum; }
  for (int dd = threadIdx.x; dd < hd; dd += blockDim.x) {
    float a = 0.f;
#pragma unroll
    for (int w = 0; w < TAIL_WARPS; ++w) a += (ml[2 * w] == -INFINITY) ? 0.f : accs[w * hd + dd] * __expf(ml[2 * w] - M);
    dst[2 + dd] = a;
  }
}

template <typename T>
__global__ void tail_attention_merge_kernel(const float *__restrict__ scratch, T *__restrict__ out, int n_q, int hd,
                                            int n_splits) {
  const int h = blockIdx.x, b = blockIdx.y;
  const float *src = scratch + ((size_t)b * n_q + h) * n_splits * (hd + 2);
  float M = -INFINITY;
  for (int s = 0; s < n_splits; ++s) M = fmaxf(M, src[(size_t)s * (hd + 2)]);
  float L = 0.f;
  for (int s = 0; s < n_splits; ++s) {
    const float ms = src[(size_t)s * (hd + 2)];
    L += (ms == -INFINITY) ? 0.f : src[(size_t)s * (hd + 2) + 1] * __expf(ms - M);
  }
  for (int dd = threadIdx.x; dd < hd; dd += blockDim.x) {
    float a = 0.f;
    for (int s = 0; s < n_splits; ++s) {
      const float ms = src[(size_t)s * (hd + 2)];
      if (ms != -INFINITY) a += src[(size_t)s * (hd + 2) + 2 + dd] * __expf(ms - M);
    }
    out[((size_t)b * n_q + h) * hd + dd] = from_f<T>(a / L);
  }
}

size_t tail_attention_scratch_bytes(int max_seqs, int n_q, int hd, int max_tokens) {
  const int chunk = tail_chunk(max_tokens);
  const int n_splits = (max_tokens + chunk - 1) / chunk;
  return (size_t)max_seqs * n_q * n_splits * (hd + 2) * sizeof(float);
}

template <typename T>
void launch_tail_attention(const T *q, const T *kc, const T *vc, T *out, const int32_t *cu_seqlens, int n_seqs,
                           int max_seq_len, int n_q, int n_kv, int hd, float *scratch, cudaStream_t st) {
  if (n_seqs <= 0) return;
  const int chunk = tail_chunk(max_seq_len);
  const int n_splits = (max_seq_len + chunk - 1) / chunk;
  const float scale = 1.0f / sqrtf((float)hd);
  const size_t smem = (size_t)(hd + 2 * TAIL_WARPS + TAIL_WARPS * hd) * sizeof(float);
  dim3 grid(n_splits, n_q, n_seqs);
  if (hd <= 32) tail_attention_partial_kernel<T, 1><<<grid, TAIL_WARPS * 32, smem, st>>>(q, kc, vc, cu_seqlens, n_q, n_kv, hd, chunk, n_splits, scale, scratch);
  else if (hd <= 64) tail_attention_partial_kernel<T, 2><<<grid, TAIL_WARPS * 32, smem, st>>>(q, kc, vc, cu_seqlens, n_q, n_kv, hd, chunk, n_splits, scale, scratch);
  else if (hd <= 128) tail_attention_partial_kernel<T, 4><<<grid, TAIL_WARPS * 32, smem, st>>>(q, kc, vc, cu_seqlens, n_q, n_kv, hd, chunk, n_splits, scale, scratch);
  else tail_attention_partial_kernel<T, 8><<<grid, TAIL_WARPS * 32, smem, st>>>(q, kc, vc, cu_seqlens, n_q, n_kv, hd, chunk, n_splits, scale, scratch);
  tail_attention_merge_kernel<T><<<dim3(n_q, n_seqs), 128, 0, st>>>(scratch, out, n_q, hd, n_splits);
}
template void launch_tail_attention<float>(const float *, const float *, const float *, float *, const int32_t *, int,
                                           int, int, int, int, float *, cudaStream_t);
template void launch_tail_attention<bf16>(const bf16 *, const bf16 *, const bf16 *, bf16 *, const int32_t *, int, int,
                                          int, int, int, float *, cudaStream_t);

}  // namespace skv
