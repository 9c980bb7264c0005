// Per-token FP8 (e4m3) KV-cache rows: quantization of freshly projected K / V rows into the cache, and dequantized
// packed copies for the attention kernels (the paper's appendix on KV quantization combines SwiftKV / AcrossKV with a
// per-token FP8 cache).  Both kernels are bandwidth-bound row passes: one block per (row, plane).
#include "common.cuh"

namespace skv {
namespace {

constexpr int QT = 128;   // threads per row

__device__ __forceinline__ float block_max(float v, float *red) {
  v = warp_max(v);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  float m = red[0];
#pragma unroll
  for (int w = 1; w < QT / 32; ++w) m = fmaxf(m, red[w]);
  return m;
}

// every arithmetic step that decides a code is a single correctly rounded fp32 operation
__device__ __forceinline__ uint8_t encode_e4m3(float x, float scale) {
  return (uint8_t)__nv_cvt_float_to_fp8(__fdiv_rn(x, scale), __NV_SATFINITE, __NV_E4M3);
}

template <typename TI, typename TO>
__global__ void __launch_bounds__(QT) quantize_rows_kernel(const TI *__restrict__ src, int width,
                                                           const int32_t *__restrict__ slot_map, uint8_t *__restrict__ codes,
                                                           float *__restrict__ scale_out, TO *__restrict__ deq) {
  __shared__ float red[QT / 32];
  const int r = blockIdx.x;
  const TI *x = src + (size_t)r * width;
  float amax = 0.f;
  for (int i = threadIdx.x; i < width; i += QT) amax = fmaxf(amax, fabsf(to_f(x[i])));
  amax = block_max(amax, red);
  const float scale = __fdiv_rn(fmaxf(amax, FP8_AMAX_FLOOR), FP8_MAX);
  const size_t orow = slot_map ? (size_t)slot_map[r] : (size_t)r;
  if (threadIdx.x == 0) scale_out[orow] = scale;
  uint8_t *c = codes + orow * width;
  for (int i = threadIdx.x; i < width; i += QT) {
    const uint8_t code = encode_e4m3(to_f(x[i]), scale);
    c[i] = code;
    if (deq) deq[(size_t)r * width + i] = from_f<TO>(__fmul_rn(to_f(fp8e4{code}), scale));
  }
}

template <typename TO>
__global__ void __launch_bounds__(QT) gather_dequant_kernel(const uint8_t *__restrict__ k_codes, const uint8_t *__restrict__ v_codes,
                                                            const float *__restrict__ k_scale, const float *__restrict__ v_scale,
                                                            TO *__restrict__ k_out, TO *__restrict__ v_out,
                                                            const int32_t *__restrict__ row0, const int32_t *__restrict__ len,
                                                            const int32_t *__restrict__ kcu, const int32_t *__restrict__ blk,
                                                            int blk_stride, int dkv) {
  const int b = blockIdx.y, p = blockIdx.x;
  if (p >= len[b]) return;
  const size_t row = kv_row_of(blk, blk_stride, b, row0[b], p);
  const size_t orow = (size_t)kcu[b] + p;
  const bool is_v = blockIdx.z != 0;
  const uint8_t *c = (is_v ? v_codes : k_codes) + row * dkv;
  const float s = (is_v ? v_scale : k_scale)[row];
  TO *o = (is_v ? v_out : k_out) + orow * dkv;
  for (int i = threadIdx.x; i < dkv; i += QT) o[i] = from_f<TO>(__fmul_rn(to_f(fp8e4{c[i]}), s));
}

}  // namespace

template <typename TI, typename TO>
void launch_quantize_rows_fp8(const TI *src, int rows, int width, const int32_t *slot_map, uint8_t *codes, float *scale,
                              TO *deq, cudaStream_t st) {
  if (rows <= 0) return;
  quantize_rows_kernel<TI, TO><<<rows, QT, 0, st>>>(src, width, slot_map, codes, scale, deq);
}
template void launch_quantize_rows_fp8<float, float>(const float *, int, int, const int32_t *, uint8_t *, float *, float *, cudaStream_t);
template void launch_quantize_rows_fp8<bf16, bf16>(const bf16 *, int, int, const int32_t *, uint8_t *, float *, bf16 *, cudaStream_t);
template void launch_quantize_rows_fp8<bf16, __half>(const bf16 *, int, int, const int32_t *, uint8_t *, float *, __half *, cudaStream_t);

template <typename TO>
void launch_gather_dequant_fp8(const uint8_t *k_codes, const uint8_t *v_codes, const float *k_scale, const float *v_scale,
                               TO *k_out, TO *v_out, const int32_t *row0, const int32_t *len, const int32_t *kcu,
                               const int32_t *blk, int blk_stride, int n_seqs, int max_len, int dkv, cudaStream_t st) {
  if (n_seqs <= 0 || max_len <= 0) return;
  gather_dequant_kernel<TO><<<dim3(max_len, n_seqs, 2), QT, 0, st>>>(k_codes, v_codes, k_scale, v_scale, k_out, v_out, row0, len,
                                                                      kcu, blk, blk_stride, dkv);
}
template void launch_gather_dequant_fp8<float>(const uint8_t *, const uint8_t *, const float *, const float *, float *, float *,
                                               const int32_t *, const int32_t *, const int32_t *, const int32_t *, int, int, int,
                                               int, cudaStream_t);
template void launch_gather_dequant_fp8<bf16>(const uint8_t *, const uint8_t *, const float *, const float *, bf16 *, bf16 *,
                                              const int32_t *, const int32_t *, const int32_t *, const int32_t *, int, int, int,
                                              int, cudaStream_t);
template void launch_gather_dequant_fp8<__half>(const uint8_t *, const uint8_t *, const float *, const float *, __half *, __half *,
                                                const int32_t *, const int32_t *, const int32_t *, const int32_t *, int, int, int,
                                                int, cudaStream_t);

}  // namespace skv
