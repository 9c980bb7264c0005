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

// 16-bit rows whose width is a multiple of 8 and at most 32 * 8 * VEC_CHUNKS: one warp per row, every lane keeps its
// elements in registers between the maximum and the conversion (128-bit loads, 64-bit code stores, no block barrier)
constexpr int VEC_CHUNKS = 8;
constexpr int VEC_ROWS = 8;      // rows (warps) per block
template <typename TO, int CHUNKS>
__global__ void __launch_bounds__(VEC_ROWS * 32) quantize_rows_vec_kernel(const bf16 *__restrict__ src, int rows, int width,
                                                                         const int32_t *__restrict__ slot_map,
                                                                         uint8_t *__restrict__ codes, float *__restrict__ scale_out,
                                                                         TO *__restrict__ deq) {
  const int r = blockIdx.x * VEC_ROWS + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (r >= rows) return;
  const uint4 *x = reinterpret_cast<const uint4 *>(src + (size_t)r * width);
  const int n_vec = width >> 3;
  uint4 raw[CHUNKS];
  float amax = 0.f;
#pragma unroll
  for (int c = 0; c < CHUNKS; ++c) {
    const int i = lane + c * 32;
    if (i < n_vec) {
      raw[c] = __ldcs(x + i);
      const bf16 *e = reinterpret_cast<const bf16 *>(&raw[c]);
#pragma unroll
      for (int k = 0; k < 8; ++k) amax = fmaxf(amax, fabsf(__bfloat162float(e[k])));
    }
  }
  amax = warp_max(amax);
  const float scale = __fdiv_rn(fmaxf(amax, FP8_AMAX_FLOOR), FP8_MAX);
  const size_t orow = slot_map ? (size_t)slot_map[r] : (size_t)r;
  if (lane == 0) scale_out[orow] = scale;
  uint2 *c_out = reinterpret_cast<uint2 *>(codes + orow * width);
#pragma unroll
  for (int c = 0; c < CHUNKS; ++c) {
    const int i = lane + c * 32;
    if (i < n_vec) {
      const bf16 *e = reinterpret_cast<const bf16 *>(&raw[c]);
      uint8_t q[8];
      TO d[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        q[k] = encode_e4m3(__bfloat162float(e[k]), scale);
        d[k] = from_f<TO>(__fmul_rn(to_f(fp8e4{q[k]}), scale));
      }
      c_out[i] = *reinterpret_cast<const uint2 *>(q);
      if (deq) reinterpret_cast<uint4 *>(deq + (size_t)r * width)[i] = *reinterpret_cast<const uint4 *>(d);
    }
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

// A decode minibatch's new K / V rows (fp32, one row per sequence) into the FP8 cache in one pass: rotary embedding on K (the
// arithmetic of rope_kernel), rounding to the model dtype (the cache is defined as the quantized model-dtype row), per-row
// scale and codes (the arithmetic of quantize_rows_kernel).  Block (row, K or V); the rounded row waits in shared memory
// between the maximum and the encoding.
template <typename T>
__global__ void __launch_bounds__(QT) store_kv_rows_fp8_kernel(const float *__restrict__ ky, const float *__restrict__ vy,
                                                               const int32_t *__restrict__ slot_map, const int32_t *__restrict__ positions,
                                                               const float *__restrict__ cos_tab, const float *__restrict__ sin_tab,
                                                               int n_heads, int hd, uint8_t *__restrict__ k_codes,
                                                               float *__restrict__ k_scale, uint8_t *__restrict__ v_codes,
                                                               float *__restrict__ v_scale) {
  extern __shared__ float row_s[];
  __shared__ float red[QT / 32];
  const int r = blockIdx.x, width = n_heads * hd, half = hd >> 1;
  const bool is_v = blockIdx.y != 0;
  const float *src = (is_v ? vy : ky) + (size_t)r * width;
  float amax = 0.f;
  if (!is_v) {
    const int p = positions[r];
    for (int idx = threadIdx.x; idx < n_heads * half; idx += QT) {
      const int h = idx / half, i = idx % half;
      const float c = cos_tab[(size_t)p * half + i], s = sin_tab[(size_t)p * half + i];
      const float a = src[h * hd + i], b = src[h * hd + i + half];
      const float x0 = to_f(from_f<T>(a * c - b * s)), x1 = to_f(from_f<T>(b * c + a * s));
      row_s[h * hd + i] = x0;
      row_s[h * hd + i + half] = x1;
      amax = fmaxf(amax, fmaxf(fabsf(x0), fabsf(x1)));
    }
  } else {
    for (int i = threadIdx.x; i < width; i += QT) {
      const float x = to_f(from_f<T>(src[i]));
      row_s[i] = x;
      amax = fmaxf(amax, fabsf(x));
    }
  }
  amax = block_max(amax, red);      // (its barrier also publishes row_s)
  const float scale = __fdiv_rn(fmaxf(amax, FP8_AMAX_FLOOR), FP8_MAX);
  const size_t orow = (size_t)slot_map[r];
  if (threadIdx.x == 0) (is_v ? v_scale : k_scale)[orow] = scale;
  uint8_t *c = (is_v ? v_codes : k_codes) + orow * width;
  for (int i = threadIdx.x; i < width; i += QT) c[i] = encode_e4m3(row_s[i], scale);
}

}  // namespace

template <typename T>
void launch_store_kv_rows_fp8(const float *ky, const float *vy, const int32_t *slot_map, const int32_t *positions, const float *cos_tab,
                              const float *sin_tab, int rows, int n_heads, int hd, uint8_t *k_codes, float *k_scale, uint8_t *v_codes,
                              float *v_scale, cudaStream_t st) {
  if (rows <= 0) return;
  store_kv_rows_fp8_kernel<T><<<dim3((unsigned)rows, 2), QT, (size_t)n_heads * hd * sizeof(float), st>>>(
      ky, vy, slot_map, positions, cos_tab, sin_tab, n_heads, hd, k_codes, k_scale, v_codes, v_scale);
}
template void launch_store_kv_rows_fp8<bf16>(const float *, const float *, const int32_t *, const int32_t *, const float *, const float *, int,
                                             int, int, uint8_t *, float *, uint8_t *, float *, cudaStream_t);
template void launch_store_kv_rows_fp8<float>(const float *, const float *, const int32_t *, const int32_t *, const float *, const float *, int,
                                              int, int, uint8_t *, float *, uint8_t *, float *, cudaStream_t);

template <typename TI, typename TO>
void launch_quantize_rows_fp8(const TI *src, int rows, int width, const int32_t *slot_map, uint8_t *codes, float *scale,
                              TO *deq, cudaStream_t st) {
  if (rows <= 0) return;
  if constexpr (sizeof(TI) == 2 && sizeof(TO) == 2) {
    const bool aligned = ((reinterpret_cast<uintptr_t>(src) | reinterpret_cast<uintptr_t>(deq)) & 15) == 0 &&
                         (reinterpret_cast<uintptr_t>(codes) & 7) == 0;
    if (width % 8 == 0 && width <= 32 * 8 * VEC_CHUNKS && aligned) {
      const int blocks = (rows + VEC_ROWS - 1) / VEC_ROWS;
      if (width <= 32 * 8 * 4) quantize_rows_vec_kernel<TO, 4><<<blocks, VEC_ROWS * 32, 0, st>>>(src, rows, width, slot_map, codes, scale, deq);
      else quantize_rows_vec_kernel<TO, VEC_CHUNKS><<<blocks, VEC_ROWS * 32, 0, st>>>(src, rows, width, slot_map, codes, scale, deq);
      return;
    }
  }
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
