// Memory-bound kernels of the SwiftKV prefill path: embedding gather, RMSNorm, rotary embedding, SwiGLU,
// last-token gather, RoPE table, and the one-time gain fold of the SingleInputKV weight (Sec. 3.5).
// All use 128-bit global accesses where the row length allows and warp-shuffle reductions.
#include <type_traits>

#include "common.cuh"

namespace skv {

// a thread's running "had to clamp a half store" note: `hit` collects, `report` raises the status bit once per thread
template <typename T>
__device__ __forceinline__ void note_overflow(float v, bool &hit) {
  if constexpr (std::is_same<T, __half>::value) hit |= fabsf(v) >= HALF_OVERFLOW;
}
__device__ __forceinline__ void report_overflow(bool hit, unsigned int *status) {
  if (hit && status) atomicOr(status, STATUS_ACT_OVERFLOW);
}

// ---------------------------------------------------------------------------------------------------------
// embedding gather: x[t, :] = float(E[tok[t], :])      (Sec. 3.1: X are the input embeddings)
// ---------------------------------------------------------------------------------------------------------
template <typename T>
__global__ void embed_kernel(const T *__restrict__ embed, const int32_t *__restrict__ tokens, float *__restrict__ x,
                             int d, int vocab, unsigned int *status) {
  const int t = blockIdx.x;
  int id = tokens[t];
  if (id < 0 || id >= vocab) {
    if (threadIdx.x == 0) atomicOr(status, STATUS_BAD_TOKEN);
    id = min(max(id, 0), vocab - 1);
  }
  const T *src = embed + (size_t)id * d;
  float *dst = x + (size_t)t * d;
  if constexpr (sizeof(T) == 2) {
    if ((d & 7) == 0) {
      for (int i = threadIdx.x * 8; i < d; i += blockDim.x * 8) {
        uint4 raw = *reinterpret_cast<const uint4 *>(src + i);
        const bf16 *e = reinterpret_cast<const bf16 *>(&raw);
        float4 a = make_float4(to_f(e[0]), to_f(e[1]), to_f(e[2]), to_f(e[3]));
        float4 b = make_float4(to_f(e[4]), to_f(e[5]), to_f(e[6]), to_f(e[7]));
        *reinterpret_cast<float4 *>(dst + i) = a;
        *reinterpret_cast<float4 *>(dst + i + 4) = b;
      }
      return;
    }
  }
  for (int i = threadIdx.x; i < d; i += blockDim.x) dst[i] = to_f(src[i]);
}

template <typename T>
void launch_embed(const T *embed, const int32_t *tokens, float *x, int n_tokens, int d, int vocab,
                  unsigned int *status, cudaStream_t st) {
  if (n_tokens <= 0) return;
  embed_kernel<T><<<n_tokens, 128, 0, st>>>(embed, tokens, x, d, vocab, status);
}
template void launch_embed<float>(const float *, const int32_t *, float *, int, int, int, unsigned int *, cudaStream_t);
template void launch_embed<bf16>(const bf16 *, const int32_t *, float *, int, int, int, unsigned int *, cudaStream_t);

// ---------------------------------------------------------------------------------------------------------
// positions[t] = t - cu_seqlens[b(t)]  (positions restart at 0 for each prompt); last_idx[b] = cu[b+1]-1
// ---------------------------------------------------------------------------------------------------------
__global__ void positions_kernel(const int32_t *__restrict__ cu, int n_seqs, int32_t *__restrict__ pos,
                                 int32_t *__restrict__ last_idx, int n_tokens) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t < n_seqs) last_idx[t] = cu[t + 1] - 1;
  if (t >= n_tokens) return;
  int lo = 0, hi = n_seqs;   // find b with cu[b] <= t < cu[b+1]
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (cu[mid] <= t) lo = mid; else hi = mid;
  }
  pos[t] = t - cu[lo];
}
void launch_positions(const int32_t *cu_seqlens, int n_seqs, int32_t *positions, int32_t *last_idx, int n_tokens,
                      cudaStream_t st) {
  const int n = n_tokens > n_seqs ? n_tokens : n_seqs;
  positions_kernel<<<(n + 255) / 256, 256, 0, st>>>(cu_seqlens, n_seqs, positions, last_idx, n_tokens);
}

// ---------------------------------------------------------------------------------------------------------
// RMSNorm: out = x / sqrt(mean(x^2) + eps) * gamma, one block per row, fp32 statistics.
// The residual stream x is fp32; the output is the model dtype.  gamma == nullptr gives the unit-rms row that
// feeds the gain-folded SingleInputKV projection (one statistic shared by every later layer).
// ---------------------------------------------------------------------------------------------------------
template <typename TG, typename T>
__global__ void __launch_bounds__(256) rmsnorm_kernel(const float *__restrict__ x, const TG *__restrict__ gamma,
                                                      T *__restrict__ out, int d, float eps, unsigned int *status, int split) {
  bool hit = false;
  const size_t row = blockIdx.x;
  const float *xr = x + row * d;
  // split (IEEE-half output only): the row is written as [hi(d) | lo(d)], lo = what the rounding to half left over
  T *orow = out + row * d * (split ? 2 : 1);
  __shared__ float red[8];
  float ss = 0.f;
  const bool vec = (d & 3) == 0;
  if (vec) {
    for (int i = threadIdx.x * 4; i < d; i += blockDim.x * 4) {
      const float4 v = *reinterpret_cast<const float4 *>(xr + i);
      ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
    }
  } else {
    for (int i = threadIdx.x; i < d; i += blockDim.x) ss += xr[i] * xr[i];
  }
  ss = warp_sum(ss);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int w = 0; w < 8; ++w) tot += (w < (blockDim.x >> 5)) ? red[w] : 0.f;
  const float rstd = rsqrtf(tot / (float)d + eps);
  if (vec) {
    for (int i = threadIdx.x * 4; i < d; i += blockDim.x * 4) {
      const float4 v = *reinterpret_cast<const float4 *>(xr + i);   // second read hits L1/L2
      float g0 = 1.f, g1 = 1.f, g2 = 1.f, g3 = 1.f;
      if (gamma) { g0 = to_f(gamma[i]); g1 = to_f(gamma[i + 1]); g2 = to_f(gamma[i + 2]); g3 = to_f(gamma[i + 3]); }
      if constexpr (sizeof(T) == 2) {
        const float y0 = v.x * rstd * g0, y1 = v.y * rstd * g1, y2 = v.z * rstd * g2, y3 = v.w * rstd * g3;
        note_overflow<T>(y0, hit); note_overflow<T>(y1, hit); note_overflow<T>(y2, hit); note_overflow<T>(y3, hit);
        T o4[4] = {from_f<T>(y0), from_f<T>(y1), from_f<T>(y2), from_f<T>(y3)};
        *reinterpret_cast<uint2 *>(orow + i) = *reinterpret_cast<uint2 *>(o4);
        if (split) {
          T l4[4] = {from_f<T>(y0 - to_f(o4[0])), from_f<T>(y1 - to_f(o4[1])), from_f<T>(y2 - to_f(o4[2])), from_f<T>(y3 - to_f(o4[3]))};
          *reinterpret_cast<uint2 *>(orow + d + i) = *reinterpret_cast<uint2 *>(l4);
        }
      } else {
        *reinterpret_cast<float4 *>(orow + i) = make_float4(v.x * rstd * g0, v.y * rstd * g1, v.z * rstd * g2, v.w * rstd * g3);
      }
    }
  } else {
    for (int i = threadIdx.x; i < d; i += blockDim.x) {
      const float y = xr[i] * rstd * (gamma ? to_f(gamma[i]) : 1.f);
      note_overflow<T>(y, hit);
      orow[i] = from_f<T>(y);
      if (split) orow[d + i] = from_f<T>(y - to_f(orow[i]));
    }
  }
  report_overflow(hit, status);
}
// Rows of exactly 256 * 4 * NV floats (4096: NV = 4, 8192: NV = 8) with 16-bit output: each thread keeps its NV float4
// in registers between the sum of squares and the scaling, so the row is read from global memory exactly once.
template <typename TG, typename T, int NV, bool SPLIT>
__global__ void __launch_bounds__(256) rmsnorm_reg_kernel(const float *__restrict__ x, const TG *__restrict__ gamma,
                                                          T *__restrict__ out, float eps, unsigned int *status) {
  bool hit = false;
  constexpr int D = 256 * 4 * NV;
  const size_t row = blockIdx.x;
  const float4 *xr = reinterpret_cast<const float4 *>(x + row * D);
  __shared__ float red[8];
  float4 v[NV];
  float ss = 0.f;
#pragma unroll
  for (int k = 0; k < NV; ++k) {
    v[k] = xr[threadIdx.x + 256 * k];
    ss += v[k].x * v[k].x + v[k].y * v[k].y + v[k].z * v[k].z + v[k].w * v[k].w;
  }
  ss = warp_sum(ss);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int w = 0; w < 8; ++w) tot += red[w];
  const float rstd = rsqrtf(tot / (float)D + eps);
  uint2 *orow = reinterpret_cast<uint2 *>(out + row * D * (SPLIT ? 2 : 1));
#pragma unroll
  for (int k = 0; k < NV; ++k) {
    const int i4 = threadIdx.x + 256 * k;
    float g0 = 1.f, g1 = 1.f, g2 = 1.f, g3 = 1.f;
    if (gamma) {
      const uint2 graw = *reinterpret_cast<const uint2 *>(gamma + 4 * i4);       // TG is a 16-bit type here
      const TG *g = reinterpret_cast<const TG *>(&graw);
      g0 = to_f(g[0]); g1 = to_f(g[1]); g2 = to_f(g[2]); g3 = to_f(g[3]);
    }
    const float y0 = v[k].x * rstd * g0, y1 = v[k].y * rstd * g1, y2 = v[k].z * rstd * g2, y3 = v[k].w * rstd * g3;
    note_overflow<T>(y0, hit); note_overflow<T>(y1, hit); note_overflow<T>(y2, hit); note_overflow<T>(y3, hit);
    T o4[4] = {from_f<T>(y0), from_f<T>(y1), from_f<T>(y2), from_f<T>(y3)};
    orow[i4] = *reinterpret_cast<uint2 *>(o4);
    if constexpr (SPLIT) {           // [hi(D) | lo(D)]: the low halves follow the row's high halves
      T l4[4] = {from_f<T>(y0 - to_f(o4[0])), from_f<T>(y1 - to_f(o4[1])), from_f<T>(y2 - to_f(o4[2])), from_f<T>(y3 - to_f(o4[3]))};
      orow[D / 4 + i4] = *reinterpret_cast<uint2 *>(l4);
    }
  }
  report_overflow(hit, status);
}
template <typename TG, typename TO>
void launch_rmsnorm(const float *x, const TG *gamma, TO *out, int rows, int d, float eps, cudaStream_t st, unsigned int *status,
                    bool split) {
  if (rows <= 0) return;
  if constexpr (!std::is_same<TO, __half>::value) split = false;      // hi + lo pairs exist for IEEE halves only
  if constexpr (sizeof(TG) == 2 && sizeof(TO) == 2) {
    if constexpr (std::is_same<TO, __half>::value) {
      if (split && d == 4096) { rmsnorm_reg_kernel<TG, TO, 4, true><<<rows, 256, 0, st>>>(x, gamma, out, eps, status); return; }
      if (split && d == 8192) { rmsnorm_reg_kernel<TG, TO, 8, true><<<rows, 256, 0, st>>>(x, gamma, out, eps, status); return; }
    }
    if (!split && d == 4096) { rmsnorm_reg_kernel<TG, TO, 4, false><<<rows, 256, 0, st>>>(x, gamma, out, eps, status); return; }
    if (!split && d == 8192) { rmsnorm_reg_kernel<TG, TO, 8, false><<<rows, 256, 0, st>>>(x, gamma, out, eps, status); return; }
  }
  rmsnorm_kernel<TG, TO><<<rows, 256, 0, st>>>(x, gamma, out, d, eps, status, split ? 1 : 0);
}
template void launch_rmsnorm<float, float>(const float *, const float *, float *, int, int, float, cudaStream_t, unsigned int *, bool);
template void launch_rmsnorm<bf16, bf16>(const float *, const bf16 *, bf16 *, int, int, float, cudaStream_t, unsigned int *, bool);
template void launch_rmsnorm<bf16, __half>(const float *, const bf16 *, __half *, int, int, float, cudaStream_t, unsigned int *, bool);

// ---------------------------------------------------------------------------------------------------------
// Rotary embedding, rotate-half pairing (i, i + hd/2), in place.  One thread per pair.
// ---------------------------------------------------------------------------------------------------------
template <typename T>
__global__ void rope_kernel(T *__restrict__ x, long long batch_stride, const int32_t *__restrict__ positions,
                            const int32_t *__restrict__ slot_map, const float *__restrict__ cos_tab,
                            const float *__restrict__ sin_tab, int rows, int n_heads, int hd, unsigned int *status) {
  const int half = hd >> 1;
  const long long per_row = (long long)n_heads * half;
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= per_row * rows) return;
  const int row = (int)(idx / per_row);
  const int rem = (int)(idx % per_row);
  const int h = rem / half, i = rem % half;
  const int p = positions[row];
  const float c = cos_tab[(size_t)p * half + i], s = sin_tab[(size_t)p * half + i];
  const size_t trow = slot_map ? (size_t)slot_map[row] : (size_t)row;
  T *base = x + (size_t)blockIdx.y * batch_stride + (trow * n_heads + h) * hd;
  const float a = to_f(base[i]), b = to_f(base[i + half]);
  bool hit = false;
  note_overflow<T>(a * c - b * s, hit);
  note_overflow<T>(b * c + a * s, hit);
  base[i] = from_f<T>(a * c - b * s);
  base[i + half] = from_f<T>(b * c + a * s);
  report_overflow(hit, status);
}
template <typename T>
void launch_rope(T *x, long long batch_stride, int n_batches, const int32_t *positions, const int32_t *slot_map,
                 const float *cos_tab, const float *sin_tab, int rows, int n_heads, int hd, cudaStream_t st, unsigned int *status) {
  const long long n = (long long)rows * n_heads * (hd / 2);
  if (n <= 0 || n_batches <= 0) return;
  dim3 grid((unsigned)((n + 255) / 256), (unsigned)n_batches);
  rope_kernel<T><<<grid, 256, 0, st>>>(x, batch_stride, positions, slot_map, cos_tab, sin_tab, rows, n_heads, hd, status);
}
template void launch_rope<float>(float *, long long, int, const int32_t *, const int32_t *, const float *, const float *, int, int, int, cudaStream_t, unsigned int *);
template void launch_rope<bf16>(bf16 *, long long, int, const int32_t *, const int32_t *, const float *, const float *, int, int, int, cudaStream_t, unsigned int *);
template void launch_rope<__half>(__half *, long long, int, const int32_t *, const int32_t *, const float *, const float *, int, int, int, cudaStream_t, unsigned int *);

// cos/sin of p * theta^(-2i/hd), evaluated in double precision and rounded once to fp32.
__global__ void rope_table_kernel(float *cos_tab, float *sin_tab, int max_pos, int half, double log_theta, int hd) {
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (long long)max_pos * half) return;
  const int p = (int)(idx / half), i = (int)(idx % half);
  const double inv_freq = exp(-2.0 * (double)i / (double)hd * log_theta);
  double s, c;
  sincos((double)p * inv_freq, &s, &c);
  cos_tab[idx] = (float)c;
  sin_tab[idx] = (float)s;
}
void launch_rope_table(float *cos_tab, float *sin_tab, int max_pos, int hd, double theta, cudaStream_t st) {
  const long long n = (long long)max_pos * (hd / 2);
  if (n <= 0) return;
  rope_table_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(cos_tab, sin_tab, max_pos, hd / 2, log(theta), hd);
}

// ---------------------------------------------------------------------------------------------------------
// SwiGLU: out = silu(gate) * up      (Sec. 3.1 MLP; fp32 arithmetic, model-dtype storage)
// ---------------------------------------------------------------------------------------------------------
template <typename T>
__global__ void swiglu_kernel(const T *__restrict__ gate, const T *__restrict__ up, T *__restrict__ out, long long n,
                              unsigned int *status) {
  bool hit = false;
  const long long stride = (long long)gridDim.x * blockDim.x;
  constexpr int V = 16 / sizeof(T);
  const long long nv = n / V;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < nv; i += stride) {
    uint4 g = reinterpret_cast<const uint4 *>(gate)[i];
    uint4 u = reinterpret_cast<const uint4 *>(up)[i];
    uint4 o;
    const T *ge = reinterpret_cast<const T *>(&g);
    const T *ue = reinterpret_cast<const T *>(&u);
    T *oe = reinterpret_cast<T *>(&o);
#pragma unroll
    for (int k = 0; k < V; ++k) {
      const float z = to_f(ge[k]);
      const float y = z / (1.f + __expf(-z)) * to_f(ue[k]);
      note_overflow<T>(y, hit);
      oe[k] = from_f<T>(y);
    }
    reinterpret_cast<uint4 *>(out)[i] = o;
  }
  for (long long i = nv * V + (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
    const float z = to_f(gate[i]);
    const float y = z / (1.f + __expf(-z)) * to_f(up[i]);
    note_overflow<T>(y, hit);
    out[i] = from_f<T>(y);
  }
  report_overflow(hit, status);
}
template <typename T>
void launch_swiglu(const T *gate, const T *up, T *out, long long n, cudaStream_t st, unsigned int *status) {
  if (n <= 0) return;
  long long blocks = (n / (16 / sizeof(T)) + 255) / 256;
  if (blocks < 1) blocks = 1;
  if (blocks > 148 * 16) blocks = 148 * 16;
  swiglu_kernel<T><<<(unsigned)blocks, 256, 0, st>>>(gate, up, out, n, status);
}
template void launch_swiglu<float>(const float *, const float *, float *, long long, cudaStream_t, unsigned int *);
template void launch_swiglu<bf16>(const bf16 *, const bf16 *, bf16 *, long long, cudaStream_t, unsigned int *);
template void launch_swiglu<__half>(const __half *, const __half *, __half *, long long, cudaStream_t, unsigned int *);

// y[b, :] = x[idx[b], :]   (the tokens that continue past layer l: the last token of each prompt)
__global__ void gather_rows_kernel(const float *__restrict__ x, const int32_t *__restrict__ idx, float *__restrict__ y, int d) {
  const float *src = x + (size_t)idx[blockIdx.x] * d;
  float *dst = y + (size_t)blockIdx.x * d;
  for (int i = threadIdx.x; i < d; i += blockDim.x) dst[i] = src[i];
}
void launch_gather_rows(const float *x, const int32_t *idx, float *y, int n_rows, int d, cudaStream_t st) {
  if (n_rows <= 0) return;
  gather_rows_kernel<<<n_rows, 256, 0, st>>>(x, idx, y, d);
}

// fp32 rows -> rows slot_map[r] (null: r) of a plane in the cache's element type (a decode step's new K / V rows)
template <typename T>
__global__ void scatter_rows_kernel(const float *__restrict__ src, T *__restrict__ dst, const int32_t *__restrict__ slot_map,
                                    int width) {
  const size_t orow = slot_map ? (size_t)slot_map[blockIdx.x] : (size_t)blockIdx.x;
  const float *s = src + (size_t)blockIdx.x * width;
  T *d = dst + orow * width;
  for (int i = threadIdx.x; i < width; i += blockDim.x) d[i] = from_f<T>(s[i]);
}
template <typename T>
void launch_scatter_rows(const float *src, T *dst, const int32_t *slot_map, int rows, int width, cudaStream_t st) {
  if (rows > 0) scatter_rows_kernel<T><<<rows, 256, 0, st>>>(src, dst, slot_map, width);
}
template void launch_scatter_rows<float>(const float *, float *, const int32_t *, int, int, cudaStream_t);
template void launch_scatter_rows<bf16>(const float *, bf16 *, const int32_t *, int, int, cudaStream_t);

template <typename T>
__global__ void __launch_bounds__(256) store_kv_rows_kernel(const float *__restrict__ ky, const float *__restrict__ vy,
                                                            T *__restrict__ k_plane, T *__restrict__ v_plane,
                                                            const int32_t *__restrict__ slot_map, const int32_t *__restrict__ pos,
                                                            const float *__restrict__ cos_tab, const float *__restrict__ sin_tab,
                                                            int n_heads, int hd) {
  const int r = blockIdx.x, half = hd >> 1, width = n_heads * hd;
  const size_t orow = slot_map ? (size_t)slot_map[r] : (size_t)r;
  const float *k = ky + (size_t)r * width, *v = vy + (size_t)r * width;
  T *ko = k_plane + orow * width, *vo = v_plane + orow * width;
  const int p = pos[r];
  for (int idx = threadIdx.x; idx < n_heads * half; idx += blockDim.x) {     // same arithmetic as rope_kernel
    const int h = idx / half, i = idx % half;
    const float c = cos_tab[(size_t)p * half + i], s = sin_tab[(size_t)p * half + i];
    const float a = k[h * hd + i], b = k[h * hd + i + half];
    ko[h * hd + i] = from_f<T>(a * c - b * s);
    ko[h * hd + i + half] = from_f<T>(b * c + a * s);
  }
  for (int i = threadIdx.x; i < width; i += blockDim.x) vo[i] = from_f<T>(v[i]);
}
template <typename T>
void launch_store_kv_rows(const float *ky, const float *vy, T *k_plane, T *v_plane, const int32_t *slot_map, const int32_t *pos,
                          const float *cos_tab, const float *sin_tab, int rows, int n_heads, int hd, cudaStream_t st) {
  if (rows > 0) store_kv_rows_kernel<T><<<rows, 256, 0, st>>>(ky, vy, k_plane, v_plane, slot_map, pos, cos_tab, sin_tab, n_heads, hd);
}
template void launch_store_kv_rows<float>(const float *, const float *, float *, float *, const int32_t *, const int32_t *,
                                          const float *, const float *, int, int, int, cudaStream_t);
template void launch_store_kv_rows<bf16>(const float *, const float *, bf16 *, bf16 *, const int32_t *, const int32_t *,
                                         const float *, const float *, int, int, int, cudaStream_t);

// dst[r, c] = w[r, c] * gamma[c], product in fp32, one rounding to the output type
template <typename T, typename TO>
__global__ void fold_kernel(const T *__restrict__ w, const T *__restrict__ gamma, TO *__restrict__ dst, long long n, int cols) {
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride)
    dst[i] = from_f<TO>(to_f(w[i]) * to_f(gamma[i % cols]));
}
template <typename T, typename TO>
void launch_fold(const T *w, const T *gamma, TO *dst, int rows, int cols, cudaStream_t st) {
  const long long n = (long long)rows * cols;
  if (n <= 0) return;
  long long blocks = (n + 255) / 256;
  if (blocks > 148 * 8) blocks = 148 * 8;
  fold_kernel<T, TO><<<(unsigned)blocks, 256, 0, st>>>(w, gamma, dst, n, cols);
}
template void launch_fold<float, float>(const float *, const float *, float *, int, int, cudaStream_t);
template void launch_fold<bf16, bf16>(const bf16 *, const bf16 *, bf16 *, int, int, cudaStream_t);
template void launch_fold<bf16, __half>(const bf16 *, const bf16 *, __half *, int, int, cudaStream_t);

__global__ void gather_kv_half_kernel(const bf16 *__restrict__ k, const bf16 *__restrict__ v, __half *__restrict__ k16,
                                      __half *__restrict__ v16, const int32_t *__restrict__ row0,
                                      const int32_t *__restrict__ len, const int32_t *__restrict__ kcu,
                                      const int32_t *__restrict__ blk, int blk_stride, int dkv, unsigned int *status) {
  const int b = blockIdx.y, r = blockIdx.x;
  if (r >= len[b]) return;
  bool hit = false;
  auto cvt = [&](__nv_bfloat162 x) {       // bf16 pair -> half pair, clamped to the half range (a bf16 may lie beyond it)
    float2 f = __bfloat1622float2(x);
    hit |= fabsf(f.x) >= HALF_OVERFLOW || fabsf(f.y) >= HALF_OVERFLOW;
    f.x = fminf(fmaxf(f.x, -65504.f), 65504.f);
    f.y = fminf(fmaxf(f.y, -65504.f), 65504.f);
    return __float22half2_rn(f);
  };
  const size_t src = kv_row_of(blk, blk_stride, b, row0[b], r) * dkv, dst = ((size_t)kcu[b] + r) * dkv;
  for (int i = threadIdx.x * 8; i < dkv; i += blockDim.x * 8) {
    const uint4 kr = *reinterpret_cast<const uint4 *>(k + src + i), vr = *reinterpret_cast<const uint4 *>(v + src + i);
    const __nv_bfloat162 *k2 = reinterpret_cast<const __nv_bfloat162 *>(&kr), *v2 = reinterpret_cast<const __nv_bfloat162 *>(&vr);
    uint4 ko, vo;
    __half2 *ko2 = reinterpret_cast<__half2 *>(&ko), *vo2 = reinterpret_cast<__half2 *>(&vo);
#pragma unroll
    for (int q = 0; q < 4; ++q) { ko2[q] = cvt(k2[q]); vo2[q] = cvt(v2[q]); }
    *reinterpret_cast<uint4 *>(k16 + dst + i) = ko;
    *reinterpret_cast<uint4 *>(v16 + dst + i) = vo;
  }
  report_overflow(hit, status);
}
void launch_gather_kv_half(const bf16 *k, const bf16 *v, __half *k16, __half *v16, const int32_t *row0, const int32_t *len,
                           const int32_t *kcu, const int32_t *blk, int blk_stride, int n_seqs, int max_len, int dkv,
                           cudaStream_t st, unsigned int *status) {
  if (n_seqs <= 0 || max_len <= 0) return;
  gather_kv_half_kernel<<<dim3(max_len, n_seqs), 128, 0, st>>>(k, v, k16, v16, row0, len, kcu, blk, blk_stride, dkv, status);
}

// bfloat16 -> IEEE half copy of a weight matrix (exact for |w| >= 2^-17, absolute error <= 2^-25 below), 128-bit accesses
__global__ void bf16_to_f16_kernel(const bf16 *__restrict__ src, __half *__restrict__ dst, long long n, unsigned int *status) {
  bool hit = false;
  const long long stride = (long long)gridDim.x * blockDim.x;
  const long long nv = n / 8;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < nv; i += stride) {
    const uint4 raw = __ldcs(reinterpret_cast<const uint4 *>(src) + i);
    const __nv_bfloat162 *in2 = reinterpret_cast<const __nv_bfloat162 *>(&raw);
    uint4 o;
    __half2 *o2 = reinterpret_cast<__half2 *>(&o);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      float2 f = __bfloat1622float2(in2[k]);
      hit |= fabsf(f.x) >= HALF_OVERFLOW || fabsf(f.y) >= HALF_OVERFLOW;     // a weight beyond the half range: clamped
      f.x = fminf(fmaxf(f.x, -65504.f), 65504.f);
      f.y = fminf(fmaxf(f.y, -65504.f), 65504.f);
      o2[k] = __float22half2_rn(f);
    }
    reinterpret_cast<uint4 *>(dst)[i] = o;
  }
  for (long long i = nv * 8 + (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
    const float f = __bfloat162float(src[i]);
    hit |= fabsf(f) >= HALF_OVERFLOW;
    dst[i] = __float2half_rn(fminf(fmaxf(f, -65504.f), 65504.f));
  }
  report_overflow(hit, status);
}
void launch_bf16_to_f16(const bf16 *src, __half *dst, long long n, cudaStream_t st, unsigned int *status) {
  if (n <= 0) return;
  long long blocks = (n / 8 + 255) / 256;
  if (blocks < 1) blocks = 1;
  if (blocks > 148 * 16) blocks = 148 * 16;
  bf16_to_f16_kernel<<<(unsigned)blocks, 256, 0, st>>>(src, dst, n, status);
}

}  // namespace skv
