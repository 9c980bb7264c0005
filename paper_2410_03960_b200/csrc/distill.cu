// Knowledge-recovery step of SwiftKV (Sec. 3.4, Eq. 3): the unmodified model (teacher) and the re-wired model (student:
// SingleInputKV / AcrossKV of Sec. 3.2 - 3.3 with its own copies of W_Q, W_K, W_V of the layers > l) share one frozen set of
// weights; every prompt token runs every layer in both modes, the loss is the distillation loss on the two logit tensors
// at temperature tau (tau^2 * mean over tokens of KL(softmax(y_t / tau) || softmax(y_s / tau))), and the gradient is taken
// with respect to the student's W_Q, W_K, W_V only.  Layers 1..l are identical in both modes and run once.
//
// fp32 data throughout (a bf16 model's frozen weights are widened to fp32 copies in the workspace first, the student's copies
// and the gradients are fp32 either way).  The GEMMs -- every projection forward, every data gradient, the three weight
// gradients -- run on the CUDA cores (precision 0) or on the tensor cores through the tcgen05 GEMM's kind::tf32 form
// (precision 1: operands as exact sums of two tf32 numbers, three products, fp32-grade; precision 2: one product, 10
// mantissa bits per operand); attention forward / backward, norms, SwiGLU, RoPE and the loss stay fp32 CUDA-core kernels.
// Every output element is owned by one thread block and summed in a fixed order, so gradients repeat bit for bit.
#include <algorithm>
#include <cmath>
#include <vector>

#include "common.cuh"

namespace skv {
namespace {

__global__ void transpose_kernel(const float *__restrict__ in, float *__restrict__ out, int rows, int cols) {
  __shared__ float tile[32][33];
  const int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
  for (int i = threadIdx.y; i < 32; i += blockDim.y) {
    const int r = r0 + i, c = c0 + threadIdx.x;
    if (r < rows && c < cols) tile[i][threadIdx.x] = in[(size_t)r * cols + c];
  }
  __syncthreads();
  for (int i = threadIdx.y; i < 32; i += blockDim.y) {
    const int c = c0 + i, r = r0 + threadIdx.x;
    if (r < rows && c < cols) out[(size_t)c * rows + r] = tile[threadIdx.x][i];
  }
}
void transpose(const float *in, float *out, int rows, int cols, cudaStream_t st) {
  transpose_kernel<<<dim3((cols + 31) / 32, (rows + 31) / 32), dim3(32, 8), 0, st>>>(in, out, rows, cols);
}

__device__ __forceinline__ float block_sum(float v, float *sh) {
  v = warp_sum(v);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = (blockDim.x + 31) >> 5;
  __syncthreads();
  if (lane == 0) sh[warp] = v;
  __syncthreads();
  float t = 0.f;
  for (int w = 0; w < nw; ++w) t += sh[w];
  return t;
}
__device__ __forceinline__ float block_max(float v, float *sh) {
  v = warp_max(v);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = (blockDim.x + 31) >> 5;
  __syncthreads();
  if (lane == 0) sh[warp] = v;
  __syncthreads();
  float t = -INFINITY;
  for (int w = 0; w < nw; ++w) t = fmaxf(t, sh[w]);
  return t;
}

// y = x * r * gamma, r = (mean(x^2) + eps)^(-1/2):  dx = r * (gamma dy) - x * r^3 * mean(x * gamma dy);  out (+)= dx
__global__ void __launch_bounds__(256) rmsnorm_bwd_kernel(const float *__restrict__ x, const float *__restrict__ gamma,
                                                          const float *__restrict__ dy, float *__restrict__ out, int d, float eps,
                                                          int accumulate) {
  __shared__ float sh[8];
  const size_t row = blockIdx.x;
  const float *xr = x + row * d, *dr = dy + row * d;
  float ss = 0.f, sg = 0.f;
  for (int i = threadIdx.x; i < d; i += blockDim.x) {
    const float xv = xr[i];
    ss = fmaf(xv, xv, ss);
    sg = fmaf(xv, gamma[i] * dr[i], sg);
  }
  ss = block_sum(ss, sh);
  sg = block_sum(sg, sh);
  const float r = rsqrtf(ss / (float)d + eps);
  const float coef = r * r * r * (sg / (float)d);
  for (int i = threadIdx.x; i < d; i += blockDim.x) {
    const float v = r * gamma[i] * dr[i] - xr[i] * coef;
    float *o = out + row * d + i;
    *o = accumulate ? *o + v : v;
  }
}

// act = silu(gate) * up:  dgate = dact * up * s (1 + gate (1 - s)),  dup = dact * silu(gate),  s = sigmoid(gate)
__global__ void swiglu_bwd_kernel(const float *__restrict__ gate, const float *__restrict__ up, const float *__restrict__ dact,
                                  float *__restrict__ dgate, float *__restrict__ dup, long long n) {
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
    const float g = gate[i], s = 1.f / (1.f + expf(-g)), da = dact[i];
    dgate[i] = da * up[i] * s * (1.f + g * (1.f - s));
    dup[i] = da * g * s;
  }
}

// transpose of the rotary embedding (rotate-half pairs (i, i + hd/2)): the rotation by the negated angle, in place
__global__ void rope_bwd_kernel(float *__restrict__ x, const int32_t *__restrict__ pos, const float *__restrict__ cos_tab,
                                const float *__restrict__ sin_tab, int rows, int n_heads, int hd) {
  const int half = hd >> 1;
  const long long total = (long long)rows * n_heads * half;
  for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (long long)gridDim.x * blockDim.x) {
    const int i = (int)(idx % half);
    const long long rh = idx / half;
    const int row = (int)(rh / n_heads);
    float *p = x + rh * hd;
    const size_t t = (size_t)pos[row] * half + i;
    const float c = cos_tab[t], s = sin_tab[t];
    const float a = p[i], b = p[i + half];
    p[i] = a * c + b * s;
    p[i + half] = b * c - a * s;
  }
}

__global__ void add_kernel(float *__restrict__ dst, const float *__restrict__ src, long long n) {
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) dst[i] += src[i];
}

// Causal attention forward: one warp per (four consecutive query tokens, query head), a single pass over the prompt's keys
// with a running maximum, sum and output per row.  Every K / V row is read once for the four queries (a warp per single query
// re-read the whole prefix from L2 and was bound by that); rows of the group that belong to another prompt than its first
// row are done in a pass of their own.  Writes the output rows and each row's (maximum, sum) for the backward pass.
template <int MAX_E>
__global__ void __launch_bounds__(128) attn_fwd_kernel(const float *__restrict__ q, const float *__restrict__ k,
                                                       const float *__restrict__ v, float *__restrict__ o, float *__restrict__ stat,
                                                       const int32_t *__restrict__ pos, int n_tokens, int n_q, int n_kv, int hd,
                                                       float scale) {
  constexpr int R = 4;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_groups = (n_tokens + R - 1) / R;
  const long long item = (long long)blockIdx.x * 4 + warp;
  if (item >= (long long)n_groups * n_q) return;
  const int grp = (int)(item / n_q), h = (int)(item % n_q), kvh = h / (n_q / n_kv);
  const int tok0 = grp * R;
  int p_r[R], first_r[R];
#pragma unroll
  for (int r = 0; r < R; ++r) {
    const int tok = tok0 + r;
    p_r[r] = tok < n_tokens ? pos[tok] : -1;
    first_r[r] = tok - p_r[r];
  }
  unsigned todo = 0;
#pragma unroll
  for (int r = 0; r < R; ++r) if (p_r[r] >= 0) todo |= 1u << r;
  while (todo) {
    const int lead = __ffs(todo) - 1;
    const int first = first_r[lead];
    unsigned act = 0;
    int p_max = 0;
#pragma unroll
    for (int r = 0; r < R; ++r)
      if (((todo >> r) & 1u) && first_r[r] == first) { act |= 1u << r; p_max = max(p_max, p_r[r]); }
    todo &= ~act;
    float qe[R][MAX_E], acc[R][MAX_E], m[R], l[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
      m[r] = -INFINITY; l[r] = 0.f;
#pragma unroll
      for (int e = 0; e < MAX_E; ++e) {
        const int dd = lane + 32 * e;
        qe[r][e] = (((act >> r) & 1u) && dd < hd) ? q[((size_t)(tok0 + r) * n_q + h) * hd + dd] * scale : 0.f;
        acc[r][e] = 0.f;
      }
    }
    for (int j = 0; j <= p_max; ++j) {
      const float *kr = k + ((size_t)(first + j) * n_kv + kvh) * hd, *vr = v + ((size_t)(first + j) * n_kv + kvh) * hd;
      float ke[MAX_E], ve[MAX_E], s[R];
#pragma unroll
      for (int e = 0; e < MAX_E; ++e) {
        const int dd = lane + 32 * e;
        ke[e] = dd < hd ? kr[dd] : 0.f;
        ve[e] = dd < hd ? vr[dd] : 0.f;
      }
#pragma unroll
      for (int r = 0; r < R; ++r) {
        s[r] = 0.f;
#pragma unroll
        for (int e = 0; e < MAX_E; ++e) s[r] = fmaf(qe[r][e], ke[e], s[r]);
      }
#pragma unroll
      for (int r = 0; r < R; ++r) s[r] = warp_sum(s[r]);
#pragma unroll
      for (int r = 0; r < R; ++r) {
        if (((act >> r) & 1u) && j <= p_r[r]) {
          const float m_new = fmaxf(m[r], s[r]), corr = expf(m[r] - m_new), pj = expf(s[r] - m_new);
          l[r] = l[r] * corr + pj;
#pragma unroll
          for (int e = 0; e < MAX_E; ++e) acc[r][e] = fmaf(pj, ve[e], acc[r][e] * corr);
          m[r] = m_new;
        }
      }
    }
#pragma unroll
    for (int r = 0; r < R; ++r) {
      if ((act >> r) & 1u) {
        const int tok = tok0 + r;
        const float inv = 1.f / l[r];
#pragma unroll
        for (int e = 0; e < MAX_E; ++e) { const int dd = lane + 32 * e; if (dd < hd) o[((size_t)tok * n_q + h) * hd + dd] = acc[r][e] * inv; }
        if (lane == 0 && stat) {
          float *st = stat + ((size_t)tok * n_q + h) * 3;
          st[0] = m[r]; st[1] = l[r];
        }
      }
    }
  }
}

// Backward, query side: one warp per (query token, query head), with the forward pass's (maximum, sum) of the row; writes dq
// and D = dO . O next to them for the key-side kernel.
template <int MAX_E>
__global__ void __launch_bounds__(128) attn_bwd_q_kernel(const float *__restrict__ q, const float *__restrict__ k,
                                                         const float *__restrict__ v, const float *__restrict__ o,
                                                         const float *__restrict__ d_o, float *__restrict__ dq,
                                                         float *__restrict__ stat, const int32_t *__restrict__ pos, int n_tokens,
                                                         int n_q, int n_kv, int hd, float scale) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long item = (long long)blockIdx.x * 4 + warp;
  if (item >= (long long)n_tokens * n_q) return;
  const int tok = (int)(item / n_q), h = (int)(item % n_q), kvh = h / (n_q / n_kv);
  const int p = pos[tok], first = tok - p;                  // the prompt's first packed row
  float qe[MAX_E], doe[MAX_E], acc[MAX_E];
  float D = 0.f;
#pragma unroll
  for (int e = 0; e < MAX_E; ++e) {
    const int dd = lane + 32 * e;
    qe[e] = dd < hd ? q[((size_t)tok * n_q + h) * hd + dd] : 0.f;
    doe[e] = dd < hd ? d_o[((size_t)tok * n_q + h) * hd + dd] : 0.f;
    const float ov = dd < hd ? o[((size_t)tok * n_q + h) * hd + dd] : 0.f;
    D = fmaf(doe[e], ov, D);
    acc[e] = 0.f;
  }
  D = warp_sum(D);
  float *st = stat + ((size_t)tok * n_q + h) * 3;
  const float m = st[0], inv_l = 1.f / st[1];
  for (int j = 0; j <= p; ++j) {
    const float *kr = k + ((size_t)(first + j) * n_kv + kvh) * hd, *vr = v + ((size_t)(first + j) * n_kv + kvh) * hd;
    float s = 0.f, dp = 0.f;
#pragma unroll
    for (int e = 0; e < MAX_E; ++e) {
      const int dd = lane + 32 * e;
      if (dd < hd) { s = fmaf(qe[e], kr[dd], s); dp = fmaf(doe[e], vr[dd], dp); }
    }
    const float pij = expf(warp_sum(s) * scale - m) * inv_l;
    const float ds = pij * (warp_sum(dp) - D) * scale;
#pragma unroll
    for (int e = 0; e < MAX_E; ++e) { const int dd = lane + 32 * e; if (dd < hd) acc[e] = fmaf(ds, kr[dd], acc[e]); }
  }
#pragma unroll
  for (int e = 0; e < MAX_E; ++e) { const int dd = lane + 32 * e; if (dd < hd) dq[((size_t)tok * n_q + h) * hd + dd] = acc[e]; }
  if (lane == 0) st[2] = D;
}

// One warp per (key token, KV head): every later query of the prompt, every query head of the group, in a fixed order.
// dk, dv are ADDED to (the AcrossKV group's layers accumulate into one pair of buffers).
template <int MAX_E>
__global__ void __launch_bounds__(128) attn_bwd_kv_kernel(const float *__restrict__ q, const float *__restrict__ k,
                                                          const float *__restrict__ v, const float *__restrict__ d_o,
                                                          const float *__restrict__ stat, float *__restrict__ dk,
                                                          float *__restrict__ dv, const int32_t *__restrict__ pos,
                                                          const int32_t *__restrict__ seq_end, int n_tokens, int n_q, int n_kv,
                                                          int hd, float scale) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long item = (long long)blockIdx.x * 4 + warp;
  if (item >= (long long)n_tokens * n_kv) return;
  const int tok = (int)(item / n_kv), kvh = (int)(item % n_kv), rep = n_q / n_kv;
  const int end = seq_end[tok];                              // one past the prompt's last packed row
  float ke[MAX_E], ve[MAX_E], ak[MAX_E], av[MAX_E];
#pragma unroll
  for (int e = 0; e < MAX_E; ++e) {
    const int dd = lane + 32 * e;
    ke[e] = dd < hd ? k[((size_t)tok * n_kv + kvh) * hd + dd] : 0.f;
    ve[e] = dd < hd ? v[((size_t)tok * n_kv + kvh) * hd + dd] : 0.f;
    ak[e] = av[e] = 0.f;
  }
  for (int i = tok; i < end; ++i)
    for (int hr = 0; hr < rep; ++hr) {
      const int h = kvh * rep + hr;
      const float *qr = q + ((size_t)i * n_q + h) * hd, *dor = d_o + ((size_t)i * n_q + h) * hd;
      const float *st = stat + ((size_t)i * n_q + h) * 3;
      float s = 0.f, dp = 0.f;
#pragma unroll
      for (int e = 0; e < MAX_E; ++e) {
        const int dd = lane + 32 * e;
        if (dd < hd) { s = fmaf(qr[dd], ke[e], s); dp = fmaf(dor[dd], ve[e], dp); }
      }
      const float pij = expf(warp_sum(s) * scale - st[0]) / st[1];
      const float ds = pij * (warp_sum(dp) - st[2]) * scale;
#pragma unroll
      for (int e = 0; e < MAX_E; ++e) {
        const int dd = lane + 32 * e;
        if (dd < hd) { av[e] = fmaf(pij, dor[dd], av[e]); ak[e] = fmaf(ds, qr[dd], ak[e]); }
      }
    }
#pragma unroll
  for (int e = 0; e < MAX_E; ++e) {
    const int dd = lane + 32 * e;
    if (dd < hd) {
      dk[((size_t)tok * n_kv + kvh) * hd + dd] += ak[e];
      dv[((size_t)tok * n_kv + kvh) * hd + dd] += av[e];
    }
  }
}

// one block per token: p_t = softmax(y_t / tau), p_s = softmax(y_s / tau); row_loss = tau^2 * KL(p_t || p_s);
// y_s is overwritten with d loss / d y_s = (tau / T) (p_s - p_t)
__global__ void __launch_bounds__(256) kl_grad_kernel(const float *__restrict__ yt, float *__restrict__ ys, float *__restrict__ row_loss,
                                                      int vocab, float tau, int n_tokens) {
  __shared__ float sh[8];
  const size_t row = blockIdx.x;
  const float *t = yt + row * vocab;
  float *s = ys + row * vocab;
  const float inv = 1.f / tau;
  float mt = -INFINITY, ms = -INFINITY;
  for (int i = threadIdx.x; i < vocab; i += blockDim.x) { mt = fmaxf(mt, t[i] * inv); ms = fmaxf(ms, s[i] * inv); }
  mt = block_max(mt, sh);
  ms = block_max(ms, sh);
  float zt = 0.f, zs = 0.f;
  for (int i = threadIdx.x; i < vocab; i += blockDim.x) { zt += expf(t[i] * inv - mt); zs += expf(s[i] * inv - ms); }
  zt = block_sum(zt, sh);
  zs = block_sum(zs, sh);
  const float lzt = logf(zt), lzs = logf(zs);
  float kl = 0.f;
  const float coef = tau / (float)n_tokens;
  for (int i = threadIdx.x; i < vocab; i += blockDim.x) {
    const float lt = t[i] * inv - mt - lzt, ls = s[i] * inv - ms - lzs;
    const float pt = expf(lt), ps = expf(ls);
    kl = fmaf(pt, lt - ls, kl);
    s[i] = coef * (ps - pt);
  }
  kl = block_sum(kl, sh);
  if (threadIdx.x == 0) row_loss[row] = tau * tau * kl;
}
__global__ void __launch_bounds__(256) mean_kernel(const float *__restrict__ v, int n, float *__restrict__ out) {
  __shared__ double sh[256];
  double a = 0.0;
  for (int i = threadIdx.x; i < n; i += 256) a += (double)v[i];
  sh[threadIdx.x] = a;
  __syncthreads();
  for (int s = 128; s > 0; s >>= 1) {
    if ((int)threadIdx.x < s) sh[threadIdx.x] += sh[threadIdx.x + s];
    __syncthreads();
  }
  if (threadIdx.x == 0) *out = (float)(sh[0] / (double)n);
}
__global__ void seq_end_kernel(const int32_t *__restrict__ cu, int n_seqs, int32_t *__restrict__ seq_end) {
  const int b = blockIdx.x;
  for (int i = cu[b] + threadIdx.x; i < cu[b + 1]; i += blockDim.x) seq_end[i] = cu[b + 1];
}

inline int grid_for(long long n) { return (int)std::min<long long>((n + 255) / 256, 148 * 8); }

// x ~ hi + lo, both representable in tf32 (10 mantissa bits): hi = x rounded to nearest, lo = (x - hi) rounded to nearest, so
// that the tensor core's own cut of the 13 low bits changes neither.  What is lost is at most 2^-22 |x| and has no preferred
// sign (cutting instead of rounding loses up to 2^-20 |x|, always toward zero, which adds up over sums of thousands of terms).
__device__ __forceinline__ float round_tf32(float v) {
  const uint32_t u = __float_as_uint(v);
  if ((u & 0x7F800000u) == 0x7F800000u) return v;      // inf / nan pass
  return __uint_as_float((u + 0x1000u) & 0xFFFFE000u);
}
__global__ void split_tf32_kernel(const float *__restrict__ x, float *__restrict__ hi, float *__restrict__ lo, long long n) {
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
    const float v = x[i], h = round_tf32(v);
    hi[i] = h;
    lo[i] = round_tf32(v - h);
  }
}
__global__ void upcast_kernel(const bf16 *__restrict__ src, float *__restrict__ dst, long long n) {
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) dst[i] = to_f(src[i]);
}

}  // namespace

void distill_upcast(const void *src_bf16, float *dst, long long n, cudaStream_t st) {
  if (n > 0) upcast_kernel<<<grid_for(n), 256, 0, st>>>(reinterpret_cast<const bf16 *>(src_bf16), dst, n);
}

// AdamW with decoupled weight decay, step counted from 1 (bias corrections computed on the host in double):
//   p <- p (1 - lr wd);  m <- b1 m + (1 - b1) g;  v <- b2 v + (1 - b2) g^2;  p <- p - lr (m / c1) / (sqrt(v / c2) + eps)
namespace {
__global__ void adamw_kernel(float *__restrict__ p, const float *__restrict__ g, float *__restrict__ m, float *__restrict__ v,
                             long long n, float lr, float b1, float b2, float nb1, float nb2, float eps, float decay, float inv_c1,
                             float inv_c2) {
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
    const float gi = g[i];
    const float mi = b1 * m[i] + nb1 * gi;
    const float vi = b2 * v[i] + nb2 * gi * gi;
    m[i] = mi;
    v[i] = vi;
    p[i] = p[i] * decay - lr * (mi * inv_c1) / (sqrtf(vi * inv_c2) + eps);
  }
}
}  // namespace
void launch_adamw(float *p, const float *g, float *m, float *v, long long n, float lr, float b1, float b2, float eps, float wd,
                  int step, cudaStream_t st) {
  if (n <= 0) return;
  const double c1 = 1.0 - pow((double)b1, (double)step), c2 = 1.0 - pow((double)b2, (double)step);
  // (1 - beta as a float subtraction would lose half of beta2's significant digits: everything derived is rounded once, from double)
  adamw_kernel<<<grid_for(n), 256, 0, st>>>(p, g, m, v, n, lr, b1, b2, (float)(1.0 - (double)b1), (float)(1.0 - (double)b2), eps,
                                            (float)(1.0 - (double)lr * wd), (float)(1.0 / c1), (float)(1.0 / c2));
}

size_t distill_workspace_floats(const DistillDims &c, int T, int l) {
  const size_t d = c.d, dq = (size_t)c.n_q * c.hd, dkv = (size_t)c.n_kv * c.hd, F = c.F, V = c.vocab;
  const size_t per_layer = (size_t)T * (4 * d + 2 * dq + 2 * dkv + 2 * F + d + 3 * (size_t)c.n_q);   // X, h, X1, m, q, att, k, v, gate, up, hs, row statistics
  const size_t wmax = std::max(std::max(V * d, F * d), dq * d);
  const size_t amax = (size_t)T * std::max(std::max(d, dq), std::max(F, V));
  const size_t common = (size_t)T * (3 * d + 2 * V + 3 * F + 3 * dq + 4 * dkv + 3 * (size_t)c.n_q + 2 * std::max(std::max(d, dq), F)) + wmax + 2 * T +
                        2 * amax + 2 * wmax +                    // operand halves of the tensor-core modes
                        160 + 48 * (size_t)(c.L - l + 1);        // (+ the rounding of every piece to 16 bytes)
  return common + (size_t)(c.L - l) * per_layer + (size_t)T * (6 * d + 2 * dq + 2 * dkv + 3 * F + 3 * (size_t)c.n_q);   // (+ the teacher's scratch layer)
}

namespace {
struct Bump {
  float *p, *end;
  float *take(size_t n) { float *r = p; p += (n + 3) & ~(size_t)3; return p <= end ? r : nullptr; }
};
struct LayerSave { float *X, *h, *q, *att, *X1, *m, *gate, *up, *hs, *k, *v, *stat; };
}  // namespace

int run_distill(const DistillDims &c, const DistillArgs &a, const DistillLayer *layers, cudaStream_t st) {
  const int T = a.T, B = a.B, L = c.L, l = a.l, g = a.g;
  const int d = c.d, nq = c.n_q, nkv = c.n_kv, hd = c.hd, F = c.F, V = c.vocab;
  const int dq = nq * hd, dkv = nkv * hd;
  const float scale = 1.0f / sqrtf((float)hd);
  Bump ws{reinterpret_cast<float *>(a.ws), reinterpret_cast<float *>(a.ws) + a.ws_floats};
  float *X = ws.take((size_t)T * d), *Xs = ws.take((size_t)T * d), *dX = ws.take((size_t)T * d);
  float *yt = ws.take((size_t)T * V), *ys = ws.take((size_t)T * V);
  float *t_F0 = ws.take((size_t)T * F), *t_F1 = ws.take((size_t)T * F), *t_F2 = ws.take((size_t)T * F);
  float *da = ws.take((size_t)T * dq), *dqb = ws.take((size_t)T * dq), *t_q = ws.take((size_t)T * dq);
  float *dk = ws.take((size_t)T * dkv), *dv = ws.take((size_t)T * dkv), *dks = ws.take((size_t)T * dkv), *dvs = ws.take((size_t)T * dkv);
  const size_t tmax = (size_t)T * std::max(std::max(d, dq), F);
  float *trA = ws.take(tmax), *trB = ws.take(tmax);
  float *wT = ws.take(std::max(std::max((size_t)V * d, (size_t)F * d), (size_t)dq * d));
  const size_t amax = (size_t)T * std::max(std::max(d, dq), std::max(F, V));
  const size_t wmax = std::max(std::max((size_t)V * d, (size_t)F * d), (size_t)dq * d);
  float *a_hi = ws.take(amax), *a_lo = ws.take(amax), *b_hi = ws.take(wmax), *b_lo = ws.take(wmax);
  float *row_loss = ws.take(T);
  int32_t *seq_end = reinterpret_cast<int32_t *>(ws.take(T));
  std::vector<LayerSave> save(L + 1);
  for (int j = l; j <= L; ++j) {          // slot L: the teacher's scratch layer (nothing of it is kept)
    LayerSave &s = save[j];
    s.X = ws.take((size_t)T * d); s.h = ws.take((size_t)T * d); s.X1 = ws.take((size_t)T * d); s.m = ws.take((size_t)T * d);
    s.hs = ws.take((size_t)T * d);
    s.q = ws.take((size_t)T * dq); s.att = ws.take((size_t)T * dq);
    s.k = ws.take((size_t)T * dkv); s.v = ws.take((size_t)T * dkv);
    s.gate = ws.take((size_t)T * F); s.up = ws.take((size_t)T * F);
    s.stat = ws.take((size_t)T * nq * 3);
  }
  if (ws.p > ws.end) return SWIFTKV_ERR_WORKSPACE_SMALL;

  // out[M, N] (+)= A[M, K] B[N, K]^T.  precision 0: fp32 on the CUDA cores.  1: tensor cores with every operand as an exact sum
  // of two tf32 numbers, three products (the lo x lo term is below fp32 resolution) -- fp32-grade results.  2: one tf32 product
  // (operands cut to 10 mantissa bits).  Shapes the tensor-core kernel does not tile keep the CUDA-core kernel.
  auto gemm = [&](const float *A, const float *Bm, int M, int N, int K, float *out, bool accumulate) {
    if (a.precision != 0 && tc_gemm_tf32_supported(M, N, K) && (size_t)M * K <= amax && (size_t)N * K <= wmax) {
      if (a.precision == 2) { launch_gemm_tc_tf32(A, Bm, M, N, K, out, accumulate, a.status, st); return; }
      split_tf32_kernel<<<grid_for((long long)M * K), 256, 0, st>>>(A, a_hi, a_lo, (long long)M * K);
      split_tf32_kernel<<<grid_for((long long)N * K), 256, 0, st>>>(Bm, b_hi, b_lo, (long long)N * K);
      // (accumulation chains of at most 1024: longer ones lose more to the tensor core's cut-off add than the split gains)
      launch_gemm_tc_tf32(a_lo, b_hi, M, N, K, out, accumulate, a.status, st);
      launch_gemm_tc_tf32(a_hi, b_lo, M, N, K, out, true, a.status, st);
      launch_gemm_tc_tf32(a_hi, b_hi, M, N, K, out, true, a.status, st, 1024);
      return;
    }
    launch_gemm_simt<float, float>(A, Bm, M, N, K, out_plain(accumulate ? OUT_RESID_ADD_F32 : OUT_STORE_F32, out, N, N), 0, st);
  };
  auto copy = [&](float *dst, const float *src, size_t n) { cudaMemcpyAsync(dst, src, n * sizeof(float), cudaMemcpyDeviceToDevice, st); };
  // dX[M, K] (+)= dY[M, N] W[N, K]
  auto dgrad = [&](const float *dY, const float *W, int M, int N, int K, float *out, bool accumulate) {
    transpose(W, wT, N, K, st);
    gemm(dY, wT, M, K, N, out, accumulate);
  };
  // dW[N, K] = dY[M, N]^T X[M, K]
  auto wgrad = [&](const float *dY, const float *Xm, int M, int N, int K, float *out) {
    transpose(dY, trA, M, N, st);
    transpose(Xm, trB, M, K, st);
    gemm(trA, trB, N, K, M, out, false);
  };
  // one decoder layer on all tokens; student mode projects K / V from x_{l+1} with the group leader's gain and the student's
  // copies (Eq. 2); saves what the backward pass reads
  auto layer_forward = [&](int j, bool student, LayerSave &s, float *x) {
    const DistillLayer &w = layers[j];
    copy(s.X, x, (size_t)T * d);
    launch_rmsnorm<float, float>(x, w.in_norm, s.h, T, d, c.eps, st);
    gemm(s.h, student ? w.s_wq : w.wq, T, dq, d, s.q, false);
    launch_rope<float>(s.q, 0, 1, a.pos, nullptr, a.cos_tab, a.sin_tab, T, nq, hd, st);
    const float *kk, *vv;
    if (student) {
      const int r = l + ((j - l) / g) * g;
      LayerSave &ld = save[r];
      if (r == j) {
        launch_rmsnorm<float, float>(Xs, layers[r].in_norm, s.hs, T, d, c.eps, st);
        gemm(s.hs, layers[r].s_wk, T, dkv, d, s.k, false);
        gemm(s.hs, layers[r].s_wv, T, dkv, d, s.v, false);
        launch_rope<float>(s.k, 0, 1, a.pos, nullptr, a.cos_tab, a.sin_tab, T, nkv, hd, st);
      }
      kk = ld.k; vv = ld.v;
    } else {
      gemm(s.h, w.wk, T, dkv, d, s.k, false);
      gemm(s.h, w.wv, T, dkv, d, s.v, false);
      launch_rope<float>(s.k, 0, 1, a.pos, nullptr, a.cos_tab, a.sin_tab, T, nkv, hd, st);
      kk = s.k; vv = s.v;
    }
    {
      const unsigned blocks = (unsigned)(((long long)((T + 3) / 4) * nq + 3) / 4);      // a warp per (4 tokens, head), 4 warps per block
      if (hd <= 32) attn_fwd_kernel<1><<<blocks, 128, 0, st>>>(s.q, kk, vv, s.att, s.stat, a.pos, T, nq, nkv, hd, scale);
      else if (hd <= 64) attn_fwd_kernel<2><<<blocks, 128, 0, st>>>(s.q, kk, vv, s.att, s.stat, a.pos, T, nq, nkv, hd, scale);
      else if (hd <= 128) attn_fwd_kernel<4><<<blocks, 128, 0, st>>>(s.q, kk, vv, s.att, s.stat, a.pos, T, nq, nkv, hd, scale);
      else attn_fwd_kernel<8><<<blocks, 128, 0, st>>>(s.q, kk, vv, s.att, s.stat, a.pos, T, nq, nkv, hd, scale);
    }
    gemm(s.att, w.wo, T, d, dq, x, true);
    copy(s.X1, x, (size_t)T * d);
    launch_rmsnorm<float, float>(x, w.post_norm, s.m, T, d, c.eps, st);
    gemm(s.m, w.w_gate, T, F, d, s.gate, false);
    gemm(s.m, w.w_up, T, F, d, s.up, false);
    launch_swiglu<float>(s.gate, s.up, t_F0, (long long)T * F, st);
    gemm(t_F0, w.w_down, T, d, F, x, true);
  };
  auto head = [&](float *x, float *logits) {
    launch_rmsnorm<float, float>(x, a.final_norm, trA, T, d, c.eps, st);
    gemm(trA, a.lm_head, T, V, d, logits, false);
  };

  seq_end_kernel<<<B, 128, 0, st>>>(a.cu, B, seq_end);
  launch_embed<float>(a.embed, a.tokens, X, T, d, V, a.status, st);
  for (int j = 0; j < l; ++j) layer_forward(j, false, save[L], X);          // shared by both modes
  copy(Xs, X, (size_t)T * d);                                              // x_{l+1}
  // teacher: the remaining layers unmodified
  for (int j = l; j < L; ++j) layer_forward(j, false, save[L], X);
  head(X, yt);
  // student: the remaining layers re-wired
  copy(X, Xs, (size_t)T * d);
  for (int j = l; j < L; ++j) layer_forward(j, true, save[j], X);
  head(X, ys);
  // loss and d loss / d y_student (in place of y_student)
  kl_grad_kernel<<<T, 256, 0, st>>>(yt, ys, row_loss, V, a.tau, T);
  mean_kernel<<<1, 256, 0, st>>>(row_loss, T, a.loss);
  // back through the lm_head and the final norm
  dgrad(ys, a.lm_head, T, V, d, trA, false);
  rmsnorm_bwd_kernel<<<T, 256, 0, st>>>(X, a.final_norm, trA, dX, d, c.eps, 0);
  for (int j = L - 1; j >= l; --j) {
    const DistillLayer &w = layers[j];
    LayerSave &s = save[j];
    const int r = l + ((j - l) / g) * g;
    // MLP and its norm:  dX1 = dX + norm_bwd(X1, gamma_post, dm)
    dgrad(dX, w.w_down, T, d, F, t_F0, false);                                                   // d act
    swiglu_bwd_kernel<<<grid_for((long long)T * F), 256, 0, st>>>(s.gate, s.up, t_F0, t_F1, t_F2, (long long)T * F);
    dgrad(t_F1, w.w_gate, T, F, d, trA, false);
    dgrad(t_F2, w.w_up, T, F, d, trA, true);                                                      // dm
    rmsnorm_bwd_kernel<<<T, 256, 0, st>>>(s.X1, w.post_norm, trA, dX, d, c.eps, 1);               // dX is now dX1
    // attention
    dgrad(dX, w.wo, T, d, dq, da, false);
    const bool group_start = (j == L - 1) || (l + ((j + 1 - l) / g) * g != r);                    // first layer of its group met going backward
    if (group_start) {
      cudaMemsetAsync(dks, 0, (size_t)T * dkv * sizeof(float), st);
      cudaMemsetAsync(dvs, 0, (size_t)T * dkv * sizeof(float), st);
    }
    const LayerSave &ld = save[r];
#define SKV_ATT_BWD(E)                                                                                                          \
    do {                                                                                                                        \
      attn_bwd_q_kernel<E><<<(unsigned)(((long long)T * nq + 3) / 4), 128, 0, st>>>(s.q, ld.k, ld.v, s.att, da, dqb, s.stat, a.pos, T, nq, \
                                                                                     nkv, hd, scale);                           \
      attn_bwd_kv_kernel<E><<<(unsigned)(((long long)T * nkv + 3) / 4), 128, 0, st>>>(s.q, ld.k, ld.v, da, s.stat, dks, dvs, a.pos,  \
                                                                                       seq_end, T, nq, nkv, hd, scale);         \
    } while (0)
    if (hd <= 32) SKV_ATT_BWD(1); else if (hd <= 64) SKV_ATT_BWD(2); else if (hd <= 128) SKV_ATT_BWD(4); else SKV_ATT_BWD(8);
#undef SKV_ATT_BWD
    // query path: dW_Q, and on into the residual stream
    rope_bwd_kernel<<<grid_for((long long)T * nq * hd / 2), 256, 0, st>>>(dqb, a.pos, a.cos_tab, a.sin_tab, T, nq, hd);
    wgrad(dqb, s.h, T, dq, d, w.g_wq);
    dgrad(dqb, w.s_wq, T, dq, d, trA, false);
    rmsnorm_bwd_kernel<<<T, 256, 0, st>>>(s.X, w.in_norm, trA, dX, d, c.eps, 1);                  // dX: gradient at the layer's input
    // key / value path: at the group leader, from the whole group's sum (x_{l+1} itself has no trainable producer)
    if (j == r) {
      rope_bwd_kernel<<<grid_for((long long)T * nkv * hd / 2), 256, 0, st>>>(dks, a.pos, a.cos_tab, a.sin_tab, T, nkv, hd);
      wgrad(dks, s.hs, T, dkv, d, w.g_wk);
      wgrad(dvs, s.hs, T, dkv, d, w.g_wv);
    } else {
      cudaMemsetAsync(w.g_wk, 0, (size_t)dkv * d * sizeof(float), st);
      cudaMemsetAsync(w.g_wv, 0, (size_t)dkv * d * sizeof(float), st);
    }
  }
  (void)dk; (void)dv; (void)t_q;
  return cudaGetLastError() == cudaSuccess ? SWIFTKV_OK : SWIFTKV_ERR_CUDA;
}

}  // namespace skv
