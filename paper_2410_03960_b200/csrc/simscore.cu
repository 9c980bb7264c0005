// SimScore (Sec. 3.2, Eq. 1): the average cosine similarity between the input of layer l and the inputs of all later
// layers, averaged over tokens -- the paper's motivation for projecting every later layer's K/V from one hidden state.
// The layer inputs x_1..x_L of the unmodified model are captured during a full-depth prefill ([L][T][d] fp32); one
// kernel then reduces every (l, j > l, token) cosine.
#include "common.cuh"

namespace skv {
namespace {

__device__ __forceinline__ float block_sum_256(float v, float *red) {
  v = warp_sum(v);
  __syncthreads();                       // red is reused from the previous call
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  float t = 0.f;
#pragma unroll
  for (int w = 0; w < 8; ++w) t += red[w];
  return t;
}

// block (token i, earlier layer l0): cos(x_{l0}[i], x_{j0}[i]) for every later j0, added into sums[l0][j0] (double, so the
// order of the atomic additions does not show in the rounded result)
__global__ void __launch_bounds__(256) simscore_pairs_kernel(const float *__restrict__ xs, int L, int T, int d,
                                                             double *__restrict__ sums) {
  __shared__ float red[8];
  const int i = blockIdx.x, l0 = blockIdx.y;
  const float *a = xs + ((size_t)l0 * T + i) * d;
  float na = 0.f;
  for (int c = threadIdx.x; c < d; c += 256) na = fmaf(a[c], a[c], na);
  na = block_sum_256(na, red);
  for (int j0 = l0 + 1; j0 < L; ++j0) {
    const float *b = xs + ((size_t)j0 * T + i) * d;
    float dot = 0.f, nb = 0.f;
    for (int c = threadIdx.x; c < d; c += 256) {
      const float av = a[c], bv = b[c];          // a stays in L1 across the later layers
      dot = fmaf(av, bv, dot);
      nb = fmaf(bv, bv, nb);
    }
    dot = block_sum_256(dot, red);
    nb = block_sum_256(nb, red);
    if (threadIdx.x == 0) atomicAdd(&sums[(size_t)l0 * L + j0], (double)dot / sqrt((double)na * (double)nb));
  }
}

// sim[l0][j0] = sums / T (upper triangle; symmetric fill, diagonal 1); simscore[l0] = mean over j0 > l0
__global__ void simscore_finish_kernel(const double *__restrict__ sums, int L, int T, float *__restrict__ sim,
                                       float *__restrict__ simscore) {
  const int l0 = blockIdx.x * blockDim.x + threadIdx.x;
  if (l0 >= L) return;
  double acc = 0.0;
  for (int j0 = l0 + 1; j0 < L; ++j0) {
    const double s = sums[(size_t)l0 * L + j0] / (double)T;
    acc += s;
    if (sim) { sim[(size_t)l0 * L + j0] = (float)s; sim[(size_t)j0 * L + l0] = (float)s; }
  }
  if (sim) sim[(size_t)l0 * L + l0] = 1.f;
  if (l0 < L - 1) simscore[l0] = (float)(acc / (double)(L - 1 - l0));
}

}  // namespace

void launch_simscore(const float *xs, int L, int T, int d, double *sums, float *sim, float *simscore, cudaStream_t st) {
  if (L < 2 || T < 1) return;
  cudaMemsetAsync(sums, 0, (size_t)L * L * sizeof(double), st);
  simscore_pairs_kernel<<<dim3((unsigned)T, (unsigned)(L - 1)), 256, 0, st>>>(xs, L, T, d, sums);
  simscore_finish_kernel<<<(L + 63) / 64, 64, 0, st>>>(sums, L, T, sim, simscore);
}

}  // namespace skv
