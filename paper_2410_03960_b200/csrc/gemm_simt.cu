// Shape-generic SIMT GEMM with fp32 accumulation: C = A[M,K] * B[N,K]^T.
// This is the fp32 model's GEMM and the bf16 model's path for shapes the tcgen05 kernels do not tile
// (K not a multiple of 64, N not a multiple of 128).  Every load is bounds-checked; no alignment assumed.
#include "common.cuh"

namespace skv {

constexpr int SBM = 64, SBN = 64, SBK = 16;

template <typename TA, typename TW>
__global__ void __launch_bounds__(256) gemm_simt_kernel(const TA *__restrict__ A, const TW *__restrict__ B, int M, int N,
                                                        int K, OutDesc out, int col0) {
  __shared__ float As[SBK][SBM + 1];
  __shared__ float Bs[SBK][SBN + 1];
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;   // 16 x 16 threads, 4 x 4 outputs each
  const int m0 = blockIdx.y * SBM, n0 = blockIdx.x * SBN;
  float acc[4][4] = {};
  for (int k0 = 0; k0 < K; k0 += SBK) {
    for (int i = threadIdx.x; i < SBM * SBK; i += 256) {
      const int r = i / SBK, c = i % SBK;
      const int gm = m0 + r, gk = k0 + c;
      As[c][r] = (gm < M && gk < K) ? to_f(A[(size_t)gm * K + gk]) : 0.f;
    }
    for (int i = threadIdx.x; i < SBN * SBK; i += 256) {
      const int r = i / SBK, c = i % SBK;
      const int gn = n0 + r, gk = k0 + c;
      Bs[c][r] = (gn < N && gk < K) ? to_f(B[(size_t)gn * K + gk]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < SBK; ++k) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[k][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = Bs[k][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int row = m0 + ty * 4 + i;
    if (row >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int col = n0 + tx * 4 + j;
      if (col < N) store_out<TA, TW>(out, row, col0 + col, acc[i][j]);
    }
  }
}

template <typename TA, typename TW>
void launch_gemm_simt(const TA *A, const TW *B, int M, int N, int K, OutDesc out, int col0, cudaStream_t st) {
  if (M <= 0 || N <= 0) return;
  dim3 grid((N + SBN - 1) / SBN, (M + SBM - 1) / SBM);
  gemm_simt_kernel<TA, TW><<<grid, 256, 0, st>>>(A, B, M, N, K, out, col0);
}
template void launch_gemm_simt<float, float>(const float *, const float *, int, int, int, OutDesc, int, cudaStream_t);
template void launch_gemm_simt<bf16, bf16>(const bf16 *, const bf16 *, int, int, int, OutDesc, int, cudaStream_t);
template void launch_gemm_simt<__half, bf16>(const __half *, const bf16 *, int, int, int, OutDesc, int, cudaStream_t);

}  // namespace skv
