// The last-token path of SwiftKV prefill: only the last token of each prompt runs layers l+1..L (footnote of
// Sec. 3.2; Sec. 3.5), so every projection here has at most 8 activation rows and is bound by streaming the
// weights from HBM exactly once; attention is one query per (prompt, head) over the cache that the
// SingleInputKV projection filled.  Activations of this path stay in fp32 (they are tiny), weights and the
// cache stay in the model dtype.

#include <cooperative_groups.h>
#include <mma.h>

#include <cstdlib>

#include "common.cuh"
#include "tc_common.cuh"

namespace skv {

// ---------------------------------------------------------------------------------------------------------
// RMSNorm of the few continuing rows: fp32 in, fp32 out, gain in the model dtype
// ---------------------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) tail_rmsnorm_kernel(const float *__restrict__ y, const T *__restrict__ gamma,
                                                           float *__restrict__ out, int d, float eps) {
  const float *yr = y + (size_t)blockIdx.x * d;
  float *orow = out + (size_t)blockIdx.x * d;
  __shared__ float red[8];
  float ss = 0.f;
  const bool vec = (d & 3) == 0;
  if (vec) {
#pragma unroll 4
    for (int i = threadIdx.x * 4; i < d; i += 1024) {
      const float4 v = *reinterpret_cast<const float4 *>(yr + i);
      ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
    }
  } else {
    for (int i = threadIdx.x; i < d; i += blockDim.x) ss += yr[i] * yr[i];
  }
  ss = warp_sum(ss);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int w = 0; w < 8; ++w) tot += red[w];
  const float rstd = rsqrtf(tot / (float)d + eps);
  if (vec) {
#pragma unroll 4
    for (int i = threadIdx.x * 4; i < d; i += 1024) {
      const float4 v = *reinterpret_cast<const float4 *>(yr + i);
      *reinterpret_cast<float4 *>(orow + i) = make_float4(v.x * rstd * to_f(gamma[i]), v.y * rstd * to_f(gamma[i + 1]),
                                                          v.z * rstd * to_f(gamma[i + 2]), v.w * rstd * to_f(gamma[i + 3]));
    }
  } else {
    for (int i = threadIdx.x; i < d; i += blockDim.x) orow[i] = yr[i] * rstd * to_f(gamma[i]);
  }
}
template <typename T>
void launch_tail_rmsnorm(const float *y, const T *gamma, float *out, int rows, int d, float eps, cudaStream_t st) {
  if (rows > 0) tail_rmsnorm_kernel<T><<<rows, 256, 0, st>>>(y, gamma, out, d, eps);
}
template void launch_tail_rmsnorm<float>(const float *, const float *, float *, int, int, float, cudaStream_t);
template void launch_tail_rmsnorm<bf16>(const float *, const bf16 *, float *, int, int, float, cudaStream_t);

// ---------------------------------------------------------------------------------------------------------
// Skinny GEMM, generic: out[r, n] = sum_k act[r, k] * W[n, k] for r < n_rows <= 8; one warp per output feature.
// Used by the fp32 model and for shapes the tensor-core variant does not tile.
// mode: OUT_STORE_F32 / OUT_RESID_ADD_F32; W2 != nullptr -> out = silu(act W^T) * (act W2^T)  (SwiGLU)
// ---------------------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) skinny_generic_kernel(const float *__restrict__ act, const T *__restrict__ W,
                                                             const T *__restrict__ W2, int n_rows, int N, int K,
                                                             float *__restrict__ out, int ldo, int mode) {
  const int lane = threadIdx.x & 31;
  const int warps_total = gridDim.x * (blockDim.x >> 5);
  for (int n = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); n < N; n += warps_total) {
    float acc[MAX_TAIL_ROWS], acc2[MAX_TAIL_ROWS];
#pragma unroll
    for (int r = 0; r < MAX_TAIL_ROWS; ++r) acc[r] = acc2[r] = 0.f;
    const T *wr = W + (size_t)n * K;
    const T *wr2 = W2 ? W2 + (size_t)n * K : nullptr;
    for (int k = lane; k < K; k += 32) {
      const float w = to_f(wr[k]);
      const float w2 = wr2 ? to_f(wr2[k]) : 0.f;
#pragma unroll
      for (int r = 0; r < MAX_TAIL_ROWS; ++r)
        if (r < n_rows) {
          const float a = act[(size_t)r * K + k];
          acc[r] = fmaf(w, a, acc[r]);
          acc2[r] = fmaf(w2, a, acc2[r]);
        }
    }
#pragma unroll
    for (int r = 0; r < MAX_TAIL_ROWS; ++r) {
      if (r < n_rows) {
        float s = warp_sum(acc[r]);
        const float s2 = warp_sum(acc2[r]);
        if (lane == 0) {
          if (W2) s = s / (1.f + __expf(-s)) * s2;
          float *o = out + (size_t)r * ldo + n;
          *o = (mode == OUT_RESID_ADD_F32) ? *o + s : s;
        }
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------------------
// Skinny GEMM on tensor cores with the operands swapped: the 16 x 16 "A" tile of mma.m16n8k16 holds 16 output
// features (rows of W) and the 8-wide "B" tile holds the (at most 8) continuing tokens, so no tensor-core
// work is wasted on padding rows.  Each lane fetches 16 contiguous bytes of two W rows per 32-wide K step
// straight from global memory; the K index is permuted identically for W and the activations (a dot product
// does not care), which makes those 16 bytes exactly the lane's fragment of two MMAs.  fp32 activations are
// split into bf16 hi + lo parts (two MMAs), so the activations keep ~16 mantissa bits.
// A block = 8 warps works on one 16-feature tile with K split across the warps, then reduces in shared memory.
// Matrices with few output features (N = 4096: 256 tiles) would leave most of the GPU idle and make every warp walk
// its K range in several dependent batches of loads, so a thread-block CLUSTER of `ks` CTAs shares one tile: each CTA
// takes 1/ks of K, the partial tiles are written into the first CTA's shared memory over DSMEM and summed there in
// rank order (deterministic), and that CTA runs the epilogue.
// ---------------------------------------------------------------------------------------------------------
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void split_hi_lo(float x0, float x1, uint32_t &hi, uint32_t &lo) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(x0, x1);
  const float2 hf = __bfloat1622float2(h);
  const __nv_bfloat162 l = __floats2bfloat162_rn(x0 - hf.x, x1 - hf.y);
  hi = *reinterpret_cast<const uint32_t *>(&h);
  lo = *reinterpret_cast<const uint32_t *>(&l);
}

constexpr int SK_WARPS = 8;
constexpr int SK_MAX_CLUSTER = 8;

// EPI: 0 = one weight matrix; 1 = two, combined as silu(act W^T) * (act W2^T); 2 = two, stored to out and out2
template <int EPI>
__global__ void __launch_bounds__(SK_WARPS * 32) skinny_mma_kernel(const float *__restrict__ act, const bf16 *__restrict__ W,
                                                                   const bf16 *__restrict__ W2, int n_rows, int N, int K,
                                                                   float *__restrict__ out, float *__restrict__ out2, int ldo,
                                                                   int mode, int ks) {
  namespace cg = cooperative_groups;
  constexpr bool SWIGLU = EPI != 0;      // (two accumulators: the name is kept from the first user)
  __shared__ float red[SK_WARPS][SWIGLU ? 2 : 1][32][4];
  __shared__ float cred[SK_MAX_CLUSTER][SWIGLU ? 2 : 1][32][4];     // partial tiles of the other CTAs of the cluster
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const int rank = blockIdx.x % ks;                                 // = rank in the cluster (cluster dims (ks, 1, 1))
  const int n0 = (blockIdx.x / ks) * 16;
  const bf16 *w_lo = W + (size_t)(n0 + g) * K + 8 * t;          // row g of the tile
  const bf16 *w_hi = W + (size_t)(n0 + g + 8) * K + 8 * t;      // row g + 8
  const bf16 *u_lo = SWIGLU ? W2 + (size_t)(n0 + g) * K + 8 * t : nullptr;
  const bf16 *u_hi = SWIGLU ? W2 + (size_t)(n0 + g + 8) * K + 8 * t : nullptr;
  const float *a_row = act + (size_t)g * K + 8 * t;              // token g
  const bool tok_ok = g < n_rows;
  float c[4] = {0.f, 0.f, 0.f, 0.f}, c2[4] = {0.f, 0.f, 0.f, 0.f};
  // this CTA's share of the K steps
  const int all_steps = K / 32;
  const int step_lo = (int)((long long)all_steps * rank / ks), steps = (int)((long long)all_steps * (rank + 1) / ks);
  // software pipeline: the loads of U K-steps are issued together before any of their MMAs, so that each lane keeps
  // 2U (4U with SwiGLU) 16-byte weight loads in flight
  constexpr int U = SWIGLU ? 2 : 4;
  for (int s0 = step_lo + warp * U; s0 < steps; s0 += U * SK_WARPS) {
    uint4 wl[U], wh[U], ul[U], uh[U];
    float4 xa[U], xb[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int s = s0 + u;
      const bool on = s < steps;
      const int kb = on ? s * 32 : 0;
      const uint4 z = make_uint4(0u, 0u, 0u, 0u);
      wl[u] = on ? __ldcs(reinterpret_cast<const uint4 *>(w_lo + kb)) : z;   // weights are streamed once
      wh[u] = on ? __ldcs(reinterpret_cast<const uint4 *>(w_hi + kb)) : z;
      if (SWIGLU) {
        ul[u] = on ? __ldcs(reinterpret_cast<const uint4 *>(u_lo + kb)) : z;
        uh[u] = on ? __ldcs(reinterpret_cast<const uint4 *>(u_hi + kb)) : z;
      }
      xa[u] = make_float4(0.f, 0.f, 0.f, 0.f);
      xb[u] = xa[u];
      if (tok_ok && on) {
        xa[u] = *reinterpret_cast<const float4 *>(a_row + kb);
        xb[u] = *reinterpret_cast<const float4 *>(a_row + kb + 4);
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      uint32_t bh[4], bl[4];
      split_hi_lo(xa[u].x, xa[u].y, bh[0], bl[0]);
      split_hi_lo(xa[u].z, xa[u].w, bh[1], bl[1]);
      split_hi_lo(xb[u].x, xb[u].y, bh[2], bl[2]);
      split_hi_lo(xb[u].z, xb[u].w, bh[3], bl[3]);
      // first MMA: K slots (2t,2t+1) <- elements 0,1 and (2t+8,2t+9) <- elements 2,3; second MMA: elements 4..7
      const uint32_t a1[4] = {wl[u].x, wh[u].x, wl[u].y, wh[u].y}, a2[4] = {wl[u].z, wh[u].z, wl[u].w, wh[u].w};
      mma_bf16_16816(c, a1, bh[0], bh[1]);
      mma_bf16_16816(c, a1, bl[0], bl[1]);
      mma_bf16_16816(c, a2, bh[2], bh[3]);
      mma_bf16_16816(c, a2, bl[2], bl[3]);
      if (SWIGLU) {
        const uint32_t d1[4] = {ul[u].x, uh[u].x, ul[u].y, uh[u].y}, d2[4] = {ul[u].z, uh[u].z, ul[u].w, uh[u].w};
        mma_bf16_16816(c2, d1, bh[0], bh[1]);
        mma_bf16_16816(c2, d1, bl[0], bl[1]);
        mma_bf16_16816(c2, d2, bh[2], bh[3]);
        mma_bf16_16816(c2, d2, bl[2], bl[3]);
      }
    }
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    red[warp][0][lane][i] = c[i];
    if (SWIGLU) red[warp][SWIGLU ? 1 : 0][lane][i] = c2[i];
  }
  __syncthreads();
  float s[4] = {0.f, 0.f, 0.f, 0.f}, s2[4] = {0.f, 0.f, 0.f, 0.f};
  if (warp == 0) {
#pragma unroll
    for (int w = 0; w < SK_WARPS; ++w)
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        s[i] += red[w][0][lane][i];
        if (SWIGLU) s2[i] += red[w][SWIGLU ? 1 : 0][lane][i];
      }
  }
  if (ks > 1) {
    cg::cluster_group cluster = cg::this_cluster();
    if (warp == 0 && rank != 0) {       // hand this CTA's partial tile to the first CTA of the cluster
      float *dst = cluster.map_shared_rank(&cred[0][0][0][0], 0);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        dst[((rank * (SWIGLU ? 2 : 1) + 0) * 32 + lane) * 4 + i] = s[i];
        if (SWIGLU) dst[((rank * 2 + 1) * 32 + lane) * 4 + i] = s2[i];
      }
    }
    cluster.sync();
    if (rank != 0) return;
    if (warp == 0) {
      for (int r = 1; r < ks; ++r)      // fixed order: the sum does not depend on which CTA finished first
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          s[i] += cred[r][0][lane][i];
          if (SWIGLU) s2[i] += cred[r][SWIGLU ? 1 : 0][lane][i];
        }
    }
  }
  if (warp == 0) {
    // fragment element i: feature n0 + g + 8*(i/2), token 2t + (i%2)
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int n = n0 + g + 8 * (i >> 1), r = 2 * t + (i & 1);
      if (r < n_rows && n < N) {
        float v = s[i];
        if (EPI == 1) v = v / (1.f + __expf(-v)) * s2[i];
        float *o = out + (size_t)r * ldo + n;
        *o = (mode == OUT_RESID_ADD_F32) ? *o + v : v;
        if (EPI == 2) out2[(size_t)r * ldo + n] = s2[i];
      }
    }
  }
}

// cluster size: enough CTAs to fill the GPU several times over, at least 2 K steps per warp
static int skinny_cluster(int tiles, int steps) {
  int ks = 1;
  while (ks < SK_MAX_CLUSTER && tiles * ks < 1024 && steps / (2 * ks) >= 2 * SK_WARPS) ks *= 2;
  return ks;
}
template <int EPI>
static void launch_skinny_mma(const float *act, const bf16 *w, const bf16 *w2, int n_rows, int N, int K, float *out, float *out2,
                              int ldo, int mode, cudaStream_t st) {
  const int tiles = N / 16, ks = skinny_cluster(tiles, K / 32);
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)(tiles * ks));
  cfg.blockDim = dim3(SK_WARPS * 32);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)ks;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaLaunchKernelEx(&cfg, skinny_mma_kernel<EPI>, act, w, w2, n_rows, N, K, out, out2, ldo, mode, ks);
}

template <typename T>
void launch_skinny_gemm(const float *act, const T *W, const T *W2, int n_rows, int N, int K, float *out, int ldo,
                        int mode, cudaStream_t st) {
  if (n_rows <= 0 || N <= 0) return;
  if constexpr (sizeof(T) == 2) {
    if ((K % 32) == 0 && (N % 16) == 0) {
      const bf16 *w = reinterpret_cast<const bf16 *>(W), *w2 = reinterpret_cast<const bf16 *>(W2);
      if (W2) launch_skinny_mma<1>(act, w, w2, n_rows, N, K, out, nullptr, ldo, mode, st);
      else launch_skinny_mma<0>(act, w, w2, n_rows, N, K, out, nullptr, ldo, mode, st);
      return;
    }
  }
  int blocks = (N + 7) / 8;
  if (blocks > 148 * 8) blocks = 148 * 8;
  skinny_generic_kernel<T><<<blocks, 256, 0, st>>>(act, W, W2, n_rows, N, K, out, ldo, mode);
}
template <typename T>
void launch_skinny_gemm_dual(const float *act, const T *W, const T *W2, int n_rows, int N, int K, float *out, float *out2,
                             int ldo, cudaStream_t st) {
  if (n_rows <= 0 || N <= 0) return;
  if constexpr (sizeof(T) == 2) {
    if ((K % 32) == 0 && (N % 16) == 0) {
      launch_skinny_mma<2>(act, reinterpret_cast<const bf16 *>(W), reinterpret_cast<const bf16 *>(W2), n_rows, N, K, out, out2, ldo,
                           OUT_STORE_F32, st);
      return;
    }
  }
  launch_skinny_gemm<T>(act, W, nullptr, n_rows, N, K, out, ldo, OUT_STORE_F32, st);
  launch_skinny_gemm<T>(act, W2, nullptr, n_rows, N, K, out2, ldo, OUT_STORE_F32, st);
}
template void launch_skinny_gemm_dual<float>(const float *, const float *, const float *, int, int, int, float *, float *, int, cudaStream_t);
template void launch_skinny_gemm_dual<bf16>(const float *, const bf16 *, const bf16 *, int, int, int, float *, float *, int, cudaStream_t);
template void launch_skinny_gemm<float>(const float *, const float *, const float *, int, int, int, float *, int, int, cudaStream_t);
template void launch_skinny_gemm<bf16>(const float *, const bf16 *, const bf16 *, int, int, int, float *, int, int, cudaStream_t);

// ---------------------------------------------------------------------------------------------------------
// single-query attention over the cache, split along the keys.
//   pass 1: block (split, KV head, prompt), one warp per query head of the group, scans its key range 32 keys
//           at a time -- one key per lane for the scores (128-bit loads of the K row), online softmax, then the
//           probabilities are broadcast while the lanes accumulate their slice of the output -- and writes
//           (max, sum, acc[hd]) to scratch;
//   pass 2: block (head, prompt) merges the splits and writes the normalised fp32 output row.
// ---------------------------------------------------------------------------------------------------------
__host__ __device__ inline int tail_chunk(int max_seq_len) {
  int c = (max_seq_len + 63) / 64;          // at most 64 splits
  c = (c + 127) / 128 * 128;                // whole rounds of the block's 4 warps x 32 keys
  return c < 512 ? 512 : c;
}

template <typename T>
__device__ __forceinline__ float dot_row(const float *__restrict__ qs, const T *__restrict__ kr, int hd) {
  constexpr int V = 16 / sizeof(T);
  float dot = 0.f;
  if ((hd % V) == 0) {
    for (int i = 0; i < hd; i += V) {
      const uint4 raw = *reinterpret_cast<const uint4 *>(kr + i);
      const T *e = reinterpret_cast<const T *>(&raw);
#pragma unroll
      for (int k = 0; k < V; ++k) dot = fmaf(qs[i + k], to_f(e[k]), dot);
    }
  } else {
    for (int i = 0; i < hd; ++i) dot = fmaf(qs[i], to_f(kr[i]), dot);
  }
  return dot;
}

// Block (split, KV head, prompt), 4 warps.  Every warp walks 32-key chunks of the block's key range for ALL query heads
// of the KV head's group at once, so each K and V row is fetched once per group.  The 32 K rows and 32 V rows of a chunk
// are copied into the warp's shared-memory tiles with coalesced 16-byte cp.async (a lane-per-key read straight from
// global memory touches 16 bytes of 32 different lines per instruction and thrashes L1), one chunk ahead of the math:
//   scores : lane = key; its K row is read from the padded tile with 128-bit loads and dotted with the REP query vectors
//   softmax: online, per head, warp-wide max / sum
//   output : for each of the 32 keys the V row is read once (lane = 4 consecutive dims) and accumulated into REP x 4
//            registers with the probabilities broadcast by shuffle
// then the warps are merged in shared memory and (max, sum, acc[hd]) per head goes to scratch.
constexpr int TA_WARPS = 4;
template <typename T>
struct TailTile {
  static constexpr int ROW = 128 * (int)sizeof(T);   // bytes of one K / V row of a head (head_dim 128)
  static constexpr int KSTRIDE = ROW + 16;           // padded: lane-per-row 128-bit reads hit 32 different banks
  static constexpr int LPR = ROW / 16;               // lanes that copy one row
  static constexpr int RPI = 32 / LPR;               // rows per copy instruction
  static constexpr int NI = 32 / RPI;                // copy instructions per 32-row tile
  static constexpr int K_BYTES = 32 * KSTRIDE, V_BYTES = 32 * ROW;
};
__device__ __forceinline__ void cp_async16(void *smem, const void *gmem) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem)), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// element dd of a query row, rotated to the row's position when the caller asks for it (same arithmetic as rope_kernel)
__device__ __forceinline__ float load_query(const float *__restrict__ qr, int dd, int hd, int b, const TailOpts &rope) {
  const float v = qr[dd];
  if (!rope.pos) return v;
  const int half = hd >> 1, i = dd < half ? dd : dd - half;
  const size_t t = (size_t)rope.pos[b] * half + i;
  const float c = rope.cos_tab[t], s = rope.sin_tab[t];
  return dd < half ? v * c - qr[dd + half] * s : v * c + qr[dd - half] * s;
}

template <typename T, int REP, int HD>
__global__ void __launch_bounds__(TA_WARPS * 32) tail_attention_group_kernel(
    const float *__restrict__ q, const T *__restrict__ kc, const T *__restrict__ vc, const float *__restrict__ kscale,
    const float *__restrict__ vscale, const int32_t *__restrict__ cu, const int32_t *__restrict__ len,
    const int32_t *__restrict__ blk, int blk_stride, int n_q, int n_kv, int chunk, int n_splits, float scale,
    float *__restrict__ scratch, TailOpts rope) {
  static_assert(HD == 128, "one lane owns 4 consecutive output dims");
  using TT = TailTile<T>;
  extern __shared__ __align__(16) uint8_t ta_smem[];
  float (*qs)[HD] = reinterpret_cast<float (*)[HD]>(ta_smem);                 // [REP][HD]
  uint8_t *tiles = ta_smem + REP * HD * sizeof(float);
  // (the KV heads of one key range are neighbours in the grid: their blocks run at the same time and together read whole
  //  cache rows -- all heads of a token are contiguous -- instead of one 256-byte piece per 2 KB row each at its own time)
  const int kvh = blockIdx.x, split = blockIdx.y, b = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  uint8_t *kt = tiles + warp * (TT::K_BYTES + TT::V_BYTES), *vt = kt + TT::K_BYTES;
  const int first = cu[b], n = len ? len[b] : cu[b + 1] - cu[b];
  const int k_begin = split * chunk, k_end = min(n, k_begin + chunk);
  if (k_begin >= k_end) {             // a split past the sequence's end: an empty partial for the merge pass
    if (threadIdx.x < REP) {
      float *dst = scratch + (((size_t)b * n_q + kvh * REP + threadIdx.x) * n_splits + split) * (HD + 2);
      dst[0] = -INFINITY;
      dst[1] = 0.f;
    }
    return;
  }
  for (int i = threadIdx.x; i < REP * HD; i += blockDim.x)
    qs[i / HD][i % HD] = load_query(q + ((size_t)b * n_q + kvh * REP + i / HD) * HD, i % HD, HD, b, rope) * scale;

  // copy rows [c0, c0 + 32) of this KV head into a tile (rows past k_end are skipped and never read)
  auto issue_tile = [&](const T *base, uint8_t *tile, int stride, int c0) {
    const int sub = lane % TT::LPR;
#pragma unroll
    for (int i = 0; i < TT::NI; ++i) {
      const int r = i * TT::RPI + lane / TT::LPR, key = c0 + r;
      if (key < k_end)
        cp_async16(tile + r * stride + sub * 16,
                   reinterpret_cast<const uint8_t *>(base + (kv_row_of(blk, blk_stride, b, first, key) * n_kv + kvh) * HD) + sub * 16);
    }
    cp_async_commit();
  };
  int c0 = k_begin + warp * 32;
  if (c0 < k_end) { issue_tile(kc, kt, TT::KSTRIDE, c0); issue_tile(vc, vt, TT::ROW, c0); }
  __syncthreads();                    // qs

  float m[REP], l[REP], acc[REP][4];
#pragma unroll
  for (int r = 0; r < REP; ++r) { m[r] = -INFINITY; l[r] = 0.f; acc[r][0] = acc[r][1] = acc[r][2] = acc[r][3] = 0.f; }

  for (; c0 < k_end; c0 += TA_WARPS * 32) {
    const int next = c0 + TA_WARPS * 32;
    const bool more = next < k_end;
    const int key = c0 + lane;
    const bool valid = key < k_end;
    cp_async_wait<1>();               // pending groups: K(c0), V(c0) -> K(c0) has landed
    __syncwarp();
    float sc[REP];
#pragma unroll
    for (int r = 0; r < REP; ++r) sc[r] = 0.f;
    float v_s = 1.f;     // FP8 cache: this lane's key carries one scale for its K row and one for its V row
    if (valid) {
      const uint8_t *kr = kt + lane * TT::KSTRIDE;
      constexpr int V = 16 / sizeof(T);
#pragma unroll 4
      for (int i = 0; i < HD; i += V) {
        const uint4 raw = *reinterpret_cast<const uint4 *>(kr + i * sizeof(T));
        const T *e = reinterpret_cast<const T *>(&raw);
#pragma unroll
        for (int k = 0; k < V; ++k) {
          const float kv_ = to_f(e[k]);
#pragma unroll
          for (int r = 0; r < REP; ++r) sc[r] = fmaf(qs[r][i + k], kv_, sc[r]);
        }
      }
      if (kscale) {
        const size_t krow = kv_row_of(blk, blk_stride, b, first, key);
        const float k_s = kscale[krow];
        v_s = vscale[krow];
#pragma unroll
        for (int r = 0; r < REP; ++r) sc[r] *= k_s;
      }
    }
    __syncwarp();                     // every lane is done with the K tile
    if (more) issue_tile(kc, kt, TT::KSTRIDE, next);
    float pe[REP];
#pragma unroll
    for (int r = 0; r < REP; ++r) {
      const float s = valid ? sc[r] : -INFINITY;
      const float m_new = fmaxf(m[r], warp_max(s));
      pe[r] = valid ? __expf(s - m_new) : 0.f;
      const float corr = __expf(m[r] - m_new);
      l[r] = l[r] * corr + warp_sum(pe[r]);
      acc[r][0] *= corr; acc[r][1] *= corr; acc[r][2] *= corr; acc[r][3] *= corr;
      m[r] = m_new;
      pe[r] *= v_s;        // (after the row sum: the V row's scale rides on the probability)
    }
    if (more) cp_async_wait<1>(); else cp_async_wait<0>();     // pending: V(c0) [, K(next)] -> V(c0) has landed
    __syncwarp();
    const int n_here = min(32, k_end - c0);
#pragma unroll 4
    for (int i = 0; i < n_here; ++i) {
      const T *vr = reinterpret_cast<const T *>(vt + i * TT::ROW) + lane * 4;
      float v0, v1, v2, v3;
      if constexpr (sizeof(T) == 2) {
        const uint2 raw = *reinterpret_cast<const uint2 *>(vr);
        const T *e = reinterpret_cast<const T *>(&raw);
        v0 = to_f(e[0]); v1 = to_f(e[1]); v2 = to_f(e[2]); v3 = to_f(e[3]);
      } else if constexpr (sizeof(T) == 1) {
        const uint32_t raw = *reinterpret_cast<const uint32_t *>(vr);
        const T *e = reinterpret_cast<const T *>(&raw);
        v0 = to_f(e[0]); v1 = to_f(e[1]); v2 = to_f(e[2]); v3 = to_f(e[3]);
      } else {
        const float4 raw = *reinterpret_cast<const float4 *>(vr);
        v0 = raw.x; v1 = raw.y; v2 = raw.z; v3 = raw.w;
      }
#pragma unroll
      for (int r = 0; r < REP; ++r) {
        const float pi = __shfl_sync(0xffffffffu, pe[r], i);
        acc[r][0] = fmaf(pi, v0, acc[r][0]); acc[r][1] = fmaf(pi, v1, acc[r][1]);
        acc[r][2] = fmaf(pi, v2, acc[r][2]); acc[r][3] = fmaf(pi, v3, acc[r][3]);
      }
    }
    __syncwarp();                     // every lane is done with the V tile
    if (more) issue_tile(vc, vt, TT::ROW, next);
  }
  // merge the warps; the tiles are free now (every copy has landed and been consumed)
  __syncthreads();
  float *w_m = reinterpret_cast<float *>(tiles);                 // [TA_WARPS][REP]
  float *w_l = w_m + TA_WARPS * REP;                             // [TA_WARPS][REP]
  float *w_acc = w_l + TA_WARPS * REP;                           // [TA_WARPS][REP][HD]
#pragma unroll
  for (int r = 0; r < REP; ++r) {
    if (lane == 0) { w_m[warp * REP + r] = m[r]; w_l[warp * REP + r] = l[r]; }
    *reinterpret_cast<float4 *>(&w_acc[(warp * REP + r) * HD + lane * 4]) = make_float4(acc[r][0], acc[r][1], acc[r][2], acc[r][3]);
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < REP * HD; idx += blockDim.x) {
    const int r = idx / HD, dd = idx % HD;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < TA_WARPS; ++w) M = fmaxf(M, w_m[w * REP + r]);
    float a = 0.f, L = 0.f;
#pragma unroll
    for (int w = 0; w < TA_WARPS; ++w) {
      const float f = (w_m[w * REP + r] == -INFINITY) ? 0.f : __expf(w_m[w * REP + r] - M);
      a += w_acc[(w * REP + r) * HD + dd] * f;
      L += w_l[w * REP + r] * f;
    }
    float *dst = scratch + (((size_t)b * n_q + kvh * REP + r) * n_splits + split) * (HD + 2);
    if (dd == 0) { dst[0] = M; dst[1] = L; }
    dst[2 + dd] = a;
  }
}

// The same block / warp / tile structure with the arithmetic on the tensor cores (bf16 cache, head_dim 128, <= 8 query heads
// per KV head): the scalar form above spends ~1400 issue slots per 32-key tile and is bound by the latency of its FMA chains
// at the occupancy its shared memory allows; here a tile is 64 + 64 mma.sync.m16n8k16 plus ~100 loads.
//   scores : S[head, key] = Q K^T with the group's query rows as the A operand (rows >= REP are zero; fp32 queries as bf16
//            hi + lo, so the products carry ~16 significant bits of q against the exact bf16 keys), K rows straight from
//            the padded tile as the B operand;
//   softmax: a lane holds 8 scores of one head (row g = lane / 4), quad reductions give the row maximum and sum;
//   output : O[head, dim] += P V with the probabilities (bf16 hi + lo) re-used from the score accumulators as the A operand
//            and V read through ldmatrix.trans from a padded tile.
constexpr int TM_VSTRIDE = 256 + 16;
constexpr int TM_TILE_BYTES = 32 * (256 + 16) + 32 * TM_VSTRIDE;
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3, const void *p) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"((uint32_t)__cvta_generic_to_shared(p)));
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3, const void *p) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"((uint32_t)__cvta_generic_to_shared(p)));
}
template <int REP>
__global__ void __launch_bounds__(TA_WARPS * 32, 3) tail_attention_mma_kernel(
    const float *__restrict__ q, const bf16 *__restrict__ kc, const bf16 *__restrict__ vc, const int32_t *__restrict__ cu,
    const int32_t *__restrict__ len, const int32_t *__restrict__ blk, int blk_stride, int n_q, int n_kv, int chunk, int n_splits,
    float scale, float *__restrict__ scratch, TailOpts rope) {
  constexpr int HD = 128, KSTRIDE = 256 + 16;
  extern __shared__ __align__(16) uint8_t ta_smem[];
  float (*qs)[HD] = reinterpret_cast<float (*)[HD]>(ta_smem);                 // [REP][HD]
  uint8_t *tiles = ta_smem + REP * HD * sizeof(float);
  const int kvh = blockIdx.x, split = blockIdx.y, b = blockIdx.z;      // (KV heads fastest: see tail_attention_group_kernel)
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  uint8_t *kt = tiles + warp * TM_TILE_BYTES, *vt = kt + 32 * KSTRIDE;
  const int first = cu[b], n = len ? len[b] : cu[b + 1] - cu[b];
  const int k_begin = split * chunk, k_end = min(n, k_begin + chunk);
  if (k_begin >= k_end) {             // a split past the sequence's end: an empty partial for the merge pass
    if (threadIdx.x < REP) {
      float *dst = scratch + (((size_t)b * n_q + kvh * REP + threadIdx.x) * n_splits + split) * (HD + 2);
      dst[0] = -INFINITY;
      dst[1] = 0.f;
    }
    return;
  }
  for (int i = threadIdx.x; i < REP * HD; i += blockDim.x)
    qs[i / HD][i % HD] = load_query(q + ((size_t)b * n_q + kvh * REP + i / HD) * HD, i % HD, HD, b, rope) * scale;

  auto issue_tile = [&](const bf16 *base, uint8_t *tile, int c0) {      // rows [c0, c0 + 32) of this KV head; 16 lanes copy one row
    const int sub = lane & 15;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const int r = i * 2 + (lane >> 4), key = c0 + r;
      if (key < k_end)
        cp_async16(tile + r * KSTRIDE + sub * 16,
                   reinterpret_cast<const uint8_t *>(base + (kv_row_of(blk, blk_stride, b, first, key) * n_kv + kvh) * HD) + sub * 16);
      else
        *reinterpret_cast<uint4 *>(tile + r * KSTRIDE + sub * 16) = make_uint4(0u, 0u, 0u, 0u);      // (keeps NaN bit patterns out of P V)
    }
    cp_async_commit();
  };
  int c0 = k_begin + warp * 32;
  if (c0 < k_end) { issue_tile(kc, kt, c0); issue_tile(vc, vt, c0); }
  __syncthreads();                    // qs

  // the group's queries as A fragments (row g of the 16 x 16 tile; rows 8..15 and rows >= REP are zero)
  uint32_t qh[8][2], ql[8][2];
#pragma unroll
  for (int kk = 0; kk < 8; ++kk) {
    float x0 = 0.f, x1 = 0.f, x2 = 0.f, x3 = 0.f;
    if (g < REP) {
      x0 = qs[g][kk * 16 + 2 * t]; x1 = qs[g][kk * 16 + 2 * t + 1];
      x2 = qs[g][kk * 16 + 8 + 2 * t]; x3 = qs[g][kk * 16 + 8 + 2 * t + 1];
    }
    split_hi_lo(x0, x1, qh[kk][0], ql[kk][0]);
    split_hi_lo(x2, x3, qh[kk][1], ql[kk][1]);
  }
  float m = -INFINITY, l = 0.f;       // of head g (the four lanes of a quad hold the same values)
  float acc[16][4];
#pragma unroll
  for (int nd = 0; nd < 16; ++nd) acc[nd][0] = acc[nd][1] = acc[nd][2] = acc[nd][3] = 0.f;

  for (; c0 < k_end; c0 += TA_WARPS * 32) {
    const int next = c0 + TA_WARPS * 32;
    const bool more = next < k_end;
    cp_async_wait<1>();               // pending groups: K(c0), V(c0) -> K(c0) has landed
    __syncwarp();
    float sc[4][4];
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) {
      sc[nt][0] = sc[nt][1] = sc[nt][2] = sc[nt][3] = 0.f;
      // one ldmatrix brings the B fragments of two 16-dim steps: 8 key rows x (4 x 16 bytes)
      const uint8_t *kr = kt + (nt * 8 + (lane & 7)) * KSTRIDE + (lane >> 3) * 16;
#pragma unroll
      for (int kp = 0; kp < 4; ++kp) {
        uint32_t b[4];
        ldmatrix_x4(b[0], b[1], b[2], b[3], kr + kp * 64);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int kk = 2 * kp + h;
          const uint32_t ah[4] = {qh[kk][0], 0u, qh[kk][1], 0u}, al[4] = {ql[kk][0], 0u, ql[kk][1], 0u};
          mma_bf16_16816(sc[nt], ah, b[2 * h], b[2 * h + 1]);
          mma_bf16_16816(sc[nt], al, b[2 * h], b[2 * h + 1]);
        }
      }
    }
    __syncwarp();                     // every lane is done with the K tile
    if (more) issue_tile(kc, kt, next);
    // online softmax of head g over the tile's 32 keys: this lane holds keys nt * 8 + 2 t, + 1
    float mx = -INFINITY;
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) {
      if (c0 + nt * 8 + 2 * t >= k_end) sc[nt][0] = -INFINITY;
      if (c0 + nt * 8 + 2 * t + 1 >= k_end) sc[nt][1] = -INFINITY;
      mx = fmaxf(mx, fmaxf(sc[nt][0], sc[nt][1]));
    }
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
    const float m_new = fmaxf(m, mx);
    const float corr = __expf(m - m_new);
    float sum = 0.f;
    uint32_t ph[4], pl[4];
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) {
      const float p0 = __expf(sc[nt][0] - m_new), p1 = __expf(sc[nt][1] - m_new);
      sum += p0 + p1;
      split_hi_lo(p0, p1, ph[nt], pl[nt]);
    }
    sum += __shfl_xor_sync(0xffffffffu, sum, 1);
    sum += __shfl_xor_sync(0xffffffffu, sum, 2);
    l = l * corr + sum;
    m = m_new;
#pragma unroll
    for (int nd = 0; nd < 16; ++nd) { acc[nd][0] *= corr; acc[nd][1] *= corr; }
    if (more) cp_async_wait<1>(); else cp_async_wait<0>();     // pending: V(c0) [, K(next)] -> V(c0) has landed
    __syncwarp();
    // P V: keys in two steps of 16; ldmatrix.trans brings, per instruction, both key halves of two 8-dim column blocks
#pragma unroll
    for (int ks = 0; ks < 2; ++ks) {
      const uint32_t ah[4] = {ph[2 * ks], 0u, ph[2 * ks + 1], 0u}, al[4] = {pl[2 * ks], 0u, pl[2 * ks + 1], 0u};
      const uint8_t *vrow = vt + (ks * 16 + (lane & 7) + ((lane >> 3) & 1) * 8) * TM_VSTRIDE + (lane >> 4) * 16;
#pragma unroll
      for (int np = 0; np < 8; ++np) {
        uint32_t b00, b01, b10, b11;
        ldmatrix_x4_trans(b00, b01, b10, b11, vrow + np * 32);
        mma_bf16_16816(acc[2 * np], ah, b00, b01);
        mma_bf16_16816(acc[2 * np], al, b00, b01);
        mma_bf16_16816(acc[2 * np + 1], ah, b10, b11);
        mma_bf16_16816(acc[2 * np + 1], al, b10, b11);
      }
    }
    __syncwarp();                     // every lane is done with the V tile
    if (more) issue_tile(vc, vt, next);
  }
  // merge the warps; the tiles are free now (every copy has landed and been consumed)
  __syncthreads();
  float *w_m = reinterpret_cast<float *>(tiles);                 // [TA_WARPS][REP]
  float *w_l = w_m + TA_WARPS * REP;                             // [TA_WARPS][REP]
  float *w_acc = w_l + TA_WARPS * REP;                           // [TA_WARPS][REP][HD]
  if (g < REP) {
    if (t == 0) { w_m[warp * REP + g] = m; w_l[warp * REP + g] = l; }
#pragma unroll
    for (int nd = 0; nd < 16; ++nd)
      *reinterpret_cast<float2 *>(&w_acc[(warp * REP + g) * HD + nd * 8 + 2 * t]) = make_float2(acc[nd][0], acc[nd][1]);
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < REP * HD; idx += blockDim.x) {
    const int r = idx / HD, dd = idx % HD;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < TA_WARPS; ++w) M = fmaxf(M, w_m[w * REP + r]);
    float a = 0.f, L = 0.f;
#pragma unroll
    for (int w = 0; w < TA_WARPS; ++w) {
      const float f = (w_m[w * REP + r] == -INFINITY) ? 0.f : __expf(w_m[w * REP + r] - M);
      a += w_acc[(w * REP + r) * HD + dd] * f;
      L += w_l[w * REP + r] * f;
    }
    float *dst = scratch + (((size_t)b * n_q + kvh * REP + r) * n_splits + split) * (HD + 2);
    if (dd == 0) { dst[0] = M; dst[1] = L; }
    dst[2 + dd] = a;
  }
}

// Shape-generic form: block (split, KV head, prompt); warp w = query head kvh*rep + w of that KV head's group, so the
// K / V rows of the block's key range come from HBM once and are shared by the group's heads through L1.
template <typename T, int MAX_E>
__global__ void __launch_bounds__(256) tail_attention_partial_kernel(
    const float *__restrict__ q, const T *__restrict__ kc, const T *__restrict__ vc, const float *__restrict__ kscale,
    const float *__restrict__ vscale, const int32_t *__restrict__ cu, const int32_t *__restrict__ len,
    const int32_t *__restrict__ blk, int blk_stride, int n_q, int n_kv, int hd, int chunk, int n_splits, float scale,
    float *__restrict__ scratch, TailOpts rope) {
  extern __shared__ float sm[];   // q of each warp's head: [rep][hd]
  const int split = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rep = n_q / n_kv;
  const int first = cu[b], n = len ? len[b] : cu[b + 1] - cu[b];
  const int k_begin = split * chunk, k_end = min(n, k_begin + chunk);
  for (int hw = warp; hw < rep; hw += (blockDim.x >> 5)) {   // (more heads per group than warps: loop)
    const int h = kvh * rep + hw;
    float *qs = sm + hw * hd;
    const float *qr = q + ((size_t)b * n_q + h) * hd;
    for (int i = lane; i < hd; i += 32) qs[i] = load_query(qr, i, hd, b, rope) * scale;
    __syncwarp();
    float m = -INFINITY, l = 0.f;
    float acc[MAX_E];
#pragma unroll
    for (int e = 0; e < MAX_E; ++e) acc[e] = 0.f;
    for (int c0 = k_begin; c0 < k_end; c0 += 32) {
      const int key = c0 + lane;
      float s = -INFINITY, v_s = 1.f;
      if (key < k_end) {
        const size_t krow = kv_row_of(blk, blk_stride, b, first, key);
        s = dot_row<T>(qs, kc + (krow * n_kv + kvh) * hd, hd);
        if (kscale) { s *= kscale[krow]; v_s = vscale[krow]; }
      }
      const float m_new = fmaxf(m, warp_max(s));
      float pe = (key < k_end) ? __expf(s - m_new) : 0.f;
      const float corr = __expf(m - m_new);
      l = l * corr + warp_sum(pe);
      pe *= v_s;
#pragma unroll
      for (int e = 0; e < MAX_E; ++e) acc[e] *= corr;
      m = m_new;
      const int n_here = min(32, k_end - c0);
      for (int i = 0; i < n_here; ++i) {
        const float pi = __shfl_sync(0xffffffffu, pe, i);
        const T *vr = vc + (kv_row_of(blk, blk_stride, b, first, c0 + i) * n_kv + kvh) * hd;
#pragma unroll
        for (int e = 0; e < MAX_E; ++e) {
          const int dd = lane + 32 * e;
          if (dd < hd) acc[e] = fmaf(pi, to_f(vr[dd]), acc[e]);
        }
      }
    }
    float *dst = scratch + (((size_t)b * n_q + h) * n_splits + split) * (hd + 2);
    if (lane == 0) { dst[0] = m; dst[1] = l; }
#pragma unroll
    for (int e = 0; e < MAX_E; ++e) {
      const int dd = lane + 32 * e;
      if (dd < hd) dst[2 + dd] = acc[e];
    }
  }
}

__global__ void __launch_bounds__(128) tail_attention_merge_kernel(const float *__restrict__ scratch, float *__restrict__ out,
                                                                   int n_q, int hd, int n_splits) {
  // block (head, prompt): warp 0 turns the splits' (max, sum) pairs into weights -- all loads issued together --, then
  // every thread combines its output dims with independent loads (a serial walk over the splits costs a dependent
  // global-memory round trip per split)
  __shared__ float wgt[64];
  __shared__ float inv_l;
  const int h = blockIdx.x, b = blockIdx.y;
  const float *src = scratch + ((size_t)b * n_q + h) * n_splits * (hd + 2);
  if (threadIdx.x < 32) {
    const int lane = threadIdx.x;
    float ms[2], ls[2];
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const int s = lane + 32 * k;
      ms[k] = s < n_splits ? src[(size_t)s * (hd + 2)] : -INFINITY;
      ls[k] = s < n_splits ? src[(size_t)s * (hd + 2) + 1] : 0.f;
    }
    const float M = warp_max(fmaxf(ms[0], ms[1]));
    float L = 0.f;
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const float w = (ms[k] == -INFINITY) ? 0.f : __expf(ms[k] - M);
      if (lane + 32 * k < 64) wgt[lane + 32 * k] = w;
      L += ls[k] * w;
    }
    L = warp_sum(L);
    if (lane == 0) inv_l = L > 0.f ? 1.f / L : 0.f;     // a sequence without keys: every split is empty, the row is zeros
  }
  __syncthreads();
  for (int dd = threadIdx.x; dd < hd; dd += blockDim.x) {
    float a = 0.f;
#pragma unroll 8
    for (int s = 0; s < n_splits; ++s) {
      const float w = wgt[s];
      if (w != 0.f) a = fmaf(src[(size_t)s * (hd + 2) + 2 + dd], w, a);
    }
    out[((size_t)b * n_q + h) * hd + dd] = a * inv_l;
  }
}

// Most splits any launch with max_seq_len <= max_tokens can use.  The split count ceil(n / tail_chunk(n)) is NOT
// monotonic in n (the chunk is rounded up to whole rounds of 128 keys), so a buffer sized from max_tokens' own split
// count can be too small for a shorter maximum; but chunks are at least 512 keys and tail_chunk never gives more than
// 64 splits, and a launch only ever coarsens the split it starts from.
int tail_max_splits(int max_tokens) {
  const int by_chunk = (max_tokens + 511) / 512;
  return by_chunk < 64 ? by_chunk : 64;
}
size_t tail_attention_scratch_bytes(int max_seqs, int n_q, int hd, int max_tokens) {
  const int rows = max_seqs < MAX_TAIL_ROWS ? max_seqs : MAX_TAIL_ROWS;
  return (size_t)rows * n_q * tail_max_splits(max_tokens) * (hd + 2) * sizeof(float);
}

// (SWIFTKV_TAIL_ATTENTION_SCALAR=1 keeps the scalar kernel: A/B and debugging)
static bool tail_attention_use_mma() {
  static int v = -1;
  if (v < 0) { const char *e = getenv("SWIFTKV_TAIL_ATTENTION_SCALAR"); v = (e && e[0] == '1') ? 0 : 1; }
  return v == 1;
}

template <typename T>
void launch_tail_attention(const float *q, const T *kc, const T *vc, const float *kscale, const float *vscale, float *out,
                           const int32_t *cu_seqlens, const int32_t *len, const int32_t *blk, int blk_stride, int n_seqs,
                           int max_seq_len, int n_q, int n_kv, int hd, float *scratch, cudaStream_t st, TailOpts rope) {
  if (n_seqs <= 0) return;
  int chunk = tail_chunk(max_seq_len);
  if (rope.total_len > 0 && hd == 128) {
    // blocks of `c` keys: about total_len / c + half a ragged block per sequence, times the KV heads; three blocks of the
    // grouped kernel fit an SM.  Cost of a split = waves x keys per block; the coarsest split of the cheapest cost wins.
    static int n_sms = 0;
    if (n_sms == 0) { int dev = 0; cudaGetDevice(&dev); cudaDeviceGetAttribute(&n_sms, cudaDevAttrMultiProcessorCount, dev); if (n_sms < 1) n_sms = 1; }
    const double cap = 3.0 * n_sms;
    double best = 1e300;
    for (int c = chunk; c <= ((max_seq_len + 127) / 128) * 128 && c < chunk + 4096; c += 128) {
      const double blocks = ((double)rope.total_len / c + 0.5 * n_seqs) * n_kv;
      const double cost = ceil(blocks / cap) * (c + 64);
      if (cost <= best) { best = cost; chunk = c; }
    }
  }
  const int n_splits = (max_seq_len + chunk - 1) / chunk;
  const float scale = 1.0f / sqrtf((float)hd);
  const int rep = n_q / n_kv;
  if constexpr (sizeof(T) == 2) {
    if (hd == 128 && !kscale && (rep == 1 || rep == 2 || rep == 4 || rep == 8) && tail_attention_use_mma()) {
      dim3 grid(n_kv, n_splits, n_seqs);
      const size_t smem = (size_t)rep * 128 * sizeof(float) + (size_t)TA_WARPS * TM_TILE_BYTES;
#define SKV_LAUNCH_MMA(R)                                                                                                     \
      do {                                                                                                                    \
        ensure_dynamic_smem(reinterpret_cast<const void *>(tail_attention_mma_kernel<R>), (int)smem);                         \
        tail_attention_mma_kernel<R><<<grid, TA_WARPS * 32, smem, st>>>(q, reinterpret_cast<const bf16 *>(kc),                \
                                                                        reinterpret_cast<const bf16 *>(vc), cu_seqlens, len, blk, \
                                                                        blk_stride, n_q, n_kv, chunk, n_splits, scale, scratch, rope); \
      } while (0)
      if (rep == 1) SKV_LAUNCH_MMA(1);
      else if (rep == 2) SKV_LAUNCH_MMA(2);
      else if (rep == 4) SKV_LAUNCH_MMA(4);
      else SKV_LAUNCH_MMA(8);
#undef SKV_LAUNCH_MMA
      tail_attention_merge_kernel<<<dim3(n_q, n_seqs), 128, 0, st>>>(scratch, out, n_q, hd, n_splits);
      return;
    }
  }
  if (hd == 128 && (rep == 1 || rep == 2 || rep == 4 || rep == 8)) {
    dim3 grid(n_kv, n_splits, n_seqs);
    const size_t smem = (size_t)rep * 128 * sizeof(float) + (size_t)TA_WARPS * (TailTile<T>::K_BYTES + TailTile<T>::V_BYTES);
#define SKV_LAUNCH_GROUP(R)                                                                                                   \
    do {                                                                                                                      \
      ensure_dynamic_smem(reinterpret_cast<const void *>(tail_attention_group_kernel<T, R, 128>), (int)smem);                 \
      tail_attention_group_kernel<T, R, 128><<<grid, TA_WARPS * 32, smem, st>>>(q, kc, vc, kscale, vscale, cu_seqlens, len, blk, \
                                                                                blk_stride, n_q, n_kv, chunk, n_splits, scale, \
                                                                                scratch, rope);                               \
    } while (0)
    if (rep == 1) SKV_LAUNCH_GROUP(1);
    else if (rep == 2) SKV_LAUNCH_GROUP(2);
    else if (rep == 4) SKV_LAUNCH_GROUP(4);
    else SKV_LAUNCH_GROUP(8);
#undef SKV_LAUNCH_GROUP
    tail_attention_merge_kernel<<<dim3(n_q, n_seqs), 128, 0, st>>>(scratch, out, n_q, hd, n_splits);
    return;
  }
  const int threads = 32 * (rep < 8 ? rep : 8);
  const size_t smem = (size_t)rep * hd * sizeof(float);
  dim3 grid(n_splits, n_kv, n_seqs);
  if (hd <= 32) tail_attention_partial_kernel<T, 1><<<grid, threads, smem, st>>>(q, kc, vc, kscale, vscale, cu_seqlens, len, blk, blk_stride, n_q, n_kv, hd, chunk, n_splits, scale, scratch, rope);
  else if (hd <= 64) tail_attention_partial_kernel<T, 2><<<grid, threads, smem, st>>>(q, kc, vc, kscale, vscale, cu_seqlens, len, blk, blk_stride, n_q, n_kv, hd, chunk, n_splits, scale, scratch, rope);
  else if (hd <= 128) tail_attention_partial_kernel<T, 4><<<grid, threads, smem, st>>>(q, kc, vc, kscale, vscale, cu_seqlens, len, blk, blk_stride, n_q, n_kv, hd, chunk, n_splits, scale, scratch, rope);
  else tail_attention_partial_kernel<T, 8><<<grid, threads, smem, st>>>(q, kc, vc, kscale, vscale, cu_seqlens, len, blk, blk_stride, n_q, n_kv, hd, chunk, n_splits, scale, scratch, rope);
  tail_attention_merge_kernel<<<dim3(n_q, n_seqs), 128, 0, st>>>(scratch, out, n_q, hd, n_splits);
}
template void launch_tail_attention<float>(const float *, const float *, const float *, const float *, const float *, float *,
                                           const int32_t *, const int32_t *, const int32_t *, int, int, int, int, int, int,
                                           float *, cudaStream_t, TailOpts);
template void launch_tail_attention<bf16>(const float *, const bf16 *, const bf16 *, const float *, const float *, float *,
                                          const int32_t *, const int32_t *, const int32_t *, int, int, int, int, int, int,
                                          float *, cudaStream_t, TailOpts);
template void launch_tail_attention<fp8e4>(const float *, const fp8e4 *, const fp8e4 *, const float *, const float *, float *,
                                           const int32_t *, const int32_t *, const int32_t *, int, int, int, int, int, int,
                                           float *, cudaStream_t, TailOpts);

// ---------------------------------------------------------------------------------------------------------
// Several dependent weight-streaming projections of the last-token path in ONE launch (bf16 weights): a persistent
// cooperative kernel, one CTA per SM, walks a short list of stages -- per layer
//     O projection + residual | [RMSNorm +] gate/up + SwiGLU | down projection + residual | [next layer's RMSNorm +] Q projection
// (the single-query attention between a Q and an O projection stays its own kernel) -- separated by grid-wide barriers
// instead of kernel boundaries.  Why: each stage moves 30 - 240 MB, i.e. 5 - 40 us at the HBM roofline, and a separate
// launch adds its ramp, its tail and a dependent round trip to HBM to every one of them.  Here a producer warp streams
// each CTA's weight rows AND the matching K-slice of the (at most 8) activation rows through a shared-memory ring with bulk
// asynchronous copies (row segments of 1 - 2 KB, ~170 KB in flight per SM), so the HBM pipe stays full across tiles and --
// the ring is refilled while the CTA waits at a barrier -- across stages, and the MMA warps never wait for L2.
//   * work split of a projection: 16-feature tiles, tile t belongs to CTA t % gridDim; the 8 MMA warps split every K
//     chunk of the tile (swap-AB mma.m16n8k16 as in skinny_mma_kernel, fp32 activations as bf16 hi + lo), are summed in
//     shared memory in warp order (deterministic), and warp 0 runs the epilogue;
//   * RMSNorm is folded into the projection that consumes it: every CTA recomputes the row statistics from the fp32
//     residual rows (128 KB of L2 reads, while the ring fills) and scales the activation fragments by rstd * gain;
//   * data produced inside the kernel is read with ld.global.cg or by the bulk copies, never through L1.
// Every wait -- ring barriers, the grid barrier -- is bounded: on timeout the kernel latches STATUS_TIMEOUT, raises a
// global abort word that every later wait sees at once, waits (bounded) for its own copies in flight and returns.
// ---------------------------------------------------------------------------------------------------------
namespace fused {

constexpr int CONSUMERS = 8;
constexpr int THREADS = (CONSUMERS + 1) * 32;
// ring depth: 5 stages beside 8 rows of resident activations; fewer rows leave room for more (up to 11), so that the
// producer can run further ahead while the MMA warps stand at a grid barrier or fill their activations
constexpr int MIN_STAGES = 5, MAX_STAGES = 12;
// one matrix: 16 rows x 512 columns per ring stage; two matrices (gate / up): 2 x (16 rows x 256 columns).  A stage is
// filled by ONE tiled bulk copy per matrix (a copy per row segment costs the copy engine ~60 clocks each and capped the
// stream at a third of the HBM rate): blocks of 16 lines of 128 bytes, 128-byte swizzle.
constexpr int KC1 = 512, KC2 = 256;
constexpr int STAGE_BYTES = 16 * KC1 * 2;             // 16384
constexpr int POOL_BYTES = 212992;                    // the ring (n x 16 KB) followed by the activation area
// Activations come in blocks of one 32-wide K step: [row slots][32 floats], row slots = the launch's rows rounded up to a
// power of two (1, 2, 4, 8; the padding rows are zero-filled), brought by tiled bulk copies.  K <= 4096: all K / 32 blocks
// are resident and converted IN PLACE, once per stage, into the MMA fragments [bf16 hi | bf16 lo][row][quarter]; larger K:
// the blocks of a K chunk travel with the chunk's weights through a ring of their own and are converted as they are used.
constexpr int ACT_BLOCK = 1024;                       // the largest block: 8 row slots
constexpr int RES_BYTES = 131072;                     // K * 32 <= RES_BYTES: resident (K <= 4096)
constexpr int RED_FLOATS = 2 * CONSUMERS * 2 * 32 * 4;   // two buffers of [warp][matrix][lane][4]
constexpr int SM_RED = POOL_BYTES, SM_BAR = SM_RED + RED_FLOATS * 4, SM_MISC = SM_BAR + 256;
constexpr int SMEM_BYTES = SM_MISC + 256 + 1024;      // 230912 incl. the slack to align the ring to 1024 bytes
static_assert(RES_BYTES / 32 * 2 <= RED_FLOATS * 2, "a resident stage's norm gains (2 bytes per K) fit the first reduction buffer");
static_assert(MIN_STAGES * STAGE_BYTES + RES_BYTES <= POOL_BYTES, "8 rows: 5 ring stages + 128 KB of resident activations");
constexpr long long WAIT_LIMIT = 4000000000LL;
constexpr int MAX_STAGE_LIST = 6;

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
               : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// data written with ordinary stores (by any SM, made visible by a barrier) is about to be read by a bulk copy
__device__ __forceinline__ void fence_generic_to_async() { asm volatile("fence.proxy.async;" ::: "memory"); }

// epi 0: out = A W^T (store); 1: out += A W^T; 2: out = silu(A W^T) * (A W2^T); 3: out = A W^T and out2 = A W2^T
struct Stage {
  CUtensorMap tmW, tmW2;   // [N, K] as [K / 64][N][64], box (64, 16, KC / 64)
  CUtensorMap tmA;         // [rows, K] fp32 as [K / 32][rows][32], box (32, row slots, KC / 32)
  const float *A;          // [rows, K] fp32 (produced earlier, possibly in this launch)
  const bf16 *gamma;       // non-null: A is RMS-normalised on the fly (row statistic * gain)
  float *out, *out2;
  int N, K, ldo, epi;
  // Hand-over between two adjacent stages of one launch (the second one resident and normed, reading the first one's output):
  // the first stage's epilogue also publishes its rows as the second one needs them in shared memory -- multiplied by the
  // second stage's gain, split into bf16 hi / lo, in the fragment layout of one block per 32-wide K step -- and the sum of
  // squares of each row over its 16 features; the second stage's fill is then its whole set-up (otherwise all 148 CTAs
  // repeat the same fp32 -> hi / lo pass over the whole activation vector for themselves).
  uint8_t *pub_image;          // producer: where to publish (null: do not)
  float *pub_ss;               // producer: [N / 16][8] partial sums of squares
  const bf16 *pub_gamma;       // producer: the consuming stage's gain
  int presplit;                // consumer: tmA points at the published image; the row statistics come from pre_ss
  const float *pre_ss;
};
struct Params {
  Stage st[MAX_STAGE_LIST];
  int n_stages, rows;
  int rs;                   // log2 of the row slots per activation block
  int n_ring;               // ring depth of this launch (MIN_STAGES .. MAX_STAGES - 1)
  float eps;
  long long wait_limit;     // clocks any single wait may take before the kernel gives up
  unsigned int sync_base;   // arrivals counted by earlier launches (the counter is never reset)
  unsigned int *sync;       // [0] arrivals at the grid barrier, [1] abort word
  unsigned int *status;
};

struct Ctx {
  uint8_t *smem;
  volatile int *abort_s;    // this CTA's copy of "give up"
  volatile int *open_s;     // the last stage whose inputs are complete (written by the MMA warps after the grid barrier)
  volatile int *decide_s;   // "give up", as published to all MMA warps at one point (so that they leave together)
  unsigned epoch;           // grid barriers passed
  unsigned chunk_no;        // ring chunks produced / consumed so far (same sequence in every role)
  unsigned slot, phase;     // ring slot of chunk chunk_no and the parity of its use
  unsigned fill_no;         // resident fills so far
};

__device__ __forceinline__ bool aborted(const Params &p, Ctx &c) {
  if (*c.abort_s) return true;
  if (*reinterpret_cast<volatile unsigned int *>(p.sync + 1)) { *c.abort_s = 1; return true; }
  return false;
}
__device__ __forceinline__ void give_up(const Params &p, Ctx &c) {
  *c.abort_s = 1;
  atomicOr(p.status, STATUS_TIMEOUT);
  atomicExch(p.sync + 1, 1u);
}
__device__ __forceinline__ bool ring_wait(const Params &p, Ctx &c, uint32_t bar, uint32_t parity) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (unsigned spins = 1;; ++spins) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((spins & 63u) == 0u) {
      if (aborted(p, c)) return false;
      if (clock64() - t0 > p.wait_limit) { give_up(p, c); return false; }
    }
  }
}
__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }
// all CTAs of the (cooperative, hence co-resident) grid -- their MMA warps; the producer warps never stop here, they
// keep the rings full with the next stage's weights.  Returns false when the kernel is giving up.
__device__ __forceinline__ bool grid_barrier(const Params &p, Ctx &c) {
  consumer_sync();
  if (threadIdx.x == 0) {
    __threadfence();
    const unsigned target = p.sync_base + (c.epoch + 1) * gridDim.x;
    atomicAdd(p.sync, 1u);
    const long long t0 = clock64();
    for (unsigned spins = 1;; ++spins) {
      if ((int)(*reinterpret_cast<volatile unsigned int *>(p.sync) - target) >= 0) break;
      if ((spins & 15u) == 0u) {
        if (aborted(p, c)) break;
        if (clock64() - t0 > p.wait_limit) { give_up(p, c); break; }
      }
    }
    __threadfence();
    *c.decide_s = *c.abort_s;
  }
  consumer_sync();
  c.epoch += 1;
  return !*c.decide_s;
}

// ---- producer warp (one lane): every stage's weight rows, tile by tile, chunk by chunk, through the ring -- as far ahead
//      as the ring allows, across stage boundaries.  A stage whose K is too large for resident activations also gets each
//      chunk's activation blocks, but those are requested only once the stage's inputs are complete (open_s).
__device__ void produce(const Params &p, Ctx &c) {
  uint64_t *full = reinterpret_cast<uint64_t *>(c.smem + SM_BAR), *empty = full + MAX_STAGES;
  if ((threadIdx.x & 31) != 0) return;
  const unsigned n_ring = (unsigned)p.n_ring;
  uint8_t *res = c.smem + n_ring * STAGE_BYTES;
  for (int i = 0; i < p.n_stages; ++i) {
    const Stage &sg = p.st[i];
    const bool dual = sg.epi >= 2;
    const int kc_len = dual ? KC2 : KC1;
    const int n_tiles = sg.N / 16, n_chunks = sg.K / kc_len;
    const bool resident = (long long)sg.K * 32 <= RES_BYTES;
    const uint32_t act_bytes = resident ? 0u : (uint32_t)(kc_len / 32) * (128u << p.rs);
    const uint32_t act_slot_bytes = (uint32_t)(KC1 / 32) * (128u << p.rs);
    const unsigned my_tiles = (int)blockIdx.x < n_tiles ? (unsigned)(n_tiles - 1 - (int)blockIdx.x) / gridDim.x + 1u : 0u;
    const unsigned total = my_tiles * (unsigned)n_chunks, base = c.chunk_no;
    unsigned act_j = resident ? total : 0u;       // next chunk of the stage whose activation blocks are still to be requested
    unsigned act_slot = c.slot;                   // ... and its ring slot
    int act_kc = 0;
    bool open = i == 0;
    auto request_activations = [&](unsigned issued) {
      if (act_j >= issued) return;
      if (!open) {
        if (*c.open_s < i) return;
        __threadfence();
        fence_generic_to_async();
        open = true;
      }
      for (; act_j < issued; ++act_j) {
        tc::tma_load_3d(smem_u32(res + act_slot * act_slot_bytes), &sg.tmA, smem_u32(&full[act_slot]), 0, 0, act_kc * (kc_len / 32));
        if (++act_kc == n_chunks) act_kc = 0;
        if (++act_slot == n_ring) act_slot = 0;
      }
    };
    unsigned j = 0;
    for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
      for (int kc = 0; kc < n_chunks; ++kc, ++j) {
        const unsigned slot = c.slot;
        const uint32_t ph = c.phase;
        const uint32_t eb = smem_u32(&empty[slot]);
        if (!mbar_try_wait(eb, ph ^ 1)) {
          const long long t0 = clock64();
          for (unsigned spins = 1; !mbar_try_wait(eb, ph ^ 1); ++spins) {
            request_activations(j);
            if ((spins & 63u) == 0u) {
              if (aborted(p, c)) { c.chunk_no = base + j; return; }
              if (clock64() - t0 > p.wait_limit) { give_up(p, c); c.chunk_no = base + j; return; }
            }
          }
        }
        const uint32_t fb = smem_u32(&full[slot]);
        mbar_expect_tx(fb, STAGE_BYTES + act_bytes);
        const uint32_t dst = smem_u32(c.smem + slot * STAGE_BYTES);
        tc::tma_load_3d(dst, &sg.tmW, fb, 0, tile * 16, kc * (kc_len / 64));
        if (dual) tc::tma_load_3d(dst + STAGE_BYTES / 2, &sg.tmW2, fb, 0, tile * 16, kc * (kc_len / 64));
        if (++c.slot == n_ring) { c.slot = 0; c.phase ^= 1; }
        request_activations(j + 1);
      }
    }
    c.chunk_no = base + total;
    if (act_j < total) {
      const long long t0 = clock64();
      for (unsigned spins = 1; act_j < total; ++spins) {
        request_activations(total);
        if ((spins & 63u) == 0u) {
          if (aborted(p, c)) return;
          if (clock64() - t0 > p.wait_limit) { give_up(p, c); return; }
        }
      }
    }
  }
}

// ---- MMA warps, one stage.  RESIDENT: the (gain-scaled) activations sit in shared memory as bf16 hi / lo fragments, made
//      once per stage; otherwise every chunk's fp32 blocks arrive with its weights and are split as they are used
template <bool DUAL, bool RESIDENT>
__device__ void consume(const Params &p, Ctx &c, const Stage &sg) {
  constexpr int KC = DUAL ? KC2 : KC1;
  constexpr int STEPS = KC / (CONSUMERS * 32);         // 32-wide K steps per warp and chunk: 2 (one matrix) or 1 (two)
  uint64_t *full = reinterpret_cast<uint64_t *>(c.smem + SM_BAR), *empty = full + MAX_STAGES, *afull = empty + MAX_STAGES;
  float *red = reinterpret_cast<float *>(c.smem + SM_RED);
  float *rstd_s = reinterpret_cast<float *>(c.smem + SM_MISC) + 8;
  const unsigned n_ring = (unsigned)p.n_ring;
  uint8_t *res = c.smem + n_ring * STAGE_BYTES;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int K = sg.K, n_tiles = sg.N / 16, n_chunks = K / KC;
  const int g = lane >> 2, t = lane & 3;
  const int rs = p.rs, RP = 1 << rs, AB = 128 << rs;   // row slots, bytes per activation block
  const bool row_ok = g < RP;
  // RMSNorm folded in: activations are multiplied by the gain on the way in, the row statistic 1 / rms scales the OUTPUT
  // row in the epilogue (it is a per-row scalar), so it can be accumulated in the same pass that brings the activations in
  float ss = 0.f;                                      // RESIDENT: this lane's row (g); else row (lane & 7)
  bool dead = false;
  if (RESIDENT && sg.presplit) {
    // the producing stage published hi / lo fragments and per-tile sums of squares: fill, row statistics, done
    if (threadIdx.x == 0) {
      fence_generic_to_async();
      mbar_expect_tx(smem_u32(afull), (uint32_t)(K / 32) * (uint32_t)AB);
      for (int part = 0; part < K / KC1; ++part)
        tc::tma_load_3d(smem_u32(res + part * (KC1 / 32) * AB), &sg.tmA, smem_u32(afull), 0, 0, part * (KC1 / 32));
    }
    if (warp < p.rows) {            // warp w: row w, the producer's K / 16 tiles in a fixed order
      float tot = 0.f;
      for (int tl = lane; tl < K / 16; tl += 32) tot += __ldcg(sg.pre_ss + (size_t)tl * MAX_TAIL_ROWS + warp);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) tot += __shfl_xor_sync(0xffffffffu, tot, o);
      if (lane == 0) rstd_s[warp] = rsqrtf(tot / (float)K + p.eps);
    }
    dead = !ring_wait(p, c, smem_u32(afull), c.fill_no & 1);
    c.fill_no += 1;
    cp_async_wait<0>();
  } else if (RESIDENT) {
    if (threadIdx.x == 0) {
      fence_generic_to_async();
      mbar_expect_tx(smem_u32(afull), (uint32_t)(K / 32) * (uint32_t)AB);
      for (int part = 0; part < K / KC1; ++part)
        tc::tma_load_3d(smem_u32(res + part * (KC1 / 32) * AB), &sg.tmA, smem_u32(afull), 0, 0, part * (KC1 / 32));
    }
    // (a wait that runs out never makes a warp leave early: the named barriers below count all 256 threads, so a warp that
    //  gave up keeps walking the same barriers and only skips the work)
    dead = !ring_wait(p, c, smem_u32(afull), c.fill_no & 1);
    c.fill_no += 1;
    // the norm gains were requested into the (idle) reduction area before the grid barrier: fetched from global memory one
    // pair per conversion step they cost a dependent L2 round trip per step -- 0.7 ms of a 6.4 ms decode step, measured
    cp_async_wait<0>();
    consumer_sync();
    // every warp converts, in place, exactly the blocks it will multiply with, 8 / RP blocks at a time:
    // lane = (block of the group, row, quarter)
    const int grp = g >> rs, r = g & (RP - 1), G = 8 >> rs;
    const int n_blk = K / (32 * CONSUMERS);
    for (int b = 0; b < n_blk && !dead; b += 2 * G) {
      uint8_t *blk[2];
      float x[2][8];
      uint4 gm[2];
      bool live[2];
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int bb = b + h * G + grp;
        live[h] = bb < n_blk;
        const int s = (bb / STEPS) * (CONSUMERS * STEPS) + warp * STEPS + (bb % STEPS);
        blk[h] = res + (size_t)s * AB;
        float4 xa = make_float4(0.f, 0.f, 0.f, 0.f), xb = xa;
        if (live[h]) {
          xa = *reinterpret_cast<const float4 *>(blk[h] + r * 128 + t * 32);
          xb = *reinterpret_cast<const float4 *>(blk[h] + r * 128 + t * 32 + 16);
        }
        x[h][0] = xa.x; x[h][1] = xa.y; x[h][2] = xa.z; x[h][3] = xa.w;
        x[h][4] = xb.x; x[h][5] = xb.y; x[h][6] = xb.z; x[h][7] = xb.w;
        gm[h] = make_uint4(0u, 0u, 0u, 0u);
        if (sg.gamma && live[h]) gm[h] = *reinterpret_cast<const uint4 *>(reinterpret_cast<const uint8_t *>(red) + ((size_t)s * 32 + t * 8) * 2);
      }
      __syncwarp();
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        if (sg.gamma) {
          const bf16 *ge = reinterpret_cast<const bf16 *>(&gm[h]);
#pragma unroll
          for (int e = 0; e < 8; ++e) { ss = fmaf(x[h][e], x[h][e], ss); x[h][e] *= to_f(ge[e]); }
        }
        uint4 hi, lo;
        split_hi_lo(x[h][0], x[h][1], hi.x, lo.x);
        split_hi_lo(x[h][2], x[h][3], hi.y, lo.y);
        split_hi_lo(x[h][4], x[h][5], hi.z, lo.z);
        split_hi_lo(x[h][6], x[h][7], hi.w, lo.w);
        if (live[h]) {
          *reinterpret_cast<uint4 *>(blk[h] + (4 * r + t) * 16) = hi;
          *reinterpret_cast<uint4 *>(blk[h] + (AB >> 1) + (4 * r + t) * 16) = lo;
        }
      }
      __syncwarp();
    }
    // row r's sum: over the quarters and over the blocks of a group, in a fixed order
    ss += __shfl_xor_sync(0xffffffffu, ss, 1);
    ss += __shfl_xor_sync(0xffffffffu, ss, 2);
    for (int m = 4 << rs; m < 32; m <<= 1) ss += __shfl_xor_sync(0xffffffffu, ss, m);
  } else if (sg.gamma) {
    // 4 lanes per row: quarters of the row, from L2 (the blocks in shared memory pass by only once)
    const int r = lane >> 2;
    if (r < p.rows)
      for (int i = (warp * 4 + t) * 4; i < K; i += CONSUMERS * 4 * 4) {
        const float4 v = __ldcg(reinterpret_cast<const float4 *>(sg.A + (size_t)r * K + i));
        ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
      }
    ss += __shfl_xor_sync(0xffffffffu, ss, 1);
    ss += __shfl_xor_sync(0xffffffffu, ss, 2);
  }
  if (sg.gamma && !(RESIDENT && sg.presplit)) {
    float *part = red + 2 * CONSUMERS * 2 * 32 * 4 - CONSUMERS * MAX_TAIL_ROWS;      // the tail of the second buffer: [8 warps][8 rows]
    if (t == 0 && g < (RESIDENT ? RP : MAX_TAIL_ROWS)) part[warp * MAX_TAIL_ROWS + g] = ss;
    consumer_sync();
    if (threadIdx.x < p.rows) {
      float tot = 0.f;
#pragma unroll
      for (int w = 0; w < CONSUMERS; ++w) tot += part[w * MAX_TAIL_ROWS + threadIdx.x];
      rstd_s[threadIdx.x] = rsqrtf(tot / (float)K + p.eps);
    }
  }
  consumer_sync();
  const int k_lane = warp * (STEPS * 32) + 8 * t;          // this lane's first K index inside a chunk
  int tile_no = 0;
  for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++tile_no) {
    // four independent accumulator chains per matrix
    float acc[4][4] = {}, acc2[4][4] = {};
    for (int kc = 0; kc < n_chunks; ++kc, ++c.chunk_no) {
      const int st = (int)c.slot;
      const uint32_t ph = c.phase;
      if (++c.slot == n_ring) { c.slot = 0; c.phase ^= 1; }
      uint4 gm[STEPS];
      if (!RESIDENT) {
#pragma unroll
        for (int u = 0; u < STEPS; ++u) {
          gm[u] = make_uint4(0u, 0u, 0u, 0u);
          if (sg.gamma) gm[u] = __ldg(reinterpret_cast<const uint4 *>(sg.gamma + (size_t)kc * KC + k_lane + u * 32));
        }
      }
      if (!dead && !ring_wait(p, c, smem_u32(&full[st]), ph)) dead = true;
      if (dead) continue;
      const uint8_t *sw = c.smem + st * STAGE_BYTES;
#pragma unroll
      for (int u = 0; u < STEPS; ++u) {
        uint32_t bh[4], bl[4];
        if (RESIDENT) {
          uint4 h4 = make_uint4(0u, 0u, 0u, 0u), l4 = h4;
          if (row_ok) {
            const uint8_t *fr = res + (size_t)(kc * (KC / 32) + warp * STEPS + u) * AB + (size_t)lane * 16;
            h4 = *reinterpret_cast<const uint4 *>(fr);
            l4 = *reinterpret_cast<const uint4 *>(fr + (AB >> 1));
          }
          bh[0] = h4.x; bh[1] = h4.y; bh[2] = h4.z; bh[3] = h4.w;
          bl[0] = l4.x; bl[1] = l4.y; bl[2] = l4.z; bl[3] = l4.w;
        } else {
          float4 xa = make_float4(0.f, 0.f, 0.f, 0.f), xb = xa;
          if (row_ok) {
            const uint8_t *fa = res + (size_t)st * ((KC1 / 32) * AB) + (size_t)(warp * STEPS + u) * AB + g * 128 + t * 32;
            xa = *reinterpret_cast<const float4 *>(fa);
            xb = *reinterpret_cast<const float4 *>(fa + 16);
          }
          float x[8] = {xa.x, xa.y, xa.z, xa.w, xb.x, xb.y, xb.z, xb.w};
          if (sg.gamma) {
            const bf16 *ge = reinterpret_cast<const bf16 *>(&gm[u]);
#pragma unroll
            for (int e = 0; e < 8; ++e) x[e] *= to_f(ge[e]);
          }
          split_hi_lo(x[0], x[1], bh[0], bl[0]);
          split_hi_lo(x[2], x[3], bh[1], bl[1]);
          split_hi_lo(x[4], x[5], bh[2], bl[2]);
          split_hi_lo(x[6], x[7], bh[3], bl[3]);
        }
        // K index inside the chunk -> block of 64 columns (16 lines of 128 bytes) and 16-byte unit inside the line, swizzled
        // by the line number (rows g and g + 8 share g & 7)
        const int kk = k_lane + u * 32;
        const uint32_t off = (uint32_t)(kk >> 6) * 2048u + (uint32_t)((((kk & 63) >> 3) ^ g) << 4);
        const uint4 wl = *reinterpret_cast<const uint4 *>(sw + off + g * 128);
        const uint4 wh = *reinterpret_cast<const uint4 *>(sw + off + (g + 8) * 128);
        const uint32_t a1[4] = {wl.x, wh.x, wl.y, wh.y}, a2[4] = {wl.z, wh.z, wl.w, wh.w};
        mma_bf16_16816(acc[0], a1, bh[0], bh[1]);
        mma_bf16_16816(acc[1], a1, bl[0], bl[1]);
        mma_bf16_16816(acc[2], a2, bh[2], bh[3]);
        mma_bf16_16816(acc[3], a2, bl[2], bl[3]);
        if (DUAL) {
          const uint4 ul = *reinterpret_cast<const uint4 *>(sw + STAGE_BYTES / 2 + off + g * 128);
          const uint4 uh = *reinterpret_cast<const uint4 *>(sw + STAGE_BYTES / 2 + off + (g + 8) * 128);
          const uint32_t d1[4] = {ul.x, uh.x, ul.y, uh.y}, d2[4] = {ul.z, uh.z, ul.w, uh.w};
          mma_bf16_16816(acc2[0], d1, bh[0], bh[1]);
          mma_bf16_16816(acc2[1], d1, bl[0], bl[1]);
          mma_bf16_16816(acc2[2], d2, bh[2], bh[3]);
          mma_bf16_16816(acc2[3], d2, bl[2], bl[3]);
        }
      }
      // Releasing the stage: every lane first fences its own reads of the stage (they must have been PERFORMED, not just
      // issued, before the producer may overwrite it).  __syncwarp() + one arrive alone, and also one arrive per lane, were
      // not enough: with reads still outstanding when the next copy landed, a few weight rows of a tile came out wrong
      // once in ~20 steps at the 8B widths.
      __threadfence_block();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&empty[st]));
    }
    // the 8 warps' partial tiles, summed in warp order by one warp (two buffers: one barrier per tile)
    float *buf = red + (tile_no & 1) * (CONSUMERS * 2 * 32 * 4);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      buf[((warp * 2 + 0) * 32 + lane) * 4 + i] = (acc[0][i] + acc[1][i]) + (acc[2][i] + acc[3][i]);
      if (DUAL) buf[((warp * 2 + 1) * 32 + lane) * 4 + i] = (acc2[0][i] + acc2[1][i]) + (acc2[2][i] + acc2[3][i]);
    }
    consumer_sync();
    if (warp == (tile_no & (CONSUMERS - 1)) && !*c.abort_s) {      // (the warps take turns, so that none falls a whole epilogue behind per tile)
      float s1[4] = {0.f, 0.f, 0.f, 0.f}, s2[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int w = 0; w < CONSUMERS; ++w)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          s1[i] += buf[((w * 2 + 0) * 32 + lane) * 4 + i];
          if (DUAL) s2[i] += buf[((w * 2 + 1) * 32 + lane) * 4 + i];
        }
      float pg[2] = {0.f, 0.f}, sq[2] = {0.f, 0.f};
      if (!DUAL && sg.pub_image) {
        pg[0] = to_f(sg.pub_gamma[tile * 16 + g]);
        pg[1] = to_f(sg.pub_gamma[tile * 16 + g + 8]);
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) {      // fragment element i: feature 16 tile + g + 8 (i / 2), token 2 t + (i % 2)
        const int n = tile * 16 + g + 8 * (i >> 1), r = 2 * t + (i & 1);
        if (r < p.rows) {
          const float rs = sg.gamma ? rstd_s[r] : 1.f;       // the folded norm's row statistic
          float v = s1[i] * rs;
          if (DUAL) {
            if (sg.epi == 2) v = v / (1.f + __expf(-v)) * (s2[i] * rs);
            else sg.out2[(size_t)r * sg.ldo + n] = s2[i] * rs;
          }
          float *o = sg.out + (size_t)r * sg.ldo + n;
          if (sg.epi == 1) v += __ldcg(o);
          *o = v;
          if (!DUAL && sg.pub_image) {
            // element n of row r in the consumer's block n / 32: quarter (n % 32) / 8 of the row, 16-bit slot n % 8; hi half of
            // the block, then lo half
            sq[i & 1] = fmaf(v, v, sq[i & 1]);
            const float x = v * pg[i >> 1];
            const bf16 hi = __float2bfloat16_rn(x);
            const bf16 lo = __float2bfloat16_rn(x - to_f(hi));
            uint8_t *dst = sg.pub_image + (size_t)(n >> 5) * AB + (4 * r + ((n & 31) >> 3)) * 16 + (n & 7) * 2;
            *reinterpret_cast<bf16 *>(dst) = hi;
            *reinterpret_cast<bf16 *>(dst + (AB >> 1)) = lo;
          }
        }
      }
      if (!DUAL && sg.pub_image) {       // rows 2 t, 2 t + 1: sum over the tile's 16 features (the 8 lanes that share t, two each)
#pragma unroll
        for (int rr = 0; rr < 2; ++rr) {
          sq[rr] += __shfl_xor_sync(0xffffffffu, sq[rr], 4);
          sq[rr] += __shfl_xor_sync(0xffffffffu, sq[rr], 8);
          sq[rr] += __shfl_xor_sync(0xffffffffu, sq[rr], 16);
          if (g == 0 && 2 * t + rr < p.rows) sg.pub_ss[(size_t)tile * MAX_TAIL_ROWS + 2 * t + rr] = sq[rr];
        }
      }
    }
  }
  consumer_sync();       // the statistics / resident buffers may be rewritten by the next stage
}

__global__ void __launch_bounds__(THREADS, 1) tail_fused_kernel(const __grid_constant__ Params p) {
  extern __shared__ uint8_t fsmem_raw[];
  uint8_t *fsmem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(fsmem_raw) + 1023) & ~(uintptr_t)1023);
  Ctx c;
  c.smem = fsmem;
  c.abort_s = reinterpret_cast<volatile int *>(fsmem + SM_MISC);
  c.open_s = c.abort_s + 1;
  c.decide_s = c.abort_s + 2;
  c.epoch = 0;
  c.chunk_no = 0;
  c.slot = 0;
  c.phase = 0;
  c.fill_no = 0;
  uint64_t *full = reinterpret_cast<uint64_t *>(fsmem + SM_BAR), *empty = full + MAX_STAGES, *afull = empty + MAX_STAGES;
  if (threadIdx.x == 0) {
    for (int s = 0; s < MAX_STAGES; ++s) { mbar_init(smem_u32(&full[s]), 1); mbar_init(smem_u32(&empty[s]), CONSUMERS); }
    mbar_init(smem_u32(afull), 1);
    *c.abort_s = 0;
    *c.open_s = 0;
    *c.decide_s = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if ((threadIdx.x >> 5) == CONSUMERS) {
    produce(p, c);
    // giving up: copies still in flight must land before this CTA's shared memory is released
    if (*c.abort_s && (threadIdx.x & 31) == 0) {
      const unsigned issued = c.chunk_no, n_ring = (unsigned)p.n_ring;
      for (unsigned q = issued > n_ring ? issued - n_ring : 0; q < issued; ++q) {
        const long long t0 = clock64();
        while (!mbar_try_wait(smem_u32(&full[q % n_ring]), (q / n_ring) & 1) && clock64() - t0 < 100000000LL) {}
      }
    }
  } else {
    for (int i = 0; i < p.n_stages; ++i) {
      const Stage &sg = p.st[i];
      const bool resident = (long long)sg.K * 32 <= RES_BYTES;      // 1 KB per 32-wide K step (8 row slots x (hi + lo))
      // a resident stage's norm gains (at most 8 KB, constants) travel while the CTA waits at the barrier: the reduction
      // area is idle between the previous stage's last epilogue and this stage's first
      if (resident && sg.gamma && !sg.presplit)
        for (int o = (int)threadIdx.x * 16; o < sg.K * 2; o += CONSUMERS * 32 * 16)
          cp_async16(fsmem + SM_RED + o, reinterpret_cast<const uint8_t *>(sg.gamma) + o);
      cp_async_commit();
      if (i > 0) {
        if (!grid_barrier(p, c)) break;
        if (threadIdx.x == 0) *c.open_s = i;
      }
      if (sg.epi >= 2) { if (resident) consume<true, true>(p, c, sg); else consume<true, false>(p, c, sg); }
      else { if (resident) consume<false, true>(p, c, sg); else consume<false, false>(p, c, sg); }
      if (threadIdx.x == 0) *c.decide_s = *c.abort_s;      // (consume ended with a barrier of the MMA warps)
      consumer_sync();
      if (*c.decide_s) break;
    }
    cp_async_wait<0>();      // (a gain request of a stage that was never reached)
  }
  __syncthreads();
}

}  // namespace fused

bool tail_fused_supported(int rows, int d, int dq, int F, int vocab) {
  // the grid barriers need every CTA resident at once: a device (or context) that cannot promise that keeps the
  // per-operator kernels
  static int coop = -1;
  if (coop < 0) {
    int dev = 0, v = 0, per_sm = 0;
    coop = cudaGetDevice(&dev) == cudaSuccess && cudaDeviceGetAttribute(&v, cudaDevAttrCooperativeLaunch, dev) == cudaSuccess && v &&
           ensure_dynamic_smem((const void *)fused::tail_fused_kernel, fused::SMEM_BYTES) == 0 &&
           cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fused::tail_fused_kernel, fused::THREADS, fused::SMEM_BYTES) == cudaSuccess &&
           per_sm >= 1;
  }
  return coop == 1 && rows >= 1 && rows <= MAX_TAIL_ROWS && d % fused::KC1 == 0 && dq % fused::KC1 == 0 && F % fused::KC1 == 0 &&
         vocab % 16 == 0;
}

int launch_tail_fused(const TailStage *stages, int n_stages, int rows, float eps, unsigned int *sync, unsigned int *arrivals,
                      unsigned int *status, cudaStream_t st, long long wait_limit_clocks, void *handover) {
  if (n_stages < 1 || n_stages > fused::MAX_STAGE_LIST || rows < 1 || rows > MAX_TAIL_ROWS) return SWIFTKV_ERR_UNSUPPORTED;
  fused::Params p{};
  int rs = 0;
  while ((1 << rs) < rows) ++rs;
  p.rs = rs;
  for (int i = 0; i < n_stages; ++i) {
    const TailStage &s = stages[i];
    const int kc = s.W2 ? fused::KC2 : fused::KC1;
    if (s.N % 16 || s.K % kc || (s.W2 != nullptr) != (s.epi >= 2) || (s.epi == 3 && !s.out2)) return SWIFTKV_ERR_UNSUPPORTED;
    fused::Stage &d = p.st[i];
    if (get_tmap_rows16(&d.tmW, s.W, s.N, s.K, kc / 64)) return SWIFTKV_ERR_CUDA;
    d.tmW2 = d.tmW;
    if (s.W2 && get_tmap_rows16(&d.tmW2, s.W2, s.N, s.K, kc / 64)) return SWIFTKV_ERR_CUDA;
    const bool resident = (long long)s.K * 32 <= fused::RES_BYTES;
    if (get_tmap_act_f32(&d.tmA, s.A, rows, 1u << rs, s.K, resident ? fused::KC1 / 32 : kc / 32)) return SWIFTKV_ERR_CUDA;
    d.A = s.A; d.gamma = reinterpret_cast<const bf16 *>(s.gamma); d.out = s.out; d.out2 = s.out2; d.N = s.N; d.K = s.K; d.ldo = s.ldo; d.epi = s.epi;
  }
  // a resident, normed stage that reads the output of the stage right before it takes that output pre-split from the
  // producer's epilogue (one hand-over area serves every such pair of the launch: a pair's fill is over before the next
  // producer's first epilogue, two grid barriers later)
  static int handover_on = -1;
  if (handover_on < 0) { const char *e = getenv("SWIFTKV_TAIL_HANDOVER"); handover_on = (e && e[0] == '0') ? 0 : 1; }
  if (handover && handover_on) {
    uint8_t *image = reinterpret_cast<uint8_t *>(handover);
    float *ss = reinterpret_cast<float *>(image + TAIL_HANDOVER_IMAGE_BYTES);
    for (int i = 1; i < n_stages; ++i) {
      const TailStage &a = stages[i - 1], &b = stages[i];
      const bool resident = (long long)b.K * 32 <= fused::RES_BYTES;
      if (!resident || !b.gamma || b.A != a.out || a.epi > 1 || a.N != b.K || a.ldo != b.K) continue;
      fused::Stage &pa = p.st[i - 1], &pb = p.st[i];
      if (pa.presplit) continue;      // (it still fills from the area while its own fastest CTAs would already publish into it)
      if (get_tmap_act_image(&pb.tmA, image, 1u << rs, b.K, fused::KC1 / 32)) return SWIFTKV_ERR_CUDA;
      pa.pub_image = image; pa.pub_ss = ss; pa.pub_gamma = reinterpret_cast<const bf16 *>(b.gamma);
      pb.presplit = 1; pb.pre_ss = ss;
    }
  }
  p.n_stages = n_stages; p.rows = rows; p.eps = eps; p.sync = sync; p.status = status;
  // ring depth: as many 16 KB stages as fit beside the activation area this launch needs (resident blocks of its widest
  // resident stage, or one activation slot per ring stage for a stage that streams them)
  {
    const size_t ab = (size_t)128 << rs;
    size_t resident_need = 0;
    bool streams = false;
    for (int i = 0; i < n_stages; ++i) {
      if ((long long)stages[i].K * 32 <= fused::RES_BYTES) resident_need = std::max(resident_need, (size_t)(stages[i].K / 32) * ab);
      else streams = true;
    }
    int n = fused::MIN_STAGES;
    for (int cand = fused::MAX_STAGES - 1; cand > fused::MIN_STAGES; --cand) {
      const size_t act = std::max(resident_need, streams ? (size_t)cand * (fused::KC1 / 32) * ab : (size_t)0);
      if ((size_t)cand * fused::STAGE_BYTES + act <= (size_t)fused::POOL_BYTES) { n = cand; break; }
    }
    p.n_ring = n;
  }
  p.sync_base = *arrivals;
  p.wait_limit = wait_limit_clocks > 0 ? wait_limit_clocks : fused::WAIT_LIMIT;
  int dev = 0, n_sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n_sms < 1)
    return SWIFTKV_ERR_CUDA;
  const void *kern = (const void *)fused::tail_fused_kernel;
  if (ensure_dynamic_smem(kern, fused::SMEM_BYTES)) return SWIFTKV_ERR_CUDA;
  void *args[] = {&p};
  if (cudaLaunchCooperativeKernel(kern, dim3((unsigned)n_sms), dim3(fused::THREADS), args, (size_t)fused::SMEM_BYTES, st) != cudaSuccess)
    return SWIFTKV_ERR_CUDA;
  *arrivals += (unsigned)(n_stages - 1) * (unsigned)n_sms;
  return SWIFTKV_OK;
}

}  // namespace skv
