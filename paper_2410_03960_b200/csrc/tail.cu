// The last-token path of SwiftKV prefill: only the last token of each prompt runs layers l+1..L (footnote of
// Sec. 3.2; Sec. 3.5), so every projection here has at most 8 activation rows and is bound by streaming the
// weights from HBM exactly once; attention is one query per (prompt, head) over the cache that the
// SingleInputKV projection filled.  Activations of this path stay in fp32 (they are tiny), weights and the
// cache stay in the model dtype.
#include <cooperative_groups.h>
#include <mma.h>

#include "common.cuh"

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
  const int split = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;
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
  if (hd == 128 && (rep == 1 || rep == 2 || rep == 4 || rep == 8)) {
    dim3 grid(n_splits, n_kv, n_seqs);
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

}  // namespace skv
