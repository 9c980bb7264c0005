// bf16 GEMMs of the prefill path on the 5th-generation tensor cores: C = A[M,K] * B[N,K]^T, fp32 accumulation.
//
// One persistent CTA per SM, 192 threads in three roles:
//   warp 0      : TMA producer -- streams 128x64 A tiles and BNx64 B tiles (128-byte swizzle) through a
//                 shared-memory ring guarded by full/empty mbarriers;
//   warp 1      : MMA issuer -- one thread issues tcgen05.mma (128 x BN x 16 per instruction) into one of two
//                 tensor-memory accumulators and commits ring slots / accumulators back through mbarriers;
//   warps 2..5  : epilogue -- read the finished accumulator from tensor memory (tcgen05.ld, one row per
//                 thread), apply the fused epilogue and write to global memory while the MMA warp already
//                 works on the next tile in the other accumulator.
// Epilogues: store bf16 (optionally scattered into K/V cache planes), accumulate into the fp32 residual
// stream, or SwiGLU with the gate and up tiles of the same features side by side in one accumulator.
// Every mbarrier wait is bounded: on timeout the kernel sets a status bit and every role leaves its loop.
#include <cstdlib>
#include <mutex>
#include <unordered_map>

#include "common.cuh"
#include "tc_common.cuh"

namespace skv {

// ---------------------------------------------------------------------------------------------------------
// host: tensor-map encoding through the driver entry point (no link-time dependency on libcuda)
// ---------------------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void *p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  });
  return fn;
}

int make_tmap_2d_bf16(CUtensorMap *out, const void *base, uint64_t rows, uint64_t cols, uint64_t ld,
                      uint32_t box_rows, uint32_t box_cols) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return -1;
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {ld * 2};
  cuuint32_t box[2] = {box_cols, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? 0 : -2;
}
int make_tmap_3d_bf16(CUtensorMap *out, const void *base, uint64_t d0, uint64_t d1, uint64_t d2, uint64_t s1,
                      uint64_t s2, uint32_t b0, uint32_t b1, uint32_t b2) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return -1;
  cuuint64_t dims[3] = {d0, d1, d2};
  cuuint64_t strides[2] = {s1 * 2, s2 * 2};
  cuuint32_t box[3] = {b0, b1, b2};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? 0 : -2;
}

namespace {
// tensor maps are pure functions of (pointer, shape, box): cache them
struct TmapKey {
  const void *p; uint64_t rows, cols, ld; uint32_t br, bc;
  bool operator==(const TmapKey &o) const { return p == o.p && rows == o.rows && cols == o.cols && ld == o.ld && br == o.br && bc == o.bc; }
};
struct TmapKeyHash {
  size_t operator()(const TmapKey &k) const {
    size_t h = reinterpret_cast<size_t>(k.p);
    h = h * 1000003u ^ k.rows; h = h * 1000003u ^ k.cols; h = h * 1000003u ^ k.ld; h = h * 1000003u ^ (k.br * 1024u + k.bc);
    return h;
  }
};
std::mutex g_tmap_mu;
std::unordered_map<TmapKey, CUtensorMap, TmapKeyHash> g_tmaps;

}  // namespace

int get_tmap(CUtensorMap *out, const void *p, uint64_t rows, uint64_t cols, uint64_t ld, uint32_t br, uint32_t bc) {
  TmapKey k{p, rows, cols, ld, br, bc};
  std::lock_guard<std::mutex> g(g_tmap_mu);
  auto it = g_tmaps.find(k);
  if (it != g_tmaps.end()) { *out = it->second; return 0; }
  if (g_tmaps.size() > 65536) g_tmaps.clear();
  CUtensorMap m;
  int rc = make_tmap_2d_bf16(&m, p, rows, cols, ld, br, bc);
  if (rc) return rc;
  g_tmaps.emplace(k, m);
  *out = m;
  return 0;
}

// A weight matrix [N, K] seen as [K / 64][N][64]: one copy brings 16 rows x (64 * chunks) columns as `chunks` blocks of
// 16 swizzled 128-byte lines (the weight-streaming kernels' ring stage).  Cached like the 2D maps.
int get_tmap_rows16(CUtensorMap *out, const void *p, uint64_t N, uint64_t K, uint32_t chunks) {
  TmapKey k{p, N, K, 0xFFFFFFFFull, 16, chunks};
  std::lock_guard<std::mutex> g(g_tmap_mu);
  auto it = g_tmaps.find(k);
  if (it != g_tmaps.end()) { *out = it->second; return 0; }
  if (g_tmaps.size() > 65536) g_tmaps.clear();
  CUtensorMap m;
  int rc = make_tmap_3d_bf16(&m, p, 64, N, K / 64, K, 64, 64, 16, chunks);
  if (rc) return rc;
  g_tmaps.emplace(k, m);
  *out = m;
  return 0;
}

// fp32 activations [rows, K] (rows <= 8) seen as [K / 32][rows][32]: one copy brings `steps` blocks of [row_slots][32
// floats], rows beyond `rows` zero-filled (the fused last-token kernel's activation blocks).
int get_tmap_act_f32(CUtensorMap *out, const float *p, uint32_t rows, uint32_t row_slots, uint64_t K, uint32_t steps) {
  TmapKey k{p, rows, K, 0xFFFFFFFEull, row_slots, steps};
  std::lock_guard<std::mutex> g(g_tmap_mu);
  auto it = g_tmaps.find(k);
  if (it != g_tmaps.end()) { *out = it->second; return 0; }
  if (g_tmaps.size() > 65536) g_tmaps.clear();
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return -1;
  CUtensorMap m;
  cuuint64_t dims[3] = {32, rows, K / 32};
  cuuint64_t strides[2] = {K * 4, 128};
  cuuint32_t box[3] = {32, row_slots, steps};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(&m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float *>(p), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return -2;
  g_tmaps.emplace(k, m);
  *out = m;
  return 0;
}

// the same blocks already laid out as the kernel keeps them in shared memory: [K / 32][row slots][32 words], contiguous
int get_tmap_act_image(CUtensorMap *out, const void *p, uint32_t row_slots, uint64_t K, uint32_t steps) {
  TmapKey k{p, row_slots, K, 0xFFFFFFFCull, row_slots, steps};
  std::lock_guard<std::mutex> g(g_tmap_mu);
  auto it = g_tmaps.find(k);
  if (it != g_tmaps.end()) { *out = it->second; return 0; }
  if (g_tmaps.size() > 65536) g_tmaps.clear();
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return -1;
  CUtensorMap m;
  cuuint64_t dims[3] = {32, row_slots, K / 32};
  cuuint64_t strides[2] = {128, (cuuint64_t)row_slots * 128};
  cuuint32_t box[3] = {32, row_slots, steps};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(&m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<void *>(p), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return -2;
  g_tmaps.emplace(k, m);
  *out = m;
  return 0;
}

// fp32 matrix [rows, cols] row-major: tiles of box_rows x 32 elements (128 bytes), 128-byte swizzle (the tf32 GEMM's operands)
int get_tmap_f32(CUtensorMap *out, const float *p, uint64_t rows, uint64_t cols, uint32_t box_rows, uint64_t ld) {
  if (ld == 0) ld = cols;
  TmapKey k{p, rows, cols, (0xFDull << 56) | ld, box_rows, 32};
  std::lock_guard<std::mutex> g(g_tmap_mu);
  auto it = g_tmaps.find(k);
  if (it != g_tmaps.end()) { *out = it->second; return 0; }
  if (g_tmaps.size() > 65536) g_tmaps.clear();
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return -1;
  CUtensorMap m;
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {ld * 4};
  cuuint32_t box[2] = {32, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(&m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float *>(p), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return -2;
  g_tmaps.emplace(k, m);
  *out = m;
  return 0;
}

int ensure_dynamic_smem(const void *kernel, int bytes) {
  static std::mutex mu;
  static std::unordered_map<const void *, unsigned long long> done;   // kernel -> bit mask of devices already set
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return -1;
  const unsigned long long bit = 1ull << (dev & 63);
  std::lock_guard<std::mutex> lock(mu);
  unsigned long long &mask = done[kernel];
  if (mask & bit) return 0;
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return -1;
  mask |= bit;
  return 0;
}

int num_sms() {
  static int n = 0;
  if (!n) {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
    if (n <= 0) n = 148;
  }
  return n;
}

namespace {
// ---------------------------------------------------------------------------------------------------------
// device
// ---------------------------------------------------------------------------------------------------------
constexpr int BM = 128, BK = 64, UMMA_K = 16;
constexpr int GEMM_THREADS = 192;
// tile rasterisation: bands of group_m row-blocks, column-blocks outer, rows inner (GemmTcParams::group_m)

struct GemmTcParams {
  int M, N, K;
  int nB0, nB1;          // columns [0,nB0) from B0, [nB0,nB0+nB1) from B1, rest from B2
  int num_m_blocks, num_n_blocks;
  int group_m;           // raster band height in 128-row blocks
  OutDesc out;
  bf16 *act;             // SwiGLU output [M, F]
  int F;
  int f16;               // A, B and the columns below out.n0 (and the SwiGLU output) hold IEEE halves (else bfloat16)
  int kb_wrap;           // K blocks of B.  Equal to K / 64 normally; half of it when A holds [hi | lo] halves side by side
                         // along K (K = 2 x B's K): the second half of the K loop multiplies A's lo part with B again
  __half *lo_p0;         // split output: the low halves (value - float(high half)) of the columns below out.n0 ...
  __half *lo_dup;        // ... and of the even-numbered segments' half copies (K planes), row stride out.seg_w
  int lo_act;            // ... and of the SwiGLU output: its rows are then [hi(F) | lo(F)], 2F elements apart
  __half *dup_base;      // optional second copy (halves) of the columns routed to segments
  long long dup_stride;
  const int32_t *rope_pos;   // EPI_ROPE: position of every row; cos/sin tables [pos][64]
  const float *cos_tab, *sin_tab;
  unsigned int *status;
};
enum { EPI_PLAIN = 0, EPI_SWIGLU = 1, EPI_ROPE = 2 };

template <int BN, int STAGES>
struct SmemLayout {
  static constexpr int A_BYTES = BM * BK * 2;
  static constexpr int B_BYTES = BN * BK * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int BAR_OFFSET = STAGES * STAGE_BYTES;
  static constexpr int TOTAL = BAR_OFFSET + 256 + 1024;   // barriers + slack for 1024-byte alignment
};

__device__ __forceinline__ void tile_coords(int tile, int num_m_blocks, int num_n_blocks, int group_m, int &m_blk, int &n_blk) {
  const int band_tiles = group_m * num_n_blocks;
  const int band = tile / band_tiles;
  const int r = tile - band * band_tiles;
  const int band_h = min(group_m, num_m_blocks - band * group_m);
  n_blk = r / band_h;
  m_blk = band * group_m + (r - n_blk * band_h);
}

__device__ __forceinline__ bool wait_or_abort(uint32_t bar, uint32_t parity, volatile int *abort_flag, unsigned int *status,
                                              long long limit = tc::WAIT_LIMIT_CLOCKS) {
  if (tc::mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (!tc::mbar_try_wait(bar, parity)) {
    if (*abort_flag) return false;
    if (clock64() - t0 > limit) {
      *abort_flag = 1;
      atomicOr(status, STATUS_TIMEOUT);
      return false;
    }
  }
  return true;
}

// low halves of a pair: what the high halves (already packed) left of a and b, as halves again
__device__ __forceinline__ uint32_t pack_f16x2_lo(float a, float b, uint32_t hi_packed) {
  const float2 h = __half22float2(*reinterpret_cast<const __half2 *>(&hi_packed));
  return tc::pack_f16x2(a - h.x, b - h.y);
}

// One thread = one accumulator row (TMEM lane): apply the epilogue to the BN columns at t_row and write them out.
// Warp-collective (tcgen05.ld): every lane of the warp must call it, also for rows beyond M.
// amax: running maximum magnitude of the values this thread stored as IEEE halves (checked against the half range once,
// when the CTA is done)
template <int BN, int EPI>
__device__ __forceinline__ void epilogue_rows(const GemmTcParams &p, uint32_t t_row, int row, int n_blk, float &amax) {
  constexpr bool SWIGLU = (EPI == EPI_SWIGLU);
  if constexpr (SWIGLU) {
    constexpr int HALF = BN / 2;
#pragma unroll 1
    for (int c = 0; c < HALF / 32; ++c) {
      uint32_t g[32], u[32];
      tc::tmem_ld_32x32b_x32(t_row + c * 32, g);
      tc::tmem_ld_32x32b_x32(t_row + HALF + c * 32, u);
      tc::tmem_ld_wait();
      if (row < p.M) {
        uint32_t pk[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const float g0 = __uint_as_float(g[2 * i]), g1 = __uint_as_float(g[2 * i + 1]);
          const float u0 = __uint_as_float(u[2 * i]), u1 = __uint_as_float(u[2 * i + 1]);
          const float y0 = g0 / (1.f + __expf(-g0)) * u0, y1 = g1 / (1.f + __expf(-g1)) * u1;
          amax = fmaxf(amax, fmaxf(fabsf(y0), fabsf(y1)));
          pk[i] = tc::pack_act(y0, y1, p.f16 != 0);
        }
        const size_t act_ld = p.lo_act ? 2 * (size_t)p.F : (size_t)p.F;
        // (streaming stores: the [T, F] output is far larger than the L2 and is read once, by the next kernel; kept out of the
        // way, the band of A rows that every column block re-reads stays resident)
        uint4 *dst = reinterpret_cast<uint4 *>(p.act + (size_t)row * act_ld + (size_t)n_blk * HALF + c * 32);
#pragma unroll
        for (int i = 0; i < 4; ++i) __stcs(dst + i, make_uint4(pk[4 * i], pk[4 * i + 1], pk[4 * i + 2], pk[4 * i + 3]));
        if (p.lo_act) {      // split output: the low halves, recomputed from the same fp32 values
          uint32_t lo[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const float g0 = __uint_as_float(g[2 * i]), g1 = __uint_as_float(g[2 * i + 1]);
            const float u0 = __uint_as_float(u[2 * i]), u1 = __uint_as_float(u[2 * i + 1]);
            lo[i] = pack_f16x2_lo(g0 / (1.f + __expf(-g0)) * u0, g1 / (1.f + __expf(-g1)) * u1, pk[i]);
          }
          uint4 *dl = reinterpret_cast<uint4 *>(p.act + (size_t)row * act_ld + p.F + (size_t)n_blk * HALF + c * 32);
#pragma unroll
          for (int i = 0; i < 4; ++i) dl[i] = make_uint4(lo[4 * i], lo[4 * i + 1], lo[4 * i + 2], lo[4 * i + 3]);
        }
      }
    }
  } else if constexpr (EPI == EPI_ROPE) {
    // head-aligned tiles (head_dim 128): rotate pairs (i, i + 64) of the q / K heads in fp32 before the one
    // rounding to bf16; V heads are stored as they are
    const int pos = row < p.M ? p.rope_pos[row] : 0;
    const float4 *ct = reinterpret_cast<const float4 *>(p.cos_tab + (size_t)pos * 64);
    const float4 *sn = reinterpret_cast<const float4 *>(p.sin_tab + (size_t)pos * 64);
#pragma unroll 1
    for (int hh = 0; hh < BN / 128; ++hh) {
      const int col_h = n_blk * BN + hh * 128;
      bf16 *dstp;
      __half *dupp = nullptr, *lop = nullptr;      // lop: where the low halves of this head go (split output), if anywhere
      bool rope, f16 = false;
      if (col_h < p.out.n0) {
        dstp = reinterpret_cast<bf16 *>(p.out.p0) + (size_t)row * p.out.ld0 + col_h;
        rope = true;
        f16 = p.f16 != 0;
        if (p.lo_p0) lop = p.lo_p0 + (size_t)row * p.out.ld0 + col_h;
      } else {
        const int cc = col_h - p.out.n0;
        const int seg = cc / p.out.seg_w, within = cc - seg * p.out.seg_w;
        const size_t srow = (p.out.slot_map && row < p.M) ? (size_t)p.out.slot_map[row] : (size_t)row;
        dstp = reinterpret_cast<bf16 *>(p.out.seg_base) + (size_t)seg * p.out.seg_stride + srow * p.out.seg_w + within;
        if (p.dup_base) dupp = p.dup_base + (size_t)seg * p.dup_stride + (size_t)row * p.out.seg_w + within;
        rope = (seg & 1) == 0;      // segments alternate K (rotated) and V (not)
        if (p.lo_dup && dupp && seg == 0) lop = p.lo_dup + (size_t)row * p.out.seg_w + within;
      }
#pragma unroll 1
      for (int c = 0; c < 2; ++c) {
        uint32_t a[32], bq[32];
        tc::tmem_ld_32x32b_x32(t_row + hh * 128 + c * 32, a);
        tc::tmem_ld_32x32b_x32(t_row + hh * 128 + 64 + c * 32, bq);
        tc::tmem_ld_wait();
        if (row < p.M) {
          if (rope) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const float4 cv = ct[c * 8 + i], sv = sn[c * 8 + i];
              const float cc4[4] = {cv.x, cv.y, cv.z, cv.w}, ss4[4] = {sv.x, sv.y, sv.z, sv.w};
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const float x = __uint_as_float(a[4 * i + e]), y = __uint_as_float(bq[4 * i + e]);
                a[4 * i + e] = __float_as_uint(x * cc4[e] - y * ss4[e]);
                bq[4 * i + e] = __float_as_uint(y * cc4[e] + x * ss4[e]);
              }
            }
          }
          if (f16 || dupp) {
#pragma unroll
            for (int i = 0; i < 32; ++i) amax = fmaxf(amax, fmaxf(fabsf(__uint_as_float(a[i])), fabsf(__uint_as_float(bq[i]))));
          }
          uint4 *d0 = reinterpret_cast<uint4 *>(dstp + c * 32);
          uint4 *d1 = reinterpret_cast<uint4 *>(dstp + 64 + c * 32);
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            d0[i] = make_uint4(tc::pack_act(__uint_as_float(a[8 * i]), __uint_as_float(a[8 * i + 1]), f16),
                               tc::pack_act(__uint_as_float(a[8 * i + 2]), __uint_as_float(a[8 * i + 3]), f16),
                               tc::pack_act(__uint_as_float(a[8 * i + 4]), __uint_as_float(a[8 * i + 5]), f16),
                               tc::pack_act(__uint_as_float(a[8 * i + 6]), __uint_as_float(a[8 * i + 7]), f16));
            d1[i] = make_uint4(tc::pack_act(__uint_as_float(bq[8 * i]), __uint_as_float(bq[8 * i + 1]), f16),
                               tc::pack_act(__uint_as_float(bq[8 * i + 2]), __uint_as_float(bq[8 * i + 3]), f16),
                               tc::pack_act(__uint_as_float(bq[8 * i + 4]), __uint_as_float(bq[8 * i + 5]), f16),
                               tc::pack_act(__uint_as_float(bq[8 * i + 6]), __uint_as_float(bq[8 * i + 7]), f16));
          }
          if (lop) {    // low halves of q (or of K's half copy): value - float(high half), from the same fp32 accumulators
            uint4 *l0 = reinterpret_cast<uint4 *>(lop + c * 32);
            uint4 *l1 = reinterpret_cast<uint4 *>(lop + 64 + c * 32);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              uint32_t wa[4], wb[4];
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const float a0 = __uint_as_float(a[8 * i + 2 * e]), a1 = __uint_as_float(a[8 * i + 2 * e + 1]);
                const float b0 = __uint_as_float(bq[8 * i + 2 * e]), b1 = __uint_as_float(bq[8 * i + 2 * e + 1]);
                wa[e] = pack_f16x2_lo(a0, a1, tc::pack_f16x2(a0, a1));
                wb[e] = pack_f16x2_lo(b0, b1, tc::pack_f16x2(b0, b1));
              }
              l0[i] = make_uint4(wa[0], wa[1], wa[2], wa[3]);
              l1[i] = make_uint4(wb[0], wb[1], wb[2], wb[3]);
            }
          }
          if (dupp) {   // the same values once more as halves, straight from the fp32 accumulators
            uint4 *e0 = reinterpret_cast<uint4 *>(dupp + c * 32);
            uint4 *e1 = reinterpret_cast<uint4 *>(dupp + 64 + c * 32);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              e0[i] = make_uint4(tc::pack_f16x2(__uint_as_float(a[8 * i]), __uint_as_float(a[8 * i + 1])),
                                 tc::pack_f16x2(__uint_as_float(a[8 * i + 2]), __uint_as_float(a[8 * i + 3])),
                                 tc::pack_f16x2(__uint_as_float(a[8 * i + 4]), __uint_as_float(a[8 * i + 5])),
                                 tc::pack_f16x2(__uint_as_float(a[8 * i + 6]), __uint_as_float(a[8 * i + 7])));
              e1[i] = make_uint4(tc::pack_f16x2(__uint_as_float(bq[8 * i]), __uint_as_float(bq[8 * i + 1])),
                                 tc::pack_f16x2(__uint_as_float(bq[8 * i + 2]), __uint_as_float(bq[8 * i + 3])),
                                 tc::pack_f16x2(__uint_as_float(bq[8 * i + 4]), __uint_as_float(bq[8 * i + 5])),
                                 tc::pack_f16x2(__uint_as_float(bq[8 * i + 6]), __uint_as_float(bq[8 * i + 7])));
            }
          }
        }
      }
    }
  } else {
#pragma unroll 1
    for (int c = 0; c < BN / 32; ++c) {
      uint32_t r[32];
      tc::tmem_ld_32x32b_x32(t_row + c * 32, r);
      tc::tmem_ld_wait();
      if (row < p.M) {
        const int col = n_blk * BN + c * 32;
        if (p.out.mode == OUT_RESID_ADD_F32) {
          float4 *px = reinterpret_cast<float4 *>(reinterpret_cast<float *>(p.out.p0) + (size_t)row * p.out.ld0 + col);
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            float4 v = __ldcs(px + i);          // streamed once per projection: do not displace the weight tiles in L2
            v.x += __uint_as_float(r[4 * i]); v.y += __uint_as_float(r[4 * i + 1]);
            v.z += __uint_as_float(r[4 * i + 2]); v.w += __uint_as_float(r[4 * i + 3]);
            __stcs(px + i, v);
          }
        } else {
          bf16 *dstp;
          bool f16 = false;
          if (col < p.out.n0) {
            dstp = reinterpret_cast<bf16 *>(p.out.p0) + (size_t)row * p.out.ld0 + col;
            f16 = p.f16 != 0;
          } else {
            const int cc = col - p.out.n0;
            const int seg = cc / p.out.seg_w, within = cc - seg * p.out.seg_w;
            const size_t srow = p.out.slot_map ? (size_t)p.out.slot_map[row] : (size_t)row;
            dstp = reinterpret_cast<bf16 *>(p.out.seg_base) + (size_t)seg * p.out.seg_stride + srow * p.out.seg_w + within;
          }
          if (f16) {
#pragma unroll
            for (int i = 0; i < 32; ++i) amax = fmaxf(amax, fabsf(__uint_as_float(r[i])));
          }
          uint4 *dst = reinterpret_cast<uint4 *>(dstp);
#pragma unroll
          for (int i = 0; i < 4; ++i)
            dst[i] = make_uint4(tc::pack_act(__uint_as_float(r[8 * i]), __uint_as_float(r[8 * i + 1]), f16),
                                tc::pack_act(__uint_as_float(r[8 * i + 2]), __uint_as_float(r[8 * i + 3]), f16),
                                tc::pack_act(__uint_as_float(r[8 * i + 4]), __uint_as_float(r[8 * i + 5]), f16),
                                tc::pack_act(__uint_as_float(r[8 * i + 6]), __uint_as_float(r[8 * i + 7]), f16));
        }
      }
    }
  }
}

// TF32: A and B hold fp32 (tensor maps of fp32 elements, 32 per 128-byte tile row instead of 64; p.K counts 16-bit units, i.e.
// twice the fp32 K), the MMAs are kind::tf32; everything else -- tile bytes, descriptors, ring, epilogues -- is the same.
template <int BN, int STAGES, int EPI, bool TF32 = false>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB0,
               const __grid_constant__ CUtensorMap tmB1, const __grid_constant__ CUtensorMap tmB2, GemmTcParams p) {
  using L = SmemLayout<BN, STAGES>;
  constexpr int KSTEP = TF32 ? BK / 2 : BK;      // elements of the operand type per K block
  constexpr bool SWIGLU = (EPI == EPI_SWIGLU);
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t *bars = reinterpret_cast<uint64_t *>(smem + L::BAR_OFFSET);
  uint64_t *full_bar = bars;                  // [STAGES]
  uint64_t *empty_bar = bars + STAGES;        // [STAGES]
  uint64_t *tfull_bar = bars + 2 * STAGES;    // [2]
  uint64_t *tempty_bar = bars + 2 * STAGES + 2;   // [2]
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * STAGES + 4);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr uint32_t TMEM_COLS = 2 * BN;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { tc::mbar_init(tc::smem_u32(&full_bar[s]), 1); tc::mbar_init(tc::smem_u32(&empty_bar[s]), 1); }
    for (int a = 0; a < 2; ++a) { tc::mbar_init(tc::smem_u32(&tfull_bar[a]), 1); tc::mbar_init(tc::smem_u32(&tempty_bar[a]), 4); }
    *abort_flag = 0;
    tc::fence_barrier_init();
    tc::tma_prefetch_desc(&tmA);
    tc::tma_prefetch_desc(&tmB0);
  }
  if (warp == 1) tc::tmem_alloc(tc::smem_u32(tmem_slot), TMEM_COLS);
  tc::tc_fence_before_sync();
  __syncthreads();
  tc::tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  const int num_tiles = p.num_m_blocks * p.num_n_blocks;
  const int num_kb = p.K / BK;

  if (warp == 0) {
    if (lane == 0) {
      // ------------------------------------------------ TMA producer
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
        int m_blk, n_blk;
        tile_coords(tile, p.num_m_blocks, p.num_n_blocks, p.group_m, m_blk, n_blk);
        const CUtensorMap *tb = &tmB0;
        int b_row = n_blk * BN;
        if constexpr (SWIGLU) {
          b_row = n_blk * (BN / 2);
        } else {
          if (b_row >= p.nB0 + p.nB1) { tb = &tmB2; b_row -= p.nB0 + p.nB1; }
          else if (b_row >= p.nB0) { tb = &tmB1; b_row -= p.nB0; }
        }
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!wait_or_abort(tc::smem_u32(&empty_bar[stage]), phase ^ 1, abort_flag, p.status)) { ok = false; break; }
          const uint32_t fb = tc::smem_u32(&full_bar[stage]);
          uint8_t *sa = smem + stage * L::STAGE_BYTES;
          uint8_t *sb = sa + L::A_BYTES;
          tc::mbar_expect_tx(fb, L::STAGE_BYTES);
          tc::tma_load_2d(tc::smem_u32(sa), &tmA, fb, kb * KSTEP, m_blk * BM);
          const int kx = (kb >= p.kb_wrap ? kb - p.kb_wrap : kb) * KSTEP;      // B's K coordinate (wraps for a split A)
          if constexpr (SWIGLU) {
            tc::tma_load_2d(tc::smem_u32(sb), &tmB0, fb, kx, b_row);                     // gate rows
            tc::tma_load_2d(tc::smem_u32(sb + L::B_BYTES / 2), &tmB1, fb, kx, b_row);   // up rows
          } else {
            tc::tma_load_2d(tc::smem_u32(sb), tb, fb, kx, b_row);
          }
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ------------------------------------------------ MMA issuer
      const uint32_t idesc = TF32 ? tc::umma_idesc_tf32(BM, BN) : tc::umma_idesc(BM, BN, 0, 0, p.f16, p.f16);
      int stage = 0;
      uint32_t phase = 0;
      int it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++it) {
        const int acc = it & 1;
        const uint32_t acc_phase = (it >> 1) & 1;
        if (!wait_or_abort(tc::smem_u32(&tempty_bar[acc]), acc_phase ^ 1, abort_flag, p.status)) break;
        tc::tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + acc * BN;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!wait_or_abort(tc::smem_u32(&full_bar[stage]), phase, abort_flag, p.status)) { ok = false; break; }
          tc::tc_fence_after_sync();
          const uint32_t a_addr = tc::smem_u32(smem + stage * L::STAGE_BYTES);
          const uint32_t b_addr = a_addr + L::A_BYTES;
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            const uint64_t ad = tc::umma_desc_sw128(a_addr + k * UMMA_K * 2, 16, 1024);
            const uint64_t bd = tc::umma_desc_sw128(b_addr + k * UMMA_K * 2, 16, 1024);
            if constexpr (TF32) tc::umma_ss_tf32(d_tmem, ad, bd, idesc, (kb | k) != 0 ? 1u : 0u);
            else tc::umma_ss(d_tmem, ad, bd, idesc, (kb | k) != 0 ? 1u : 0u);
          }
          tc::umma_commit(tc::smem_u32(&empty_bar[stage]));   // frees the ring slot when these MMAs retire
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
        if (ok) tc::umma_commit(tc::smem_u32(&tfull_bar[acc]));   // accumulator complete
      }
    }
  } else {
    // -------------------------------------------------- epilogue warps (2..5)
    const int quarter = warp & 3;   // the TMEM lane quarter this warp may read
    int it = 0;
    float amax = 0.f;
    for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x, ++it) {
      int m_blk, n_blk;
      tile_coords(tile, p.num_m_blocks, p.num_n_blocks, p.group_m, m_blk, n_blk);
      const int acc = it & 1;
      const uint32_t acc_phase = (it >> 1) & 1;
      if (!wait_or_abort(tc::smem_u32(&tfull_bar[acc]), acc_phase, abort_flag, p.status)) break;
      tc::tc_fence_after_sync();
      const int row = m_blk * BM + quarter * 32 + lane;
      const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * BN;
      epilogue_rows<BN, EPI>(p, t_row, row, n_blk, amax);
      tc::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) tc::mbar_arrive(tc::smem_u32(&tempty_bar[acc]));
    }
    if ((p.f16 || p.dup_base) && amax >= HALF_OVERFLOW) atomicOr(p.status, STATUS_ACT_OVERFLOW);   // a half store was clamped
  }
  tc::tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc::tc_fence_after_sync();
    tc::tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

// ---------------------------------------------------------------------------------------------------------
// CTA-pair variant (cta_group::2): a cluster of two CTAs on neighbouring SMs computes one 256 x 256 tile.  Each CTA
// stages its own 128 rows of A and its own 128 rows (N half) of B -- half the B traffic per SM of the single-CTA
// kernel --, the even-ranked CTA issues 256 x 256 x 16 MMAs that read both CTAs' shared memory and write 128
// accumulator rows into each CTA's tensor memory, and both CTAs run the epilogue on their own rows.
// Barriers: the leader's full[] collects the bytes of both CTAs' TMA loads; every commit is multicast to the
// barriers of both CTAs; the accumulator-empty barrier lives in the leader and takes 8 warp arrivals.
// ---------------------------------------------------------------------------------------------------------
constexpr int PAIR_BN = 256;

template <int STAGES>
struct PairSmem {
  static constexpr int A_BYTES = BM * BK * 2;          // this CTA's 128 rows of A
  static constexpr int B_BYTES = 128 * BK * 2;         // this CTA's 128 rows of B
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int BAR_OFFSET = STAGES * STAGE_BYTES;
  static constexpr int TOTAL = BAR_OFFSET + 256 + 1024;
};

template <int STAGES, int EPI>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(GEMM_THREADS, 1)
gemm_tc_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB0,
                    const __grid_constant__ CUtensorMap tmB1, const __grid_constant__ CUtensorMap tmB2, GemmTcParams p) {
  using L = PairSmem<STAGES>;
  constexpr bool SWIGLU = (EPI == EPI_SWIGLU);
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t *bars = reinterpret_cast<uint64_t *>(smem + L::BAR_OFFSET);
  uint64_t *full_bar = bars;
  uint64_t *empty_bar = bars + STAGES;
  uint64_t *tfull_bar = bars + 2 * STAGES;
  uint64_t *tempty_bar = bars + 2 * STAGES + 2;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * STAGES + 4);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = tc::cluster_ctarank();
  const bool leader = rank == 0;
  constexpr uint32_t TMEM_COLS = 2 * PAIR_BN;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { tc::mbar_init(tc::smem_u32(&full_bar[s]), 1); tc::mbar_init(tc::smem_u32(&empty_bar[s]), 1); }
    for (int a = 0; a < 2; ++a) { tc::mbar_init(tc::smem_u32(&tfull_bar[a]), 1); tc::mbar_init(tc::smem_u32(&tempty_bar[a]), 8); }
    *abort_flag = 0;
    tc::fence_barrier_init();
    tc::tma_prefetch_desc(&tmA);
    tc::tma_prefetch_desc(&tmB0);
  }
  if (warp == 1) tc::tmem_alloc_pair(tc::smem_u32(tmem_slot), TMEM_COLS);
  tc::tc_fence_before_sync();
  __syncthreads();
  tc::cluster_sync_all();          // both CTAs' barriers are initialised before anyone signals across the pair
  tc::tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  const int num_pairs = gridDim.x >> 1, pair = blockIdx.x >> 1;
  const int num_m2 = (p.M + 2 * BM - 1) / (2 * BM);
  const int num_n = SWIGLU ? p.F / 128 : p.N / PAIR_BN;
  const int num_tiles = num_m2 * num_n;
  const int num_kb = p.K / BK;
  auto coords = [&](int tile, int &m2, int &n_blk) {
    const int gm2 = max(1, p.group_m >> 1);
    const int band_tiles = gm2 * num_n;
    const int band = tile / band_tiles;
    const int r = tile - band * band_tiles;
    const int band_h = min(gm2, num_m2 - band * gm2);
    n_blk = r / band_h;
    m2 = band * gm2 + (r - n_blk * band_h);
  };

  if (warp == 0) {
    if (lane == 0) {
      // ------------------------------------------------ TMA producer (both CTAs, each its own halves)
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = pair; tile < num_tiles && ok; tile += num_pairs) {
        int m2, n_blk;
        coords(tile, m2, n_blk);
        const CUtensorMap *tb = &tmB0;
        int b_row;
        if constexpr (SWIGLU) {
          tb = leader ? &tmB0 : &tmB1;                 // leader stages the gate rows, its peer the up rows
          b_row = n_blk * 128;
        } else {
          b_row = n_blk * PAIR_BN;
          if (b_row >= p.nB0 + p.nB1) { tb = &tmB2; b_row -= p.nB0 + p.nB1; }
          else if (b_row >= p.nB0) { tb = &tmB1; b_row -= p.nB0; }
          b_row += rank * 128;
        }
        const int a_row = m2 * 2 * BM + rank * BM;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!wait_or_abort(tc::smem_u32(&empty_bar[stage]), phase ^ 1, abort_flag, p.status)) { ok = false; break; }
          const uint32_t own_full = tc::smem_u32(&full_bar[stage]);
          const uint32_t leader_full = tc::mapa_shared(own_full, 0);
          uint8_t *sa = smem + stage * L::STAGE_BYTES;
          uint8_t *sb = sa + L::A_BYTES;
          if (leader) tc::mbar_expect_tx(own_full, 2 * L::STAGE_BYTES);   // bytes of both CTAs' loads
          tc::tma_load_2d_pair(tc::smem_u32(sa), &tmA, leader_full, kb * BK, a_row);
          tc::tma_load_2d_pair(tc::smem_u32(sb), tb, leader_full, (kb >= p.kb_wrap ? kb - p.kb_wrap : kb) * BK, b_row);
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && leader) {
      // ------------------------------------------------ MMA issuer (leader CTA only)
      const uint32_t idesc = tc::umma_idesc(2 * BM, PAIR_BN, 0, 0, p.f16, p.f16);
      int stage = 0;
      uint32_t phase = 0;
      int it = 0;
      bool ok = true;
      for (int tile = pair; tile < num_tiles && ok; tile += num_pairs, ++it) {
        const int acc = it & 1;
        const uint32_t acc_phase = (it >> 1) & 1;
        if (!wait_or_abort(tc::smem_u32(&tempty_bar[acc]), acc_phase ^ 1, abort_flag, p.status)) break;
        tc::tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + acc * PAIR_BN;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!wait_or_abort(tc::smem_u32(&full_bar[stage]), phase, abort_flag, p.status)) { ok = false; break; }
          tc::tc_fence_after_sync();
          const uint32_t a_addr = tc::smem_u32(smem + stage * L::STAGE_BYTES);
          const uint32_t b_addr = a_addr + L::A_BYTES;
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            const uint64_t ad = tc::umma_desc_sw128(a_addr + k * UMMA_K * 2, 16, 1024);
            const uint64_t bd = tc::umma_desc_sw128(b_addr + k * UMMA_K * 2, 16, 1024);
            tc::umma_ss_pair(d_tmem, ad, bd, idesc, (kb | k) != 0 ? 1u : 0u);
          }
          tc::umma_commit_pair(tc::smem_u32(&empty_bar[stage]), 3);     // frees the slot in both CTAs
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
        if (ok) tc::umma_commit_pair(tc::smem_u32(&tfull_bar[acc]), 3);  // accumulator complete, both CTAs
      }
    }
  } else {
    // -------------------------------------------------- epilogue warps (2..5) of both CTAs, own 128 rows each
    const int quarter = warp & 3;
    const uint32_t leader_tempty0 = tc::mapa_shared(tc::smem_u32(&tempty_bar[0]), 0);
    const uint32_t leader_tempty1 = tc::mapa_shared(tc::smem_u32(&tempty_bar[1]), 0);
    int it = 0;
    float amax = 0.f;
    for (int tile = pair; tile < num_tiles; tile += num_pairs, ++it) {
      int m2, n_blk;
      coords(tile, m2, n_blk);
      const int acc = it & 1;
      const uint32_t acc_phase = (it >> 1) & 1;
      if (!wait_or_abort(tc::smem_u32(&tfull_bar[acc]), acc_phase, abort_flag, p.status)) break;
      tc::tc_fence_after_sync();
      const int row = m2 * 2 * BM + rank * BM + quarter * 32 + lane;
      const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * PAIR_BN;
      epilogue_rows<PAIR_BN, EPI>(p, t_row, row, n_blk, amax);
      tc::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) tc::mbar_arrive_cluster(acc ? leader_tempty1 : leader_tempty0);
    }
    if ((p.f16 || p.dup_base) && amax >= HALF_OVERFLOW) atomicOr(p.status, STATUS_ACT_OVERFLOW);
  }
  tc::tc_fence_before_sync();
  __syncthreads();
  tc::cluster_sync_all();          // neither CTA leaves while its peer may still signal its barriers or read its smem
  if (warp == 1) {
    __syncwarp();
    tc::tc_fence_after_sync();
    tc::tmem_dealloc_pair(tmem_base, TMEM_COLS);
  }
}

// see launch_bounded_wait_probe
__global__ void __launch_bounds__(64) bounded_wait_probe_kernel(long long limit, unsigned int *status, unsigned int *outcome) {
  __shared__ uint64_t bar;
  __shared__ int abort_word;
  volatile int *abort_flag = &abort_word;
  if (threadIdx.x == 0) {
    tc::mbar_init(tc::smem_u32(&bar), 1);      // one arrival expected; nobody will ever arrive
    abort_word = 0;
    tc::fence_barrier_init();
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    // the role that runs out of patience: same wait as every role of the GEMM kernels, short limit
    const bool ok = wait_or_abort(tc::smem_u32(&bar), 0, abort_flag, status, limit);
    outcome[0] = ok ? 0u : 1u;
  } else if (threadIdx.x == 32) {
    // a role with the full limit: it must leave because the first role raised the abort flag, not by its own clock
    const long long t0 = clock64();
    const bool ok = wait_or_abort(tc::smem_u32(&bar), 0, abort_flag, status);
    outcome[1] = (!ok && clock64() - t0 < 2 * limit + 10000000) ? 1u : 0u;
  }
}

template <int STAGES, int EPI>
int launch_pair(const CUtensorMap &a, const CUtensorMap &b0, const CUtensorMap &b1, const CUtensorMap &b2,
                const GemmTcParams &p, int tiles, cudaStream_t st) {
  using L = PairSmem<STAGES>;
  auto kern = gemm_tc_pair_kernel<STAGES, EPI>;
  if (ensure_dynamic_smem(reinterpret_cast<const void *>(kern), L::TOTAL)) return SWIFTKV_ERR_CUDA;
  int pairs = num_sms() / 2;
  if (tiles < pairs) pairs = tiles;
  kern<<<2 * pairs, GEMM_THREADS, L::TOTAL, st>>>(a, b0, b1, b2, p);
  return cudaGetLastError() == cudaSuccess ? SWIFTKV_OK : SWIFTKV_ERR_CUDA;
}

template <int BN, int STAGES, int EPI>
int launch_cfg(const CUtensorMap &a, const CUtensorMap &b0, const CUtensorMap &b1, const CUtensorMap &b2,
               const GemmTcParams &p, cudaStream_t st) {
  using L = SmemLayout<BN, STAGES>;
  auto kern = gemm_tc_kernel<BN, STAGES, EPI>;
  if (ensure_dynamic_smem(reinterpret_cast<const void *>(kern), L::TOTAL)) return SWIFTKV_ERR_CUDA;
  const int tiles = p.num_m_blocks * p.num_n_blocks;
  const int grid = tiles < num_sms() ? tiles : num_sms();
  kern<<<grid, GEMM_THREADS, L::TOTAL, st>>>(a, b0, b1, b2, p);
  return cudaGetLastError() == cudaSuccess ? SWIFTKV_OK : SWIFTKV_ERR_CUDA;
}

}  // namespace

// fp32 operands on the tensor cores (kind::tf32): out[M, N] (+)= A[M, K] B[N, K]^T, fp32 in and out.  N % 128 == 0, K % 32 == 0.
bool tc_gemm_tf32_supported(int M, int N, int K) { return M >= 1 && K >= 32 && (K % 32) == 0 && (N % 128) == 0; }
int launch_gemm_tc_tf32(const float *A, const float *B, int M, int N, int K, float *out, bool accumulate, unsigned int *status,
                        cudaStream_t st, int k_chunk) {
  if (!tc_gemm_tf32_supported(M, N, K)) return SWIFTKV_ERR_UNSUPPORTED;
  if (k_chunk < 0 || (k_chunk % 32) != 0) return SWIFTKV_ERR_INVALID_ARG;
  constexpr int BN = 128, STAGES = 6;
  if (!accumulate && cudaMemsetAsync(out, 0, (size_t)M * N * sizeof(float), st) != cudaSuccess) return SWIFTKV_ERR_CUDA;
  using L = SmemLayout<BN, STAGES>;
  auto kern = gemm_tc_kernel<BN, STAGES, EPI_PLAIN, true>;
  if (ensure_dynamic_smem(reinterpret_cast<const void *>(kern), L::TOTAL)) return SWIFTKV_ERR_CUDA;
  // The tensor core adds into its fp32 accumulator by cutting, not rounding (measured: with exactly representable operands
  // the result falls short by 2^-24 per accumulation step on average, 7e-6 relative at K = 1024 and 5e-4 at K = 65536 on
  // same-sign data).  k_chunk > 0 keeps every accumulation chain that short: one launch per chunk of the inner dimension,
  // the chunks meeting in the epilogue's fp32 add (round to nearest).
  const int step = k_chunk > 0 ? k_chunk : K;
  for (int k0 = 0; k0 < K; k0 += step) {
    const int kc = K - k0 < step ? K - k0 : step;
    CUtensorMap ta, tb;
    if (get_tmap_f32(&ta, A + k0, M, kc, BM, K) || get_tmap_f32(&tb, B + k0, N, kc, BN, K)) return SWIFTKV_ERR_CUDA;
    GemmTcParams p{};
    p.M = M; p.N = N; p.K = 2 * kc; p.nB0 = N; p.nB1 = 0;
    p.kb_wrap = 2 * kc / BK;
    p.num_m_blocks = (M + BM - 1) / BM; p.num_n_blocks = N / BN;
    p.group_m = 32;
    p.out = out_plain(OUT_RESID_ADD_F32, out, N, N, status);
    p.status = status;
    const int tiles = p.num_m_blocks * p.num_n_blocks;
    const int grid = tiles < num_sms() ? tiles : num_sms();
    kern<<<grid, GEMM_THREADS, L::TOTAL, st>>>(ta, tb, tb, tb, p);
    if (cudaGetLastError() != cudaSuccess) return SWIFTKV_ERR_CUDA;
  }
  return SWIFTKV_OK;
}

int launch_bounded_wait_probe(long long limit_clocks, unsigned int *status, unsigned int *outcome, cudaStream_t st) {
  bounded_wait_probe_kernel<<<1, 64, 0, st>>>(limit_clocks, status, outcome);
  return cudaGetLastError() == cudaSuccess ? SWIFTKV_OK : SWIFTKV_ERR_CUDA;
}

bool tc_gemm_supported(int M, int N, int K) { return M >= 1 && K >= 64 && (K % 64) == 0 && (N % 128) == 0 && N >= 128; }
bool tc_swiglu_supported(int M, int F, int K) { return M >= 1 && K >= 64 && (K % 64) == 0 && (F % 128) == 0 && F >= 128; }

// Raster band height in 128-row blocks.  A band's A rows (band x K x 2 bytes) are re-walked for every column block, so they
// must stay in L2 next to the streaming weights and output: 4096 rows for K <= 4096 (33 MB of A), 2048 rows for longer K.
static int group_m_setting(int K) {
  static int v = 0, v_long = 0;
  if (!v) {
    const char *e = getenv("SWIFTKV_GROUP_M"), *el = getenv("SWIFTKV_GROUP_M_LONGK");
    v_long = el ? atoi(el) : (e ? atoi(e) : 16);
    if (v_long < 1) v_long = 16;
    v = e ? atoi(e) : 32;
    if (v < 1) v = 32;
  }
  return K > 4096 ? v_long : v;
}
static bool g_use_pairs = true, g_swiglu_pairs = false;
void tc_gemm_use_cta_pairs(bool on, bool swiglu_too) { g_use_pairs = on; g_swiglu_pairs = swiglu_too; }

int launch_gemm_tc(const void *A, bool f16, int M, int K, const void *B0, int nB0, const void *B1, int nB1, const void *B2,
                   int nB2, OutDesc out, void *dup_base, long long dup_stride, const RopeSpec *rope, unsigned int *status,
                   cudaStream_t st, const GemmSplit *split) {
  const int N = nB0 + nB1 + nB2;
  const bool a_split = split && split->a_split;
  if (split && !f16) return SWIFTKV_ERR_UNSUPPORTED;            // hi + lo pairs exist for IEEE halves only
  if (split && (split->lo_p0 || split->lo_dup) && !rope) return SWIFTKV_ERR_UNSUPPORTED;
  if (!tc_gemm_supported(M, N, K)) return SWIFTKV_ERR_UNSUPPORTED;
  if (out.mode == OUT_STORE_F32) return SWIFTKV_ERR_UNSUPPORTED;
  int BN = 256;
  if ((N % 256) || (nB1 + nB2 > 0 && ((nB0 % 256) || (nB1 % 256)))) BN = 128;
  if (nB1 + nB2 > 0 && ((nB0 % BN) || (nB1 % BN))) return SWIFTKV_ERR_UNSUPPORTED;
  if (out.mode == OUT_STORE && ((out.n0 % 32) || (out.n0 < N && (out.seg_w % 32)))) return SWIFTKV_ERR_UNSUPPORTED;
  CUtensorMap ta, tb0, tb1, tb2;
  const int KA = a_split ? 2 * K : K;      // A's row: [hi | lo] side by side along K when split
  if (get_tmap(&ta, A, M, KA, KA, BM, BK)) return SWIFTKV_ERR_CUDA;
  if (get_tmap(&tb0, B0, nB0, K, K, BN, BK)) return SWIFTKV_ERR_CUDA;
  tb1 = tb0; tb2 = tb0;
  if (nB1 > 0 && get_tmap(&tb1, B1, nB1, K, K, BN, BK)) return SWIFTKV_ERR_CUDA;
  if (nB2 > 0 && get_tmap(&tb2, B2, nB2, K, K, BN, BK)) return SWIFTKV_ERR_CUDA;
  GemmTcParams p{};
  p.M = M; p.N = N; p.K = KA; p.nB0 = nB0; p.nB1 = nB1;
  p.kb_wrap = K / BK;
  p.lo_p0 = split ? reinterpret_cast<__half *>(split->lo_p0) : nullptr;
  p.lo_dup = split ? reinterpret_cast<__half *>(split->lo_dup) : nullptr;
  p.lo_act = 0;
  p.num_m_blocks = (M + BM - 1) / BM;
  p.num_n_blocks = N / BN;
  p.out = out; p.act = nullptr; p.F = 0; p.status = status; p.group_m = group_m_setting(K);
  p.f16 = f16; p.dup_base = reinterpret_cast<__half *>(dup_base); p.dup_stride = dup_stride;
  if (dup_base && !rope) return SWIFTKV_ERR_UNSUPPORTED;
  const bool pairs = g_use_pairs && BN == 256 && M > 128;
  CUtensorMap tb0h = tb0, tb1h = tb1, tb2h = tb2;      // pair kernel: each CTA loads 128-row halves of a B tile
  if (pairs) {
    if (get_tmap(&tb0h, B0, nB0, K, K, 128, BK)) return SWIFTKV_ERR_CUDA;
    tb1h = tb0h; tb2h = tb0h;
    if (nB1 > 0 && get_tmap(&tb1h, B1, nB1, K, K, 128, BK)) return SWIFTKV_ERR_CUDA;
    if (nB2 > 0 && get_tmap(&tb2h, B2, nB2, K, K, 128, BK)) return SWIFTKV_ERR_CUDA;
  }
  const int pair_tiles = ((M + 255) / 256) * (N / 256);
  // Few rows: a launch whose CTA pairs would cover less than half of the SMs runs as single CTAs on 128 x 128 tiles instead
  // (four times as many CTAs, each with a quarter of a pair's work) -- e.g. 512 rows x 4096 features: 128 CTAs instead of 64;
  // same accumulation order, same bits.  Only for long inner dimensions, where the launch is bound by streaming the weights
  // (a 256-token prompt at the 8B widths: 7.5 -> 7.2 ms); short ones are launch-latency either way.
  static int small_m_single = -1;
  if (small_m_single < 0) { const char *e = getenv("SWIFTKV_SMALL_M_SINGLE"); small_m_single = (e && e[0] == '0') ? 0 : 1; }
  if (pairs && small_m_single && K >= 2048 && 4 * pair_tiles <= num_sms()) {
    p.num_n_blocks = N / 128;
    if (rope) {
      if (rope->hd != 128 || out.mode != OUT_STORE || (out.n0 % 128) || (out.n0 < N && (out.seg_w % 128)))
        return SWIFTKV_ERR_UNSUPPORTED;
      p.rope_pos = rope->positions; p.cos_tab = rope->cos_tab; p.sin_tab = rope->sin_tab;
      return launch_cfg<128, 6, EPI_ROPE>(ta, tb0h, tb1h, tb2h, p, st);
    }
    return launch_cfg<128, 6, EPI_PLAIN>(ta, tb0h, tb1h, tb2h, p, st);
  }
  if (rope) {
    // fused rotary embedding needs head-aligned tiles of 128-wide heads and a bf16 store
    if (rope->hd != 128 || out.mode != OUT_STORE || (out.n0 % 128) || (out.n0 < N && (out.seg_w % 128)))
      return SWIFTKV_ERR_UNSUPPORTED;
    p.rope_pos = rope->positions; p.cos_tab = rope->cos_tab; p.sin_tab = rope->sin_tab;
    if (pairs) return launch_pair<6, EPI_ROPE>(ta, tb0h, tb1h, tb2h, p, pair_tiles, st);
    if (BN == 256) return launch_cfg<256, 4, EPI_ROPE>(ta, tb0, tb1, tb2, p, st);
    return launch_cfg<128, 6, EPI_ROPE>(ta, tb0, tb1, tb2, p, st);
  }
  if (pairs) return launch_pair<6, EPI_PLAIN>(ta, tb0h, tb1h, tb2h, p, pair_tiles, st);
  if (BN == 256) return launch_cfg<256, 4, EPI_PLAIN>(ta, tb0, tb1, tb2, p, st);
  return launch_cfg<128, 6, EPI_PLAIN>(ta, tb0, tb1, tb2, p, st);
}

int launch_gemm_tc_swiglu(const void *A, bool f16, int M, int K, const void *Wg, const void *Wu, int F, void *act,
                          unsigned int *status, cudaStream_t st, bool a_split, bool out_split) {
  if (!tc_swiglu_supported(M, F, K)) return SWIFTKV_ERR_UNSUPPORTED;
  if ((a_split || out_split) && !f16) return SWIFTKV_ERR_UNSUPPORTED;
  CUtensorMap ta, tg, tu;
  const int KA = a_split ? 2 * K : K;
  if (get_tmap(&ta, A, M, KA, KA, BM, BK)) return SWIFTKV_ERR_CUDA;
  if (get_tmap(&tg, Wg, F, K, K, 128, BK)) return SWIFTKV_ERR_CUDA;
  if (get_tmap(&tu, Wu, F, K, K, 128, BK)) return SWIFTKV_ERR_CUDA;
  GemmTcParams p{};
  p.M = M; p.N = 2 * F; p.K = KA; p.nB0 = F; p.nB1 = F;
  p.kb_wrap = K / BK;
  p.lo_p0 = nullptr; p.lo_dup = nullptr; p.lo_act = out_split ? 1 : 0;
  p.num_m_blocks = (M + BM - 1) / BM;
  p.num_n_blocks = F / 128;
  p.out = OutDesc{}; p.act = reinterpret_cast<bf16 *>(act); p.F = F; p.status = status; p.group_m = group_m_setting(K);
  p.f16 = f16; p.dup_base = nullptr; p.dup_stride = 0;
  // measured on the 8B shape under the power cap: the single-CTA form is 3 % faster for this launch (it already keeps
  // the tensor pipe 85 % busy), while the pair form wins 7-10 % on the N = 4096 / 6144 projections
  if (g_swiglu_pairs && g_use_pairs && M > 128)
    return launch_pair<6, EPI_SWIGLU>(ta, tg, tu, tu, p, ((M + 255) / 256) * (F / 128), st);
  return launch_cfg<256, 4, EPI_SWIGLU>(ta, tg, tu, tu, p, st);
}

}  // namespace skv
