// Shared declarations of the SwiftKV prefill library (host + device helpers, launch prototypes).
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_fp8.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/swiftkv.h"

namespace skv {

// ---- device status word -------------------------------------------------------------------------------
// Kernels never trap: a bounded wait that runs out, or a bad token id, sets a bit here and carries on.
// STATUS_ACT_OVERFLOW: a value that had to be stored as IEEE half lay beyond the half range (|v| >= 65520 would round to
// infinity) and was clamped to +-65504.
enum : unsigned int { STATUS_TIMEOUT = 1u, STATUS_BAD_TOKEN = 2u, STATUS_ACT_OVERFLOW = 4u };
constexpr float HALF_OVERFLOW = 65520.f;

// ---- element types ---------------------------------------------------------------------------------------
using bf16 = __nv_bfloat16;

template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<bf16>(bf16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f<bf16>(float v) { return __float2bfloat16_rn(v); }
// IEEE half: the precise storage format for activations of a bf16 model; conversion saturates at +-65504
template <> __device__ __forceinline__ float to_f<__half>(__half v) { return __half2float(v); }
template <> __device__ __forceinline__ __half from_f<__half>(float v) {
  return __float2half_rn(fminf(fmaxf(v, -65504.f), 65504.f));
}

// one stored element of the FP8 cache (e4m3: 4 exponent bits, bias 7, 3 mantissa bits, finite only); its value is the
// decoded number times the fp32 scale of its token row (appendix "KV quantization": per-token FP8 quantization)
struct fp8e4 { uint8_t x; };
template <> __device__ __forceinline__ float to_f<fp8e4>(fp8e4 v) {
  return __half2float(__half(__nv_cvt_fp8_to_halfraw((__nv_fp8_storage_t)v.x, __NV_E4M3)));
}
constexpr float FP8_MAX = 448.f;
constexpr float FP8_AMAX_FLOOR = 5.421010862427522e-20f;   // 2^-64: an all-zero row still gets a normal scale

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// ---- where a GEMM writes its result ----------------------------------------------------------------------
// Columns [0, n0) go to p0 (row stride ld0).  Columns >= n0 are cut into segments of seg_w columns; segment i
// goes to seg_base + i*seg_stride (row stride seg_w): this is how one projection lands directly in the
// K / V planes of the cache (QKV projection of a layer, and the fused SingleInputKV projection of Sec. 3.5).
enum OutMode : int { OUT_STORE = 0, OUT_RESID_ADD_F32 = 1, OUT_STORE_F32 = 2 };
struct OutDesc {
  int mode;
  void *p0;
  long long ld0;
  int n0;
  void *seg_base;
  long long seg_stride;   // elements
  int seg_w;
  const int32_t *slot_map;   // optional: GEMM row r lands in row slot_map[r] of a segment (cache row of token r)
  unsigned int *status;      // optional: receives STATUS_ACT_OVERFLOW when a half store had to clamp
};
inline OutDesc out_plain(int mode, void *p, long long ld, int n, unsigned int *status = nullptr) {
  return OutDesc{mode, p, ld, n, nullptr, 0, 1, nullptr, status};
}

// ---- paged cache rows ------------------------------------------------------------------------------------
// A sequence's token p lives in cache row first + p (contiguous region), or -- with a block table -- in row
// blk[b * stride + p / PAGE_ROWS] * PAGE_ROWS + p % PAGE_ROWS.
constexpr int PAGE_ROWS = 128;
#ifdef __CUDACC__
__device__ __forceinline__ size_t kv_row_of(const int32_t *blk, int stride, int b, int first, int p) {
  return blk ? (size_t)blk[(size_t)b * stride + (p >> 7)] * PAGE_ROWS + (p & (PAGE_ROWS - 1)) : (size_t)first + p;
}
// write one fp32 accumulator where the descriptor says (device side)
// TP: element type of the p0 region; TS: element type of the segments (K / V cache planes)
template <typename TP, typename TS>
__device__ __forceinline__ void store_out(const OutDesc &o, int row, int col, float acc) {
  if (o.mode == OUT_RESID_ADD_F32) {
    float *p = reinterpret_cast<float *>(o.p0) + (size_t)row * o.ld0 + col;
    *p += acc;
  } else if (o.mode == OUT_STORE_F32) {
    reinterpret_cast<float *>(o.p0)[(size_t)row * o.ld0 + col] = acc;
  } else if (col < o.n0) {
    if constexpr (sizeof(TP) == 2 && !__is_same(TP, bf16)) {
      if (fabsf(acc) >= HALF_OVERFLOW && o.status) atomicOr(o.status, STATUS_ACT_OVERFLOW);
    }
    reinterpret_cast<TP *>(o.p0)[(size_t)row * o.ld0 + col] = from_f<TP>(acc);
  } else {
    const int c = col - o.n0;
    const int seg = c / o.seg_w, within = c % o.seg_w;
    const size_t srow = o.slot_map ? (size_t)o.slot_map[row] : (size_t)row;
    reinterpret_cast<TS *>(o.seg_base)[(size_t)seg * o.seg_stride + srow * o.seg_w + within] = from_f<TS>(acc);
  }
}
#endif

// raises a kernel's dynamic shared-memory limit once per (device, kernel) -- the attribute belongs to the device's copy of
// the function, so a process that drives several GPUs sets it on each; returns 0 on success
int ensure_dynamic_smem(const void *kernel, int bytes);

// sets the calling thread's swiftkv_last_error() text and returns `code` (defined with the C ABI)
int32_t report_error(int32_t code, const char *msg);

// ---- launch prototypes (each queues work on `st`, no synchronisation) -------------------------------------
// elementwise.cu
template <typename T>
void launch_embed(const T *embed, const int32_t *tokens, float *x, int n_tokens, int d, int vocab,
                  unsigned int *status, cudaStream_t st);
void launch_positions(const int32_t *cu_seqlens, int n_seqs, int32_t *positions, int32_t *last_idx, int n_tokens,
                      cudaStream_t st);
// y = x * rsqrt(mean(x^2)+eps) * gamma (gamma may be null: unit-rms only).  x fp32 [rows, d] -> out TO [rows, d]
// status (nullable): receives STATUS_ACT_OVERFLOW when TO is IEEE half and a value had to be clamped (the same holds for
// the other launches below that take a status word)
template <typename TG, typename TO>
// split (TO = IEEE half only): out is [rows, 2d], each row [hi(d) | lo(d)] with lo = y - float(hi): the A operand of a
// GEMM launched with GemmSplit::a_split
void launch_rmsnorm(const float *x, const TG *gamma, TO *out, int rows, int d, float eps, cudaStream_t st,
                    unsigned int *status = nullptr, bool split = false);
// in-place rotary embedding on `n_batches` tensors [*, n_heads, hd] spaced batch_stride elements apart; logical row r
// (position positions[r]) lives in tensor row slot_map[r] (null: row r)
template <typename T>
void launch_rope(T *x, long long batch_stride, int n_batches, const int32_t *positions, const int32_t *slot_map,
                 const float *cos_tab, const float *sin_tab, int rows, int n_heads, int hd, cudaStream_t st,
                 unsigned int *status = nullptr);
// packs each sequence's cache rows [row0[b], row0[b] + len[b]) of one layer's K and V planes (bf16) into contiguous half
// copies starting at row kcu[b]: the tensor-core attention kernel's operands in a chunked step with half activations
void launch_gather_kv_half(const bf16 *k, const bf16 *v, __half *k16, __half *v16, const int32_t *row0, const int32_t *len,
                           const int32_t *kcu, const int32_t *blk, int blk_stride, int n_seqs, int max_len, int dkv,
                           cudaStream_t st, unsigned int *status = nullptr);
// kv_fp8.cu : per-token FP8 cache rows.  One scale per row of `width` elements: scale = max(amax, 2^-64) / 448,
// code = e4m3(x / scale) (correctly rounded fp32 divisions, round to nearest even, saturating).  Row r of `src` goes to row
// slot_map[r] (null: r) of `codes` / `scale`; deq (nullable, row r) receives value(code) * scale in type TO.
// the new K / V rows of a decode minibatch (fp32, one per sequence) -> FP8 cache rows slot_map[r]: rotary embedding on K, rounding
// to the model dtype T, per-row scale, codes -- one launch
template <typename T>
void launch_store_kv_rows_fp8(const float *ky, const float *vy, const int32_t *slot_map, const int32_t *positions, const float *cos_tab,
                              const float *sin_tab, int rows, int n_heads, int hd, uint8_t *k_codes, float *k_scale, uint8_t *v_codes,
                              float *v_scale, cudaStream_t st);
template <typename TI, typename TO>
void launch_quantize_rows_fp8(const TI *src, int rows, int width, const int32_t *slot_map, uint8_t *codes, float *scale,
                              TO *deq, cudaStream_t st);
// dequantized, packed copies of each sequence's cache rows (K and V planes of one slot): sequence b's key p goes to row
// kcu[b] + p of k_out / v_out.  Row addressing as in launch_gather_kv_half.
template <typename TO>
void launch_gather_dequant_fp8(const uint8_t *k_codes, const uint8_t *v_codes, const float *k_scale, const float *v_scale,
                               TO *k_out, TO *v_out, const int32_t *row0, const int32_t *len, const int32_t *kcu,
                               const int32_t *blk, int blk_stride, int n_seqs, int max_len, int dkv, cudaStream_t st);
template <typename T>
void launch_swiglu(const T *gate, const T *up, T *out, long long n, cudaStream_t st, unsigned int *status = nullptr);
void launch_gather_rows(const float *x, const int32_t *idx, float *y, int n_rows, int d, cudaStream_t st);
// fp32 rows -> rows slot_map[r] (null: r) of a [*, width] plane of type T
template <typename T>
void launch_scatter_rows(const float *src, T *dst, const int32_t *slot_map, int rows, int width, cudaStream_t st);
// a decode step's new K / V rows (fp32, K not yet rotated) -> rotary embedding of K at pos[r] -> rows slot_map[r] of the
// K and V planes in the cache's element type, one launch
template <typename T>
void launch_store_kv_rows(const float *ky, const float *vy, T *k_plane, T *v_plane, const int32_t *slot_map, const int32_t *pos,
                          const float *cos_tab, const float *sin_tab, int rows, int n_heads, int hd, cudaStream_t st);
void launch_rope_table(float *cos_tab, float *sin_tab, int max_pos, int hd, double theta, cudaStream_t st);
// dst[r, c] = w[r, c] * gamma[c]   (gain of the input norm folded into a projection weight, Sec. 3.5)
template <typename T, typename TO>
void launch_fold(const T *w, const T *gamma, TO *dst, int rows, int cols, cudaStream_t st);
// IEEE-half copy of a bf16 matrix (the compute copy of a layer's weights when activations are kept in half)
void launch_bf16_to_f16(const bf16 *src, __half *dst, long long n, cudaStream_t st, unsigned int *status = nullptr);

// gemm_simt.cu : C = A[M,K] * B[N,K]^T with fp32 accumulation, any shape; result column c is written as
// column col0 + c of `out` (p0 region in the activation type TA, segments in the weight / cache type TW)
template <typename TA, typename TW>
void launch_gemm_simt(const TA *A, const TW *B, int M, int N, int K, OutDesc out, int col0, cudaStream_t st);

// gemm_tc.cu : tcgen05 / TMEM / TMA GEMMs (bf16)
struct TcGemmPlan;   // host object holding tensor maps
bool tc_gemm_supported(int M, int N, int K);
// fp32 operands on the tensor cores (kind::tf32, 10 mantissa bits of each operand): out[M, N] (+)= A[M, K] B[N, K]^T
bool tc_gemm_tf32_supported(int M, int N, int K);
// k_chunk > 0 (a multiple of 32): one launch per k_chunk of the inner dimension, summed by the epilogue's fp32 add -- the tensor
// core's own accumulation cuts instead of rounding, an error that grows with the length of the chain
int launch_gemm_tc_tf32(const float *A, const float *B, int M, int N, int K, float *out, bool accumulate, unsigned int *status,
                        cudaStream_t st, int k_chunk = 0);
// CTA-pair (cta_group::2) kernels on / off (default on)
void tc_gemm_use_cta_pairs(bool on, bool swiglu_too);
// generic: B rows come from up to three matrices stacked along N: [0,nB0) from B0, [nB0, nB0+nB1) from B1, rest B2
// rope != nullptr: the rotary embedding (rotate-half pairs (i, i + hd/2)) is applied in the epilogue, in fp32,
// to the columns below out.n0 and to the even-numbered segments above it (K planes; odd ones are V planes)
struct RopeSpec {
  const int32_t *positions;
  const float *cos_tab, *sin_tab;   // [position][hd/2]
  int hd;
};
// f16: A, every B and the columns below out.n0 hold IEEE halves instead of bfloat16 (same type on both operands);
// columns routed to segments (the K / V cache planes) are always stored as bfloat16, and -- if dup_base is given --
// stored a second time as halves at dup_base + segment * dup_stride (the attention kernel's operand copy)
// split (optional, IEEE-half operands only): extended-precision activations as pairs of halves, value = hi + lo.
//   a_split : A is [M, 2K], each row [hi(K) | lo(K)]; the product is A_hi B^T + A_lo B^T in one accumulator (the K loop
//             runs twice over B), so A enters with ~22 significant bits at twice the tensor-core time;
//   lo_p0   : the epilogue also writes the low halves of the columns below out.n0 (same layout as out.p0);
//   lo_dup  : ... and the low halves of segment 0's half copy (a layer's K plane), row stride out.seg_w.
struct GemmSplit {
  bool a_split = false;
  void *lo_p0 = nullptr, *lo_dup = nullptr;
};
int launch_gemm_tc(const void *A, bool f16, int M, int K, const void *B0, int nB0, const void *B1, int nB1, const void *B2,
                   int nB2, OutDesc out, void *dup_base, long long dup_stride, const RopeSpec *rope, unsigned int *status,
                   cudaStream_t st, const GemmSplit *split = nullptr);
// act[M, F] = silu(A Wg^T) * (A Wu^T), gate/up tiles paired inside one CTA tile; f16: all three in IEEE half
// a_split: A is [M, 2K] = [hi | lo] as above; out_split: act is [M, 2F], each row [hi(F) | lo(F)] (the split A operand of
// the down projection)
int launch_gemm_tc_swiglu(const void *A, bool f16, int M, int K, const void *Wg, const void *Wu, int F, void *act,
                          unsigned int *status, cudaStream_t st, bool a_split = false, bool out_split = false);
bool tc_swiglu_supported(int M, int F, int K);
// Failure-detection self-check: one CTA whose consumer role waits -- with the GEMM kernels' own bounded wait, but a
// limit of `limit_clocks` -- on a barrier that nothing ever completes, and whose second role watches the CTA's abort
// flag.  The wait runs out, STATUS_TIMEOUT is set in *status, both roles leave their loops, the kernel returns.
// outcome[0] = 1 if the waiting role gave up at its limit, outcome[1] = 1 if the second role left through the abort flag.
int launch_bounded_wait_probe(long long limit_clocks, unsigned int *status, unsigned int *outcome, cudaStream_t st);

// attention.cu
// k_row0 / kv_len as for launch_attention_tc
template <typename TQ, typename TKV>
void launch_attention_simple(const TQ *q, const TKV *k, const TKV *v, TQ *out, const int32_t *cu_seqlens, int n_seqs,
                             const int32_t *k_row0, const int32_t *kv_len, const int32_t *blk, int blk_stride,
                             int n_tokens, int n_q, int n_kv, int hd, cudaStream_t st);
bool tc_attention_supported(int n_q, int n_kv, int hd);
// f16: q, k, v and out all hold IEEE halves (else all bfloat16).  cu_seqlens: offsets of each sequence's new tokens
// (queries) in q / out; k_row0 / kv_len (both nullable): first K / V row and number of keys (cached + new) of each
// sequence -- null means a plain prefill whose K / V rows are packed like q; kv_rows: rows of k / v that hold data;
// max_seq_len bounds the new tokens of one sequence
// blk / blk_stride (nullable): block tables of a paged cache, see kv_row_of (then k_row0 is ignored)
// sched (optional, device arrays): a host-balanced assignment of the work items to n_ctas persistent CTAs -- CTA c runs
// items[off[c] .. off[c + 1]), each the item's index in the order (query tile descending, sequence, head pair) over
// ceil(max_seq_len / 128) query tiles; see attention_schedule()
struct AttnSchedule {
  const int32_t *off = nullptr, *items = nullptr;
  int n_ctas = 0;
};
int launch_attention_tc(const void *q, bool f16, const void *k, const void *v, void *out, const int32_t *cu_seqlens,
                        const int32_t *k_row0, const int32_t *kv_len, const int32_t *blk, int blk_stride, int n_seqs,
                        int n_tokens, int kv_rows, int max_seq_len, int n_q, int n_kv, int hd, unsigned int *status,
                        cudaStream_t st, AttnSchedule sched = AttnSchedule());
// Plain prefill (every sequence starts at position 0, K / V rows packed like q) with extended-precision scores: q and K
// as pairs of half tensors (value = hi + lo), S = Q K^T from three tensor-core passes; v, out in IEEE half.  out_split: out
// is [T, 2 * n_q * hd], each row [hi | lo] (the split A operand of the O projection); else [T, n_q * hd].  One CTA per item.
int launch_attention_tc_split(const void *q_hi, const void *q_lo, const void *k_hi, const void *k_lo, const void *v, void *out,
                              bool out_split, const int32_t *cu_seqlens, int n_seqs, int n_tokens, int max_seq_len, int n_q, int n_kv,
                              int hd, unsigned int *status, cudaStream_t st);
// host side of the persistent attention kernel: items of sequences with n_new[b] new tokens after n_past[b] cached ones,
// longest first, each to the least loaded of n_ctas CTAs; writes off[n_ctas + 1] and items[], returns the item count
int attention_schedule(const int32_t *n_new, const int32_t *n_past, int n_seqs, int n_q, int n_ctas, int32_t *off, int32_t *items);

// simscore.cu : Eq. 1 over captured layer inputs xs [L][T][d] (fp32).  sums: [L][L] doubles of scratch; sim (nullable):
// [L][L] average cosines (symmetric, diagonal 1); simscore: [L-1], entry l-1 = SimScore(x_l)
void launch_simscore(const float *xs, int L, int T, int d, double *sums, float *sim, float *simscore, cudaStream_t st);

// tail.cu : the last-token path (at most MAX_TAIL_ROWS activation rows per launch, fp32 activations)
constexpr int MAX_TAIL_ROWS = 8;
template <typename T>
void launch_tail_rmsnorm(const float *y, const T *gamma, float *out, int rows, int d, float eps, cudaStream_t st);
// out[r, n] = sum_k act[r, k] * W[n, k]  (mode OUT_STORE_F32 or OUT_RESID_ADD_F32);
// with W2: out[r, n] = silu(act W^T) * (act W2^T)
template <typename T>
void launch_skinny_gemm(const float *act, const T *W, const T *W2, int n_rows, int N, int K, float *out, int ldo,
                        int mode, cudaStream_t st);
// two projections of the same rows in one launch: out[r, n] = act W^T, out2[r, n] = act W2^T (a decode step's K and V)
template <typename T>
void launch_skinny_gemm_dual(const float *act, const T *W, const T *W2, int n_rows, int N, int K, float *out, float *out2,
                             int ldo, cudaStream_t st);
// options of the single-query attention inside a prefill / step.  pos != null: rotary embedding of the query rows in the
// kernel (row b sits at position pos[b]; the tables are those of launch_rope), which saves a launch per layer.
// total_len > 0: the sum of the sequences' key counts, known to the host, from which the key split is chosen so that the
// blocks fill whole waves of the GPU (never finer than the default split, so the scratch always suffices).
struct TailOpts {
  const int32_t *pos = nullptr;
  const float *cos_tab = nullptr, *sin_tab = nullptr;
  int total_len = 0;
};
// one query token per sequence against that sequence's cache rows [row0[b], row0[b] + len[b]); len == nullptr means
// row0 is a cu_seqlens array (len[b] = row0[b+1] - row0[b]); scratch holds split partials
size_t tail_attention_scratch_bytes(int max_seqs, int n_q, int hd, int max_tokens);
// upper bound of the key splits of any launch whose max_seq_len is at most max_tokens (what the scratch is sized for)
int tail_max_splits(int max_tokens);
// T = fp8e4: kc / vc hold FP8 codes and kscale / vscale the fp32 scale of every cache row (null for other types)
template <typename T>
void launch_tail_attention(const float *q, const T *kc, const T *vc, const float *kscale, const float *vscale, float *out,
                           const int32_t *row0, const int32_t *len, const int32_t *blk, int blk_stride, int n_seqs,
                           int max_seq_len, int n_q, int n_kv, int hd, float *scratch, cudaStream_t st, TailOpts rope = TailOpts());

// Several dependent projections of the last-token path (at most 6) as one persistent cooperative launch with grid-wide
// barriers between them (bf16 weights).  Stage: out (+)= A W^T with A [rows, K] fp32, W [N, K]; epi 0 store, 1 accumulate
// into out, 2 out = silu(A W^T) * (A W2^T), 3 out = A W^T and out2 = A W2^T; gamma != null: A is RMS-normalised on the fly (the norm that precedes the
// projection is folded in).  sync: two words of device scratch; status: the model's status word.
struct TailStage {
  const float *A;
  const void *gamma, *W, *W2;
  float *out;
  int N, K, ldo, epi;
  float *out2 = nullptr;     // epi 3 (two projections of the same input, e.g. K and V of a decode token): W2's result
};
bool tail_fused_supported(int rows, int d, int dq, int F, int vocab);

// distill.cu : loss of Eq. 3 and its gradients with respect to the student's W_Q, W_K, W_V (fp32 models)
struct DistillDims { int vocab, d, L, n_q, n_kv, hd, F; float eps; };
struct DistillLayer {
  const float *in_norm, *wq, *wk, *wv, *wo, *post_norm, *w_gate, *w_up, *w_down;   // the frozen model
  const float *s_wq, *s_wk, *s_wv;                                                 // the student's copies (layers >= l)
  float *g_wq, *g_wk, *g_wv;                                                       // their gradients (written)
};
struct DistillArgs {
  const float *embed, *final_norm, *lm_head;
  const int32_t *tokens, *cu, *pos;      // device: packed token ids, sequence offsets [B + 1], position of every token in its prompt
  const float *cos_tab, *sin_tab;
  int T, B, l, g;
  int precision;                         // 0 fp32 CUDA cores; 1 tensor cores, split tf32 operands (fp32-grade); 2 tensor cores, plain tf32
  float tau;
  float *loss;                           // device scalar
  unsigned int *status;
  void *ws;
  size_t ws_floats;
};
size_t distill_workspace_floats(const DistillDims &c, int T, int l);
void distill_upcast(const void *src_bf16, float *dst, long long n, cudaStream_t st);
void launch_adamw(float *p, const float *g, float *m, float *v, long long n, float lr, float b1, float b2, float eps, float wd,
                  int step, cudaStream_t st);
int run_distill(const DistillDims &c, const DistillArgs &a, const DistillLayer *layers, cudaStream_t st);
// arrivals: the host's count of barrier arrivals on sync[0] so far (the counter is never reset between launches; zero both
// together).
// wait_limit_clocks: how long any single wait inside the kernel (ring stage, grid barrier) may take before the kernel latches
// STATUS_TIMEOUT and every role leaves (0: the default of about two seconds).
// handover: TAIL_HANDOVER_BYTES of device scratch (or null): where a stage publishes its output rows pre-split for the resident,
// normed stage that follows it in the same launch (SWIFTKV_TAIL_HANDOVER=0 keeps every stage converting for itself).
constexpr size_t TAIL_HANDOVER_IMAGE_BYTES = 131072;                       // K <= 4096, 8 row slots, hi + lo
constexpr size_t TAIL_HANDOVER_BYTES = TAIL_HANDOVER_IMAGE_BYTES + 256 * MAX_TAIL_ROWS * sizeof(float);
int launch_tail_fused(const TailStage *stages, int n_stages, int rows, float eps, unsigned int *sync, unsigned int *arrivals,
                      unsigned int *status, cudaStream_t st, long long wait_limit_clocks = 0, void *handover = nullptr);

}  // namespace skv
