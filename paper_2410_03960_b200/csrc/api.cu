// C ABI and host-side prefill schedule of the SwiftKV prefill library.
//
// The schedule follows the paper's inference procedure (Sec. 3.5): layers 1..l on every prompt token, then --
// immediately after layer l -- the KV caches of all later layers from one fused, gain-folded projection of
// the layer-l output (Eq. 2; AcrossKV groups, Sec. 3.3, share one cache slot), then only the last token of
// each prompt through layers l+1..L and the lm_head.
#include <algorithm>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <string>
#include <type_traits>
#include <vector>

#include "common.cuh"

using namespace skv;

// ---------------------------------------------------------------------------------------------------------
// errors
// ---------------------------------------------------------------------------------------------------------
static thread_local std::string g_last_error;
static int32_t fail(int32_t code, const char *fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof buf, fmt, ap);
  va_end(ap);
  g_last_error = buf;
  return code;
}
namespace skv {
// records the calling thread's last-error text for entry points defined in other translation units
int32_t report_error(int32_t code, const char *msg) { return fail(code, "%s", msg); }
}  // namespace skv
#define CUDA_TRY(expr)                                                                                   \
  do {                                                                                                   \
    cudaError_t e__ = (expr);                                                                            \
    if (e__ != cudaSuccess) return fail(SWIFTKV_ERR_CUDA, "%s failed: %s", #expr, cudaGetErrorString(e__)); \
  } while (0)

// ---------------------------------------------------------------------------------------------------------
// model object
// ---------------------------------------------------------------------------------------------------------
struct Carve {   // walks a buffer handing out 256-byte aligned regions; with base == nullptr it only measures
  uint8_t *base;
  size_t off = 0;
  explicit Carve(void *b) : base(reinterpret_cast<uint8_t *>(b)) {}
  void *take(size_t bytes) {
    off = (off + 255) & ~(size_t)255;
    void *p = base ? base + off : nullptr;
    off += bytes;
    return p;
  }
};

struct Buffers {
  float *x;                 // fp32 residual stream [T, d]
  void *h, *q, *attn;       // normed hidden [T, d]; queries [T, d_q]; attention output [T, d_q]
  void *gate, *up;          // unfused MLP scratch [mlp_chunk, F] each
  void *act;                // SwiGLU output [T, F]
  void *wfold;              // folded, concatenated SingleInputKV weight [n_groups*2*d_kv, d]
  void *w16;                // bf16 models: IEEE-half compute copy of ONE layer's seven matrices (refilled per layer)
  void *kv16;               // bf16 models: half copies of the current layer's K and V, [2][T, d_kv]
  void *kvst;               // FP8 cache: the projections' K / V rows of one layer before quantization, [2][T, d_kv] model dtype
  void *kvdq;               // FP8 cache: dequantized K / V of one layer for the attention kernels (fp32 models; 16-bit
                            //   models use kv16)
  float *y;                 // continuing tokens' residual [B, d]
  float *hy, *qy, *ay, *acty;  // the continuing tokens' activations stay in fp32
  float *ky, *vy;           // a decode step's new K / V rows before they go to the cache, KV_STAGE_SLOTS x [8, d_kv] each
  float *tail_scratch;
  void *tail_handover;      // the fused last-token launch: rows published pre-split from one stage to the next
  float *logits;            // [B, vocab]
  int32_t *tokens, *cu, *pos, *last_idx, *last_pos;
  int32_t *att_off, *att_items;   // schedule of the persistent attention kernel: [ATT_MAX_CTAS + 1] offsets, items
  int32_t *slot;            // [T] cache row of every new token
  int32_t *kv_row0, *kv_len;   // [B] first cache row / number of cached + new tokens of every sequence
  int32_t *kcu;             // [B+1] offsets of the sequences in the gathered half K / V copy (chunked steps)
  int32_t *emit_row0, *emit_len;   // [B] cache range of the sequences whose last new token continues
  int32_t *blk, *blk_emit;  // [B][pages] block tables of a paged step, and the rows of the emitting sequences
  unsigned int *status;
  float *cos_tab, *sin_tab;
};

static const int MLP_CHUNK_ROWS = 8192;

struct swiftkv_model {
  swiftkv_config cfg;
  std::vector<swiftkv_layer_weights> layers;
  const void *embed, *final_norm, *lm_head;
  int max_tokens, max_seqs;
  size_t esize;
  size_t fold_capacity_elems;   // elements reserved for the folded weight
  int slot_capacity;            // cache slots the KV buffer holds
  uint8_t *kv;
  Buffers b;
  int device;
  // state of the last prefill
  bool ready = false;
  int n_tokens = 0, n_seqs = 0, cur_l = 0, cur_g = 1;   // rows in use per cache plane, sequences with logits
  int fold_l = -1, fold_g = -1, fold_fmt = -1;
  int launches = 0;
  int kernel_mask = 119;
  int n_sms = 0;
  int act_format = SWIFTKV_ACT_F16;
  float *capture = nullptr;     // while set: layer j's input (the residual stream before layer j) is copied to capture[j][T][d]
  int split_mask = 0;           // SWIFTKV_SPLIT_* bits: which operands travel as half pairs (SWIFTKV_ACT_F16_SPLIT)
  // profiling
  bool profiling = false;
  std::vector<cudaEvent_t> pool;
  struct Rec { cudaEvent_t a, b; int cls; };
  std::vector<Rec> recs;
  std::vector<int32_t> host_meta;
  // side stream on which the next layer's weights are copied to half while the current layer computes
  cudaStream_t side = nullptr;
  cudaEvent_t ev_start = nullptr, ev_ready[2] = {nullptr, nullptr}, ev_free[2] = {nullptr, nullptr};
  // optional caller-owned room for the half copies of the first layers' matrices, kept from step to step
  // (swiftkv_set_half_weight_cache): capacity and number of layers whose copies are current
  __half *w16_cache = nullptr;
  int w16_cache_cap = 0, w16_cache_valid = 0;
};

static size_t dsize(int dtype) { return dtype == SWIFTKV_DTYPE_BF16 ? 2 : 4; }
static int n_groups(int L, int l, int g) { return (L - l + g - 1) / g; }

static int32_t check_cfg(const swiftkv_config *c, int max_tokens, int max_seqs, int l, int g) {
  if (!c) return fail(SWIFTKV_ERR_INVALID_ARG, "config is null");
  if (c->vocab < 1 || c->hidden < 1 || c->n_layers < 1 || c->n_q_heads < 1 || c->n_kv_heads < 1 || c->head_dim < 2 || c->ffn < 1)
    return fail(SWIFTKV_ERR_INVALID_ARG, "non-positive model dimension");
  if (c->n_q_heads % c->n_kv_heads) return fail(SWIFTKV_ERR_INVALID_ARG, "n_q_heads must be a multiple of n_kv_heads");
  if (c->head_dim % 2 || c->head_dim > 256) return fail(SWIFTKV_ERR_INVALID_ARG, "head_dim must be even and <= 256");
  if (c->dtype != SWIFTKV_DTYPE_F32 && c->dtype != SWIFTKV_DTYPE_BF16) return fail(SWIFTKV_ERR_INVALID_ARG, "unknown dtype");
  if (c->kv_format != SWIFTKV_KV_MODEL_DTYPE && c->kv_format != SWIFTKV_KV_FP8) return fail(SWIFTKV_ERR_INVALID_ARG, "unknown kv_format");
  if (!(c->rope_theta > 0.f) || !(c->rms_eps >= 0.f)) return fail(SWIFTKV_ERR_INVALID_ARG, "bad rope_theta / rms_eps");
  if (max_tokens < 1 || max_seqs < 1) return fail(SWIFTKV_ERR_INVALID_ARG, "max_tokens and max_seqs must be positive");
  if (l < 1 || l > c->n_layers) return fail(SWIFTKV_ERR_INVALID_ARG, "swift_layer %d outside [1, %d]", l, c->n_layers);
  if (g < 1) return fail(SWIFTKV_ERR_INVALID_ARG, "acrosskv_group must be >= 1");
  return SWIFTKV_OK;
}

// persistent attention kernel: at most this many CTAs; one item per (128-query tile, pair of query heads)
constexpr int ATT_MAX_CTAS = 1024;
// staging rows for the K / V projections of a decode step: this many AcrossKV groups' rows per fused launch
constexpr int KV_STAGE_SLOTS = 6;
static size_t att_max_items(const swiftkv_config &c, int T, int B) {
  return ((size_t)T / 128 + (size_t)B) * (size_t)((c.n_q_heads + 1) / 2);
}
static void carve_all(const swiftkv_config &c, int T, int B, size_t fold_elems, Carve &cv, Buffers &b) {
  const size_t E = dsize(c.dtype);
  const size_t d = c.hidden, dq = (size_t)c.n_q_heads * c.head_dim, F = c.ffn;
  const size_t chunk = std::min<size_t>(T, MLP_CHUNK_ROWS);
  // (a 16-bit model's activation buffers hold two halves per element, so that the half-pair format fits)
  const size_t P2 = c.dtype == SWIFTKV_DTYPE_BF16 ? 2 : 1;
  b.x = (float *)cv.take((size_t)T * d * 4);
  b.h = cv.take((size_t)T * d * E * P2);
  b.q = cv.take((size_t)T * dq * E * P2);
  b.attn = cv.take((size_t)T * dq * E * P2);
  b.gate = cv.take(chunk * F * E);
  b.up = cv.take(chunk * F * E);
  b.act = cv.take((size_t)T * F * E * P2);
  b.wfold = cv.take(fold_elems * E);
  const size_t dkv_ = (size_t)c.n_kv_heads * c.head_dim;
  const bool bf = c.dtype == SWIFTKV_DTYPE_BF16;
  b.w16 = cv.take(bf ? 2 * (2 * d * dq + 2 * d * dkv_ + 3 * d * F) * 2 : 0);   // two layers: double buffer
  b.kv16 = cv.take(bf ? (size_t)3 * T * dkv_ * 2 : 0);      // K, V and (half pairs) the low halves of K
  const bool fp8 = c.kv_format == SWIFTKV_KV_FP8;
  b.kvst = cv.take(fp8 ? (size_t)2 * T * dkv_ * E : 0);
  b.kvdq = cv.take(fp8 && !bf ? (size_t)2 * T * dkv_ * 4 : 0);
  b.y = (float *)cv.take((size_t)B * d * 4);
  const size_t R = std::min<size_t>(B, MAX_TAIL_ROWS);
  b.hy = (float *)cv.take(R * std::max(d, dq) * 4);
  b.qy = (float *)cv.take(R * dq * 4);
  b.ay = (float *)cv.take(R * dq * 4);
  b.acty = (float *)cv.take(R * F * 4);
  b.ky = (float *)cv.take(KV_STAGE_SLOTS * R * dkv_ * 4);      // (several AcrossKV groups' rows per fused launch)
  b.vy = (float *)cv.take(KV_STAGE_SLOTS * R * dkv_ * 4);
  b.tail_scratch = (float *)cv.take(tail_attention_scratch_bytes(B, c.n_q_heads, c.head_dim, T));
  b.tail_handover = cv.take(TAIL_HANDOVER_BYTES);
  b.logits = (float *)cv.take((size_t)B * c.vocab * 4);
  b.tokens = (int32_t *)cv.take((size_t)T * 4);
  b.cu = (int32_t *)cv.take((size_t)(B + 1) * 4);
  b.pos = (int32_t *)cv.take((size_t)T * 4);
  b.last_idx = (int32_t *)cv.take((size_t)B * 4);
  b.last_pos = (int32_t *)cv.take((size_t)B * 4);
  b.slot = (int32_t *)cv.take((size_t)T * 4);
  b.kv_row0 = (int32_t *)cv.take((size_t)B * 4);
  b.kv_len = (int32_t *)cv.take((size_t)B * 4);
  b.kcu = (int32_t *)cv.take((size_t)(B + 1) * 4);
  b.emit_row0 = (int32_t *)cv.take((size_t)B * 4);
  b.emit_len = (int32_t *)cv.take((size_t)B * 4);
  const size_t pages = ((size_t)T + PAGE_ROWS - 1) / PAGE_ROWS;
  b.blk = (int32_t *)cv.take((size_t)B * pages * 4);
  b.blk_emit = (int32_t *)cv.take((size_t)B * pages * 4);
  b.att_off = (int32_t *)cv.take((size_t)(ATT_MAX_CTAS + 1) * 4);
  b.att_items = (int32_t *)cv.take(att_max_items(c, T, B) * 4);
  b.status = (unsigned int *)cv.take(256);
  b.cos_tab = (float *)cv.take((size_t)T * (c.head_dim / 2) * 4);
  b.sin_tab = (float *)cv.take((size_t)T * (c.head_dim / 2) * 4);
}

static size_t fold_elems_for(const swiftkv_config &c, int l, int g) {
  return (size_t)n_groups(c.n_layers, l, g) * 2 * c.n_kv_heads * c.head_dim * c.hidden;
}
static size_t slot_elems(const swiftkv_config &c, int T) { return (size_t)2 * T * c.n_kv_heads * c.head_dim; }
// FP8 cache slot: K codes | V codes | K scales | V scales, every part padded to 256 bytes
static size_t fp8_code_plane(const swiftkv_config &c, int T) { return ((size_t)T * c.n_kv_heads * c.head_dim + 255) & ~(size_t)255; }
static size_t fp8_scale_plane(int T) { return ((size_t)T * 4 + 255) & ~(size_t)255; }
static size_t slot_bytes_of(const swiftkv_config &c, int T) {
  if (c.kv_format == SWIFTKV_KV_FP8) return 2 * fp8_code_plane(c, T) + 2 * fp8_scale_plane(T);
  return slot_elems(c, T) * dsize(c.dtype);
}

// ---------------------------------------------------------------------------------------------------------
extern "C" int32_t swiftkv_version(void) { return 100; }
extern "C" const char *swiftkv_last_error(void) { return g_last_error.c_str(); }

extern "C" int32_t swiftkv_workspace_bytes(const swiftkv_config *cfg, int32_t max_tokens, int32_t max_seqs,
                                           int32_t swift_layer, int32_t acrosskv_group, size_t *workspace_bytes,
                                           size_t *kv_cache_bytes) {
  int32_t rc = check_cfg(cfg, max_tokens, max_seqs, swift_layer, acrosskv_group);
  if (rc) return rc;
  if (!workspace_bytes || !kv_cache_bytes) return fail(SWIFTKV_ERR_INVALID_ARG, "output pointer is null");
  Carve cv(nullptr);
  Buffers b;
  carve_all(*cfg, max_tokens, max_seqs, fold_elems_for(*cfg, swift_layer, acrosskv_group), cv, b);
  *workspace_bytes = ((cv.off + 255) & ~(size_t)255) + 512;
  const int slots = swift_layer + n_groups(cfg->n_layers, swift_layer, acrosskv_group);
  *kv_cache_bytes = (size_t)slots * slot_bytes_of(*cfg, max_tokens);
  return SWIFTKV_OK;
}

extern "C" void swiftkv_model_free(swiftkv_model *m);

extern "C" int32_t swiftkv_model_load(const swiftkv_config *cfg, const swiftkv_weights *w, void *workspace,
                                      size_t workspace_bytes, void *kv_cache, size_t kv_cache_bytes,
                                      int32_t max_tokens, int32_t max_seqs, swiftkv_model **out) {
  if (!out) return fail(SWIFTKV_ERR_INVALID_ARG, "out is null");
  *out = nullptr;
  int32_t rc = check_cfg(cfg, max_tokens, max_seqs, 1, 1);
  if (rc) return rc;
  if (!w || !w->embed || !w->final_norm || !w->lm_head || !w->layers) return fail(SWIFTKV_ERR_INVALID_ARG, "a weight pointer is null");
  if (!workspace || !kv_cache) return fail(SWIFTKV_ERR_INVALID_ARG, "workspace / kv_cache is null");
  if ((reinterpret_cast<uintptr_t>(workspace) & 255) || (reinterpret_cast<uintptr_t>(kv_cache) & 255))
    return fail(SWIFTKV_ERR_INVALID_ARG, "workspace and kv_cache must be 256-byte aligned");
  for (int j = 0; j < cfg->n_layers; ++j) {
    const swiftkv_layer_weights &lw = w->layers[j];
    const void *ps[9] = {lw.in_norm, lw.wq, lw.wk, lw.wv, lw.wo, lw.post_norm, lw.w_gate, lw.w_up, lw.w_down};
    for (const void *p : ps) {
      if (!p) return fail(SWIFTKV_ERR_INVALID_ARG, "layer %d: a weight pointer is null", j);
      if (reinterpret_cast<uintptr_t>(p) & 15) return fail(SWIFTKV_ERR_INVALID_ARG, "layer %d: weights must be 16-byte aligned", j);
    }
  }
  // smallest workspace: no folded weight at all (l = L)
  Carve measure(nullptr);
  Buffers tmp;
  carve_all(*cfg, max_tokens, max_seqs, 0, measure, tmp);
  const size_t base_need = (measure.off + 255) & ~(size_t)255;
  if (workspace_bytes < base_need) return fail(SWIFTKV_ERR_WORKSPACE_SMALL, "workspace %zu < %zu bytes", workspace_bytes, base_need);
  const size_t E = dsize(cfg->dtype);
  const size_t slot_bytes = slot_bytes_of(*cfg, max_tokens);
  if (kv_cache_bytes < slot_bytes) return fail(SWIFTKV_ERR_WORKSPACE_SMALL, "kv cache smaller than one slot");

  swiftkv_model *m = new (std::nothrow) swiftkv_model();
  if (!m) return fail(SWIFTKV_ERR_CUDA, "out of host memory");
  m->cfg = *cfg;
  m->layers.assign(w->layers, w->layers + cfg->n_layers);
  m->embed = w->embed; m->final_norm = w->final_norm; m->lm_head = w->lm_head;
  m->max_tokens = max_tokens; m->max_seqs = max_seqs; m->esize = E;
  // everything beyond the base need is room for the folded weight (kept 256-byte slack for alignment)
  m->fold_capacity_elems = workspace_bytes - base_need > 256 ? (workspace_bytes - base_need - 256) / E : 0;
  m->slot_capacity = (int)std::min<size_t>(kv_cache_bytes / slot_bytes, 1u << 20);
  m->kv = reinterpret_cast<uint8_t *>(kv_cache);
  Carve cv(workspace);
  carve_all(*cfg, max_tokens, max_seqs, m->fold_capacity_elems, cv, m->b);
  if (cudaGetDevice(&m->device) != cudaSuccess) { delete m; return fail(SWIFTKV_ERR_CUDA, "cudaGetDevice failed"); }
  if (cudaDeviceGetAttribute(&m->n_sms, cudaDevAttrMultiProcessorCount, m->device) != cudaSuccess || m->n_sms < 1) {
    delete m;
    return fail(SWIFTKV_ERR_CUDA, "cannot read the SM count");
  }
  // the cache starts as zeros: attention tiles may touch rows past a sequence's end (masked to probability 0), which
  // must never hold NaN / Inf bit patterns
  cudaError_t e = cudaMemsetAsync(kv_cache, 0, (size_t)m->slot_capacity * slot_bytes, 0);
  if (e == cudaSuccess) e = cudaMemsetAsync(m->b.status, 0, 256, 0);
  if (e == cudaSuccess) {
    launch_rope_table(m->b.cos_tab, m->b.sin_tab, max_tokens, cfg->head_dim, (double)cfg->rope_theta, 0);
    e = cudaGetLastError();
  }
  if (e == cudaSuccess) e = cudaStreamSynchronize(0);
  if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&m->side, cudaStreamNonBlocking);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&m->ev_start, cudaEventDisableTiming);
  for (int i = 0; i < 2 && e == cudaSuccess; ++i) {
    e = cudaEventCreateWithFlags(&m->ev_ready[i], cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&m->ev_free[i], cudaEventDisableTiming);
  }
  if (e != cudaSuccess) { swiftkv_model_free(m); return fail(SWIFTKV_ERR_CUDA, "model_load: %s", cudaGetErrorString(e)); }
  *out = m;
  return SWIFTKV_OK;
}

extern "C" void swiftkv_model_free(swiftkv_model *m) {
  if (!m) return;
  for (cudaEvent_t ev : m->pool) cudaEventDestroy(ev);
  for (auto &r : m->recs) { cudaEventDestroy(r.a); cudaEventDestroy(r.b); }
  if (m->side) { cudaStreamSynchronize(m->side); cudaStreamDestroy(m->side); }
  if (m->ev_start) cudaEventDestroy(m->ev_start);
  for (int i = 0; i < 2; ++i) {
    if (m->ev_ready[i]) cudaEventDestroy(m->ev_ready[i]);
    if (m->ev_free[i]) cudaEventDestroy(m->ev_free[i]);
  }
  delete m;
}

// ---------------------------------------------------------------------------------------------------------
// launch bookkeeping: counts launches; with profiling on, brackets each launch with events
// ---------------------------------------------------------------------------------------------------------
struct Scope {
  swiftkv_model *m; cudaStream_t st; int cls; cudaEvent_t a = nullptr, b = nullptr;
  static cudaEvent_t get(swiftkv_model *m) {
    if (!m->pool.empty()) { cudaEvent_t e = m->pool.back(); m->pool.pop_back(); return e; }
    cudaEvent_t e; cudaEventCreate(&e); return e;
  }
  bool timed;
  // timed = false: count the launches only (work on the side stream overlaps the main stream's kernels, so its
  // wall time is not part of any class)
  Scope(swiftkv_model *m_, cudaStream_t s, int c, int n_launches = 1, bool timed_ = true) : m(m_), st(s), cls(c) {
    m->launches += n_launches;
    timed = timed_ && m->profiling;
    if (timed) { a = get(m); b = get(m); cudaEventRecord(a, st); }
  }
  ~Scope() {
    if (timed) { cudaEventRecord(b, st); m->recs.push_back({a, b, cls}); }
  }
};

// ---------------------------------------------------------------------------------------------------------
// the schedule
// ---------------------------------------------------------------------------------------------------------
// TA: storage type of the activations that feed GEMMs and attention (h, q, attention output, SwiGLU output):
//     float for an fp32 model; for a bf16 model either bf16 or IEEE half (8x finer rounding, saturating).
// TW: storage type of weights and of the KV cache (the model dtype).
// rope_fused (optional): in: request the rotary embedding in the epilogue; out: whether it was applied
// Bh0..2 (optional): IEEE-half copies of B0..2, used by the tensor-core path when TA is half (both MMA operands must
// have the same 16-bit type); dup: half copy of the segment columns (see launch_gemm_tc)
template <typename TA, typename TW>
static int32_t gemm_any(swiftkv_model *m, const TA *A, int M, int K, const TW *B0, int n0, const TW *B1, int n1,
                        const TW *B2, int n2, const OutDesc &out, cudaStream_t st, const __half *Bh0 = nullptr,
                        const __half *Bh1 = nullptr, const __half *Bh2 = nullptr, const RopeSpec *rope = nullptr,
                        bool *rope_fused = nullptr, void *dup = nullptr, long long dup_stride = 0, const GemmSplit *split = nullptr) {
  Scope sc(m, st, SWIFTKV_KC_GEMM, 0);
  if (rope_fused) *rope_fused = false;
  if (split && !split->a_split && !split->lo_p0 && !split->lo_dup) split = nullptr;
  if constexpr (sizeof(TW) == 2) {
    constexpr bool f16 = std::is_same<TA, __half>::value;
    const bool have_b = !f16 || (Bh0 && (n1 == 0 || Bh1) && (n2 == 0 || Bh2));
    if ((m->kernel_mask & 1) && have_b && tc_gemm_supported(M, n0 + n1 + n2, K)) {
      const void *b0 = f16 ? (const void *)Bh0 : (const void *)B0;
      const void *b1 = f16 ? (const void *)Bh1 : (const void *)B1;
      const void *b2 = f16 ? (const void *)Bh2 : (const void *)B2;
      int rc = SWIFTKV_ERR_UNSUPPORTED;
      if (rope && rope_fused) {
        rc = launch_gemm_tc(A, f16, M, K, b0, n0, b1, n1, b2, n2, out, dup, dup_stride, rope, m->b.status, st, split);
        if (rc == SWIFTKV_OK) *rope_fused = true;
      }
      const bool split_out = split && (split->lo_p0 || split->lo_dup);      // low halves come from the rotary epilogue only
      if (rc == SWIFTKV_ERR_UNSUPPORTED && !split_out)
        rc = launch_gemm_tc(A, f16, M, K, b0, n0, b1, n1, b2, n2, out, nullptr, 0, nullptr, m->b.status, st, split);
      if (rc == SWIFTKV_OK) { m->launches += 1; return rc; }
      if (rc != SWIFTKV_ERR_UNSUPPORTED) return fail(rc, "tensor-core GEMM launch failed: %s", cudaGetErrorString(cudaGetLastError()));
    }
  }
  if (split) return fail(SWIFTKV_ERR_UNSUPPORTED, "half-pair operands need the tensor-core GEMM (shape %d x %d x %d)", M, n0 + n1 + n2, K);
  OutDesc o = out;
  o.status = m->b.status;      // a clamped half store is reported like on the tensor-core path
  launch_gemm_simt<TA, TW>(A, B0, M, n0, K, o, 0, st);
  m->launches += 1;
  if (n1 > 0) { launch_gemm_simt<TA, TW>(A, B1, M, n1, K, o, n0, st); m->launches += 1; }
  if (n2 > 0) { launch_gemm_simt<TA, TW>(A, B2, M, n2, K, o, n0 + n1, st); m->launches += 1; }
  return SWIFTKV_OK;
}

// One forward pass over a minibatch (Sec. 3.5).  `plain`: every sequence starts at position 0 and its cache rows are
// its rows in the packed batch (a whole-prompt prefill); otherwise sequences carry cached prefixes (chunked prefill,
// decode tokens) and new tokens are scattered to slot[t].
struct Batch {
  int T_tok, B, n_emit;
  int max_new;        // longest run of new tokens
  int max_kv;         // longest cached + new length
  int total_kv;       // sum of cached + new lengths
  bool plain;
  int att_ctas;       // > 0: the device holds a schedule for that many persistent attention CTAs
  std::vector<int> emit_lens;   // cached + new length of every emitting sequence, in their order (host copy)
  bool paged;         // sequences own lists of 128-row pages instead of one contiguous region
  int blk_stride;     // pages per sequence in the device block tables
  bool decode;        // at most 8 sequences, one new token each, all emitting: every layer runs on the weight-streaming
                      // kernels of the last-token path
};

template <typename TA, typename T>
static int32_t run_prefill(swiftkv_model *m, const Batch &bt, int l, int g, cudaStream_t st) {
  const int T_tok = bt.T_tok, B = bt.B, max_len = bt.max_kv;
  const swiftkv_config &c = m->cfg;
  Buffers &b = m->b;
  const int d = c.hidden, dq = c.n_q_heads * c.head_dim, dkv = c.n_kv_heads * c.head_dim, F = c.ffn, L = c.n_layers;
  const size_t plane = (size_t)m->max_tokens * dkv;          // elements of one K (or V) plane
  constexpr bool act_f16 = std::is_same<TA, __half>::value;
  T *kv = reinterpret_cast<T *>(m->kv);
  // FP8 cache (appendix, KV quantization): projections land in a staging pair of planes, a row pass turns them into
  // codes + per-token scales in the cache, and every attention read sees the dequantized values
  const bool fp8 = c.kv_format == SWIFTKV_KV_FP8;
  const size_t slot_b = slot_bytes_of(c, m->max_tokens), cp8 = fp8_code_plane(c, m->max_tokens), sp8 = fp8_scale_plane(m->max_tokens);
  auto k_codes = [&](int slot) { return m->kv + (size_t)slot * slot_b; };
  auto v_codes = [&](int slot) { return m->kv + (size_t)slot * slot_b + cp8; };
  auto k_scale = [&](int slot) { return reinterpret_cast<float *>(m->kv + (size_t)slot * slot_b + 2 * cp8); };
  auto v_scale = [&](int slot) { return reinterpret_cast<float *>(m->kv + (size_t)slot * slot_b + 2 * cp8 + sp8); };
  T *kst = (T *)b.kvst, *vst = kst + plane;
  TA *h = (TA *)b.h, *q = (TA *)b.q, *attn = (TA *)b.attn, *act = (TA *)b.act;
  const T *no_w = nullptr;
  int32_t rc;
  const RopeSpec rope{b.pos, b.cos_tab, b.sin_tab, c.head_dim};
  // With half activations the tensor-core kernels need both MMA operands in half: each layer's matrices are copied
  // to half right before use (one 0.4 GB pass per layer on the 8B shape, exact for |w| >= 2^-17), K / V get a half
  // copy beside the bf16 cache, and the folded SingleInputKV weight is produced in half directly.
  const bool use_w16 = act_f16 && (m->kernel_mask & 1) && tc_gemm_supported(T_tok, dq, d) && tc_gemm_supported(T_tok, d, dq) &&
                       tc_gemm_supported(T_tok, d, F) && (dkv % 256 == 0) && (dq % 256 == 0) && c.head_dim == 128;
  const bool attn_tc = sizeof(T) == 2 && (m->kernel_mask & 2) && tc_attention_supported(c.n_q_heads, c.n_kv_heads, c.head_dim);
  // half pairs (SWIFTKV_ACT_F16_SPLIT): which operands carry hi + lo halves in this pass.  Only the whole-prompt prefill on
  // the tensor-core kernels has them; chunked / decode steps and the FP8 cache run as plain SWIFTKV_ACT_F16.
  const int sm = (use_w16 && attn_tc && bt.plain && !fp8 && !bt.decode) ? m->split_mask : 0;
  const bool sp_hin = sm & SWIFTKV_SPLIT_QKV_INPUT, sp_qk = (sm & (SWIFTKV_SPLIT_SCORES | SWIFTKV_SPLIT_ATTN_OUT)) != 0,
             sp_ao = sm & SWIFTKV_SPLIT_ATTN_OUT, sp_hpost = sm & SWIFTKV_SPLIT_MLP_INPUT, sp_act = sm & SWIFTKV_SPLIT_MLP_ACT;
  AttnSchedule att_sched;
  if (bt.att_ctas > 0) { att_sched.off = b.att_off; att_sched.items = b.att_items; att_sched.n_ctas = bt.att_ctas; }
  const size_t w16_layer = (size_t)2 * d * dq + (size_t)2 * d * dkv + (size_t)3 * d * F;   // halves of one layer's copy
  __half *wq16 = nullptr, *wk16 = nullptr, *wv16 = nullptr, *wo16 = nullptr, *wg16 = nullptr, *wu16 = nullptr, *wd16 = nullptr;
  auto w16_at = [&](__half *base) {
    wq16 = base; wk16 = wq16 + (size_t)dq * d; wv16 = wk16 + (size_t)dkv * d;
    wo16 = wv16 + (size_t)dkv * d; wg16 = wo16 + (size_t)d * dq; wu16 = wg16 + (size_t)F * d; wd16 = wu16 + (size_t)F * d;
  };
  auto w16_select = [&](int buf) { w16_at((__half *)b.w16 + (size_t)buf * w16_layer); };
  // layer j's seven matrices -> the selected half copies, on stream `s`
  auto convert_into = [&](int j, cudaStream_t s, bool timed) {
    const swiftkv_layer_weights &lw = m->layers[j];
    Scope sc(m, s, SWIFTKV_KC_ELEMWISE, 7, timed);
    launch_bf16_to_f16((const bf16 *)lw.wq, wq16, (long long)dq * d, s, b.status);
    launch_bf16_to_f16((const bf16 *)lw.wk, wk16, (long long)dkv * d, s, b.status);
    launch_bf16_to_f16((const bf16 *)lw.wv, wv16, (long long)dkv * d, s, b.status);
    launch_bf16_to_f16((const bf16 *)lw.wo, wo16, (long long)d * dq, s, b.status);
    launch_bf16_to_f16((const bf16 *)lw.w_gate, wg16, (long long)F * d, s, b.status);
    launch_bf16_to_f16((const bf16 *)lw.w_up, wu16, (long long)F * d, s, b.status);
    launch_bf16_to_f16((const bf16 *)lw.w_down, wd16, (long long)d * F, s, b.status);
  };
  // layer j's copy is made on the side stream into buffer j % 2 while layer j - 1 computes on `st`
  auto convert_layer = [&](int j) {
    const int buf = j & 1;
    if (j >= 2) cudaStreamWaitEvent(m->side, m->ev_free[buf], 0);   // layer j - 2 has finished with this buffer
    w16_select(buf);
    convert_into(j, m->side, false);
    cudaEventRecord(m->ev_ready[buf], m->side);
  };
  // with room for them the copies of layers 1..l stay from step to step: made once, on `st`, by the first step that needs them
  const bool w16_resident = use_w16 && m->w16_cache && l <= m->w16_cache_cap && !bt.decode;
  if constexpr (sizeof(T) == 2) {
    if (use_w16 && l > 0 && !bt.decode && !w16_resident) {
      cudaEventRecord(m->ev_start, st);                 // the side stream starts after everything queued before
      cudaStreamWaitEvent(m->side, m->ev_start, 0);
      convert_layer(0);
    }
  }
  __half *k16 = (__half *)b.kv16, *v16 = k16 + plane, *k_lo = v16 + plane;
  __half *q_lo = (__half *)b.q + (size_t)m->max_tokens * dq;         // low halves of the queries: a second plane

  const int32_t *slot_map = bt.plain ? nullptr : b.slot;        // cache row of each new token (identity when plain)
  const int32_t *k_row0 = bt.plain ? nullptr : b.kv_row0;
  const int32_t *kv_len = bt.plain ? nullptr : b.kv_len;
  const int32_t *blk = bt.paged ? b.blk : nullptr, *blk_emit = bt.paged ? b.blk_emit : nullptr;
  { Scope s(m, st, SWIFTKV_KC_ELEMWISE); launch_embed<T>((const T *)m->embed, b.tokens, b.x, T_tok, d, c.vocab, b.status, st); }

  // one-time model transformation for this (l, g): fold each group leader's input-norm gain into its W_K, W_V
  // and stack them (Sec. 3.5)
  const int ng = n_groups(L, l, g);
  const int fold_fmt = use_w16 ? 1 : 0;
  if (!bt.decode && l < L && (m->fold_l != l || m->fold_g != g || m->fold_fmt != fold_fmt)) {
    for (int i = 0; i < ng; ++i) {
      const swiftkv_layer_weights &lw = m->layers[l + i * g];
      const size_t off = (size_t)i * 2 * dkv * d;
      if constexpr (sizeof(T) == 2) {
        if (use_w16) {
          __half *dst = (__half *)b.wfold + off;
          { Scope s(m, st, SWIFTKV_KC_ELEMWISE); launch_fold<bf16, __half>((const bf16 *)lw.wk, (const bf16 *)lw.in_norm, dst, dkv, d, st); }
          { Scope s(m, st, SWIFTKV_KC_ELEMWISE); launch_fold<bf16, __half>((const bf16 *)lw.wv, (const bf16 *)lw.in_norm, dst + (size_t)dkv * d, dkv, d, st); }
          continue;
        }
      }
      T *dst = (T *)b.wfold + off;
      { Scope s(m, st, SWIFTKV_KC_ELEMWISE); launch_fold<T, T>((const T *)lw.wk, (const T *)lw.in_norm, dst, dkv, d, st); }
      { Scope s(m, st, SWIFTKV_KC_ELEMWISE); launch_fold<T, T>((const T *)lw.wv, (const T *)lw.in_norm, dst + (size_t)dkv * d, dkv, d, st); }
    }
    m->fold_l = l; m->fold_g = g; m->fold_fmt = fold_fmt;
  }

  // kernel-mask bit 6: the dependent projections between two attention calls of the last-token / decode path -- O, gate/up,
  // down and the next layer's Q (and K / V of a decode token), or the lm_head at the end -- run as ONE persistent cooperative
  // launch with the norms folded in
  bool fused_tail = false;
  if constexpr (sizeof(T) == 2) {
    fused_tail = (m->kernel_mask & 64) && bt.n_emit > 0 && dkv % 16 == 0 &&
                 tail_fused_supported(std::min(MAX_TAIL_ROWS, bt.n_emit), d, dq, F, c.vocab);
  }
  unsigned int fused_arrivals = 0;
  if (fused_tail && cudaMemsetAsync(b.status + 32, 0, 32 * sizeof(unsigned int), st) != cudaSuccess)
    return fail(SWIFTKV_ERR_CUDA, "clearing the grid-barrier words failed");
  TailStage list[6];
  int n_list = 0;
  auto flush = [&](int rows) -> int32_t {
    if (n_list == 0) return SWIFTKV_OK;
    Scope s(m, st, SWIFTKV_KC_TAIL);
    const int frc = launch_tail_fused(list, n_list, rows, c.rms_eps, b.status + 32, &fused_arrivals, b.status, st, 0, b.tail_handover);
    n_list = 0;
    return frc == SWIFTKV_OK ? SWIFTKV_OK : fail(frc, "fused last-token launch failed: %s", cudaGetErrorString(cudaGetLastError()));
  };

  // ---- a minibatch of decode tokens (Sec. 3.5: "decode tokens complete all layers"): at most 8 rows, so every
  //      projection is bound by streaming its weights once -- layers 1..l run on the last-token path's kernels too,
  //      the new K / V rows go to the cache before the single-query attention reads it, and the rows of the later
  //      layers' caches come from each group leader's own gain and W_K, W_V applied to the layer-l output (Eq. 2)
  if (bt.decode) {
    const int rows = T_tok;
    float *hy = b.hy, *qy = b.qy, *ay = b.ay, *acty = b.acty, *ky = b.ky, *vy = b.vy, *y = b.y;
    const TailOpts q_rope{b.last_pos, b.cos_tab, b.sin_tab, bt.total_kv};     // the queries are rotated inside the attention kernel
    auto store_kv = [&](int slot, float *ky, float *vy) {      // ky -> rotary embedding, vy -> the cache rows of the new tokens in `slot`
      if (fp8) {        // (rows are quantized from the model dtype)
        Scope s(m, st, SWIFTKV_KC_TAIL);
        launch_store_kv_rows_fp8<T>(ky, vy, b.slot, b.last_pos, b.cos_tab, b.sin_tab, rows, c.n_kv_heads, c.head_dim,
                                    k_codes(slot), k_scale(slot), v_codes(slot), v_scale(slot), st);
      } else {
        Scope s(m, st, SWIFTKV_KC_TAIL);
        launch_store_kv_rows<T>(ky, vy, kv + (size_t)slot * 2 * plane, kv + (size_t)slot * 2 * plane + plane, b.slot, b.last_pos,
                                b.cos_tab, b.sin_tab, rows, c.n_kv_heads, c.head_dim, st);
      }
    };
    const int kv_launches = (sizeof(T) == 2 && d % 32 == 0 && dkv % 16 == 0) ? 1 : 2;
    auto project_kv = [&](const swiftkv_layer_weights &lw) {   // hy -> ky, vy: both projections in one launch
      Scope s(m, st, SWIFTKV_KC_TAIL, kv_launches);
      launch_skinny_gemm_dual<T>(hy, (const T *)lw.wk, (const T *)lw.wv, rows, dkv, d, ky, vy, dkv, st);
    };
    { Scope s(m, st, SWIFTKV_KC_TAIL); launch_gather_rows(b.x, b.last_idx, y, rows, d, st); }
    for (int j = 0; j < l; ++j) {
      const swiftkv_layer_weights &lw = m->layers[j];
      if (fused_tail) {      // [O, gate/up, down of the previous layer,] Q, K / V of this one: one launch
        list[n_list++] = TailStage{y, lw.in_norm, lw.wq, nullptr, qy, dq, d, dq, 0};
        list[n_list++] = TailStage{y, lw.in_norm, lw.wk, lw.wv, ky, dkv, d, dkv, 3, vy};
        if ((rc = flush(rows))) return rc;
      } else {
      { Scope s(m, st, SWIFTKV_KC_TAIL); launch_tail_rmsnorm<T>(y, (const T *)lw.in_norm, hy, rows, d, c.rms_eps, st); }
      { Scope s(m, st, SWIFTKV_KC_TAIL); launch_skinny_gemm<T>(hy, (const T *)lw.wq, nullptr, rows, dq, d, qy, dq, OUT_STORE_F32, st); }
      project_kv(lw);
      }
      store_kv(j, ky, vy);
      {
        Scope s(m, st, SWIFTKV_KC_TAIL, 2);
        if (fp8)
          launch_tail_attention<fp8e4>(qy, (const fp8e4 *)k_codes(j), (const fp8e4 *)v_codes(j), k_scale(j), v_scale(j), ay, b.emit_row0,
                                       b.emit_len, blk_emit, bt.blk_stride, rows, max_len, c.n_q_heads, c.n_kv_heads, c.head_dim,
                                       b.tail_scratch, st, q_rope);
        else
          launch_tail_attention<T>(qy, kv + (size_t)j * 2 * plane, kv + (size_t)j * 2 * plane + plane, nullptr, nullptr, ay, b.emit_row0,
                                   b.emit_len, blk_emit, bt.blk_stride, rows, max_len, c.n_q_heads, c.n_kv_heads, c.head_dim,
                                   b.tail_scratch, st, q_rope);
      }
      if (fused_tail) {      // (launched with the next layer's Q / K / V, or with the first SingleInputKV rows below)
        list[n_list++] = TailStage{ay, nullptr, lw.wo, nullptr, y, d, dq, d, 1};
        list[n_list++] = TailStage{y, lw.post_norm, lw.w_gate, lw.w_up, acty, F, d, F, 2};
        list[n_list++] = TailStage{acty, nullptr, lw.w_down, nullptr, y, d, F, d, 1};
        continue;
      }
      { Scope s(m, st, SWIFTKV_KC_TAIL); launch_skinny_gemm<T>(ay, (const T *)lw.wo, nullptr, rows, d, dq, y, d, OUT_RESID_ADD_F32, st); }
      { Scope s(m, st, SWIFTKV_KC_TAIL); launch_tail_rmsnorm<T>(y, (const T *)lw.post_norm, hy, rows, d, c.rms_eps, st); }
      { Scope s(m, st, SWIFTKV_KC_TAIL); launch_skinny_gemm<T>(hy, (const T *)lw.w_gate, (const T *)lw.w_up, rows, F, d, acty, F, OUT_STORE_F32, st); }
      { Scope s(m, st, SWIFTKV_KC_TAIL); launch_skinny_gemm<T>(acty, (const T *)lw.w_down, nullptr, rows, d, F, y, d, OUT_RESID_ADD_F32, st); }
    }
    if (fused_tail) {
      // SingleInputKV rows of the new tokens (Eq. 2, unfused: each group leader's own gain and W_K, W_V on the layer-l output):
      // as many groups per launch as the stage list and the staging rows hold, then their cache stores
      int first = 0;
      for (int i = 0; i < ng && l < L; ++i) {
        const swiftkv_layer_weights &lw = m->layers[l + i * g];
        const int k_slot = i - first;
        list[n_list++] = TailStage{y, lw.in_norm, lw.wk, lw.wv, ky + (size_t)k_slot * rows * dkv, dkv, d, dkv, 3, vy + (size_t)k_slot * rows * dkv};
        if (n_list == 6 || k_slot + 1 == KV_STAGE_SLOTS || i + 1 == ng) {
          if ((rc = flush(rows))) return rc;
          for (int q = first; q <= i; ++q) store_kv(l + q, ky + (size_t)(q - first) * rows * dkv, vy + (size_t)(q - first) * rows * dkv);
          first = i + 1;
        }
      }
      if ((rc = flush(rows))) return rc;      // (l == L: the last layer's O / gate-up / down are still pending)
    } else
    for (int i = 0; i < ng && l < L; ++i) {      // SingleInputKV rows of the new tokens, one AcrossKV group at a time
      const swiftkv_layer_weights &lw = m->layers[l + i * g];
      { Scope s(m, st, SWIFTKV_KC_TAIL); launch_tail_rmsnorm<T>(y, (const T *)lw.in_norm, hy, rows, d, c.rms_eps, st); }
      project_kv(lw);
      store_kv(l + i, ky, vy);
    }
  }

  // ---- layers 1..l on all prompt tokens (unmodified, Sec. 3.1)
  for (int j = 0; j < l && !bt.decode; ++j) {
    const swiftkv_layer_weights &lw = m->layers[j];
    T *Kj = kv + (size_t)j * 2 * plane, *Vj = Kj + plane;
    if (m->capture) {     // SimScore (Eq. 1) needs every layer's input
      Scope s(m, st, SWIFTKV_KC_ELEMWISE);
      cudaMemcpyAsync(m->capture + (size_t)j * T_tok * d, b.x, (size_t)T_tok * d * sizeof(float), cudaMemcpyDeviceToDevice, st);
    }
    if constexpr (sizeof(T) == 2) {
      if (w16_resident) {
        w16_at(m->w16_cache + (size_t)j * w16_layer);
        if (j >= m->w16_cache_valid) convert_into(j, st, true);
      } else if (use_w16) {
        if (j + 1 < l) convert_layer(j + 1);            // queued now, runs beside this layer's kernels
        w16_select(j & 1);
        cudaStreamWaitEvent(st, m->ev_ready[j & 1], 0);
      }
    }
    { Scope s(m, st, SWIFTKV_KC_ELEMWISE); launch_rmsnorm<T, TA>(b.x, (const T *)lw.in_norm, h, T_tok, d, c.rms_eps, st, b.status, sp_hin); }
    OutDesc qkv{OUT_STORE, q, dq, dq, Kj, (long long)plane, dkv, slot_map};
    const GemmSplit qkv_split{sp_hin, sp_qk ? (void *)q_lo : nullptr, sp_qk ? (void *)k_lo : nullptr};
    if (fp8) { Kj = kst; Vj = vst; qkv.seg_base = kst; qkv.slot_map = nullptr; }   // staging rows are in batch order
    bool roped = false;
    // the attention kernel reads half copies of this layer's K / V: written by the QKV epilogue for a plain prefill,
    // gathered from the cache (cached prefix + new tokens) otherwise
    const bool want_dup = use_w16 && attn_tc && bt.plain && !fp8;
    rc = gemm_any<TA, T>(m, h, T_tok, d, (const T *)lw.wq, dq, (const T *)lw.wk, dkv, (const T *)lw.wv, dkv, qkv, st,
                         use_w16 ? wq16 : nullptr, use_w16 ? wk16 : nullptr, use_w16 ? wv16 : nullptr, &rope, &roped,
                         want_dup ? k16 : nullptr, (long long)plane, &qkv_split);
    if (rc) return rc;
    if (!roped) {
      { Scope s(m, st, SWIFTKV_KC_ELEMWISE); launch_rope<TA>(q, 0, 1, b.pos, nullptr, b.cos_tab, b.sin_tab, T_tok, c.n_q_heads, c.head_dim, st, b.status); }
      { Scope s(m, st, SWIFTKV_KC_ELEMWISE); launch_rope<T>(Kj, 0, 1, b.pos, fp8 ? nullptr : slot_map, b.cos_tab, b.sin_tab, T_tok, c.n_kv_heads, c.head_dim, st); }
    }
    if (fp8) {
      // quantize this layer's rows into the cache; the attention operands are the dequantized values: written by the same
      // pass for a whole-prompt prefill, gathered from the cache (cached prefix + new rows) otherwise
      using TD = typename std::conditional<sizeof(T) == 2, TA, float>::type;   // operand type of the attention kernels
      const bool tc_path = sizeof(T) == 2 && attn_tc;
      TD *kd = sizeof(T) == 2 ? (TD *)b.kv16 : (TD *)b.kvdq, *vd = kd + plane;
      T *kd_t = (T *)kd, *vd_t = kd_t + plane;   // (SIMT attention reads operands of the cache's element type)
      {
        Scope s(m, st, SWIFTKV_KC_ELEMWISE, 2);
        if (tc_path) {
          launch_quantize_rows_fp8<T, TD>(kst, T_tok, dkv, slot_map, k_codes(j), k_scale(j), bt.plain ? kd : nullptr, st);
          launch_quantize_rows_fp8<T, TD>(vst, T_tok, dkv, slot_map, v_codes(j), v_scale(j), bt.plain ? vd : nullptr, st);
        } else {
          launch_quantize_rows_fp8<T, T>(kst, T_tok, dkv, slot_map, k_codes(j), k_scale(j), bt.plain ? kd_t : nullptr, st);
          launch_quantize_rows_fp8<T, T>(vst, T_tok, dkv, slot_map, v_codes(j), v_scale(j), bt.plain ? vd_t : nullptr, st);
        }
      }
      if (!bt.plain) {
        Scope s(m, st, SWIFTKV_KC_ELEMWISE);
        if (tc_path) launch_gather_dequant_fp8<TD>(k_codes(j), v_codes(j), k_scale(j), v_scale(j), kd, vd, b.kv_row0, b.kv_len, b.kcu, blk, bt.blk_stride, B, bt.max_kv, dkv, st);
        else launch_gather_dequant_fp8<T>(k_codes(j), v_codes(j), k_scale(j), v_scale(j), kd_t, vd_t, b.kv_row0, b.kv_len, b.kcu, blk, bt.blk_stride, B, bt.max_kv, dkv, st);
      }
      Scope s(m, st, SWIFTKV_KC_ATTENTION);
      const int32_t *kr0 = bt.plain ? nullptr : b.kcu;
      bool done = false;
      if constexpr (sizeof(T) == 2) {
        if (tc_path) {
          rc = launch_attention_tc(q, act_f16, kd, vd, attn, b.cu, kr0, kv_len, nullptr, 0, B, T_tok, bt.plain ? T_tok : bt.total_kv,
                                   bt.max_new, c.n_q_heads, c.n_kv_heads, c.head_dim, b.status, st, att_sched);
          if (rc == SWIFTKV_OK) done = true;
          else if (rc != SWIFTKV_ERR_UNSUPPORTED) return fail(rc, "attention launch failed");
        }
      }
      if (!done) {
        if (tc_path) return fail(SWIFTKV_ERR_UNSUPPORTED, "FP8 cache: tensor-core attention refused this shape");
        launch_attention_simple<TA, T>(q, kd_t, vd_t, attn, b.cu, B, kr0, kv_len, nullptr, 0, T_tok, c.n_q_heads, c.n_kv_heads, c.head_dim, st);
      }
    } else {
      Scope s(m, st, SWIFTKV_KC_ATTENTION);
      bool done = false;
      if constexpr (sizeof(T) == 2) {
        if (sp_qk) {     // scores from half pairs of q and K (three passes); output rows as [hi | lo] if the O projection wants them
          rc = launch_attention_tc_split(q, q_lo, k16, k_lo, v16, attn, sp_ao, b.cu, B, T_tok, bt.max_new, c.n_q_heads, c.n_kv_heads,
                                         c.head_dim, b.status, st);
          if (rc) return fail(rc, "half-pair attention launch failed");
          done = true;
        }
        // (half activations: the kernel needs half copies of K and V -- from the QKV epilogue, or gathered here)
        if (!done && attn_tc && (!act_f16 || (use_w16 && roped))) {
          const void *kk = Kj, *vv = Vj;
          const int32_t *kr0 = k_row0;
          int kv_rows = bt.plain ? T_tok : m->max_tokens;
          if (act_f16) {
            kk = k16; vv = v16;
            if (!bt.plain) {
              Scope s2(m, st, SWIFTKV_KC_ELEMWISE);
              launch_gather_kv_half((const bf16 *)Kj, (const bf16 *)Vj, k16, v16, b.kv_row0, b.kv_len, b.kcu, blk, bt.blk_stride, B, bt.max_kv, dkv, st, b.status);
              kr0 = b.kcu;
              kv_rows = bt.total_kv;
            }
          }
          // (the gathered half copies are contiguous: only a direct read of the cache follows the block tables)
          const int32_t *ablk = (act_f16 && !bt.plain) ? nullptr : blk;
          rc = launch_attention_tc(q, act_f16, kk, vv, attn, b.cu, kr0, kv_len, ablk, bt.blk_stride, B, T_tok, kv_rows, bt.max_new, c.n_q_heads,
                                   c.n_kv_heads, c.head_dim, b.status, st, att_sched);
          if (rc == SWIFTKV_OK) done = true;
          else if (rc != SWIFTKV_ERR_UNSUPPORTED) return fail(rc, "attention launch failed");
        }
      }
      if (!done) launch_attention_simple<TA, T>(q, Kj, Vj, attn, b.cu, B, k_row0, kv_len, blk, bt.blk_stride, T_tok, c.n_q_heads, c.n_kv_heads, c.head_dim, st);
    }
    const GemmSplit o_split{sp_ao, nullptr, nullptr}, down_split{sp_act, nullptr, nullptr};
    rc = gemm_any<TA, T>(m, attn, T_tok, dq, (const T *)lw.wo, d, no_w, 0, no_w, 0, out_plain(OUT_RESID_ADD_F32, b.x, d, d), st,
                         use_w16 ? wo16 : nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, 0, &o_split);
    if (rc) return rc;
    { Scope s(m, st, SWIFTKV_KC_ELEMWISE); launch_rmsnorm<T, TA>(b.x, (const T *)lw.post_norm, h, T_tok, d, c.rms_eps, st, b.status, sp_hpost); }
    bool fused = false;
    if constexpr (sizeof(T) == 2) {
      if ((m->kernel_mask & 1) && tc_swiglu_supported(T_tok, F, d) && (!act_f16 || use_w16)) {
        Scope s(m, st, SWIFTKV_KC_SWIGLU);
        const void *wg = act_f16 ? (const void *)wg16 : lw.w_gate, *wu = act_f16 ? (const void *)wu16 : lw.w_up;
        rc = launch_gemm_tc_swiglu(h, act_f16, T_tok, d, wg, wu, F, act, b.status, st, sp_hpost, sp_act);
        if (rc == SWIFTKV_OK) fused = true;
        else if (rc != SWIFTKV_ERR_UNSUPPORTED) return fail(rc, "SwiGLU GEMM launch failed");
      }
    }
    if (!fused && (sp_hpost || sp_act)) return fail(SWIFTKV_ERR_UNSUPPORTED, "half-pair MLP operands need the fused gate/up kernel");
    if (!fused) {
      for (int r0 = 0; r0 < T_tok; r0 += MLP_CHUNK_ROWS) {
        const int rows = std::min(MLP_CHUNK_ROWS, T_tok - r0);
        rc = gemm_any<TA, T>(m, h + (size_t)r0 * d, rows, d, (const T *)lw.w_gate, F, no_w, 0, no_w, 0, out_plain(OUT_STORE, b.gate, F, F), st,
                             use_w16 ? wg16 : nullptr);
        if (rc) return rc;
        rc = gemm_any<TA, T>(m, h + (size_t)r0 * d, rows, d, (const T *)lw.w_up, F, no_w, 0, no_w, 0, out_plain(OUT_STORE, b.up, F, F), st,
                             use_w16 ? wu16 : nullptr);
        if (rc) return rc;
        Scope s(m, st, SWIFTKV_KC_ELEMWISE);
        launch_swiglu<TA>((const TA *)b.gate, (const TA *)b.up, act + (size_t)r0 * F, (long long)rows * F, st, b.status);
      }
    }
    rc = gemm_any<TA, T>(m, act, T_tok, F, (const T *)lw.w_down, d, no_w, 0, no_w, 0, out_plain(OUT_RESID_ADD_F32, b.x, d, d), st,
                         use_w16 ? wd16 : nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, 0, &down_split);
    if (rc) return rc;
    if (w16_resident) m->w16_cache_valid = std::max(m->w16_cache_valid, j + 1);
    else if (use_w16) cudaEventRecord(m->ev_free[j & 1], st);   // this layer's half copies may be overwritten
  }

  // ---- SingleInputKV (+ AcrossKV): one projection of s = x_{l+1} fills the caches of layers l+1..L (Eq. 2)
  if (l < L && !bt.decode) {
    { Scope s(m, st, SWIFTKV_KC_ELEMWISE); launch_rmsnorm<T, TA>(b.x, (const T *)nullptr, h, T_tok, d, c.rms_eps, st, b.status, sp_hin); }
    const GemmSplit kv_split{sp_hin, nullptr, nullptr};
    if (fp8) {
      // one group at a time through the staging planes: projection (+ RoPE on K), then the quantizing row pass into the
      // group's cache slot
      for (int i = 0; i < ng; ++i) {
        const size_t woff = (size_t)i * 2 * dkv * d;
        OutDesc o{OUT_STORE, nullptr, 0, 0, kst, (long long)plane, dkv, nullptr};
        bool roped = false;
        rc = gemm_any<TA, T>(m, h, T_tok, d, (const T *)b.wfold + woff, 2 * dkv, no_w, 0, no_w, 0, o, st,
                             use_w16 ? (const __half *)b.wfold + woff : nullptr, nullptr, nullptr, &rope, &roped);
        if (rc) return rc;
        if (use_w16 && !roped) return fail(SWIFTKV_ERR_UNSUPPORTED, "half-folded SingleInputKV weight needs the tensor-core GEMM");
        if (!roped) { Scope s(m, st, SWIFTKV_KC_ELEMWISE); launch_rope<T>(kst, 0, 1, b.pos, nullptr, b.cos_tab, b.sin_tab, T_tok, c.n_kv_heads, c.head_dim, st); }
        Scope s(m, st, SWIFTKV_KC_ELEMWISE, 2);
        launch_quantize_rows_fp8<T, T>(kst, T_tok, dkv, slot_map, k_codes(l + i), k_scale(l + i), (T *)nullptr, st);
        launch_quantize_rows_fp8<T, T>(vst, T_tok, dkv, slot_map, v_codes(l + i), v_scale(l + i), (T *)nullptr, st);
      }
    } else {
    T *slot_l = kv + (size_t)l * 2 * plane;
    OutDesc o{OUT_STORE, nullptr, 0, 0, slot_l, (long long)plane, dkv, slot_map};
    bool roped = false;
    rc = gemm_any<TA, T>(m, h, T_tok, d, (const T *)b.wfold, ng * 2 * dkv, no_w, 0, no_w, 0, o, st,
                         use_w16 ? (const __half *)b.wfold : nullptr, nullptr, nullptr, &rope, &roped, nullptr, 0, &kv_split);
    if (rc) return rc;
    if (use_w16 && !roped) return fail(SWIFTKV_ERR_UNSUPPORTED, "half-folded SingleInputKV weight needs the tensor-core GEMM");
    if (!roped) { Scope s(m, st, SWIFTKV_KC_ELEMWISE); launch_rope<T>(slot_l, (long long)(2 * plane), ng, b.pos, slot_map, b.cos_tab, b.sin_tab, T_tok, c.n_kv_heads, c.head_dim, st); }
    }
  }

  // ---- the tokens that must produce output -- the last token of a prompt (footnote of Sec. 3.2), decode tokens
  //      (Sec. 3.5) -- continue through layers l+1..L
  for (int r0 = 0; r0 < bt.n_emit; r0 += MAX_TAIL_ROWS) {
    const int rows = std::min(MAX_TAIL_ROWS, bt.n_emit - r0);
    float *hy = b.hy, *qy = b.qy, *ay = b.ay, *acty = b.acty;
    float *y = b.y + (size_t)r0 * d;
    if (!bt.decode) { Scope s(m, st, SWIFTKV_KC_TAIL); launch_gather_rows(b.x, b.last_idx + r0, y, rows, d, st); }
    const int32_t *be = blk_emit ? blk_emit + (size_t)r0 * bt.blk_stride : nullptr;
    int emit_kv = 0;
    for (int r = r0; r < r0 + rows; ++r) emit_kv += bt.emit_lens[r];
    const TailOpts q_rope{b.last_pos + r0, b.cos_tab, b.sin_tab, emit_kv};    // the queries are rotated inside the attention kernel
    auto attention = [&](int slot) {
      Scope s(m, st, SWIFTKV_KC_TAIL, 2);
      if (fp8)
        launch_tail_attention<fp8e4>(qy, (const fp8e4 *)k_codes(slot), (const fp8e4 *)v_codes(slot), k_scale(slot), v_scale(slot), ay,
                                     b.emit_row0 + r0, b.emit_len + r0, be, bt.blk_stride, rows, max_len, c.n_q_heads,
                                     c.n_kv_heads, c.head_dim, b.tail_scratch, st, q_rope);
      else
        launch_tail_attention<T>(qy, kv + (size_t)slot * 2 * plane, kv + (size_t)slot * 2 * plane + plane, nullptr, nullptr, ay,
                                 b.emit_row0 + r0, b.emit_len + r0, be, bt.blk_stride, rows, max_len, c.n_q_heads, c.n_kv_heads,
                                 c.head_dim, b.tail_scratch, st, q_rope);
    };
    if (fused_tail) {
      for (int j = l; j < L; ++j) {
        const swiftkv_layer_weights &lw = m->layers[j];
        list[n_list++] = TailStage{y, lw.in_norm, lw.wq, nullptr, qy, dq, d, dq, 0};
        if ((rc = flush(rows))) return rc;
        attention(l + (j - l) / g);
        list[n_list++] = TailStage{ay, nullptr, lw.wo, nullptr, y, d, dq, d, 1};
        list[n_list++] = TailStage{y, lw.post_norm, lw.w_gate, lw.w_up, acty, F, d, F, 2};
        list[n_list++] = TailStage{acty, nullptr, lw.w_down, nullptr, y, d, F, d, 1};
        if (j + 1 == L) list[n_list++] = TailStage{y, m->final_norm, m->lm_head, nullptr, b.logits + (size_t)r0 * c.vocab, c.vocab, d, c.vocab, 0};
      }
      if (l == L) list[n_list++] = TailStage{y, m->final_norm, m->lm_head, nullptr, b.logits + (size_t)r0 * c.vocab, c.vocab, d, c.vocab, 0};
      if ((rc = flush(rows))) return rc;
      continue;
    }
    for (int j = l; j < L; ++j) {
      const swiftkv_layer_weights &lw = m->layers[j];
      { Scope s(m, st, SWIFTKV_KC_TAIL); launch_tail_rmsnorm<T>(y, (const T *)lw.in_norm, hy, rows, d, c.rms_eps, st); }
      { Scope s(m, st, SWIFTKV_KC_TAIL); launch_skinny_gemm<T>(hy, (const T *)lw.wq, nullptr, rows, dq, d, qy, dq, OUT_STORE_F32, st); }
      attention(l + (j - l) / g);
      { Scope s(m, st, SWIFTKV_KC_TAIL); launch_skinny_gemm<T>(ay, (const T *)lw.wo, nullptr, rows, d, dq, y, d, OUT_RESID_ADD_F32, st); }
      { Scope s(m, st, SWIFTKV_KC_TAIL); launch_tail_rmsnorm<T>(y, (const T *)lw.post_norm, hy, rows, d, c.rms_eps, st); }
      { Scope s(m, st, SWIFTKV_KC_TAIL); launch_skinny_gemm<T>(hy, (const T *)lw.w_gate, (const T *)lw.w_up, rows, F, d, acty, F, OUT_STORE_F32, st); }
      { Scope s(m, st, SWIFTKV_KC_TAIL); launch_skinny_gemm<T>(acty, (const T *)lw.w_down, nullptr, rows, d, F, y, d, OUT_RESID_ADD_F32, st); }
    }
    { Scope s(m, st, SWIFTKV_KC_TAIL); launch_tail_rmsnorm<T>(y, (const T *)m->final_norm, hy, rows, d, c.rms_eps, st); }
    { Scope s(m, st, SWIFTKV_KC_TAIL); launch_skinny_gemm<T>(hy, (const T *)m->lm_head, nullptr, rows, c.vocab, d,
                                                              b.logits + (size_t)r0 * c.vocab, c.vocab, OUT_STORE_F32, st); }
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail(SWIFTKV_ERR_CUDA, "kernel launch failed: %s", cudaGetErrorString(e));
  return SWIFTKV_OK;
}

static int32_t forward_common(swiftkv_model *m, const int32_t *tokens, bool tokens_on_device, const swiftkv_seq_step *seqs,
                              int32_t n_seqs, bool plain, int32_t l, int32_t g, void *stream) {
  const swiftkv_config &c = m->cfg;
  if (l < 1 || l > c.n_layers) return fail(SWIFTKV_ERR_INVALID_ARG, "swift_layer %d outside [1, %d]", l, c.n_layers);
  if (g < 1) return fail(SWIFTKV_ERR_INVALID_ARG, "acrosskv_group must be >= 1");
  if (n_seqs < 1 || n_seqs > m->max_seqs) return fail(SWIFTKV_ERR_INVALID_ARG, "n_seqs %d outside [1, %d]", n_seqs, m->max_seqs);
  Batch bt{};
  bt.B = n_seqs; bt.plain = plain;
  bt.paged = seqs[0].block_table != nullptr;
  bt.blk_stride = (m->max_tokens + PAGE_ROWS - 1) / PAGE_ROWS;
  const int n_pages = m->max_tokens / PAGE_ROWS;          // whole pages inside a cache plane
  std::vector<char> page_used(bt.paged ? n_pages : 0, 0);
  long long total = 0, total_kv = 0;
  int rows_used = 0;
  for (int i = 0; i < n_seqs; ++i) {
    const swiftkv_seq_step &s = seqs[i];
    if (s.n_new < 1) return fail(SWIFTKV_ERR_INVALID_ARG, "sequence %d: n_new = %d < 1", i, s.n_new);
    if (s.n_past < 0 || s.cache_row < 0) return fail(SWIFTKV_ERR_INVALID_ARG, "sequence %d: negative n_past / cache_row", i);
    if ((s.block_table != nullptr) != bt.paged) return fail(SWIFTKV_ERR_INVALID_ARG, "either every sequence has a block table or none");
    long long end = (long long)s.cache_row + s.n_past + s.n_new;
    if (bt.paged) {
      const int need = (s.n_past + s.n_new + PAGE_ROWS - 1) / PAGE_ROWS;
      if (s.n_blocks < need) return fail(SWIFTKV_ERR_INVALID_ARG, "sequence %d: %d pages listed, %d needed", i, s.n_blocks, need);
      end = 0;
      for (int k = 0; k < need; ++k) {
        const int pg = s.block_table[k];
        if (pg < 0 || pg >= n_pages) return fail(SWIFTKV_ERR_INVALID_ARG, "sequence %d: page %d outside [0, %d)", i, pg, n_pages);
        if (page_used[pg]) return fail(SWIFTKV_ERR_INVALID_ARG, "page %d is listed twice", pg);
        page_used[pg] = 1;
        end = std::max(end, (long long)(pg + 1) * PAGE_ROWS);
      }
    } else {
      if (end > m->max_tokens) return fail(SWIFTKV_ERR_INVALID_ARG, "sequence %d: cache rows up to %lld exceed max_tokens %d", i, end, m->max_tokens);
      for (int k = 0; k < i; ++k) {   // regions of different sequences must not overlap
        const long long a0 = seqs[k].cache_row, a1 = a0 + seqs[k].n_past + seqs[k].n_new;
        if (s.cache_row < a1 && a0 < end) return fail(SWIFTKV_ERR_INVALID_ARG, "cache rows of sequences %d and %d overlap", k, i);
      }
    }
    total += s.n_new;
    total_kv += s.n_past + s.n_new;
    bt.max_new = std::max(bt.max_new, s.n_new);
    bt.max_kv = std::max(bt.max_kv, s.n_past + s.n_new);
    rows_used = std::max(rows_used, (int)end);
    if (s.emit) bt.n_emit += 1;
  }
  if (total > m->max_tokens || total_kv > m->max_tokens)
    return fail(SWIFTKV_ERR_INVALID_ARG, "%lld new / %lld cached+new tokens > max_tokens %d", total, total_kv, m->max_tokens);
  // (no emitting sequence is fine: a minibatch of inner prefill chunks fills caches only and skips layers l+1..L)
  if (plain && bt.n_emit < 1) return fail(SWIFTKV_ERR_INVALID_ARG, "no sequence is marked to emit logits");
  bt.T_tok = (int)total; bt.total_kv = (int)total_kv;
  bt.decode = !plain && total == n_seqs && bt.n_emit == n_seqs && n_seqs <= MAX_TAIL_ROWS && (m->kernel_mask & 32);
  if (!tokens_on_device)
    for (long long t = 0; t < total; ++t)
      if (tokens[t] < 0 || tokens[t] >= c.vocab) return fail(SWIFTKV_ERR_INVALID_ARG, "token %lld = %d outside [0, %d)", t, tokens[t], c.vocab);
  if (l < c.n_layers && fold_elems_for(c, l, g) > m->fold_capacity_elems)
    return fail(SWIFTKV_ERR_WORKSPACE_SMALL, "workspace too small for the folded weight of (l=%d, g=%d)", l, g);
  if (l + n_groups(c.n_layers, l, g) > m->slot_capacity)
    return fail(SWIFTKV_ERR_WORKSPACE_SMALL, "kv cache holds %d slots, (l=%d, g=%d) needs %d", m->slot_capacity, l, g,
                l + n_groups(c.n_layers, l, g));
  int dev = -1;
  CUDA_TRY(cudaGetDevice(&dev));
  if (dev != m->device) return fail(SWIFTKV_ERR_INVALID_ARG, "current device %d is not the model's device %d", dev, m->device);

  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  tc_gemm_use_cta_pairs((m->kernel_mask & 4) != 0, (m->kernel_mask & 8) != 0);
  m->ready = false;
  m->launches = 0;
  // host-side metadata -> one staging vector -> device arrays
  const int B = n_seqs, T = bt.T_tok;
  std::vector<int32_t> &hm = m->host_meta;
  hm.assign((size_t)(B + 1) + 2 * (size_t)T + 2 * B + (B + 1) + 4 * (size_t)B, 0);
  int32_t *cu = hm.data(), *pos = cu + B + 1, *slot = pos + T, *row0 = slot + T, *klen = row0 + B, *kcu = klen + B;
  int32_t *last_idx = kcu + B + 1, *last_pos = last_idx + B, *e_row0 = last_pos + B, *e_len = e_row0 + B;
  int ne = 0;
  for (int i = 0; i < B; ++i) {
    const swiftkv_seq_step &s = seqs[i];
    cu[i + 1] = cu[i] + s.n_new;
    row0[i] = s.cache_row;
    klen[i] = s.n_past + s.n_new;
    kcu[i + 1] = kcu[i] + klen[i];
    for (int k = 0; k < s.n_new; ++k) {
      const int pp = s.n_past + k;
      pos[cu[i] + k] = pp;
      slot[cu[i] + k] = bt.paged ? s.block_table[pp / PAGE_ROWS] * PAGE_ROWS + pp % PAGE_ROWS : s.cache_row + pp;
    }
    if (s.emit) {
      last_idx[ne] = cu[i + 1] - 1; last_pos[ne] = klen[i] - 1; e_row0[ne] = s.cache_row; e_len[ne] = klen[i]; ++ne;
      bt.emit_lens.push_back(klen[i]);
    }
  }
  Buffers &b = m->b;
  if (bt.paged) {   // block tables of all sequences, and once more for the emitting ones in their order
    std::vector<int32_t> tb((size_t)B * bt.blk_stride, 0), te((size_t)B * bt.blk_stride, 0);
    int e = 0;
    for (int i = 0; i < B; ++i) {
      const int need = (klen[i] + PAGE_ROWS - 1) / PAGE_ROWS;
      for (int k = 0; k < need; ++k) tb[(size_t)i * bt.blk_stride + k] = seqs[i].block_table[k];
      if (seqs[i].emit) { std::copy_n(&tb[(size_t)i * bt.blk_stride], need, &te[(size_t)e * bt.blk_stride]); ++e; }
    }
    CUDA_TRY(cudaMemcpyAsync(b.blk, tb.data(), tb.size() * 4, cudaMemcpyHostToDevice, st));
    CUDA_TRY(cudaMemcpyAsync(b.blk_emit, te.data(), te.size() * 4, cudaMemcpyHostToDevice, st));
  }
  bt.att_ctas = 0;
  if ((m->kernel_mask & 16) && (m->kernel_mask & 2) && !bt.decode && c.dtype == SWIFTKV_DTYPE_BF16 &&
      tc_attention_supported(c.n_q_heads, c.n_kv_heads, c.head_dim)) {
    // the persistent attention kernel's work list, balanced here where the lengths are known
    const int n_ctas = std::min(m->n_sms, ATT_MAX_CTAS);
    std::vector<int32_t> n_new(B), n_past(B), off(n_ctas + 1), items(att_max_items(c, m->max_tokens, m->max_seqs));
    for (int i = 0; i < B; ++i) { n_new[i] = seqs[i].n_new; n_past[i] = seqs[i].n_past; }
    const int n_items = attention_schedule(n_new.data(), n_past.data(), B, c.n_q_heads, n_ctas, off.data(), items.data());
    CUDA_TRY(cudaMemcpyAsync(b.att_off, off.data(), off.size() * 4, cudaMemcpyHostToDevice, st));
    if (n_items > 0) CUDA_TRY(cudaMemcpyAsync(b.att_items, items.data(), (size_t)n_items * 4, cudaMemcpyHostToDevice, st));
    bt.att_ctas = n_ctas;
  }
  CUDA_TRY(cudaMemcpyAsync(b.cu, cu, (size_t)(B + 1) * 4, cudaMemcpyHostToDevice, st));
  CUDA_TRY(cudaMemcpyAsync(b.pos, pos, (size_t)T * 4, cudaMemcpyHostToDevice, st));
  CUDA_TRY(cudaMemcpyAsync(b.slot, slot, (size_t)T * 4, cudaMemcpyHostToDevice, st));
  CUDA_TRY(cudaMemcpyAsync(b.kv_row0, row0, (size_t)B * 4, cudaMemcpyHostToDevice, st));
  CUDA_TRY(cudaMemcpyAsync(b.kv_len, klen, (size_t)B * 4, cudaMemcpyHostToDevice, st));
  CUDA_TRY(cudaMemcpyAsync(b.kcu, kcu, (size_t)(B + 1) * 4, cudaMemcpyHostToDevice, st));
  if (ne > 0) CUDA_TRY(cudaMemcpyAsync(b.last_idx, last_idx, (size_t)ne * 4, cudaMemcpyHostToDevice, st));
  if (ne > 0) CUDA_TRY(cudaMemcpyAsync(b.last_pos, last_pos, (size_t)ne * 4, cudaMemcpyHostToDevice, st));
  if (ne > 0) CUDA_TRY(cudaMemcpyAsync(b.emit_row0, e_row0, (size_t)ne * 4, cudaMemcpyHostToDevice, st));
  if (ne > 0) CUDA_TRY(cudaMemcpyAsync(b.emit_len, e_len, (size_t)ne * 4, cudaMemcpyHostToDevice, st));
  CUDA_TRY(cudaMemcpyAsync(b.tokens, tokens, (size_t)total * 4,
                           tokens_on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice, st));
  int32_t rc;
  if (c.dtype == SWIFTKV_DTYPE_F32) rc = run_prefill<float, float>(m, bt, l, g, st);
  else if (m->act_format == SWIFTKV_ACT_F16) rc = run_prefill<__half, bf16>(m, bt, l, g, st);
  else rc = run_prefill<bf16, bf16>(m, bt, l, g, st);
  if (rc) return rc;
  m->n_tokens = plain ? T : std::max(rows_used, m->n_tokens);
  m->n_seqs = ne; m->cur_l = l; m->cur_g = g; m->ready = true;
  return SWIFTKV_OK;
}

static int32_t prefill_common(swiftkv_model *m, const int32_t *tokens, bool tokens_on_device, const int32_t *seq_lens,
                              int32_t n_seqs, int32_t l, int32_t g, void *stream) {
  if (!m) return fail(SWIFTKV_ERR_INVALID_ARG, "model is null");
  if (!tokens || !seq_lens) return fail(SWIFTKV_ERR_INVALID_ARG, "tokens / seq_lens is null");
  if (n_seqs < 1 || n_seqs > m->max_seqs) return fail(SWIFTKV_ERR_INVALID_ARG, "n_seqs %d outside [1, %d]", n_seqs, m->max_seqs);
  std::vector<swiftkv_seq_step> seqs(n_seqs);
  long long row = 0;
  for (int i = 0; i < n_seqs; ++i) {
    if (seq_lens[i] < 1) return fail(SWIFTKV_ERR_INVALID_ARG, "seq_lens[%d] = %d < 1", i, seq_lens[i]);
    if (row + seq_lens[i] > m->max_tokens) return fail(SWIFTKV_ERR_INVALID_ARG, "more than max_tokens %d tokens", m->max_tokens);
    seqs[i] = swiftkv_seq_step{seq_lens[i], 0, (int32_t)row, 1, nullptr, 0};   // whole prompt, packed rows, last token emits
    row += seq_lens[i];
  }
  return forward_common(m, tokens, tokens_on_device, seqs.data(), n_seqs, true, l, g, stream);
}

extern "C" int32_t swiftkv_prefill(swiftkv_model *m, const int32_t *tokens, const int32_t *seq_lens, int32_t n_seqs,
                                   int32_t swift_layer, int32_t acrosskv_group, void *cuda_stream) {
  return prefill_common(m, tokens, false, seq_lens, n_seqs, swift_layer, acrosskv_group, cuda_stream);
}
extern "C" int32_t swiftkv_prefill_device_tokens(swiftkv_model *m, const int32_t *tokens_dev, const int32_t *seq_lens,
                                                 int32_t n_seqs, int32_t swift_layer, int32_t acrosskv_group,
                                                 void *cuda_stream) {
  return prefill_common(m, tokens_dev, true, seq_lens, n_seqs, swift_layer, acrosskv_group, cuda_stream);
}

extern "C" int32_t swiftkv_step(swiftkv_model *m, const int32_t *tokens, const swiftkv_seq_step *seqs, int32_t n_seqs,
                                int32_t swift_layer, int32_t acrosskv_group, void *cuda_stream) {
  if (!m) return fail(SWIFTKV_ERR_INVALID_ARG, "model is null");
  if (!tokens || !seqs) return fail(SWIFTKV_ERR_INVALID_ARG, "tokens / seqs is null");
  return forward_common(m, tokens, false, seqs, n_seqs, false, swift_layer, acrosskv_group, cuda_stream);
}

static size_t simscore_bytes(const swiftkv_config &c, int n_tokens) {
  const size_t xs = ((size_t)c.n_layers * n_tokens * c.hidden * sizeof(float) + 255) & ~(size_t)255;
  return xs + (size_t)c.n_layers * c.n_layers * sizeof(double);
}
extern "C" size_t swiftkv_simscore_scratch_bytes(const swiftkv_model *m, int32_t n_tokens) {
  if (!m || n_tokens < 1) return 0;
  return simscore_bytes(m->cfg, n_tokens);
}
extern "C" int32_t swiftkv_simscore(swiftkv_model *m, const int32_t *tokens, const int32_t *seq_lens, int32_t n_seqs,
                                    void *scratch, size_t scratch_bytes, float *sim, float *simscore, void *cuda_stream) {
  if (!m || !tokens || !seq_lens || !scratch || !simscore) return fail(SWIFTKV_ERR_INVALID_ARG, "null argument");
  if (m->cfg.n_layers < 2) return fail(SWIFTKV_ERR_INVALID_ARG, "SimScore needs at least two layers");
  if ((reinterpret_cast<uintptr_t>(scratch) & 255)) return fail(SWIFTKV_ERR_INVALID_ARG, "scratch must be 256-byte aligned");
  if (n_seqs < 1) return fail(SWIFTKV_ERR_INVALID_ARG, "n_seqs < 1");
  long long T = 0;
  for (int i = 0; i < n_seqs; ++i) T += seq_lens[i] > 0 ? seq_lens[i] : 0;
  if (T < 1 || T > m->max_tokens) return fail(SWIFTKV_ERR_INVALID_ARG, "token count outside [1, max_tokens]");
  if (scratch_bytes < simscore_bytes(m->cfg, (int)T))
    return fail(SWIFTKV_ERR_WORKSPACE_SMALL, "scratch %zu < %zu bytes", scratch_bytes, simscore_bytes(m->cfg, (int)T));
  const int L = m->cfg.n_layers;
  m->capture = reinterpret_cast<float *>(scratch);
  const int32_t rc = prefill_common(m, tokens, false, seq_lens, n_seqs, L, 1, cuda_stream);   // the unmodified model
  m->capture = nullptr;
  if (rc) return rc;
  const size_t xs = ((size_t)L * T * m->cfg.hidden * sizeof(float) + 255) & ~(size_t)255;
  launch_simscore(reinterpret_cast<const float *>(scratch), L, (int)T, m->cfg.hidden,
                  reinterpret_cast<double *>(reinterpret_cast<uint8_t *>(scratch) + xs), sim, simscore,
                  reinterpret_cast<cudaStream_t>(cuda_stream));
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail(SWIFTKV_ERR_CUDA, "launch failed: %s", cudaGetErrorString(e));
  m->launches += 3;
  return SWIFTKV_OK;
}

static DistillDims distill_dims(const swiftkv_config &c) {
  return DistillDims{c.vocab, c.hidden, c.n_layers, c.n_q_heads, c.n_kv_heads, c.head_dim, c.ffn, c.rms_eps};
}
// fp32 copies of a bf16 model's frozen weights (the step computes in fp32): floats per layer / for embedding, final norm, lm_head
static size_t distill_layer_weight_floats(const swiftkv_config &c) {
  const size_t d = c.hidden, dq = (size_t)c.n_q_heads * c.head_dim, dkv = (size_t)c.n_kv_heads * c.head_dim, F = c.ffn;
  return 2 * d + 2 * dq * d + 2 * dkv * d + 3 * F * d + 9 * 4;
}
static size_t distill_weight_floats(const swiftkv_config &c) {
  if (c.dtype != SWIFTKV_DTYPE_BF16) return 0;
  return (size_t)c.n_layers * distill_layer_weight_floats(c) + 2 * (size_t)c.vocab * c.hidden + c.hidden + 3 * 4;
}
extern "C" size_t swiftkv_distill_workspace_bytes(const swiftkv_model *m, int32_t total_tokens, int32_t swift_layer) {
  if (!m || total_tokens < 1 || swift_layer < 1 || swift_layer > m->cfg.n_layers) return 0;
  return (distill_workspace_floats(distill_dims(m->cfg), total_tokens, swift_layer) + distill_weight_floats(m->cfg)) * sizeof(float);
}
extern "C" int32_t swiftkv_distill_grads(swiftkv_model *m, const int32_t *tokens, const int32_t *seq_lens, int32_t n_seqs,
                                         int32_t l, int32_t g, float temperature, int32_t precision, const void *const *student_wq,
                                         const void *const *student_wk, const void *const *student_wv, void *const *grad_wq,
                                         void *const *grad_wk, void *const *grad_wv, float *loss, void *workspace,
                                         size_t workspace_bytes, void *cuda_stream) {
  if (!m || !tokens || !seq_lens || !student_wq || !student_wk || !student_wv || !grad_wq || !grad_wk || !grad_wv || !loss || !workspace)
    return fail(SWIFTKV_ERR_INVALID_ARG, "null argument");
  const swiftkv_config &c = m->cfg;
  if (l < 1 || l > c.n_layers) return fail(SWIFTKV_ERR_INVALID_ARG, "swift_layer %d outside [1, %d]", l, c.n_layers);
  if (g < 1) return fail(SWIFTKV_ERR_INVALID_ARG, "acrosskv_group must be >= 1");
  if (!(temperature > 0.f)) return fail(SWIFTKV_ERR_INVALID_ARG, "temperature must be positive");
  if (precision < 0 || precision > 2) return fail(SWIFTKV_ERR_INVALID_ARG, "precision must be SWIFTKV_DISTILL_FP32, _TF32X3 or _TF32");
  if (n_seqs < 1 || n_seqs > m->max_seqs) return fail(SWIFTKV_ERR_INVALID_ARG, "n_seqs %d outside [1, %d]", n_seqs, m->max_seqs);
  if ((reinterpret_cast<uintptr_t>(workspace) & 255)) return fail(SWIFTKV_ERR_INVALID_ARG, "workspace must be 256-byte aligned");
  std::vector<int32_t> cu(n_seqs + 1, 0);
  for (int i = 0; i < n_seqs; ++i) {
    if (seq_lens[i] < 1) return fail(SWIFTKV_ERR_INVALID_ARG, "sequence %d: length %d < 1", i, seq_lens[i]);
    cu[i + 1] = cu[i] + seq_lens[i];
  }
  const int T = cu[n_seqs];
  if (T > m->max_tokens) return fail(SWIFTKV_ERR_INVALID_ARG, "%d tokens > max_tokens %d", T, m->max_tokens);
  const DistillDims dims = distill_dims(c);
  const size_t main_floats = distill_workspace_floats(dims, T, l);
  const size_t need = (main_floats + distill_weight_floats(c)) * sizeof(float);
  if (workspace_bytes < need) return fail(SWIFTKV_ERR_WORKSPACE_SMALL, "workspace %zu < %zu bytes", workspace_bytes, need);
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  // a bf16 model: fp32 copies of the frozen weights behind the step's own workspace
  const bool widen = c.dtype == SWIFTKV_DTYPE_BF16;
  float *wcopy = reinterpret_cast<float *>(workspace) + main_floats;
  auto f32 = [&](const void *p, size_t n) -> const float * {
    if (!widen) return reinterpret_cast<const float *>(p);
    float *dst = wcopy;
    wcopy += (n + 3) & ~(size_t)3;
    distill_upcast(p, dst, (long long)n, st);
    return dst;
  };
  const size_t dd = c.hidden, dq_ = (size_t)c.n_q_heads * c.head_dim, dkv_ = (size_t)c.n_kv_heads * c.head_dim, F_ = c.ffn;
  std::vector<DistillLayer> layers(c.n_layers);
  for (int j = 0; j < c.n_layers; ++j) {
    const swiftkv_layer_weights &w = m->layers[j];
    DistillLayer &d = layers[j];
    d = DistillLayer{f32(w.in_norm, dd), f32(w.wq, dq_ * dd), f32(w.wk, dkv_ * dd), f32(w.wv, dkv_ * dd), f32(w.wo, dd * dq_),
                     f32(w.post_norm, dd), f32(w.w_gate, F_ * dd), f32(w.w_up, F_ * dd), f32(w.w_down, dd * F_),
                     nullptr, nullptr, nullptr, nullptr, nullptr, nullptr};
    if (j >= l) {
      if (!student_wq[j] || !student_wk[j] || !student_wv[j] || !grad_wq[j] || !grad_wk[j] || !grad_wv[j])
        return fail(SWIFTKV_ERR_INVALID_ARG, "layer %d: null student weight or gradient pointer", j);
      d.s_wq = (const float *)student_wq[j]; d.s_wk = (const float *)student_wk[j]; d.s_wv = (const float *)student_wv[j];
      d.g_wq = (float *)grad_wq[j]; d.g_wk = (float *)grad_wk[j]; d.g_wv = (float *)grad_wv[j];
    }
  }
  Buffers &b = m->b;
  // sequence offsets to the device (a few bytes: a blocking copy keeps the host vector's lifetime out of the picture)
  CUDA_TRY(cudaStreamSynchronize(st));
  CUDA_TRY(cudaMemcpy(b.cu, cu.data(), (size_t)(n_seqs + 1) * 4, cudaMemcpyHostToDevice));
  launch_positions(b.cu, n_seqs, b.pos, b.last_idx, T, st);
  DistillArgs a{f32(m->embed, (size_t)c.vocab * dd), f32(m->final_norm, dd), f32(m->lm_head, (size_t)c.vocab * dd), tokens, b.cu, b.pos, b.cos_tab,
                b.sin_tab, T, n_seqs, l, g, precision, temperature, loss, b.status, workspace, main_floats};
  const int rc = run_distill(dims, a, layers.data(), st);
  if (rc) return fail(rc, "distillation step failed: %s", cudaGetErrorString(cudaGetLastError()));
  m->ready = false;      // the prefill state (positions, offsets) has been overwritten
  return SWIFTKV_OK;
}

extern "C" int32_t swiftkv_adamw_update(float *param, const float *grad, float *exp_avg, float *exp_avg_sq, int64_t n, int32_t step,
                                        float lr, float beta1, float beta2, float eps, float weight_decay, void *cuda_stream) {
  if (!param || !grad || !exp_avg || !exp_avg_sq) return fail(SWIFTKV_ERR_INVALID_ARG, "null argument");
  if (n < 0 || step < 1) return fail(SWIFTKV_ERR_INVALID_ARG, "n must be >= 0 and step >= 1");
  if (!(lr >= 0.f) || !(beta1 >= 0.f && beta1 < 1.f) || !(beta2 >= 0.f && beta2 < 1.f) || !(eps > 0.f) || !(weight_decay >= 0.f))
    return fail(SWIFTKV_ERR_INVALID_ARG, "bad hyper-parameter");
  launch_adamw(param, grad, exp_avg, exp_avg_sq, (long long)n, lr, beta1, beta2, eps, weight_decay, step, reinterpret_cast<cudaStream_t>(cuda_stream));
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail(SWIFTKV_ERR_CUDA, "launch failed: %s", cudaGetErrorString(e));
  return SWIFTKV_OK;
}

extern "C" int32_t swiftkv_kv_cache_view(const swiftkv_model *m, int32_t layer, swiftkv_kv_view *out) {
  if (!m || !out) return fail(SWIFTKV_ERR_INVALID_ARG, "null argument");
  if (layer < 0 || layer >= m->cfg.n_layers) return fail(SWIFTKV_ERR_INVALID_ARG, "layer %d outside [0, %d)", layer, m->cfg.n_layers);
  if (!m->ready) return fail(SWIFTKV_ERR_NOT_READY, "no prefill has been run");
  const int l = m->cur_l, g = m->cur_g;
  const int dkv = m->cfg.n_kv_heads * m->cfg.head_dim;
  const size_t plane = (size_t)m->max_tokens * dkv;
  int slot = layer, owner = layer;
  if (layer >= l) { slot = l + (layer - l) / g; owner = l + ((layer - l) / g) * g; }
  const uint8_t *kp = m->kv + (size_t)slot * slot_bytes_of(m->cfg, m->max_tokens);
  out->k = kp;
  out->k_scale = out->v_scale = nullptr;
  if (m->cfg.kv_format == SWIFTKV_KV_FP8) {
    const size_t cp = fp8_code_plane(m->cfg, m->max_tokens), sp = fp8_scale_plane(m->max_tokens);
    out->v = kp + cp;
    out->k_scale = reinterpret_cast<const float *>(kp + 2 * cp);
    out->v_scale = reinterpret_cast<const float *>(kp + 2 * cp + sp);
    out->dtype = SWIFTKV_DTYPE_FP8_E4M3;
  } else {
    out->v = kp + plane * m->esize;
    out->dtype = m->cfg.dtype;
  }
  out->token_stride = dkv;
  out->head_stride = m->cfg.head_dim;
  out->n_tokens = m->n_tokens;
  out->owner_layer = owner;
  return SWIFTKV_OK;
}

extern "C" int32_t swiftkv_first_logits(const swiftkv_model *m, const float **logits, int32_t *n_seqs) {
  if (!m || !logits) return fail(SWIFTKV_ERR_INVALID_ARG, "null argument");
  if (!m->ready) return fail(SWIFTKV_ERR_NOT_READY, "no prefill has been run");
  *logits = m->b.logits;
  if (n_seqs) *n_seqs = m->n_seqs;
  return SWIFTKV_OK;
}

extern "C" int32_t swiftkv_status(swiftkv_model *m, void *cuda_stream) {
  if (!m) return fail(SWIFTKV_ERR_INVALID_ARG, "model is null");
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  unsigned int word = 0;
  CUDA_TRY(cudaMemcpyAsync(&word, m->b.status, 4, cudaMemcpyDeviceToHost, st));
  CUDA_TRY(cudaMemsetAsync(m->b.status, 0, 4, st));
  CUDA_TRY(cudaStreamSynchronize(st));
  if (word & STATUS_TIMEOUT) return fail(SWIFTKV_ERR_DEVICE_TIMEOUT, "a bounded wait inside a kernel ran out");
  if (word & STATUS_ACT_OVERFLOW)
    return fail(SWIFTKV_ERR_ACT_OVERFLOW, "an activation (or weight) beyond the IEEE-half range was clamped to +-65504: results are "
                                          "wrong; run this model with swiftkv_set_activation_format(SWIFTKV_ACT_BF16)");
  if (word & STATUS_BAD_TOKEN) return fail(SWIFTKV_ERR_BAD_TOKEN, "a token id outside [0, vocab) was clamped");
  return SWIFTKV_OK;
}

extern "C" int32_t swiftkv_profile_enable(swiftkv_model *m, int32_t on) {
  if (!m) return fail(SWIFTKV_ERR_INVALID_ARG, "model is null");
  m->profiling = on != 0;
  return SWIFTKV_OK;
}
extern "C" int32_t swiftkv_profile_read(swiftkv_model *m, void *cuda_stream, float *ms, int32_t *launches) {
  if (!m || !ms || !launches) return fail(SWIFTKV_ERR_INVALID_ARG, "null argument");
  CUDA_TRY(cudaStreamSynchronize(reinterpret_cast<cudaStream_t>(cuda_stream)));
  for (int i = 0; i < SWIFTKV_KC_COUNT; ++i) { ms[i] = 0.f; launches[i] = 0; }
  for (auto &r : m->recs) {
    float t = 0.f;
    if (cudaEventElapsedTime(&t, r.a, r.b) == cudaSuccess) { ms[r.cls] += t; launches[r.cls] += 1; }
    m->pool.push_back(r.a);
    m->pool.push_back(r.b);
  }
  m->recs.clear();
  return SWIFTKV_OK;
}
extern "C" int32_t swiftkv_last_launch_count(const swiftkv_model *m) { return m ? m->launches : 0; }
extern "C" int32_t swiftkv_set_kernel_mask(swiftkv_model *m, int32_t mask) {
  if (!m) return 0;
  m->kernel_mask = mask & 127;
  return m->kernel_mask;
}

extern "C" int32_t swiftkv_set_activation_format(swiftkv_model *m, int32_t format) {
  if (!m) return fail(SWIFTKV_ERR_INVALID_ARG, "model is null");
  if (format != SWIFTKV_ACT_BF16 && format != SWIFTKV_ACT_F16 && format != SWIFTKV_ACT_F16_SPLIT)
    return fail(SWIFTKV_ERR_INVALID_ARG, "unknown activation format");
  m->act_format = format == SWIFTKV_ACT_F16_SPLIT ? SWIFTKV_ACT_F16 : format;
  m->split_mask = format == SWIFTKV_ACT_F16_SPLIT ? SWIFTKV_SPLIT_DEFAULT : 0;
  return SWIFTKV_OK;
}

extern "C" int64_t swiftkv_half_weight_cache_bytes(const swiftkv_config *cfg, int32_t n_layers) {
  if (!cfg || n_layers < 0 || cfg->hidden < 1 || cfg->ffn < 1 || cfg->head_dim < 1 || cfg->n_q_heads < 1 || cfg->n_kv_heads < 1) return -1;
  const long long d = cfg->hidden, dq = (long long)cfg->n_q_heads * cfg->head_dim, dkv = (long long)cfg->n_kv_heads * cfg->head_dim, F = cfg->ffn;
  return (int64_t)((2 * d * dq + 2 * d * dkv + 3 * d * F) * 2 * n_layers);
}

extern "C" int32_t swiftkv_set_half_weight_cache(swiftkv_model *m, void *buffer, int64_t bytes) {
  if (!m) return fail(SWIFTKV_ERR_INVALID_ARG, "model is null");
  if ((buffer == nullptr) != (bytes == 0) || bytes < 0) return fail(SWIFTKV_ERR_INVALID_ARG, "buffer and bytes must both be given or both be zero");
  if (reinterpret_cast<uintptr_t>(buffer) & 255) return fail(SWIFTKV_ERR_INVALID_ARG, "buffer must be 256-byte aligned");
  const int64_t per_layer = swiftkv_half_weight_cache_bytes(&m->cfg, 1);
  m->w16_cache = reinterpret_cast<__half *>(buffer);
  m->w16_cache_cap = buffer ? (int)std::min<int64_t>(bytes / per_layer, m->cfg.n_layers) : 0;
  m->w16_cache_valid = 0;
  return SWIFTKV_OK;
}

extern "C" int32_t swiftkv_set_split_mask(swiftkv_model *m, int32_t mask) {
  if (!m) return fail(SWIFTKV_ERR_INVALID_ARG, "model is null");
  if (mask < 0 || mask > 31) return fail(SWIFTKV_ERR_INVALID_ARG, "split mask outside [0, 31]");
  if (mask && m->act_format != SWIFTKV_ACT_F16) return fail(SWIFTKV_ERR_INVALID_ARG, "half pairs need IEEE-half activations");
  m->split_mask = mask;
  return SWIFTKV_OK;
}

// ---------------------------------------------------------------------------------------------------------
// stand-alone operators
// ---------------------------------------------------------------------------------------------------------
// a device word for the stand-alone entry points' bounded waits
static __device__ unsigned int g_op_status[64];
// the word's address on the CURRENT device (every device that loads the library has its own copy of the symbol)
static unsigned int *op_status_word() {
  constexpr int MAX_DEVICES = 64;
  static std::mutex mu;
  static unsigned int *ptr[MAX_DEVICES] = {};
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return nullptr;
  std::lock_guard<std::mutex> lock(mu);
  if (!ptr[dev]) {
    void *p = nullptr;
    if (cudaGetSymbolAddress(&p, g_op_status) == cudaSuccess) ptr[dev] = reinterpret_cast<unsigned int *>(p);
  }
  return ptr[dev];
}

extern "C" int32_t swiftkv_op_status(void *cuda_stream) {
  unsigned int *status = op_status_word();
  if (!status) return fail(SWIFTKV_ERR_CUDA, "no status word");
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  unsigned int word = 0;
  CUDA_TRY(cudaMemcpyAsync(&word, status, 4, cudaMemcpyDeviceToHost, st));
  CUDA_TRY(cudaMemsetAsync(status, 0, 4, st));
  CUDA_TRY(cudaStreamSynchronize(st));
  if (word & STATUS_TIMEOUT) return fail(SWIFTKV_ERR_DEVICE_TIMEOUT, "a bounded wait inside a stand-alone operator ran out");
  if (word & STATUS_ACT_OVERFLOW) return fail(SWIFTKV_ERR_ACT_OVERFLOW, "a half store of a stand-alone operator was clamped");
  return SWIFTKV_OK;
}

extern "C" int32_t swiftkv_debug_bounded_wait(swiftkv_model *m, int64_t limit_clocks, int32_t *outcome, void *cuda_stream) {
  if (!m || !outcome) return fail(SWIFTKV_ERR_INVALID_ARG, "null argument");
  if (limit_clocks < 1 || limit_clocks > 100000000LL) return fail(SWIFTKV_ERR_INVALID_ARG, "limit_clocks outside [1, 1e8]");
  int rc = launch_bounded_wait_probe((long long)limit_clocks, m->b.status, m->b.status + 8, reinterpret_cast<cudaStream_t>(cuda_stream));
  if (rc) return fail(rc, "launch failed: %s", cudaGetErrorString(cudaGetLastError()));
  CUDA_TRY(cudaMemcpyAsync(outcome, m->b.status + 8, 2 * sizeof(int32_t), cudaMemcpyDeviceToHost, reinterpret_cast<cudaStream_t>(cuda_stream)));
  CUDA_TRY(cudaStreamSynchronize(reinterpret_cast<cudaStream_t>(cuda_stream)));
  return SWIFTKV_OK;
}

extern "C" int32_t swiftkv_debug_fused_barrier_wait(swiftkv_model *m, int64_t limit_clocks, void *cuda_stream) {
  if (!m) return fail(SWIFTKV_ERR_INVALID_ARG, "null argument");
  if (limit_clocks < 1 || limit_clocks > 100000000LL) return fail(SWIFTKV_ERR_INVALID_ARG, "limit_clocks outside [1, 1e8]");
  const swiftkv_config &c = m->cfg;
  const int d = c.hidden, dq = c.n_q_heads * c.head_dim, F = c.ffn;
  if (c.dtype != SWIFTKV_DTYPE_BF16 || !tail_fused_supported(1, d, dq, F, c.vocab))
    return fail(SWIFTKV_ERR_UNSUPPORTED, "the fused last-token launch does not run this model");
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  Buffers &b = m->b;
  const swiftkv_layer_weights &lw = m->layers[0];
  CUDA_TRY(cudaMemsetAsync(b.status + 32, 0, 32 * sizeof(unsigned int), st));
  CUDA_TRY(cudaMemsetAsync(b.ay, 0, (size_t)dq * sizeof(float), st));
  CUDA_TRY(cudaMemsetAsync(b.y, 0, (size_t)d * sizeof(float), st));
  // two stages of layer 1 on one zero row; the host claims one barrier arrival that never happened, so the grid barrier
  // between the stages can never complete and every CTA's wait runs out at the limit
  TailStage list[2] = {TailStage{b.ay, nullptr, lw.wo, nullptr, b.y, d, dq, d, 1},
                       TailStage{b.y, lw.post_norm, lw.w_gate, lw.w_up, b.acty, F, d, F, 2}};
  unsigned int arrivals = 1;
  const int rc = launch_tail_fused(list, 2, 1, c.rms_eps, b.status + 32, &arrivals, b.status, st, (long long)limit_clocks);
  if (rc) return fail(rc, "launch failed: %s", cudaGetErrorString(cudaGetLastError()));
  CUDA_TRY(cudaStreamSynchronize(st));
  m->ready = false;
  return SWIFTKV_OK;
}

extern "C" int32_t swiftkv_gemm_tc(const void *A, const void *B, void *C, int32_t M, int32_t N, int32_t K,
                                   int32_t dtype, void *cuda_stream) {
  const int32_t act_dtype = dtype;
  if (!A || !B || !C || M < 1 || N < 1 || K < 1) return fail(SWIFTKV_ERR_INVALID_ARG, "bad argument");
  if (act_dtype != SWIFTKV_DTYPE_BF16 && act_dtype != SWIFTKV_DTYPE_F16) return fail(SWIFTKV_ERR_INVALID_ARG, "act_dtype must be bf16 or f16");
  if (((uintptr_t)A | (uintptr_t)B | (uintptr_t)C) & 15) return fail(SWIFTKV_ERR_INVALID_ARG, "pointers must be 16-byte aligned");
  if (!tc_gemm_supported(M, N, K)) return fail(SWIFTKV_ERR_UNSUPPORTED, "needs K %% 64 == 0 and N %% 128 == 0");
  unsigned int *status = op_status_word();
  if (!status) return fail(SWIFTKV_ERR_CUDA, "no status word");
  const bool f16 = act_dtype == SWIFTKV_DTYPE_F16;
  int rc = launch_gemm_tc(A, f16, M, K, B, N, nullptr, 0, nullptr, 0, out_plain(OUT_STORE, C, N, N), nullptr, 0, nullptr,
                          status, reinterpret_cast<cudaStream_t>(cuda_stream));
  if (rc) return fail(rc, "launch failed: %s", cudaGetErrorString(cudaGetLastError()));
  return SWIFTKV_OK;
}

extern "C" int32_t swiftkv_gemm_tf32(const float *A, const float *B, float *C, int32_t M, int32_t N, int32_t K, int32_t accumulate,
                                     void *cuda_stream) {
  if (!A || !B || !C || M < 1 || N < 1 || K < 1) return fail(SWIFTKV_ERR_INVALID_ARG, "bad argument");
  if (((uintptr_t)A | (uintptr_t)B | (uintptr_t)C) & 15) return fail(SWIFTKV_ERR_INVALID_ARG, "pointers must be 16-byte aligned");
  if (!tc_gemm_tf32_supported(M, N, K)) return fail(SWIFTKV_ERR_UNSUPPORTED, "needs K %% 32 == 0 and N %% 128 == 0");
  unsigned int *status = op_status_word();
  if (!status) return fail(SWIFTKV_ERR_CUDA, "no status word");
  int rc = launch_gemm_tc_tf32(A, B, M, N, K, C, accumulate != 0, status, reinterpret_cast<cudaStream_t>(cuda_stream));
  if (rc) return fail(rc, "launch failed: %s", cudaGetErrorString(cudaGetLastError()));
  return SWIFTKV_OK;
}

extern "C" int32_t swiftkv_gemm_tc_split(const void *A2, const void *B, float *C, int32_t M, int32_t N, int32_t K,
                                         void *cuda_stream) {
  if (!A2 || !B || !C || M < 1 || N < 1 || K < 1) return fail(SWIFTKV_ERR_INVALID_ARG, "bad argument");
  if (((uintptr_t)A2 | (uintptr_t)B | (uintptr_t)C) & 15) return fail(SWIFTKV_ERR_INVALID_ARG, "pointers must be 16-byte aligned");
  if (!tc_gemm_supported(M, N, K)) return fail(SWIFTKV_ERR_UNSUPPORTED, "needs K %% 64 == 0 and N %% 128 == 0");
  unsigned int *status = op_status_word();
  if (!status) return fail(SWIFTKV_ERR_CUDA, "no status word");
  const GemmSplit split{true, nullptr, nullptr};
  int rc = launch_gemm_tc(A2, true, M, K, B, N, nullptr, 0, nullptr, 0, out_plain(OUT_RESID_ADD_F32, C, N, N), nullptr, 0, nullptr,
                          status, reinterpret_cast<cudaStream_t>(cuda_stream), &split);
  if (rc) return fail(rc, "launch failed: %s", cudaGetErrorString(cudaGetLastError()));
  return SWIFTKV_OK;
}

extern "C" int32_t swiftkv_attention_prefill_split(const void *q_hi, const void *q_lo, const void *k_hi, const void *k_lo,
                                                   const void *v, void *out, int32_t out_split, const int32_t *cu_seqlens,
                                                   int32_t n_seqs, int32_t total_tokens, int32_t max_seq_len, int32_t n_q_heads,
                                                   int32_t n_kv_heads, int32_t head_dim, void *cuda_stream) {
  if (!q_hi || !q_lo || !k_hi || !k_lo || !v || !out || !cu_seqlens) return fail(SWIFTKV_ERR_INVALID_ARG, "null argument");
  if (n_seqs < 1 || total_tokens < 1 || max_seq_len < 1 || n_q_heads < 1 || n_kv_heads < 1 || n_q_heads % n_kv_heads)
    return fail(SWIFTKV_ERR_INVALID_ARG, "bad shape");
  if (!tc_attention_supported(n_q_heads, n_kv_heads, head_dim))
    return fail(SWIFTKV_ERR_UNSUPPORTED, "needs head_dim 128 and an even number of query heads per KV head");
  unsigned int *status = op_status_word();
  if (!status) return fail(SWIFTKV_ERR_CUDA, "no status word");
  int rc = launch_attention_tc_split(q_hi, q_lo, k_hi, k_lo, v, out, out_split != 0, cu_seqlens, n_seqs, total_tokens, max_seq_len,
                                     n_q_heads, n_kv_heads, head_dim, status, reinterpret_cast<cudaStream_t>(cuda_stream));
  if (rc) return fail(rc, "attention launch failed");
  return SWIFTKV_OK;
}

extern "C" int32_t swiftkv_attention_prefill(const void *q, const void *k, const void *v, void *out,
                                             const int32_t *cu_seqlens, int32_t n_seqs, int32_t total_tokens,
                                             int32_t max_seq_len, int32_t n_q_heads, int32_t n_kv_heads,
                                             int32_t head_dim, int32_t q_dtype, int32_t kv_dtype,
                                             int32_t use_tensor_cores, void *cuda_stream) {
  if (!q || !k || !v || !out || !cu_seqlens) return fail(SWIFTKV_ERR_INVALID_ARG, "null argument");
  if (n_seqs < 1 || total_tokens < 1 || n_q_heads < 1 || n_kv_heads < 1 || n_q_heads % n_kv_heads || head_dim < 2 || head_dim > 256)
    return fail(SWIFTKV_ERR_INVALID_ARG, "bad shape");
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  const bool q16 = q_dtype == SWIFTKV_DTYPE_BF16 || q_dtype == SWIFTKV_DTYPE_F16;
  if (use_tensor_cores) {
    if (kv_dtype != q_dtype || !q16 || !tc_attention_supported(n_q_heads, n_kv_heads, head_dim))
      return fail(SWIFTKV_ERR_UNSUPPORTED, "tensor-core attention needs q, K, V of one 16-bit type, head_dim 128, an even group size");
    unsigned int *status = op_status_word();
    if (!status) return fail(SWIFTKV_ERR_CUDA, "no status word");
    int rc = launch_attention_tc(q, q_dtype == SWIFTKV_DTYPE_F16, k, v, out, cu_seqlens, nullptr, nullptr, nullptr, 0, n_seqs,
                                 total_tokens, total_tokens, max_seq_len, n_q_heads, n_kv_heads, head_dim, status, st);
    if (rc) return fail(rc, "attention launch failed");
    return SWIFTKV_OK;
  }
  if (q_dtype == SWIFTKV_DTYPE_BF16 && kv_dtype == SWIFTKV_DTYPE_BF16)
    launch_attention_simple<bf16, bf16>((const bf16 *)q, (const bf16 *)k, (const bf16 *)v, (bf16 *)out, cu_seqlens, n_seqs, nullptr, nullptr, nullptr, 0,
                                        total_tokens, n_q_heads, n_kv_heads, head_dim, st);
  else if (q_dtype == SWIFTKV_DTYPE_F16 && kv_dtype == SWIFTKV_DTYPE_BF16)
    launch_attention_simple<__half, bf16>((const __half *)q, (const bf16 *)k, (const bf16 *)v, (__half *)out, cu_seqlens, n_seqs,
                                          nullptr, nullptr, nullptr, 0, total_tokens, n_q_heads, n_kv_heads, head_dim, st);
  else if (q_dtype == SWIFTKV_DTYPE_F32 && kv_dtype == SWIFTKV_DTYPE_F32)
    launch_attention_simple<float, float>((const float *)q, (const float *)k, (const float *)v, (float *)out, cu_seqlens, n_seqs,
                                          nullptr, nullptr, nullptr, 0, total_tokens, n_q_heads, n_kv_heads, head_dim, st);
  else
    return fail(SWIFTKV_ERR_INVALID_ARG, "unsupported dtype combination");
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail(SWIFTKV_ERR_CUDA, "launch failed: %s", cudaGetErrorString(e));
  return SWIFTKV_OK;
}

extern "C" size_t swiftkv_tail_attention_scratch_bytes(int32_t n_seqs, int32_t n_q_heads, int32_t head_dim,
                                                       int32_t max_seq_len) {
  if (n_seqs < 1 || n_q_heads < 1 || head_dim < 1 || max_seq_len < 1) return 0;
  return tail_attention_scratch_bytes(n_seqs, n_q_heads, head_dim, max_seq_len);
}

extern "C" int32_t swiftkv_tail_attention(const float *q, const void *k_cache, const void *v_cache, float *out,
                                          const int32_t *cu_seqlens, int32_t n_seqs, int32_t max_seq_len,
                                          int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim, int32_t dtype,
                                          void *scratch, size_t scratch_bytes, void *cuda_stream) {
  if (!q || !k_cache || !v_cache || !out || !cu_seqlens || !scratch) return fail(SWIFTKV_ERR_INVALID_ARG, "null argument");
  if (n_seqs < 1 || n_seqs > MAX_TAIL_ROWS || max_seq_len < 1 || n_q_heads < 1 || n_kv_heads < 1 || n_q_heads % n_kv_heads ||
      head_dim < 2 || head_dim > 256)
    return fail(SWIFTKV_ERR_INVALID_ARG, "bad shape (n_seqs must be in [1, %d])", MAX_TAIL_ROWS);
  if (scratch_bytes < tail_attention_scratch_bytes(n_seqs, n_q_heads, head_dim, max_seq_len))
    return fail(SWIFTKV_ERR_WORKSPACE_SMALL, "scratch %zu < %zu bytes", scratch_bytes,
                tail_attention_scratch_bytes(n_seqs, n_q_heads, head_dim, max_seq_len));
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  if (dtype == SWIFTKV_DTYPE_BF16)
    launch_tail_attention<bf16>(q, (const bf16 *)k_cache, (const bf16 *)v_cache, nullptr, nullptr, out, cu_seqlens, nullptr, nullptr, 0, n_seqs, max_seq_len, n_q_heads,
                                n_kv_heads, head_dim, (float *)scratch, st);
  else if (dtype == SWIFTKV_DTYPE_F32)
    launch_tail_attention<float>(q, (const float *)k_cache, (const float *)v_cache, nullptr, nullptr, out, cu_seqlens, nullptr, nullptr, 0, n_seqs, max_seq_len,
                                 n_q_heads, n_kv_heads, head_dim, (float *)scratch, st);
  else
    return fail(SWIFTKV_ERR_INVALID_ARG, "unknown dtype");
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail(SWIFTKV_ERR_CUDA, "launch failed: %s", cudaGetErrorString(e));
  return SWIFTKV_OK;
}

extern "C" int32_t swiftkv_quantize_rows_fp8(const float *x, int32_t rows, int32_t width, uint8_t *codes, float *scales,
                                             float *deq, void *cuda_stream) {
  if (!x || !codes || !scales) return fail(SWIFTKV_ERR_INVALID_ARG, "null argument");
  if (rows < 1 || width < 1) return fail(SWIFTKV_ERR_INVALID_ARG, "rows and width must be positive");
  launch_quantize_rows_fp8<float, float>(x, rows, width, nullptr, codes, scales, deq, reinterpret_cast<cudaStream_t>(cuda_stream));
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail(SWIFTKV_ERR_CUDA, "launch failed: %s", cudaGetErrorString(e));
  return SWIFTKV_OK;
}

extern "C" int32_t swiftkv_tail_attention_fp8(const float *q, const uint8_t *k_codes, const uint8_t *v_codes, const float *k_scale,
                                              const float *v_scale, float *out, const int32_t *cu_seqlens, int32_t n_seqs,
                                              int32_t max_seq_len, int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim,
                                              void *scratch, size_t scratch_bytes, void *cuda_stream) {
  if (!q || !k_codes || !v_codes || !k_scale || !v_scale || !out || !cu_seqlens || !scratch) return fail(SWIFTKV_ERR_INVALID_ARG, "null argument");
  if (n_seqs < 1 || n_seqs > MAX_TAIL_ROWS || max_seq_len < 1 || n_q_heads < 1 || n_kv_heads < 1 || n_q_heads % n_kv_heads ||
      head_dim < 4 || head_dim > 256 || head_dim % 4)
    return fail(SWIFTKV_ERR_INVALID_ARG, "bad shape (n_seqs must be in [1, %d], head_dim a multiple of 4)", MAX_TAIL_ROWS);
  if (scratch_bytes < tail_attention_scratch_bytes(n_seqs, n_q_heads, head_dim, max_seq_len))
    return fail(SWIFTKV_ERR_WORKSPACE_SMALL, "scratch %zu < %zu bytes", scratch_bytes,
                tail_attention_scratch_bytes(n_seqs, n_q_heads, head_dim, max_seq_len));
  launch_tail_attention<fp8e4>(q, (const fp8e4 *)k_codes, (const fp8e4 *)v_codes, k_scale, v_scale, out, cu_seqlens, nullptr, nullptr, 0,
                               n_seqs, max_seq_len, n_q_heads, n_kv_heads, head_dim, (float *)scratch,
                               reinterpret_cast<cudaStream_t>(cuda_stream));
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail(SWIFTKV_ERR_CUDA, "launch failed: %s", cudaGetErrorString(e));
  return SWIFTKV_OK;
}
