/*
 * swiftkv.h -- C ABI of the SwiftKV prefill library for NVIDIA B200 (sm_100a).
 *
 * The library runs the prefill of a Llama-style decoder (RMSNorm, rotary embedding, causal grouped-query
 * attention, SwiGLU MLP; paper Sec. 3.1) re-wired by SwiftKV:
 *   - SingleInputKV (Sec. 3.2, Eq. 2): layers 1..l run unchanged on every prompt token; the output of
 *     layer l (the paper's x_{l+1}) is projected ONCE through the K/V projections of every later layer,
 *     which fills their KV caches; prompt tokens skip every other operation of layers l+1..L.
 *   - AcrossKV (Sec. 3.3): groups of g consecutive later layers share the K/V computed by the first layer of
 *     the group and one cache allocation.
 *   - The last token of each prompt continues through layers l+1..L to give the first output token's
 *     logits (footnote of Sec. 3.2; Sec. 3.5: only the tokens that must produce output are propagated).
 *   - The K/V projections of all later layers run as a single fused GEMM over a concatenated weight with
 *     each layer's input-norm gain folded in (Sec. 3.5).
 *
 * Conventions
 *   - Every function returns an int32 status (SWIFTKV_OK = 0, errors < 0), never throws, never aborts.
 *     swiftkv_last_error() returns a thread-local description of the last failure in this thread.
 *   - "device" pointers are CUDA device memory of the current device; "host" pointers are ordinary host
 *     memory.  All buffers are CALLER-OWNED; the library allocates no device memory.  Device buffers must be
 *     256-byte aligned unless stated.
 *   - Weight matrices are [out_features, in_features] row-major in the model dtype (bf16 or fp32), gains
 *     are vectors in the model dtype.  They must outlive the model and are never written by the library.
 *   - swift_layer l is a COUNT: layers 1..l (0-based 0..l-1) run on all tokens; l = n_layers is the
 *     unmodified model.  acrosskv_group g >= 1; groups are aligned at layer l+1; a short last group is allowed.
 *   - Work is queued on the CUDA stream passed to swiftkv_prefill and is not synchronised by the library
 *     unless stated; results are ordered after that stream.
 */
#ifndef SWIFTKV_H_
#define SWIFTKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SWIFTKV_OK                    0
#define SWIFTKV_ERR_INVALID_ARG      -1
#define SWIFTKV_ERR_WORKSPACE_SMALL  -2
#define SWIFTKV_ERR_NOT_READY        -3
#define SWIFTKV_ERR_CUDA             -4
#define SWIFTKV_ERR_DEVICE_TIMEOUT   -5   /* a bounded wait inside a kernel ran out                      */
#define SWIFTKV_ERR_BAD_TOKEN        -6   /* a token id outside [0, vocab) was met on the device         */
#define SWIFTKV_ERR_UNSUPPORTED      -7
#define SWIFTKV_ERR_ACT_OVERFLOW     -8   /* a value beyond the IEEE-half range was clamped (SWIFTKV_ACT_F16)   */

#define SWIFTKV_DTYPE_F32  0
#define SWIFTKV_DTYPE_BF16 1
#define SWIFTKV_DTYPE_F16  2   /* IEEE half: only as the activation type of the stand-alone operators */
#define SWIFTKV_DTYPE_FP8_E4M3 3   /* element type of the FP8 cache's code planes (see SWIFTKV_KV_FP8)      */

typedef struct swiftkv_model swiftkv_model;   /* opaque, library-owned host object */

typedef struct {
  int32_t vocab, hidden, n_layers, n_q_heads, n_kv_heads, head_dim, ffn;
  float   rope_theta, rms_eps;
  int32_t dtype;                               /* SWIFTKV_DTYPE_F32 / BF16: storage type of weights, activations, KV cache */
  int32_t kv_format;                           /* SWIFTKV_KV_*: how cache rows are stored                          */
} swiftkv_config;

/*
 * Cache formats.  SWIFTKV_KV_MODEL_DTYPE: rows in the model dtype.  SWIFTKV_KV_FP8: the per-token FP8 cache that the
 * paper combines with AcrossKV (appendix "KV quantization"; 62.5 % / 68.75 % cache reduction with 2- / 4-way sharing):
 * every token's K row and V row ([n_kv_heads * head_dim] values) of a layer is stored as e4m3 codes (1 sign, 4
 * exponent bits with bias 7, 3 mantissa bits, finite only, largest value 448) plus one fp32 scale,
 *     scale = max(max|x|, 2^-64) / 448,   code = e4m3(x / scale)   (fp32, round to nearest even, saturating),
 * and every attention read -- the prefill attention of layers <= l included -- sees value(code) * scale, so chunked
 * and one-shot prefill stay identical.  A cache slot is then  K codes | V codes | K scales | V scales  (each part
 * padded to 256 bytes); swiftkv_workspace_bytes and swiftkv_kv_cache_view account for it.
 */
#define SWIFTKV_KV_MODEL_DTYPE 0
#define SWIFTKV_KV_FP8         1

typedef struct {                               /* one decoder layer; all device pointers                */
  const void *in_norm;                         /* [hidden]                 gain of the input RMSNorm    */
  const void *wq, *wk, *wv;                    /* [n_q*hd, hidden], [n_kv*hd, hidden] x 2               */
  const void *wo;                              /* [hidden, n_q*hd]                                      */
  const void *post_norm;                       /* [hidden]                 gain of the post-attention RMSNorm */
  const void *w_gate, *w_up;                   /* [ffn, hidden] x 2                                     */
  const void *w_down;                          /* [hidden, ffn]                                         */
} swiftkv_layer_weights;

typedef struct {
  const void *embed;                           /* device [vocab, hidden]                                */
  const void *final_norm;                      /* device [hidden]                                       */
  const void *lm_head;                         /* device [vocab, hidden]                                */
  const swiftkv_layer_weights *layers;         /* HOST array of n_layers entries (copied by model_load) */
} swiftkv_weights;

/* Library version (major*10000 + minor*100 + patch). */
int32_t swiftkv_version(void);

/* Thread-local text of the last error raised in the calling thread ("" if none). */
const char *swiftkv_last_error(void);

/*
 * Bytes the caller must provide for a model that will prefill at most max_tokens packed prompt tokens in at
 * most max_seqs prompts with (swift_layer, acrosskv_group).
 *   workspace_bytes : activations, metadata, the RoPE table, the folded SingleInputKV weight (Sec. 3.5).
 *   kv_cache_bytes  : (l + ceil((L-l)/g)) cache slots of 2 * max_tokens * n_kv*hd elements: layers of one
 *                     AcrossKV group share one slot, which is how the memory saving of Sec. 3.3 is realised
 *                     ((L-l)/L * (1-1/g) of the unmodified model's cache when g divides L-l).
 * A model loaded with these sizes also accepts any later (l', g') whose needs do not exceed them.
 * Errors: INVALID_ARG (null pointers, non-positive sizes, l outside [1, L], g < 1, n_q % n_kv != 0, odd head_dim).
 */
int32_t swiftkv_workspace_bytes(const swiftkv_config *cfg, int32_t max_tokens, int32_t max_seqs,
                                int32_t swift_layer, int32_t acrosskv_group,
                                size_t *workspace_bytes, size_t *kv_cache_bytes);

/*
 * Create a model over caller-owned device buffers.  Records the (borrowed) weight pointers and fills the RoPE
 * table (cos/sin of p * theta^(-2i/hd), evaluated in
 * double precision, rotate-half pairing (i, i + hd/2)) on the current device's default stream, then
 * synchronises that stream.  The device current at this call is the model's device.
 * Errors: INVALID_ARG (as above, or a null / misaligned pointer), WORKSPACE_SMALL, CUDA.
 */
int32_t swiftkv_model_load(const swiftkv_config *cfg, const swiftkv_weights *weights,
                           void *workspace, size_t workspace_bytes,
                           void *kv_cache, size_t kv_cache_bytes,
                           int32_t max_tokens, int32_t max_seqs, swiftkv_model **out);

/*
 * SwiftKV prefill of a packed batch (Sec. 3.2 Eq. 2, Sec. 3.3, Sec. 3.5).
 *   tokens   : HOST int32 [sum(seq_lens)], prompt-major; ids in [0, vocab)
 *   seq_lens : HOST int32 [n_seqs], each >= 1
 * Copies the ids to the device on `cuda_stream` (a cudaStream_t, may be 0), then queues every kernel of the
 * path on that stream and returns without synchronising.  After the stream completes, the KV cache of every
 * layer holds K (after RoPE) and V of every prompt token and the first-token logits are available.
 * The first call with a new (swift_layer, acrosskv_group) also folds and concatenates the later layers' K/V
 * weights (once; cached until another pair is used).
 * Errors: INVALID_ARG (l, g, n_seqs, lengths, token range, totals beyond max_tokens / max_seqs),
 *         WORKSPACE_SMALL ((l, g) needs more than the model was sized for), CUDA.
 */
int32_t swiftkv_prefill(swiftkv_model *m, const int32_t *tokens, const int32_t *seq_lens, int32_t n_seqs,
                        int32_t swift_layer, int32_t acrosskv_group, void *cuda_stream);

/*
 * Same, with the token ids already resident on the device (DEVICE int32 [sum(seq_lens)]); seq_lens stays a
 * HOST array.  Ids cannot be range-checked on the host: a bad id is clamped, recorded in the device status
 * word and reported by swiftkv_status() as SWIFTKV_ERR_BAD_TOKEN.
 */
int32_t swiftkv_prefill_device_tokens(swiftkv_model *m, const int32_t *tokens_dev, const int32_t *seq_lens,
                                      int32_t n_seqs, int32_t swift_layer, int32_t acrosskv_group,
                                      void *cuda_stream);

/*
 * One sequence's part of a mixed minibatch (Sec. 3.5: "chunks of prefill tokens and decode tokens in each minibatch").
 */
typedef struct {
  int32_t n_new;       /* new tokens of this sequence in this step (>= 1): a prefill chunk, or 1 for a decode token   */
  int32_t n_past;      /* tokens of this sequence already in the cache (0 for the first chunk of a prompt)            */
  int32_t cache_row;   /* first row of the sequence's region in every cache plane: token p of the sequence lives in
                          row cache_row + p.  Regions of different sequences must not overlap and must end inside
                          max_tokens; the caller keeps a sequence's region fixed for the sequence's lifetime        */
  int32_t emit;        /* != 0: the last new token continues through layers l+1..L and gets logits (every decode
                          token; the last chunk of a prompt)                                                         */
  const int32_t *block_table;   /* paged cache (optional, HOST array): page numbers of this sequence; token p lives in
                          row block_table[p / 128] * 128 + p % 128 of every cache plane and cache_row is ignored.
                          Pages are SWIFTKV_PAGE_ROWS = 128 rows; a page belongs to one sequence; either every sequence
                          of a step has a table or none has.  With AcrossKV the layers of a group share the pages
                          (one slot per group), which is how an allocator turns the grouping into memory savings.  */
  int32_t n_blocks;    /* entries of block_table; must cover n_past + n_new tokens                                  */
} swiftkv_seq_step;
#define SWIFTKV_PAGE_ROWS 128

/*
 * One forward pass over a mixed minibatch with SwiftKV (Sec. 3.5): layers 1..l run on all new tokens, which attend to
 * their sequence's cached tokens and, causally, to themselves; right after layer l the SingleInputKV projection
 * (Eq. 2, with AcrossKV grouping) writes the new tokens' K / V of every later layer into the cache; then only the
 * emitting tokens run layers l+1..L against those caches and produce logits.  A whole-prompt swiftkv_prefill is the
 * special case n_past = 0, packed regions, every sequence emitting.
 *   tokens : HOST int32, the new tokens of all sequences packed in order (sum of n_new)
 *   seqs   : HOST array of n_seqs entries
 * swift_layer and acrosskv_group must stay the same for all steps that share cached state.  Sum of n_new and sum of
 * (n_past + n_new) must not exceed max_tokens.  swiftkv_first_logits afterwards returns one row per emitting
 * sequence, in order (none, n_seqs = 0, for a minibatch of inner prefill chunks in which nobody emits: such a step
 * fills caches only and never touches layers l+1..L); swiftkv_kv_cache_view returns whole planes (index them with
 * cache_row + position).
 * Errors: INVALID_ARG, WORKSPACE_SMALL, CUDA.
 */
int32_t swiftkv_step(swiftkv_model *m, const int32_t *tokens, const swiftkv_seq_step *seqs, int32_t n_seqs,
                     int32_t swift_layer, int32_t acrosskv_group, void *cuda_stream);

/*
 * SimScore (Sec. 3.2, Eq. 1), the paper's measure of how alike the inputs of deeper layers are -- the observation
 * SingleInputKV rests on:  SimScore(x_l) = sum_{j=l+1..L} Similarity(x_l, x_j) / (L - l),  Similarity = the cosine
 * similarity of token i's x_l and x_j averaged over all tokens; x_l is the input of (1-based) layer l of the UNMODIFIED
 * model.  Runs a full-depth prefill of the batch (as swiftkv_prefill with swift_layer = n_layers: caches and logits are
 * filled as a side effect), capturing every layer's input in `scratch` (DEVICE, caller-owned, 256-byte aligned, at least
 * swiftkv_simscore_scratch_bytes(m, total tokens) bytes = n_layers * tokens * hidden * 4 + a little), then reduces.
 *   simscore : DEVICE fp32 [n_layers - 1]; entry l-1 = SimScore(x_l), l = 1 .. n_layers - 1
 *   sim      : nullable, DEVICE fp32 [n_layers][n_layers]; sim[a][b] = Similarity(x_{a+1}, x_{b+1}) (symmetric, 1 on the
 *              diagonal)
 * tokens, seq_lens: HOST arrays as for swiftkv_prefill.  The model's cache must have room for n_layers slots.
 * Errors: INVALID_ARG, WORKSPACE_SMALL, CUDA.
 */
size_t  swiftkv_simscore_scratch_bytes(const swiftkv_model *m, int32_t n_tokens);
int32_t swiftkv_simscore(swiftkv_model *m, const int32_t *tokens, const int32_t *seq_lens, int32_t n_seqs,
                         void *scratch, size_t scratch_bytes, float *sim, float *simscore, void *cuda_stream);

/* Knowledge recovery, Sec. 3.4 Eq. 3 ("Efficient Distillation"; temperature 2.0 in the training details of the appendix):
 * one frozen copy of the model runs in two modes on the same batch --
 *     y_teacher = M(x, SwiftKV = False)   every token through every unmodified layer,
 *     y_student = M(x, SwiftKV = True)    layers > swift_layer re-wired: their K / V come from x_{l+1} through the group
 *                                         leader's input-norm gain and the STUDENT's W_K, W_V (Eq. 2, AcrossKV groups of
 *                                         Sec. 3.3), their queries from the layer's own normalised input through the
 *                                         student's W_Q; in training every prompt token runs every layer --
 * and this call returns the standard distillation loss on the two logit tensors,
 *     loss = T^2 * mean over all prompt tokens of KL( softmax(y_teacher / T) || softmax(y_student / T) ),  T = temperature,
 * and its gradient with respect to the student's W_Q, W_K, W_V of every layer > swift_layer (the only trainable
 * parameters; norm gains and everything else stay frozen).  Layers 1..swift_layer are shared by both modes and run once.
 *   tokens      : DEVICE int32 [sum(seq_lens)], packed prompt-major;  seq_lens: HOST int32 [n_seqs], every prompt >= 1 token
 *   student_w*  : HOST arrays [n_layers] of DEVICE pointers, fp32 [out_features][hidden] like the model's own matrices;
 *                 entries of layers <= swift_layer (0-based index < swift_layer) are ignored and may be null.  With
 *                 acrosskv_group > 1 only the first layer of each group projects K / V: the other layers' student W_K / W_V
 *                 are never read and their gradients are written as zeros.
 *   grad_w*     : HOST arrays [n_layers] of DEVICE pointers, fp32, same shapes, WRITTEN (not accumulated)
 *   loss        : DEVICE fp32 scalar, written
 *   workspace   : DEVICE, caller-owned, 256-byte aligned, >= swiftkv_distill_workspace_bytes(m, total tokens, swift_layer)
 * All data is fp32 whatever the model's dtype: a bf16 model's frozen weights are widened into fp32 copies inside `workspace`
 * first (its size accounts for them: 4 bytes per model parameter), the student's matrices and the gradients are fp32 either
 * way (master weights).  `precision` selects where the GEMMs (projections, data gradients, weight gradients) run:
 * SWIFTKV_DISTILL_FP32 on the CUDA cores; SWIFTKV_DISTILL_TF32X3 on the tensor cores (tcgen05 kind::tf32) with every operand
 * split into two tf32 numbers (x rounded to nearest, and the rounded remainder) and three products per GEMM -- results at fp32 accuracy; SWIFTKV_DISTILL_TF32 one
 * tf32 product per GEMM (operands cut to 10 mantissa bits, gradients good to ~1e-3).  GEMM shapes the tensor-core kernel does
 * not tile (it needs out-features % 128 == 0 and inner dimension % 32 == 0) stay on the CUDA cores.  Attention, norms, SwiGLU,
 * RoPE and the loss are fp32 CUDA-core kernels in every mode.  Gradients repeat bit for bit (no atomics).  The model's prefill state (swiftkv_kv_cache_view,
 * swiftkv_first_logits) is invalid afterwards until the next prefill.  The sequence offsets are copied with a blocking
 * copy after synchronising `cuda_stream`; everything else is queued on it.
 * Errors: INVALID_ARG, WORKSPACE_SMALL, CUDA.
 */
size_t  swiftkv_distill_workspace_bytes(const swiftkv_model *m, int32_t total_tokens, int32_t swift_layer);
#define SWIFTKV_DISTILL_FP32   0   /* every GEMM in fp32 on the CUDA cores */
#define SWIFTKV_DISTILL_TF32X3 1   /* GEMMs on the tensor cores, operands as sums of two tf32 numbers (three products): fp32-grade */
#define SWIFTKV_DISTILL_TF32   2   /* GEMMs on the tensor cores, one tf32 product (10 mantissa bits per operand) */
int32_t swiftkv_distill_grads(swiftkv_model *m, const int32_t *tokens, const int32_t *seq_lens, int32_t n_seqs,
                              int32_t swift_layer, int32_t acrosskv_group, float temperature, int32_t precision,
                              const void *const *student_wq, const void *const *student_wk, const void *const *student_wv,
                              void *const *grad_wq, void *const *grad_wk, void *const *grad_wv, float *loss,
                              void *workspace, size_t workspace_bytes, void *cuda_stream);

/* The update that goes with swiftkv_distill_grads.  The training details of the paper give a learning rate (3e-4), a weight
 * decay (0.05) and a warm-up ratio (5 %) but do not name the optimiser; this is AdamW with decoupled weight decay, one
 * elementwise pass over a parameter tensor (all DEVICE fp32 arrays of n elements; exp_avg / exp_avg_sq are the optimiser
 * state, zero before step 1; step counts from 1; the learning-rate schedule is the caller's):
 *     p <- p (1 - lr wd);  m <- b1 m + (1 - b1) g;  v <- b2 v + (1 - b2) g^2;
 *     p <- p - lr (m / (1 - b1^step)) / (sqrt(v / (1 - b2^step)) + eps).
 * Errors: INVALID_ARG, CUDA. */
int32_t swiftkv_adamw_update(float *param, const float *grad, float *exp_avg, float *exp_avg_sq, int64_t n, int32_t step,
                             float lr, float beta1, float beta2, float eps, float weight_decay, void *cuda_stream);

typedef struct {
  const void *k;            /* device, [n_tokens][n_kv_heads][head_dim], model dtype (FP8 cache: uint8 e4m3
                               codes), AFTER RoPE                                                           */
  const void *v;            /* device, same shape                                                           */
  const float *k_scale;     /* FP8 cache: device fp32 [n_tokens], scale of every K row; else null          */
  const float *v_scale;     /* FP8 cache: device fp32 [n_tokens], scale of every V row; else null          */
  int64_t token_stride;     /* elements between consecutive tokens (= n_kv_heads * head_dim)               */
  int64_t head_stride;      /* elements between consecutive KV heads (= head_dim)                          */
  int32_t n_tokens;         /* rows in use: the packed prompt tokens of the last prefill (prompt-major), or the
                               highest cache row written so far by swiftkv_step                            */
  int32_t dtype;            /* SWIFTKV_DTYPE_* (SWIFTKV_DTYPE_FP8_E4M3 for the FP8 cache)                   */
  int32_t owner_layer;      /* 0-based layer whose projection produced this cache (the AcrossKV group's
                               first layer for layers >= l; the layer itself otherwise)                    */
} swiftkv_kv_view;

/*
 * Borrowed view of one layer's cache after the last prefill (layer is 0-based).  Layers of one AcrossKV
 * group return the SAME pointers.  Valid until the next prefill or free; only ordered after the stream given
 * to that prefill.  Errors: INVALID_ARG, NOT_READY (no prefill yet).
 */
int32_t swiftkv_kv_cache_view(const swiftkv_model *m, int32_t layer, swiftkv_kv_view *out);

/*
 * Borrowed pointer to the first-token logits of the last prefill: DEVICE fp32 [n_seqs][vocab]
 * (final RMSNorm then lm_head on the last token of each prompt).  Errors: INVALID_ARG, NOT_READY.
 */
int32_t swiftkv_first_logits(const swiftkv_model *m, const float **logits, int32_t *n_seqs);

/*
 * Synchronises `cuda_stream` and returns the device status word latched by the kernels of earlier calls:
 * OK, DEVICE_TIMEOUT (a bounded in-kernel wait gave up; results are invalid), ACT_OVERFLOW (with SWIFTKV_ACT_F16 an
 * intermediate activation, a cached K / V value or a weight lay beyond +-65504 and was clamped: results are wrong,
 * select SWIFTKV_ACT_BF16 for this model), BAD_TOKEN, or CUDA.  Clears the word.
 */
int32_t swiftkv_status(swiftkv_model *m, void *cuda_stream);

/*
 * Kernel-class timing.  With profiling enabled, each prefill brackets every launch with CUDA events on the
 * prefill's stream; swiftkv_profile_read synchronises the stream and returns the device time (ms) and launch
 * count accumulated per class since the last read, then resets them.  Classes are SWIFTKV_KC_*.
 */
#define SWIFTKV_KC_GEMM      0   /* QKV / O / down / SingleInputKV GEMMs (M = all prompt tokens)          */
#define SWIFTKV_KC_ATTENTION 1   /* causal varlen GQA prefill attention                                   */
#define SWIFTKV_KC_ELEMWISE  2   /* embedding gather, RMSNorm, RoPE, SwiGLU, gathers, weight fold         */
#define SWIFTKV_KC_TAIL      3   /* last-token path of layers > l and the lm_head                         */
#define SWIFTKV_KC_SWIGLU    4   /* the fused gate/up GEMM + SwiGLU, the single largest kernel            */
#define SWIFTKV_KC_COUNT     5
int32_t swiftkv_profile_enable(swiftkv_model *m, int32_t on);
int32_t swiftkv_profile_read(swiftkv_model *m, void *cuda_stream, float *ms_per_class /*[KC_COUNT]*/,
                             int32_t *launches_per_class /*[KC_COUNT]*/);

/* Number of kernels the last prefill launched. */
int32_t swiftkv_last_launch_count(const swiftkv_model *m);

/* Select kernel families (debug / comparison): bit 0 = tensor-core GEMMs, bit 1 = tensor-core attention,
 * bit 2 = CTA-pair (cta_group::2) form of the projection GEMMs, bit 3 = CTA-pair form of the gate/up GEMM too,
 * bit 4 = the tensor-core attention runs as one persistent CTA per SM over a work list that the host balances from the
 * sequence lengths (longest item first, each to the least loaded CTA) instead of one CTA per work item,
 * bit 5 = decode minibatches (at most 8 sequences, one new token each) run every layer on the weight-streaming
 * kernels of the last-token path instead of 128-row GEMM tiles,
 * bit 6 = the projections of the last-token path between two attention calls (O, gate/up + SwiGLU, down, the next
 * layer's Q or the lm_head, norms folded in) run as ONE persistent cooperative launch (weight rows streamed through a
 * shared-memory ring, grid-wide barriers between the stages) instead of one launch per operator; bf16 models whose
 * hidden, query and FFN widths are multiples of 512.
 * Default 119: everything that the model's shape and dtype support except bit 3.  Returns the mask in effect. */
int32_t swiftkv_set_kernel_mask(swiftkv_model *m, int32_t mask);

/* Storage format of the intermediate activations of a bf16 model (normed hidden states, queries, attention
 * output, SwiGLU output, softmax probabilities) -- never of weights or the KV cache, which stay bf16.
 *   SWIFTKV_ACT_F16  (default): IEEE half, 8x finer rounding than bf16; conversions saturate at +-65504 and every
 *                      clamped store raises SWIFTKV_ERR_ACT_OVERFLOW in swiftkv_status (never silently).  Because
 *                      both operands of a tensor-core MMA must share one 16-bit type, each layer's matrices are
 *                      copied to half right before use (workspace scratch for one layer; exact for |w| >= 2^-17)
 *                      and the current layer's K / V get a half copy beside the bf16 cache.
 *   SWIFTKV_ACT_BF16          : bfloat16 end to end, for checkpoints whose activations exceed the half range.
 * Ignored by fp32 models.  Takes effect at the next prefill. */
#define SWIFTKV_ACT_BF16 0
#define SWIFTKV_ACT_F16  1
/*   SWIFTKV_ACT_F16_SPLIT     : SWIFTKV_ACT_F16 with the error-critical operands of a whole-prompt prefill carried as PAIRS
 *                      of halves, value = hi + lo (~22 significant bits), at the price of extra tensor-core passes:
 *                      a GEMM whose A operand is a pair runs its K loop twice (A_hi B^T + A_lo B^T in one fp32
 *                      accumulator), the attention scores take three passes (Q_hi K_hi^T + Q_lo K_hi^T + Q_hi K_lo^T).
 *                      Which operands: swiftkv_set_split_mask, default SWIFTKV_SPLIT_DEFAULT.  For deep models whose
 *                      softmax is so sharp that the 2^-12 rounding of h, q and K dominates the error of the logits (the
 *                      80-layer 70B shape with random weights misses the 0.1 max-abs bar with plain halves).  Chunked /
 *                      decode steps and the FP8 cache run as SWIFTKV_ACT_F16. */
#define SWIFTKV_ACT_F16_SPLIT 2
int32_t swiftkv_set_activation_format(swiftkv_model *m, int32_t format);

/* Optional room for the half copies of the weights (SWIFTKV_ACT_F16 on a bf16 model).  Without it every prefill / chunk step
 * copies each of its layers' seven matrices to half right before use (one layer of scratch, on a side stream): 2 x 2 bytes
 * per parameter of layers 1..l of HBM traffic per step, noticeable when steps are small (chunks of a few thousand tokens).
 * With a DEVICE buffer of swiftkv_half_weight_cache_bytes(cfg, n) bytes (256-byte aligned, owned by the caller, alive until
 * the model is destroyed or the cache is replaced) the copies of the first n layers are made once, by the first step that
 * needs them, and reused by every later step whose SwiftKV layer l is <= n; a step with l > n falls back to per-step copies.
 * The library cannot see the caller changing the model's weights: call swiftkv_set_half_weight_cache again (same buffer is
 * fine) after updating them, which marks every copy stale.  buffer = NULL, bytes = 0 removes the cache.  The results are
 * bit-identical with and without it.  swiftkv_half_weight_cache_bytes returns -1 for a bad config. */
int64_t swiftkv_half_weight_cache_bytes(const swiftkv_config *cfg, int32_t n_layers);
int32_t swiftkv_set_half_weight_cache(swiftkv_model *m, void *buffer, int64_t bytes);

/* Operands that travel as half pairs under SWIFTKV_ACT_F16_SPLIT (bits; call after swiftkv_set_activation_format):
 *   QKV_INPUT : the normed hidden state that feeds the Q/K/V projections and the SingleInputKV projection (those GEMMs x2)
 *   SCORES    : q and K inside the attention kernel (Q K^T x3)
 *   ATTN_OUT  : the attention output that feeds the O projection (x2; implies the half-pair attention kernel)
 *   MLP_INPUT : the normed hidden state that feeds the gate / up projections (x2)
 *   MLP_ACT   : the SwiGLU output that feeds the down projection (x2) */
#define SWIFTKV_SPLIT_QKV_INPUT 1
#define SWIFTKV_SPLIT_SCORES    2
#define SWIFTKV_SPLIT_ATTN_OUT  4
#define SWIFTKV_SPLIT_MLP_INPUT 8
#define SWIFTKV_SPLIT_MLP_ACT   16
#define SWIFTKV_SPLIT_DEFAULT   (SWIFTKV_SPLIT_QKV_INPUT | SWIFTKV_SPLIT_SCORES | SWIFTKV_SPLIT_ATTN_OUT)
int32_t swiftkv_set_split_mask(swiftkv_model *m, int32_t mask);

/* Failure-detection self-check (no counterpart in the paper).  Every wait inside the kernels is bounded: when it runs out
 * the kernel latches DEVICE_TIMEOUT in the model's status word, every role of the CTA leaves its loop and the kernel
 * returns, so the context stays usable.  This call launches one small CTA that waits, with that same bounded wait but a
 * limit of `limit_clocks` SM clocks (1 .. 1e8, i.e. at most ~50 ms), on a barrier that is never completed, synchronises
 * the stream and writes to HOST outcome[2]: [0] = 1 if the waiting role gave up at its limit, [1] = 1 if a second role
 * of the CTA left through the abort flag.  Afterwards swiftkv_status reports SWIFTKV_ERR_DEVICE_TIMEOUT once.
 * Errors: INVALID_ARG, CUDA. */
int32_t swiftkv_debug_bounded_wait(swiftkv_model *m, int64_t limit_clocks, int32_t *outcome, void *cuda_stream);
/* The same self-check for the persistent cooperative launch of the last-token path (kernel-mask bit 6): two stages of layer
 * 1 are launched on one zero row with every in-kernel wait limited to `limit_clocks` SM clocks (1 .. 1e8) and a grid barrier
 * between them that cannot complete (the host claims one arrival that never happened).  Every CTA's wait runs out, the kernel
 * latches DEVICE_TIMEOUT, raises its abort word, lets the copies in flight land, and returns; the call synchronises the
 * stream.  Afterwards swiftkv_status reports SWIFTKV_ERR_DEVICE_TIMEOUT once and the model needs a new prefill before its
 * cache / logits are read.  bf16 models whose widths the fused launch supports (UNSUPPORTED otherwise).
 * Errors: INVALID_ARG, UNSUPPORTED, CUDA. */
int32_t swiftkv_debug_fused_barrier_wait(swiftkv_model *m, int64_t limit_clocks, void *cuda_stream);

/* Synchronises `cuda_stream`, then returns and clears the current device's status word of the stand-alone operator
 * entry points below (swiftkv_gemm_tc, swiftkv_attention_prefill): OK, DEVICE_TIMEOUT, ACT_OVERFLOW or CUDA. */
int32_t swiftkv_op_status(void *cuda_stream);

/* Destroys the host object (never the caller's buffers).  Null is allowed. */
void swiftkv_model_free(swiftkv_model *m);

/*
 * Stand-alone operator entry points (the same kernels the prefill uses), for unit tests and profiling.
 * All pointers are DEVICE memory; all run on `cuda_stream` without synchronising.
 */

/* C[M,N] = A[M,K] * B[N,K]^T on the tensor cores (tcgen05), fp32 accumulation, row-major, ldc = N.  A, B and C
 * are all of `dtype` (SWIFTKV_DTYPE_BF16 or SWIFTKV_DTYPE_F16; the two operands of one MMA must share a type).
 * Needs K % 64 == 0, N % 128 == 0, 16-byte aligned pointers.  Errors: INVALID_ARG, UNSUPPORTED, CUDA. */
int32_t swiftkv_gemm_tc(const void *A, const void *B, void *C, int32_t M, int32_t N, int32_t K, int32_t dtype,
                        void *cuda_stream);

/* C[M,N] (+)= A[M,K] * B[N,K]^T with fp32 operands on the tensor cores (tcgen05 kind::tf32: sign, exponent and 10 mantissa
 * bits of every operand enter the product; fp32 accumulation), row-major, ldc = N; accumulate != 0 adds to C.  The GEMM
 * form of the knowledge-recovery step's tensor-core mode.  Needs K % 32 == 0, N % 128 == 0, 16-byte aligned pointers.
 * Errors: INVALID_ARG, UNSUPPORTED, CUDA. */
int32_t swiftkv_gemm_tf32(const float *A, const float *B, float *C, int32_t M, int32_t N, int32_t K, int32_t accumulate,
                          void *cuda_stream);

/* The half-pair operand format of SWIFTKV_ACT_F16_SPLIT, stand-alone.  C[M,N] (DEVICE fp32, row-major, ldc = N) +=
 * (A_hi + A_lo) B^T with A2 DEVICE IEEE half [M, 2K], each row [hi(K) | lo(K)], B IEEE half [N, K]; two tensor-core passes
 * into one fp32 accumulator.  Same shape rules as swiftkv_gemm_tc.  Errors: INVALID_ARG, UNSUPPORTED, CUDA. */
int32_t swiftkv_gemm_tc_split(const void *A2, const void *B, float *C, int32_t M, int32_t N, int32_t K, void *cuda_stream);

/* Causal varlen GQA attention (Sec. 3.1) with the scores computed from half pairs: q = q_hi + q_lo [T, n_q, hd] and
 * K = k_hi + k_lo [T, n_kv, hd] (all IEEE half), S = Q_hi K_hi^T + Q_lo K_hi^T + Q_hi K_lo^T; v and out IEEE half;
 * out_split != 0: out is [T, 2 * n_q * hd], each row [hi | lo].  head_dim 128, even n_q / n_kv.
 * Errors: INVALID_ARG, UNSUPPORTED, CUDA. */
int32_t swiftkv_attention_prefill_split(const void *q_hi, const void *q_lo, const void *k_hi, const void *k_lo, const void *v,
                                        void *out, int32_t out_split, const int32_t *cu_seqlens, int32_t n_seqs,
                                        int32_t total_tokens, int32_t max_seq_len, int32_t n_q_heads, int32_t n_kv_heads,
                                        int32_t head_dim, void *cuda_stream);

/* Causal varlen grouped-query attention (Sec. 3.1) on packed prompts.  q [T, n_q, hd] and out [T, n_q*hd] in
 * q_dtype, k, v [T, n_kv, hd] in kv_dtype; cu_seqlens DEVICE int32 [n_seqs+1]; softmax scale 1/sqrt(hd).
 * max_seq_len bounds the longest prompt (grid sizing).  Type pairs: (F32, F32), (BF16, BF16), (F16, BF16) on the
 * SIMT kernel; (BF16, BF16) or (F16, F16), head_dim 128 and an even n_q / n_kv on the tensor-core kernel. */
int32_t swiftkv_attention_prefill(const void *q, const void *k, const void *v, void *out,
                                  const int32_t *cu_seqlens, int32_t n_seqs, int32_t total_tokens,
                                  int32_t max_seq_len, int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim,
                                  int32_t q_dtype, int32_t kv_dtype, int32_t use_tensor_cores, void *cuda_stream);

/* Single-query attention of the last-token path (footnote of Sec. 3.2: the last prompt token still runs every
 * layer; Sec. 3.5: it attends to the caches the SingleInputKV projection filled).  One query per prompt:
 * q DEVICE fp32 [n_seqs, n_q, hd] (already rotated); k_cache, v_cache DEVICE [total_tokens, n_kv, hd] in `dtype`,
 * prompt b occupying rows [cu_seqlens[b], cu_seqlens[b+1]); out DEVICE fp32 [n_seqs, n_q*hd]; softmax scale
 * 1/sqrt(hd).  n_seqs <= 8.  The keys are split across CTAs; `scratch` (DEVICE, caller-owned, at least
 * swiftkv_tail_attention_scratch_bytes(...) bytes, 16-byte aligned) holds the per-split partial results.
 * max_seq_len must bound every prompt's length: cu_seqlens lives on the device and is not checked, and keys beyond
 * the range that max_seq_len's split covers are not read.  A prompt of length 0 gets an all-zero output row.
 * The scratch size is valid for every call with the same n_seqs / heads and any smaller max_seq_len.
 * Errors: INVALID_ARG, WORKSPACE_SMALL (scratch too small), CUDA. */
size_t  swiftkv_tail_attention_scratch_bytes(int32_t n_seqs, int32_t n_q_heads, int32_t head_dim, int32_t max_seq_len);
int32_t swiftkv_tail_attention(const float *q, const void *k_cache, const void *v_cache, float *out,
                               const int32_t *cu_seqlens, int32_t n_seqs, int32_t max_seq_len, int32_t n_q_heads,
                               int32_t n_kv_heads, int32_t head_dim, int32_t dtype, void *scratch, size_t scratch_bytes,
                               void *cuda_stream);

/* The row pass that fills the FP8 cache (SWIFTKV_KV_FP8; appendix "KV quantization", per-token FP8), stand-alone:
 * x DEVICE fp32 [rows, width]; codes DEVICE uint8 [rows, width]; scales DEVICE fp32 [rows];
 * deq (nullable) DEVICE fp32 [rows, width] receives value(code) * scale.  Per row: scale = max(max|x|, 2^-64) / 448,
 * code = e4m3(x / scale), each step one correctly rounded fp32 operation, round to nearest even, saturating --
 * so codes and scales are bit-exact functions of x.  Errors: INVALID_ARG, CUDA. */
int32_t swiftkv_quantize_rows_fp8(const float *x, int32_t rows, int32_t width, uint8_t *codes, float *scales,
                                  float *deq, void *cuda_stream);

/* swiftkv_tail_attention over an FP8 cache: k_codes, v_codes DEVICE uint8 [total_tokens, n_kv, hd], k_scale, v_scale
 * DEVICE fp32 [total_tokens] (one scale per token row and plane); everything else as swiftkv_tail_attention. */
int32_t swiftkv_tail_attention_fp8(const float *q, const uint8_t *k_codes, const uint8_t *v_codes, const float *k_scale,
                                   const float *v_scale, float *out, const int32_t *cu_seqlens, int32_t n_seqs,
                                   int32_t max_seq_len, int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim,
                                   void *scratch, size_t scratch_bytes, void *cuda_stream);

/* (No counterpart in the paper: an integration aid.)
 * swiftkv_tail_attention for callers that must not allocate device memory and have no spare buffer to lend --
 * for example a plug-in running inside a serving process whose memory pool is fully committed to weights and KV
 * cache, or code running where cudaMalloc is forbidden (between a stream-capture begin/end, in a latency-critical
 * loop, under a memory-accounting harness).  Same arguments and result as swiftkv_tail_attention minus the
 * scratch pair: the per-split partial results live in a fixed array inside the library's device image instead.
 *   - Limit: that array is SWIFTKV_NOALLOC_SCRATCH_BYTES (9 MiB); it exists once per GPU that loads the library
 *     and stays until the process exits.  A call whose partials need more (see
 *     swiftkv_tail_attention_scratch_bytes) is rejected with SWIFTKV_ERR_WORKSPACE_SMALL and does nothing.
 *   - The first call on each device looks up the array's device address (no allocation); make that first call
 *     outside any stream capture.
 *   - The array is shared by every call in the process and keeps whatever the previous call left; each call
 *     overwrites every entry it later reads, so nothing needs clearing, but two calls that overlap on the GPU
 *     (different streams, or different host threads) race on it: serialise them.
 *   - Calls no cudaMalloc / cudaFree and no allocating library routine.
 * Errors: INVALID_ARG, WORKSPACE_SMALL, CUDA. */
#define SWIFTKV_NOALLOC_SCRATCH_BYTES (9u * 1024u * 1024u)
int32_t swiftkv_tail_attention_noalloc(const float *q, const void *k_cache, const void *v_cache, float *out,
                                       const int32_t *cu_seqlens, int32_t n_seqs, int32_t max_seq_len,
                                       int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim, int32_t dtype,
                                       void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* SWIFTKV_H_ */
