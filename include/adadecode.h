/*
 * adadecode.h - C ABI of the B200 (sm_100a) layer-parallel decode library.
 *
 * The library implements the decoding loop of AdaDecode (Algorithm 1 of the paper): the newest
 * token climbs the decoder layers while the deferred upper layers of earlier early-predicted
 * tokens are processed alongside it; at chosen intermediate layers a lightweight head
 * (Section 2.1) predicts the next token and, if its probability exceeds a threshold (Eq. 1),
 * the token is emitted early; when the newest token reaches the last layer every early token
 * is verified against the full-depth argmax (Eq. 2 at temperature zero, Appendix D) and the
 * first mismatch rolls the sequence and the KV cache back.  Plain greedy decoding (Table 2,
 * "Vanilla Decoding") runs through the same kernels with one row and no heads.
 *
 * Conventions
 *   - Every function returns 0 (ADA_OK) or a negative ADA_E* code; nothing throws, aborts or
 *     traps the GPU.  ada_strerror() names a code; ada_last_cuda_error() returns the CUDA error
 *     string saved by the last ADA_ECUDA on the calling thread.
 *   - "dev" pointers are device memory owned by the CALLER (allocated e.g. through PyTorch); the
 *     library borrows them and they must outlive the object they were given to.  "host" pointers
 *     are ordinary host memory.  The library never allocates device memory itself: weights it has to
 *     repack go into an arena the caller provides, everything else into the session's scratch.
 *   - All matrices are row-major [out_features, in_features]; every tensor of a model has the
 *     model's dtype (fp32 or bf16 bit patterns).
 *   - One session is used from one host thread at a time.  All device work of a session is issued
 *     on the CUDA stream given at creation.
 */
#ifndef ADADECODE_H
#define ADADECODE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ADA_OK 0
#define ADA_EINVAL (-1)       /* bad argument */
#define ADA_ESTATE (-2)       /* call order (e.g. decode before prefill, tensor missing) */
#define ADA_ECAPACITY (-3)    /* KV pool, max_seq_len, max_early or scratch too small */
#define ADA_ECUDA (-4)        /* a CUDA call failed; see ada_last_cuda_error() */
#define ADA_ETIMEOUT (-5)     /* a bounded device-side wait expired */
#define ADA_EUNSUPPORTED (-6) /* shape or dtype outside what the kernels are built for */

#define ADA_DTYPE_FP32 0
#define ADA_DTYPE_BF16 1

#define ADA_MAX_BATCH 16
#define ADA_MAX_LAYERS 256
#define ADA_PROF_CLASSES 12

typedef struct ada_model ada_model;     /* opaque */
typedef struct ada_session ada_session; /* opaque: sequences, paged KV metadata, in-flight state */

/* Decoder shape (the Llama family the paper evaluates, Section 3).  d_model, d_ff and
   n_q_heads*head_dim must be multiples of 8; head_dim a multiple of 32, at most 256;
   n_q_heads a multiple of n_kv_heads. */
typedef struct {
    int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ff, vocab;
    int32_t dtype;        /* ADA_DTYPE_* of every tensor, of the activations fed to the GEMMs and of the KV cache */
    int32_t tied_lm_head; /* 1: the LM head E* aliases tok_embed */
    float rope_base, rms_eps;
} ada_config;

/* Counters of one or more decode calls (accumulated into the struct the caller passes).
   Definitions: a "step" is one iteration of Algorithm 1's while loop for one sequence; the
   early-exit rate is early_exits / steps; the rejection rate is rejected / (accepted + rejected);
   early predictions behind a rejection were never examined and count as discarded. */
typedef struct {
    int64_t steps, head_evals, early_exits, verify_steps, accepted, rejected, discarded;
    int64_t row_layers;      /* sum over processed layers of the rows processed there */
    int64_t truncated;       /* verified tokens dropped to end a call on the requested count */
    int64_t exits_at_layer[ADA_MAX_LAYERS]; /* indexed by 1-based exit layer */
    int64_t layer_passes;    /* decoder-layer passes launched (each streams one layer's weights once) */
    int64_t host_syncs;      /* stream synchronisations the decode loop needed */
    int64_t kernel_launches; /* kernels of this library launched by the decode calls */
    double decode_ms;        /* device time of the decode calls (CUDA events on the session stream) */
    int64_t emitted[ADA_MAX_BATCH]; /* tokens returned per sequence (fewer than asked for only after an end-of-sequence token) */
    int64_t finished;        /* sequences that ended on a verified end-of-sequence token during these calls */
    int64_t path;            /* decode path of the last call: 1 = persistent kernel, 0 = one kernel per operation */
} ada_stats;

const char *ada_strerror(int code);
const char *ada_last_cuda_error(void);

/* ---- model: "load weights" -------------------------------------------------------------- */

int ada_model_create(const ada_config *cfg, ada_model **out);

/* Lend one tensor (device pointer, exact byte size checked).  Names:
 *   tok_embed [vocab, d]         final_norm [d]          lm_head [vocab, d] (only if not tied)
 *   layers.N.attn_norm [d]       layers.N.ffn_norm [d]
 *   layers.N.wq [n_q head_dim, d]    layers.N.wk, layers.N.wv [n_kv head_dim, d]
 *   layers.N.wo [d, n_q head_dim]
 *   layers.N.w_gate, layers.N.w_up [d_ff, d]
 *   layers.N.w_down [d, d_ff]
 * and, for callers that already hold them stacked (nothing is gained or lost either way):
 *   layers.N.wqkv [(n_q+2 n_kv) head_dim, d]   rows: all q heads, then all k heads, then all v heads
 *   layers.N.w_gate_up [2 d_ff, d]             rows: gate, then up
 * Pointers must be 16-byte aligned. */
int ada_model_set_tensor(ada_model *m, const char *name, const void *dev_ptr, size_t bytes);

/* Repack on load.  The persistent decode kernel finishes q, k and v (rotary embedding, cache write)
 * in the epilogue of the QKV product, which needs the rows of every q and k head in an order that
 * puts the two partners (i, i + head_dim/2) of a rotation into one tensor-core tile.
 * ada_model_finalize() writes that reordered copy of q | k | v of every layer into an arena the
 * caller provides: ada_model_arena_bytes() device bytes, 256-byte aligned, which must outlive the
 * model (0 bytes for models the persistent kernel does not take: fp32, head_dim other than 64 / 128,
 * more than 4 q heads per kv head, d_model / n_q head_dim / d_ff not multiples of 64; such models
 * need no arena).  The lent tensors themselves are never written. */
size_t ada_model_arena_bytes(const ada_model *m);
int ada_model_set_arena(ada_model *m, void *arena_dev, size_t bytes);

/* Register the intermediate head of Section 2.1 at 1-based `layer` (1 <= layer < n_layers):
 * logits = logit_scale * E* (T RMSNorm_f(h)), E^(i) = E* T^(i).  T_dev is a dense [d, d] matrix in
 * the model dtype, or NULL for T = I. */
int ada_model_set_exit_head(ada_model *m, int32_t layer, const void *T_dev, float logit_scale);

/* Checks that every tensor is present and repacks into the arena (on the device that is current;
 * synchronises that device).  ADA_ESTATE if a tensor or a required arena is missing. */
int ada_model_finalize(ada_model *m);
void ada_model_destroy(ada_model *m);

/* ---- session ------------------------------------------------------------------------------ */

/* Device bytes of scratch a session needs (activations, partial results, state; no KV). */
size_t ada_session_scratch_bytes(const ada_model *m, int32_t batch, int32_t max_seq_len, int32_t max_early);
/* Device bytes of one KV page (page_tokens positions, all layers, K and V). */
size_t ada_kv_page_bytes(const ada_model *m, int32_t page_tokens);

/* Create a session of `batch` independent sequences.  kv_pool_dev holds kv_pool_bytes /
 * ada_kv_page_bytes() pages that the session hands to sequences on demand; page_tokens is a power
 * of two in [16, 256].  max_early bounds the early predictions in flight per sequence (the paper
 * uses 5).  scratch_dev must be 256-byte aligned and at least ada_session_scratch_bytes() long;
 * the session zero-fills what it needs of it.  cuda_stream is a cudaStream_t (0 = default). */
int ada_session_create(const ada_model *m, int32_t batch, int32_t max_seq_len, int32_t page_tokens,
                       int32_t max_early, void *kv_pool_dev, size_t kv_pool_bytes, void *scratch_dev,
                       size_t scratch_bytes, void *cuda_stream, ada_session **out);
void ada_session_destroy(ada_session *s);
/* Forget sequence `seq` (or all sequences if seq < 0) and return its pages to the pool. */
int ada_session_reset(ada_session *s, int32_t seq);

/* KV cache <- LM(x) (first line of Algorithm 1): runs the n_prompt tokens of sequence `seq`
 * through all layers (prompts of 32 tokens or more in dense blocks of 128 positions, see ada_debug_set_prefill).  The first generated token (full-depth argmax at the last prompt token)
 * becomes the sequence's pending token.  ADA_ECAPACITY if pages or max_seq_len do not suffice. */
int ada_prefill(ada_session *s, int32_t seq, const int32_t *prompt_host, int32_t n_prompt);

/* Both decode calls return the NEXT n_tokens verified generated tokens of every sequence into
 * out_host[batch][n_tokens] (counting from the first generated token, which prefill produced),
 * synchronise the stream before returning, and leave the same logical state: K/V present at all
 * layers for every token before the last returned one, which stays pending.  Calls can be chained
 * and mixed.  Every sequence must have been prefilled.
 *
 * eos_id (Algorithm 1: "while t_i != [EOS]"): a token id, or -1 for none.  A sequence ends at its first
 * VERIFIED end-of-sequence token, i.e. one that is the full-depth argmax; an early-predicted one stops
 * nothing until the verification accepts it.  The row of a sequence that ended holds its tokens up to
 * and including that token, then eos_id up to n_tokens; stats->emitted[seq] counts the real ones.
 * Later calls return only padding for it, and ADA_ESTATE once every sequence of the session has
 * ended (ada_prefill or ada_session_reset starts a sequence afresh). */
int ada_plain_decode(ada_session *s, int32_t n_tokens, int32_t eos_id, int32_t *out_host, ada_stats *stats /* nullable */);

/* Algorithm 1.  threshold = gamma of Eq. 1 (strict: exit iff p > gamma).  exit_layers: ascending
 * 1-based layers, each < n_layers, each with a registered head.  max_early <= the session's. */
int ada_adaptive_decode(ada_session *s, int32_t n_tokens, float threshold, const int32_t *exit_layers,
                        int32_t n_exit_layers, int32_t max_early, int32_t eos_id, int32_t *out_host, ada_stats *stats);

/* Algorithm 1 with SAMPLED tokens (Eq. 1: "any sampling strategy can be employed"; here: the softmax of the head's logits
 * over `temperature` > 0) and the stochastic form of Eq. 2.  At an exit layer the successor t of the newest token is
 * drawn from the head's distribution q and emitted early iff q(t) > threshold.  At the last layer every early-predicted
 * token, in sequence order, is accepted with probability min{1, p*(t) / q(t)} (p* = the full model's distribution at
 * the same temperature); the first one that is not is replaced by a draw from Normalize(max(0, p* - q)), the K/V of
 * everything from its position on is dropped and generation resumes from the replacement; if all are accepted the next
 * token is drawn from p*.  n_exit_layers = 0 is plain sampling.  Draws are inverse-CDF draws in vocabulary order.
 *
 * Every random number is an input (nothing is generated inside the library): uniforms_host[batch][n_pos][8], fp32 in
 * [0, 1), row j of a sequence belonging to the token at sequence position first_pos + j (prompt included):
 * [0] its draw at the last layer, [1] its acceptance test, [2] its resampling, [3 + e] its draw at the e-th exit layer
 * of the call (at most 5 exit layers).  A position drawn again after a rollback uses its numbers again.  Rows must cover
 * every position from each sequence's current length to one past the call's last token; ADA_EINVAL otherwise.
 * With threshold 0 the verified tokens are distributed exactly as plain sampling; for threshold > 0 the draft is
 * consulted only where q(t) > threshold and the law differs slightly from p* (the paper states the rule, not this
 * consequence).  The first token after the prompt is the prompt pass's argmax.  Persistent decode path only
 * (ADA_EUNSUPPORTED otherwise); end-of-sequence handling, return layout and statistics as for ada_adaptive_decode. */
int ada_sampling_decode(ada_session *s, int32_t n_tokens, float temperature, float threshold, const int32_t *exit_layers,
                        int32_t n_exit_layers, int32_t max_early, int32_t eos_id, const float *uniforms_host,
                        int32_t first_pos, int32_t n_pos, int32_t *out_host, ada_stats *stats);

/* ---- test hooks --------------------------------------------------------------------------- */

/* Record the final-layer logits of every verified generated token of sequence 0 into dev_buf
 * [max_tokens][vocab] fp32 (device memory), from the next prefill/decode on; NULL stops. */
int ada_debug_capture_logits(ada_session *s, float *dev_buf, int32_t max_tokens);
int ada_debug_logits_captured(ada_session *s, int32_t *n_out);
/* Record every intermediate-head evaluation as 4 floats (step, layer, token, p) into host_buf
 * (copied at the end of each adaptive call); NULL stops. */
int ada_debug_capture_heads(ada_session *s, float *host_buf, int32_t max_evals, int32_t *n_out);
/* Force exit decisions: entry i is consumed by the i-th head evaluation of sequence 0 of the next
 * adaptive call; 0 = continue, 1 = exit, other = follow Eq. 1.  Past the end: Eq. 1. */
int ada_debug_set_exit_tape(ada_session *s, const uint8_t *tape_host, int32_t n);
/* Read back per-layer fill levels (positions with valid K/V) and the length of sequence seq. */
int ada_debug_get_state(ada_session *s, int32_t seq, int32_t *len_out, int32_t *fill_out /*[n_layers]*/);
/* Copy K (which=0) or V (which=1) of one cached position of one layer into host_out
 * [n_kv_heads*head_dim] as fp32. */
int ada_debug_read_kv(ada_session *s, int32_t seq, int32_t which, int32_t layer0, int32_t pos, float *host_out);
/* Per-kernel-class device timing (path 0: CUDA events around every launch, which slows the run;
 * path 1: the persistent kernel's own per-phase timers, read in CTA 0, always running).  Classes: 0 step set-up and control, 1 RMSNorm, 2 QKV GEMM, 3 RoPE + KV write, 4 attention,
 * 5 O-proj GEMM, 6 gate/up GEMM, 7 SwiGLU, 8 down GEMM, 9 LM-head stream, 10 head transformation T,
 * 11 other.  ada_debug_profile_read returns, accumulated since profiling was switched on, the device
 * milliseconds, launch counts and algorithmic HBM bytes (weights or KV the launch must read) per class. */
int ada_debug_profile(ada_session *s, int32_t on);
int ada_debug_profile_read(ada_session *s, double *ms_out, int64_t *launches_out, double *bytes_out);
/* Select the decode path: 1 = the persistent kernel (one cooperative launch runs many steps of
 * Algorithm 1; bf16 models, at most 8 tokens per pass, 64-token KV pages, head_dim 64
 * or 128, at most 4 q heads per kv head, d_model / n_q_heads*head_dim / d_ff multiples of 64); it is
 * the default wherever a session qualifies; a session that qualifies but cannot be set up fails in
 * ada_session_create instead of taking the other path).  0 = one kernel per operation on CUDA cores
 * (any dtype, any batch; sequences of a batch share every layer pass).  On path 1 the sequences of a batch are
 * decoded one after another, each streaming the weights for itself.  ADA_EUNSUPPORTED if path 1 is asked of a
 * session that does not qualify.
 * ada_stats.path reports the path a decode call ran on. */
int ada_debug_set_path(ada_session *s, int32_t path);
int ada_debug_get_path(ada_session *s, int32_t *path_out);
/* How ada_prefill runs prompts of 32 tokens or more.  1 (the default wherever it is available: bf16 models of
 * the shapes the persistent kernel takes, on sm_100): the dense pass, blocks of 128 positions, every weight
 * matrix streamed once per block through a tcgen05 GEMM with its accumulator in tensor memory.  0: through
 * the decode path itself (passes of eight positions in the persistent kernel, or one kernel per operation).
 * ADA_EUNSUPPORTED if the dense pass is asked of a session that cannot run it. */
int ada_debug_set_prefill(ada_session *s, int32_t dense);
/* Steps of Algorithm 1 one launch of the persistent kernel may start before it returns to the host
 * (default 256; the host relaunches until the call is complete). */
int ada_debug_set_launch_steps(ada_session *s, int32_t steps);
/* Every wait inside the persistent kernel (on a shared-memory barrier, on the grid-wide counter, on
 * another CTA's partial sums) gives up after `ns` nanoseconds (default 2 s): the kernel then sets an
 * error word, lets every other wait fall through, ends, and the decode call returns ADA_ETIMEOUT.
 * The sequence state is undefined after that; ada_session_reset + ada_prefill make the session
 * usable again.  A limit shorter than a grid-wide wait normally lasts (a few microseconds) makes the
 * next decode call time out: that is how the give-up path is tested. */
int ada_debug_set_wait_limit(ada_session *s, uint64_t ns);
/* Event trace of the persistent kernel: while the kernel runs the steps [step0, step1) of a launch
 * (counted from 0 in every launch), every CTA appends (nanosecond timestamp, code) pairs of
 * uint64 to its own region of dev_buf [SMs][cap_events][2]; code = CTA << 32 | argument << 8 | event (1 phase begin, 2
 * first activation stage landed, 3 first weight stage landed, 4 last tile group multiplied, 5
 * epilogue done, 6 / 7 weight producer starts / ends a phase, 8 attention item done, 9 attention
 * chunks merged, 10 barrier arrival, 11.. attention sub-steps).  count_dev [SMs] receives the number of
 * events of each CTA in the last traced launch.  NULL stops. */
int ada_debug_trace(ada_session *s, uint64_t *dev_buf, uint32_t *count_dev, uint32_t cap_events, int32_t step0, int32_t step1);

/* Host-only: how the streaming GEMM of shape N x K (mode as in ada_debug_gemm) divides its work
 * over `grid` CTAs, for CTA `cta`.  out9 (host) receives {split, t0, t1, n, ta, tb, s0_own_k0,
 * s0_pub_k1, sl_k1}: split == 0: whole 16-row tiles [t0, t1); split == 1 (only if `split` is
 * nonzero and the shape allows it): one group of n tile slots, slot s holding tile ta + s, where
 * slot 0 multiplies k chunks >= s0_own_k0 of its tile and, before them, chunks < s0_pub_k1 of
 * tile tb (published to the next CTA), and the last slot (if not slot 0) only chunks < sl_k1.
 * A k chunk is 512 wide.  No GPU is touched.  ADA_EINVAL on bad arguments. */
int ada_debug_gemm_plan(int32_t N, int32_t K, int32_t mode, int32_t grid, int32_t cta, int32_t split, int32_t *out9);

/* Run the weight-streaming skinny GEMM of the decode kernel by itself (the kernel behind the QKV,
 * O, gate/up, down and LM-head products of a layer pass, Algorithm 1 "process all tokens in P[l]
 * in parallel"): bf16 weights W_dev [N, K] row-major, fp32 activations X_dev [cols, K], 1 <= cols
 * <= 8, fp32 result Y_dev [cols, ldy].
 *   mode 0: Y[c][n] = sum_k W[n][k] X[c][k], n < N.
 *   mode 1: W stacks a gate matrix over an up matrix (N/2 rows each, N/2 a multiple of 16):
 *           Y[c][n] = silu(gate_n . X[c]) * (up_n . X[c]), n < N/2.
 * K must be a multiple of 64.  work_dev is device scratch of at least ada_debug_gemm_work_bytes(K)
 * bytes, 256-byte aligned.  The product is launched `repeat` >= 1 times back to back inside one
 * kernel; *ms_out (nullable) receives the device time of that kernel.  All pointers except ms_out
 * are device pointers.  Returns ADA_ETIMEOUT if a bounded device-side wait expired. */
size_t ada_debug_gemm_work_bytes(int32_t K);
int ada_debug_gemm(const void *W_dev, int32_t N, int32_t K, int32_t mode, const float *X_dev, int32_t cols,
                   void *work_dev, size_t work_bytes, float *Y_dev, int32_t ldy, int32_t repeat, void *cuda_stream,
                   float *ms_out);

/* Run the dense GEMM of the prompt pass by itself (Algorithm 1, first line: all prompt tokens go through the
 * model at once): Y[m][n] = (or +=, if `accumulate`) sum_k X[m][k] W[n][k] for up to 128 rows m, on tcgen05
 * tensor cores with the accumulator in tensor memory.  W_dev bf16 [N, K] row-major, X_dev fp32 [rows, K],
 * Y_dev fp32 [rows, ldy] (16-byte aligned, ldy a multiple of 4), K a multiple of 64; work_dev: device scratch
 * of ada_debug_dense_gemm_work_bytes(K) bytes, 256-byte aligned.  sm_100 only (ADA_EUNSUPPORTED elsewhere).
 * Synchronises the stream; ADA_ETIMEOUT if a bounded device-side wait expired. */
size_t ada_debug_dense_gemm_work_bytes(int32_t K);
int ada_debug_dense_gemm(const void *W_dev, int32_t N, int32_t K, const float *X_dev, int32_t rows, float *Y_dev, int32_t ldy,
                         int32_t accumulate, void *work_dev, size_t work_bytes, void *cuda_stream);

/* The same streaming GEMM as ada_debug_gemm (modes, shapes and layouts as described there, one
 * product per call), for callers that have no device memory to lend and must not allocate any.
 * (The paper has no counterpart to this call; it exists for deployment.)  Think of a serving
 * process whose framework has already handed every byte of HBM to its KV-cache pool, or of code
 * running where a device allocation would stall every stream of the process: such a caller can
 * still pass the weights, the activations and the output, and this call brings its own scratch.
 *
 * The scratch (activations re-laid for the tensor cores, an error word, a tensor map) is a fixed
 * array of 512.5 KB inside the library image; every GPU that loads the library holds it until the
 * process exits.  It bounds the depth: K <= 16384, larger K returns ADA_ECAPACITY.  The call
 * performs no cudaMalloc / cudaFree and creates no events.
 *
 * The scratch comes into being when the library's device code is first used on a GPU (the driver
 * then places the array and the kernels there; that one-time placement is the driver's, not a call
 * this function makes).  The first call on each device also looks up the array's device address and
 * configures the kernel: make that first call before any stream capture begins.  Every call, the
 * first and the later ones alike, waits for `cuda_stream` twice and copies an error word back to
 * the host before it returns.  All calls on a device share the one array:
 * it keeps the previous call's contents (the call clears the word that has to start at zero and
 * rewrites the rest), and two calls whose kernels overlap on the GPU (different streams, or
 * different host threads) race on it.
 * W_dev, X_dev, Y_dev are device pointers as in ada_debug_gemm. */
int ada_gemm_noalloc(const void *W_dev, int32_t N, int32_t K, int32_t mode, const float *X_dev, int32_t cols, float *Y_dev,
                     int32_t ldy, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* ADADECODE_H */
