/*
 * fastcot.h - C ABI of the Jacobi-window decode step (FastCoT, arXiv 2311.08263) for NVIDIA B200.
 *
 * One step = one causal decoder forward over (committed prefix held in a K/V cache) + (a window
 * of c tokens: the pending exact token followed by c-1 approximate tokens), greedy argmax at
 * every window row, verification of the previous guesses one by one, K/V commit of the accepted
 * rows and shift + refill of the window (paper, Method, "Approximate Rationale Generation": Eq. 4
 * inference, Eq. 5 verification, "Cache Update"; buffer and index vector: "Approximate Tokens
 * Buffer").  With c = 1 the step is plain greedy autoregressive decoding (Eq. 1).
 *
 * Conventions
 *   - "host"/"device" on every pointer says where the memory lives.  The library allocates NO
 *     device memory: weights, K/V slab and workspace are caller-owned device buffers, BORROWED for
 *     the lifetime of the context.  fc_destroy frees host state only.
 *   - All matrices are row-major [out_features, in_features] in the model dtype.
 *   - Every call returns FC_OK (0) or a negative fc_status; nothing aborts or throws and no device
 *     trap is used.  A call refused for its arguments (FC_ERR_ARG, _CAPACITY, _TOKEN_RANGE, _BAD_WINDOW,
 *     _STATE) leaves the committed state (tokens, kv_len) unchanged, with one exception: fc_prefill
 *     drops the previous sequences as soon as its arguments are accepted.  After FC_ERR_DEVICE_TIMEOUT
 *     or FC_ERR_CUDA from a call that launched kernels, the sequences are lost: call fc_prefill again.
 *   - Calls are synchronous with respect to their host outputs: they wait on the context's stream.
 *   - A context is bound to one device and one stream and is not re-entrant.
 */
#ifndef FASTCOT_H_
#define FASTCOT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct fc_ctx fc_ctx;

typedef enum { FC_F32 = 0, FC_BF16 = 1 } fc_dtype;

/* How window slots that no forward has predicted yet are filled ("Approximate Tokens Buffer": the
 * buffer is initialised from the prompt's own token ids; a pad token is the alternative it mentions). */
typedef enum { FC_REFILL_PROMPT_CYCLE = 0, FC_REFILL_PAD = 1 } fc_refill;

typedef enum {
  FC_OK = 0,
  FC_ERR_ARG = -1,            /* NULL pointer, non-positive size, bad enum */
  FC_ERR_SHAPE = -2,          /* model shape the kernels cannot run (see fc_init) */
  FC_ERR_CAPACITY = -3,       /* kv_len + c > max_seq, batch > max_batch, c > max_c, buffer too small */
  FC_ERR_TOKEN_RANGE = -4,    /* token id outside [0, vocab) */
  FC_ERR_STATE = -5,          /* step/generate before prefill */
  FC_ERR_BAD_WINDOW = -6,     /* window_in[b][0] is not the pending exact token */
  FC_ERR_DEVICE_TIMEOUT = -7, /* a bounded device-side wait expired; context must be re-prefilled */
  FC_ERR_CUDA = -8            /* a CUDA runtime/driver call failed; see fc_last_cuda_error */
} fc_status;

enum {                        /* fc_model_shape.flags */
  FC_FLAG_SIMT_GEMM = 1,      /* run projections on the plain FMA kernels even for bf16 (debug aid) */
  FC_FLAG_NO_PDL = 4,         /* launch every kernel fully serialised (no programmatic dependent launch) */
  FC_FLAG_NO_CHAIN = 8,       /* one launch per projection instead of one chained launch per layer */
  FC_FLAG_NO_FFN_SPLIT = 16,  /* chained launch: gate/up and down as one phase each instead of two halves of d_ffn */
  FC_FLAG_NO_CTA_PAIRS = 32   /* more than 64 rows: one CTA per weight tile instead of a pair of CTAs per 256-row tile */
};

typedef struct {
  int32_t n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ffn, vocab;
  int32_t dtype;              /* fc_dtype of the weights and of the K/V cache */
  float rms_eps, rope_theta;  /* RMSNorm epsilon; rotary base (half-split pairing i <-> i+head_dim/2) */
  int32_t max_batch, max_c;   /* capacity: sequences per step, window rows per sequence */
  int32_t max_seq;            /* K/V capacity per sequence: committed tokens + window rows */
  float bias_beta;            /* synthetic-workload logit bonus on token bias_perm[input]; 0 disables */
  int32_t flags;
} fc_model_shape;

typedef struct {              /* DEVICE pointers, borrowed */
  const void *tok_emb;                                   /* [vocab, d_model] */
  const void *const *wq, *const *wk, *const *wv, *const *wo;   /* HOST arrays of n_layers device ptrs */
  const void *const *w_gate, *const *w_up, *const *w_down;
  const void *const *g_attn, *const *g_ffn;              /* RMSNorm gains [d_model] */
  const void *g_final, *lm_head;                         /* [d_model], [vocab, d_model] */
  const int32_t *bias_perm;                              /* device [vocab] or NULL */
} fc_weights;

typedef struct {              /* filled by fc_generate */
  int64_t steps, tokens;      /* forwards run; tokens committed over all sequences */
  int32_t accept_hist[65];    /* accept_hist[k] = (sequence, step) pairs that accepted k tokens; k>64 -> [64] */
  float ms_prefill, ms_steps; /* device time of the most recent fc_prefill and of this call's iterations */
} fc_stats;

/* Bytes the caller must provide.  K/V slab layout: [layer][K|V][max_batch][n_kv_heads][max_seq][head_dim]
 * in the model dtype.  Both return 0 for an invalid shape. */
size_t fc_kv_bytes(const fc_model_shape *shape);
size_t fc_workspace_bytes(const fc_model_shape *shape);

/* Create a context: the decode state of "Approximate Tokens Buffer" (buffer Y as window + committed tokens,
 * index vector I as kv_len per sequence) and the K/V cache of the exact prefix, all empty.
 * shape, weights: host structs (copied).  kv, ws: device, >= the sizes above,
 * 256-byte aligned.  cuda_stream: a cudaStream_t (NULL = default stream).  Shape limits:
 * head_dim in {32, 64, 128}; n_heads % n_kv_heads == 0; d_model, d_ffn, n_heads*head_dim multiples of 8;
 * max_c <= 64.  The bf16 tensor-core path needs an sm_100a device; FC_F32 runs on FMA kernels. */
int fc_init(fc_ctx **out, const fc_model_shape *shape, const fc_weights *weights,
            void *kv, size_t kv_bytes, void *ws, size_t ws_bytes, void *cuda_stream);

/* Start `batch` sequences (dropping any previous ones).  prompt_ids: host [batch, p_stride]; prompt_lens:
 * host [batch], each >= 1.  Caches K/V of prompt[0 .. P-2] in blocks of at least 128 rows per forward;
 * prompt[P-1] becomes the pending exact token (window slot 0); slots 1..c-1 are filled by the refill rule.
 * "Overview of FastCoT": the prompt and the window taken from the buffer form the first input. */
int fc_prefill(fc_ctx *ctx, int32_t batch, const int32_t *prompt_ids, int32_t p_stride,
               const int32_t *prompt_lens, int32_t c, int32_t refill, int32_t pad_id);

/* One Jacobi-window iteration for every live sequence (Eq. 4, Eq. 5, cache update).
 * window_in: host [batch, c] or NULL (keep the internal window); slot 0 of each row must be the
 * pending exact token.  Outputs (host, each nullable): accepted_count [batch] (k in [1, c]; 0 for a
 * finished sequence), accepted_tokens [batch, c] (first k valid), window_out [batch, c].
 * Sequences that fc_generate has finished (max_tokens reached or EOS) take no rows of the forward: the step
 * runs over the live sequences only (the paper's "Time Analysis" counts what padded, finished batch members
 * cost; here they cost nothing). */
int fc_jacobi_step(fc_ctx *ctx, const int32_t *window_in, int32_t *accepted_count,
                   int32_t *accepted_tokens, int32_t *window_out);

/* Change the number of window rows c between iterations (the paper treats the context-window length as a free
 * parameter, "Context Window Length"): the pending token and the guesses that still fit are kept, new slots are
 * filled by the refill rule for their generated index.  1 <= c <= max_c. */
int fc_set_window(fc_ctx *ctx, int32_t c);

/* Iterate with c rows per forward (c <= 0: keep the current window size; otherwise as fc_set_window) until every
 * sequence has committed max_tokens tokens since its prefill or eos_id (eos_id < 0: never), or until max_iters
 * forwards have run (max_iters <= 0: no cap).  "Iteration Stop Condition": condition 1 is an upper bound on the
 * iterations, condition 2 a verified EOS.  Streams are cut at max_tokens and just after the first EOS.
 * out_tokens: host [batch, max_tokens], receives the tokens committed by THIS call; out_lens: host [batch];
 * stats nullable.  A later call with a larger max_tokens goes on where this one stopped (sequences that ended
 * on eos_id stay finished). */
int fc_generate(fc_ctx *ctx, int32_t max_tokens, int32_t c, int32_t eos_id, int32_t max_iters,
                int32_t *out_tokens, int32_t *out_lens, fc_stats *stats);

/* Hand-off of the approximate rationale ("Overview of FastCoT", last step; "Trigger Answer"): everything generated
 * so far - the exact tokens and the approximate tokens still in the window, taken as they are - is joined with the
 * answer trigger, and the answer is decoded greedily (Eq. 1) from there.  Per sequence the context
 * [window slot 0 .. c-1 | trigger_ids] is appended to the cache (all but its last token, which becomes the pending
 * token) and up to max_answer_tokens tokens are decoded, cut just after eos_id (eos_id < 0: never).
 * trigger_ids: host [n_trigger] (n_trigger may be 0); answer_tokens: host [batch, max_answer_tokens];
 * answer_lens: host [batch].  Needs kv_len + c + n_trigger + max_answer_tokens <= max_seq.  The Jacobi state is
 * consumed: call fc_prefill before iterating again. */
int fc_finish_with_trigger(fc_ctx *ctx, const int32_t *trigger_ids, int32_t n_trigger, int32_t max_answer_tokens,
                           int32_t eos_id, int32_t *answer_tokens, int32_t *answer_lens);

/* Benchmark/debug aids.  fc_debug_set_state: declare `batch` sequences with kv_lens[b] tokens
 * already present in the K/V slab (written by the caller) and pending tokens pending[b]; windows are
 * refilled with pad_id.  fc_debug_logits: device buffer [max_batch*max_c, vocab] fp32 that receives
 * the logits of every following step (NULL turns it off).  fc_get_state: host copies of kv_len and
 * n_gen per sequence (each nullable). */
int fc_debug_set_state(fc_ctx *ctx, int32_t batch, const int32_t *kv_lens, const int32_t *pending,
                       int32_t c, int32_t pad_id);
int fc_debug_logits(fc_ctx *ctx, float *dev_logits);
int fc_get_state(fc_ctx *ctx, int32_t *kv_lens, int32_t *n_gen);

/* Robustness aids for tests (no compute-sanitizer is assumed).  fc_debug_inject_timeout: the accept kernel of the
 * next step raises the device error word exactly as an expired bounded wait would, without any wait; that step
 * returns FC_ERR_DEVICE_TIMEOUT and the context needs fc_prefill.  fc_debug_check_guards: the workspace slices are
 * separated by canary bands written at fc_init; *n_damaged (host) receives how many of them no longer hold the
 * pattern (0 = no kernel wrote outside its slice). */
int fc_debug_inject_timeout(fc_ctx *ctx);
int fc_debug_check_guards(fc_ctx *ctx, int32_t *n_damaged);

/* Enqueue `n_steps` iterations back to back with no host round trip in between and return the
 * device time in milliseconds from the first to the last kernel (CUDA events on the context's
 * stream).  commit != 0: every step commits its accepted tokens on the device (needs
 * kv_len + n_steps * c <= max_seq; every eighth step the host re-reads kv_len to size the attention grid);
 * host mirrors are refreshed afterwards and *tokens_out (nullable)
 * gets the tokens committed over all sequences.  commit == 0: kv_len, n_gen and the window are left
 * untouched, so every step runs at the same K/V length (latency sweeps). */
int fc_bench_steps(fc_ctx *ctx, int32_t n_steps, int32_t commit, float *ms_total, int64_t *tokens_out);

/* One non-committing step with CUDA events around every launch (launches are therefore fully serialised:
 * no programmatic overlap between neighbours).  ms_by_class / launches_by_class
 * (host, FC_N_CLASSES entries each) receive device time and launch count per kernel class. */
enum { FC_CLS_EMBED = 0, FC_CLS_QKV, FC_CLS_ROPE, FC_CLS_ATTN, FC_CLS_OPROJ, FC_CLS_GATEUP, FC_CLS_DOWN,
       FC_CLS_HEAD, FC_CLS_ACCEPT, FC_CLS_CHAIN /* O + gate/up + down + next QKV in one launch */, FC_N_CLASSES };
int fc_profile_step(fc_ctx *ctx, float *ms_by_class, int32_t *launches_by_class);

/* Number of kernels the most recent step / prefill / bench call launched. */
int64_t fc_last_launch_count(const fc_ctx *ctx);

void fc_destroy(fc_ctx *ctx);
const char *fc_strerror(int status);
const char *fc_last_cuda_error(const fc_ctx *ctx);   /* text of the last CUDA failure, or "" */

/* ---- single operations of the step, for unit parity tests (all pointers DEVICE unless noted) ---- */

/* y[R, N] += x[R, K] . w[N, K]^T with fp32 x and y and weights in `dtype`; K % 8 == 0.
 * use_tensor_cores != 0 selects the tcgen05 kernel (bf16 only; K >= 64, N % 4 == 0 and y 16-byte aligned,
 * else FC_ERR_SHAPE).  The projections of the step (QKV, O, gate/up, down) are this contraction. */
int fc_op_linear(const float *x, const void *w, float *y, int32_t R, int32_t N, int32_t K,
                 int32_t dtype, int32_t use_tensor_cores, void *cuda_stream);

/* Verification + cache update on given argmax results (Eq. 5).  All arrays device int32:
 * window [batch, c] (in/out), argmax [batch, c], kv_len/n_gen [batch] (in/out),
 * accepted_count [batch], accepted_tokens [batch, c]; prompt [batch, p_stride], prompt_lens [batch]. */
int fc_op_accept(int32_t *window, const int32_t *argmax, int32_t *kv_len, int32_t *n_gen,
                 int32_t *accepted_count, int32_t *accepted_tokens, const int32_t *prompt,
                 const int32_t *prompt_lens, int32_t batch, int32_t c, int32_t p_stride,
                 int32_t refill, int32_t pad_id, void *cuda_stream);

/* Window attention of one layer (the attention inside Eq. 4's single causal forward): for sequence b,
 * window row j and query head h, softmax over keys 0 .. kv_len[b] + j of q.k / sqrt(head_dim), times V;
 * kv head = h / (n_heads / n_kv_heads).  q: [batch*c, n_heads*head_dim], kcache/vcache:
 * [batch][n_kv_heads][max_seq][head_dim], all in `dtype`, rotary embedding already applied, the window's
 * own K/V already stored at slots kv_len[b] .. kv_len[b]+c-1.  kv_len: device [batch]; max_len: host upper
 * bound on kv_len[b].  out: fp32 [batch*c, n_heads*head_dim].  scratch: device, at least
 * fc_op_window_attention_scratch_bytes(...) bytes, 256-byte aligned; it holds the per-split partial
 * results and is cleared as needed by the call. */
size_t fc_op_window_attention_scratch_bytes(int32_t batch, int32_t c, int32_t n_heads, int32_t n_kv_heads,
                                            int32_t head_dim, int32_t max_len, int32_t dtype);
int fc_op_window_attention(const void *q, const void *kcache, const void *vcache, const int32_t *kv_len,
                           float *out, int32_t batch, int32_t c, int32_t n_heads, int32_t n_kv_heads,
                           int32_t head_dim, int32_t max_seq, int32_t max_len, int32_t dtype,
                           void *scratch, size_t scratch_bytes, void *cuda_stream);

/* The attention kernel of the bf16 step as it runs inside fc_jacobi_step (head_dim 64 or 128): applies the deferred
 * RMSNorm factor 1/sqrt(sumsq[r] / d_norm + rms_eps) to the q, k and v accumulators of every window row, rotates q and k
 * at position kv_len[b] + j (pairs i <-> i + head_dim/2, angle pos * rope_theta^(-2i/head_dim)), stores the window's k and v
 * rows as bf16 at cache slots kv_len[b] .. kv_len[b]+c-1, and computes the window attention of Eq. 4's forward as
 * fc_op_window_attention does.  qkv_acc: fp32 [batch*c, (n_heads + 2 n_kv_heads) * head_dim] = (q | k | v), cleared by
 * the call; sumsq: fp32 [batch*c], cleared by the call; kcache/vcache: bf16 [batch][n_kv_heads][max_seq][head_dim],
 * in/out, 16-byte aligned (cached K/V tiles are fetched by TMA); out: fp32 [batch*c, n_heads*head_dim].  c <= 128.
 * n_splits: 0 = the grid fc_jacobi_step would choose, 1..8 forces that many CTAs (one thread-block cluster) per
 * (sequence, kv head, group of query tiles), each over a run of consecutive 64-key tiles.  q_tiles: 0 = the step's
 * choice, 1, 2 or 4 forces that many 16-row query tiles per CTA.  scratch: device, 256-byte
 * aligned, >= ..._scratch_bytes(...) (rotary table and an error word).  Returns FC_ERR_DEVICE_TIMEOUT when a bounded
 * wait inside the kernel gave up. */
size_t fc_op_fused_window_attention_scratch_bytes(int32_t batch, int32_t c, int32_t n_heads, int32_t n_kv_heads,
                                                  int32_t head_dim, int32_t max_seq, int32_t max_len);
int fc_op_fused_window_attention(float *qkv_acc, float *sumsq, float rms_eps, int32_t d_norm, float rope_theta,
                                 void *kcache, void *vcache, const int32_t *kv_len, float *out, int32_t batch,
                                 int32_t c, int32_t n_heads, int32_t n_kv_heads, int32_t head_dim, int32_t max_seq,
                                 int32_t max_len, int32_t n_splits, int32_t q_tiles, void *scratch,
                                 size_t scratch_bytes, void *cuda_stream);

/* The same window attention for callers that may not allocate device memory (the paper has no
 * counterpart; this exists for hosts whose device memory is owned by someone else, e.g. a serving
 * process with a fixed arena, or code that must stay out of the CUDA allocator after start-up).
 * Scratch is a fixed FC_NOALLOC_SCRATCH_BYTES array built into the library - every GPU that loads the
 * library holds it until the process exits - so only inputs and outputs are passed; arguments are
 * those of fc_op_window_attention.  Problems whose scratch need (fc_op_window_attention_scratch_bytes)
 * exceeds the array are refused with FC_ERR_CAPACITY and a message on stderr.  The call makes no
 * cudaMalloc/cudaFree and uses no allocating library routine.  The first call on each device looks up
 * the array's device address (cudaGetSymbolAddress) with that device current; make that first call
 * before starting any stream capture.  All calls on a device share the one array, which keeps
 * whatever the previous call left in it (the call clears the part that must start at zero): two calls
 * that overlap on the GPU - different streams or threads - race on it; serialise them. */
#define FC_NOALLOC_SCRATCH_BYTES (8u << 20)
int fc_op_window_attention_noalloc(const void *q, const void *kcache, const void *vcache,
                                   const int32_t *kv_len, float *out, int32_t batch, int32_t c,
                                   int32_t n_heads, int32_t n_kv_heads, int32_t head_dim, int32_t max_seq,
                                   int32_t max_len, int32_t dtype, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif  /* FASTCOT_H_ */
