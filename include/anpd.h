/*
 * anpd.h - C boundary of the B200 implementation of the draft-and-verify step of
 * Adaptive N-gram Parallel Decoding (ANPD, arXiv 2404.08698).
 *
 * The calls follow the paper's statement of the method:
 *   - the N-gram module's Initialize / Update / Query (Section 3.1, "Token Level
 *     N-gram Module") and its multi-level back-off (Section 3.2, Algorithm 2):
 *       anpd_ngram_update, anpd_ngram_draft
 *   - the verification stage (Section 3.1, "Parallel Decoding", item 2; the LLM(drafts)
 *     call and the accept loop of Algorithm 1):  anpd_verify
 *   - the decoding loop with inputs prompt, K, M and output O (Algorithm 1): anpd_generate
 *
 * General conventions
 *   - Every function returns an anpd_status: 0 on success, negative on failure.  Nothing
 *     aborts or throws.  On failure the caller's output arguments are left untouched.
 *   - Handles (anpd_model, anpd_kv, anpd_ngram) are opaque, owned by the library and
 *     released by the matching *_destroy.  One handle is used by one thread at a time; a kv or
 *     ngram handle belongs with its model, so one model and everything created for it stay on
 *     one thread at a time.  Different models may be used from different threads: the library
 *     keeps no mutable state outside the handles except the launch counter (atomic) and the text
 *     of the calling thread's last CUDA failure (thread-local).
 *   - A model is laid out for the device that was current when it was created (the weight
 *     blocks are ordered for that device's SM count).  Using its handles while another device
 *     is current returns ANPD_ERR_STATE.
 *   - Array arguments are caller-owned HOST memory unless the parameter comment says
 *     "device"; they are only read or written during the call.
 *   - All device work of a model, and of the kv / ngram handles used with it, is issued on
 *     the CUDA stream given at creation (0 = the default stream).  Calls that return results
 *     in host memory synchronise that stream before returning; calls marked "asynchronous"
 *     only enqueue work.
 *   - There is no CPU implementation behind any of these calls: without a CUDA device
 *     every call that needs one returns ANPD_ERR_CUDA.
 *   - Limits: draft length K <= ANPD_K_MAX (a step verifies at most K+1 = 8 rows per
 *     sequence); n-gram levels 2 <= n_min <= n_max <= ANPD_N_MAX; token ids in [0, vocab).
 */
#ifndef ANPD_H
#define ANPD_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int anpd_status;
enum {
    ANPD_OK = 0,
    ANPD_ERR_ARG = -1,      /* null pointer, non-positive size, inconsistent configuration */
    ANPD_ERR_OOM = -2,      /* host or device allocation failed */
    ANPD_ERR_CAPACITY = -3, /* context, KV cache or n-gram table would overflow */
    ANPD_ERR_RANGE = -4,    /* token id >= vocab, K > ANPD_K_MAX, n outside [2, ANPD_N_MAX] */
    ANPD_ERR_CUDA = -5,     /* a CUDA call failed, or a kernel reported an internal error */
    ANPD_ERR_STATE = -6     /* call order: e.g. verify on an empty KV cache with no prefill */
};

#define ANPD_K_MAX 7
#define ANPD_N_MAX 8
#define ANPD_ROWS 8 /* rows per sequence of every decode forward (K+1 padded to 8) */

typedef struct anpd_model anpd_model; /* weights in device memory + configuration */
typedef struct anpd_kv anpd_kv;       /* paged KV cache, per-sequence lengths, activations */
typedef struct anpd_ngram anpd_ngram; /* one sequence's token buffer + MLN tables ("Memory") */

/* LLaMA-style decoder (the paper names the family only, Section 4.1): RMSNorm, rotary
 * embedding with pairs (i, i + head_dim/2) and angle pos * theta^(-2i/head_dim), grouped-query
 * attention with softmax scale 1/sqrt(head_dim), SwiGLU FFN, no biases, untied LM head.
 * Requirements: d_model, d_ffn and n_q_heads*head_dim multiples of 8; head_dim 64 or 128;
 * 1, 2, 4 or 8 query heads per kv head; d_model <= 16384. */
typedef struct {
    int n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ffn, vocab;
    float rope_theta, rms_eps;
} anpd_model_config;

/* Query policy (the paper says Query "predicts the next token" from frequency counts, Eq. 1,
 * without fixing ties): 0 = successor with the largest count, equal counts to the one seen
 * most recently; 1 = successor of the context's most recent occurrence. */
typedef struct {
    int n_min;   /* lowest level, >= 2 */
    int n_max;   /* N of Section 3.2: levels n_min..n_max, level n keyed on n-1 tokens */
    int max_ctx; /* most tokens (prompt + generated) the context may ever hold */
    int policy;
} anpd_ngram_config;

/* One record of a level-n table: context key[0..n-2], successor, how often the n-gram
 * occurred, and the position (index into the committed token sequence) of its last
 * occurrence.  Unused key slots are -1. */
typedef struct {
    int32_t key[ANPD_N_MAX - 1];
    int32_t succ;
    int32_t count;
    int32_t last_pos;
} anpd_ngram_entry;

typedef struct {
    int steps;            /* draft-and-verify steps run */
    int drafted;          /* draft tokens proposed */
    int accepted;         /* draft tokens accepted; hit ratio alpha = accepted / drafted (Sec. 4.4) */
    int generated;        /* tokens committed by the loop (may exceed max_new by up to K) */
    int hist_accepted[8]; /* steps by accepted_len */
    int alt_wins;         /* two-candidate mode: steps whose second candidate was the one kept (else 0) */
    int reserved;
    double ms_prefill;    /* device time of the prompt forward (CUDA events) */
    double ms_decode;     /* device time of the decoding loop, first step to last */
    double bytes_per_step;/* weight + KV bytes one verify step must read, at the mean KV length */
} anpd_stats;

/* Device time by kernel class, accumulated while profiling is on (CUDA events around every
 * launch; slower than a normal run, so never mix with throughput numbers). */
typedef struct {
    double ms_gemm;   int n_gemm;     /* weight-streaming GEMMs */
    double ms_attn;   int n_attn;     /* attention partial + combine */
    double ms_other;  int n_other;    /* norms, RoPE/append, SwiGLU, argmax/accept */
    double ms_ngram;  int n_ngram;    /* n-gram update + draft */
    double gemm_bytes;                /* weight bytes read by the GEMM launches counted above */
} anpd_profile;

/* ---- model ---------------------------------------------------------------------------
 * weights: array of 1 + 9*n_layers + 2 pointers in this order:
 *   embed [vocab, d_model];
 *   per layer: attn_norm [d_model] (fp32 always), wq [n_q_heads*head_dim, d_model],
 *     wk [n_kv_heads*head_dim, d_model], wv [same], wo [d_model, n_q_heads*head_dim],
 *     ffn_norm [d_model] (fp32), w_gate [d_ffn, d_model], w_up [d_ffn, d_model],
 *     w_down [d_model, d_ffn];
 *   final_norm [d_model] (fp32), lm_head [vocab, d_model].
 * Matrices are row-major [out_features, in_features] (y = x W^T), bf16 if weights_are_bf16
 * else fp32 (rounded to bf16, nearest-even, by the library).  weights_on_device says whether
 * the pointers are device or host pointers.  The library copies everything into its own device
 * memory; the caller may free its buffers after the call returns. */
anpd_status anpd_model_create(const anpd_model_config* cfg, const void* const* weights,
                              int weights_are_bf16, int weights_on_device, void* cuda_stream,
                              anpd_model** out);
anpd_status anpd_model_destroy(anpd_model* m);

/* ---- KV cache ------------------------------------------------------------------------
 * Paged bf16 cache for `batch` independent sequences of at most max_len positions each
 * (max_len <= 32768 is rounded up to whole pages, batch <= 16; a step needs kv_len + 8 <= max_len).  Also holds the
 * activation buffers of a forward, so a kv handle is tied to the model it was created for.
 * shuffle_pages != 0 permutes the physical page order (results must not change). */
anpd_status anpd_kv_create(const anpd_model* m, int max_len, int batch, int shuffle_pages, anpd_kv** out);
anpd_status anpd_kv_destroy(anpd_kv* kv);
anpd_status anpd_kv_len(anpd_kv* kv, int seq, int* len);
/* Roll sequence `seq` back to `len` <= its current length.  Nothing is copied or cleared:
 * entries past `len` are simply overwritten by later steps (Section 3.1: rejected tokens
 * and everything after them are discarded). */
anpd_status anpd_kv_truncate(anpd_kv* kv, int seq, int len);
/* Candidates verified per step of the decoding loops (anpd_generate*): 1 (Algorithm 1 as printed) or 2.  The Conclusion
 * names, as future work, verifying several draft candidates in parallel; with 2, a step drafts the usual candidate (cut
 * to min(K, 4) tokens) and a second one of up to min(K, 3) tokens whose first token is the answer of the longest N-gram
 * level that disagrees with the first candidate's first token (continued by ordinary back-off queries; empty when no
 * level disagrees).  Both are verified by the same forward over the step's 8 rows - the second candidate's rows attend to
 * the committed context and to themselves, not to the first candidate - and the one with the longer accepted prefix is
 * committed (the first on a tie).  The output stays the model's greedy output.  anpd_stats.drafted then counts the tokens
 * of both candidates and anpd_stats.alt_wins the steps the second one won.  The staged verify calls (anpd_verify*) always
 * take one candidate.  ANPD_ERR_RANGE for any other value. */
anpd_status anpd_kv_set_candidates(anpd_kv* kv, int candidates);

/* ---- N-gram module (Sections 3.1, 3.2) ---------------------------------------------------- */
anpd_status anpd_ngram_create(const anpd_ngram_config* cfg, void* cuda_stream, anpd_ngram** out);
anpd_status anpd_ngram_reset(anpd_ngram* ctx);   /* forget all tokens and statistics */
anpd_status anpd_ngram_destroy(anpd_ngram* ctx);
anpd_status anpd_ngram_len(anpd_ngram* ctx, int* n_tokens);

/* Initialize / Update: append n_new committed tokens to the context; each is paired with its
 * previous n-1 tokens at every level n and the level's statistics are updated.  The first call
 * with the whole prompt is the paper's Initialize.  ANPD_ERR_CAPACITY if the context would
 * exceed max_ctx (nothing is changed then). */
anpd_status anpd_ngram_update(anpd_ngram* ctx, const int32_t* new_tokens, int n_new);

/* Drafting stage + Algorithm 2: K chained queries from the tail of the context, each from the
 * highest level down to the lowest, first level that knows the context answers; the answer is
 * appended to a temporary context for the next query.  Stops at the first query no level can
 * answer.  draft: int32[K]; *draft_len in [0, K].  Does not modify the statistics. */
anpd_status anpd_ngram_draft(anpd_ngram* ctx, int K, int32_t* draft, int* draft_len);

/* Test hook: all records of level n in canonical order (sorted by key, then successor).
 * out may be NULL to query the count only. */
anpd_status anpd_ngram_dump(anpd_ngram* ctx, int n, anpd_ngram_entry* out, int cap, int* n_entries);
/* Test hook: for every context of level n (sorted), the answer Query would give, in `succ`;
 * count/last_pos are those of that successor. */
anpd_status anpd_ngram_dump_best(anpd_ngram* ctx, int n, anpd_ngram_entry* out, int cap, int* n_entries);

/* ---- verification (Section 3.1 item 2; Algorithm 1's LLM(drafts) + accept loop) ----------
 * Prefill: LLM(prompt).  Runs the prompt through the decoder from an empty sequence `seq`,
 * leaves kv_len = prompt_len and returns the first generated token (argmax of the last row). */
anpd_status anpd_prefill(anpd_model* m, anpd_kv* kv, int seq, const int32_t* prompt, int prompt_len,
                         int32_t* first_tok);

/* One forward over [last_tok, draft[0..draft_len)] at positions kv_len.. of sequence 0, then
 * greedy acceptance: accepted_len = the longest prefix with draft[i] == argmax of row i's
 * logits (ties to the lowest token id); next_tok = argmax of row accepted_len; the cache is
 * committed to kv_len + accepted_len + 1.  draft_len == 0 is a plain greedy step. */
anpd_status anpd_verify(anpd_model* m, anpd_kv* kv, int32_t last_tok, const int32_t* draft,
                        int draft_len, int* accepted_len, int32_t* next_tok);

/* Batched, ragged form: one step for each of the kv handle's `batch` sequences.
 * last_tok[B], drafts[B * ANPD_K_MAX] (row b at b*ANPD_K_MAX), draft_len[B]; results [B]. */
anpd_status anpd_verify_batch(anpd_model* m, anpd_kv* kv, const int32_t* last_tok,
                              const int32_t* drafts, const int* draft_len,
                              int* accepted_len, int32_t* next_tok);

/* Parity hook: the same forward for sequence 0, logits of the draft_len+1 rows copied to
 * logits_host [(draft_len+1) * vocab] fp32; the cache length is left unchanged. */
anpd_status anpd_verify_logits(anpd_model* m, anpd_kv* kv, int32_t last_tok, const int32_t* draft,
                               int draft_len, float* logits_host);

/* Verification of two candidates in one step (the Conclusion's outlook: several candidates verified in parallel), for a
 * kv handle of batch 1, the candidates brought by the host: draft_a [len_a] and draft_b [len_b], len_a >= 1, len_b >= 1,
 * len_a + len_b <= ANPD_K_MAX (else ANPD_ERR_RANGE).  One forward over rows {last_tok, draft_a, draft_b}: the rows of
 * draft_b take the positions right after last_tok again and attend to the committed context, last_tok and themselves,
 * not to draft_a.  Each candidate's accepted prefix is found as in anpd_verify; the longer one is committed (draft_a on a
 * tie): *chosen = 0 or 1, *accepted_len its accepted length, *next_tok the model's token after it, cache length =
 * kv_len + accepted_len + 1, and the cache holds the chosen candidate's rows at their positions.  logits_host: NULL, or
 * host memory for the (1 + len_a + len_b) * vocab fp32 logits of the rows in the order above (parity hook). */
anpd_status anpd_verify_two_candidates(anpd_model* m, anpd_kv* kv, int32_t last_tok, const int32_t* draft_a, int len_a,
                                       const int32_t* draft_b, int len_b, int* accepted_len, int32_t* next_tok,
                                       int* chosen, float* logits_host);

/* Asynchronous layer under anpd_verify_batch, for timing with events on the model's stream:
 * stage copies the step's inputs for all sequences to the device; enqueue issues the forward,
 * accept and commit; result waits and reads the outcome.  enqueue may be called repeatedly
 * without re-staging, but between two enqueues the library must learn the cache lengths again:
 * either anpd_verify_result, or anpd_kv_truncate for every sequence; otherwise ANPD_ERR_STATE. */
anpd_status anpd_verify_stage(anpd_model* m, anpd_kv* kv, const int32_t* last_tok,
                              const int32_t* drafts, const int* draft_len);
anpd_status anpd_verify_enqueue(anpd_model* m, anpd_kv* kv);
anpd_status anpd_verify_result(anpd_model* m, anpd_kv* kv, int* accepted_len, int32_t* next_tok);

/* ---- Algorithm 1 ------------------------------------------------------------------------
 * prompt -> Initialize + prefill -> repeat {commit, Update, draft K, verify, accept} until
 * max_new tokens are out; the result is cut to max_new.  K == 0 is plain greedy decoding
 * through the same kernels at the same row count, so the two token streams are bit-identical.
 * kv and ctx are reset first.  out: int32[max_new]; *n_out = max_new on success.  Capacity is
 * checked before any work: the context needs prompt_len + max_new + 9 <= max_ctx and the cache
 * prompt_len + max_new + 16 <= max_len (the loop may overshoot max_new by up to K tokens and
 * every step writes 8 rows); otherwise ANPD_ERR_CAPACITY is returned with out and n_out
 * untouched.  stats may be NULL. */
anpd_status anpd_generate(anpd_model* m, anpd_kv* kv, anpd_ngram* ctx, const int32_t* prompt,
                          int prompt_len, int max_new, int K, int32_t* out, int* n_out,
                          anpd_stats* stats);

/* anpd_generate with the prompt and the output in DEVICE memory (int32 on the model's device):
 * no host buffer is touched except the few bytes of loop control read back per step.  Token ids
 * are validated on the device (ANPD_ERR_RANGE after the fact). */
anpd_status anpd_generate_dev(anpd_model* m, anpd_kv* kv, anpd_ngram* ctx, const int32_t* prompt_dev,
                              int prompt_len, int max_new, int K, int32_t* out_dev, int* n_out,
                              anpd_stats* stats);

/* Batch of independent sequences sharing one weight stream per step: ctxs[B], prompts
 * [B * prompt_len] (equal lengths), out [B * max_new], stats [B] or NULL. */
anpd_status anpd_generate_batch(anpd_model* m, anpd_kv* kv, anpd_ngram* const* ctxs,
                                const int32_t* prompts, int prompt_len, int max_new, int K,
                                int32_t* out, anpd_stats* stats);

/* ---- measurement ------------------------------------------------------------------------ */
anpd_status anpd_profile_enable(anpd_model* m, int on); /* on: time every launch with events */
anpd_status anpd_profile_read(anpd_model* m, anpd_profile* out, int reset);
/* Number of kernel launches issued by this library since the last reset (all handles). */
long long anpd_launch_count(int reset);

/* Test hook for the projections inside LLM(drafts) (Section 3.1, "Verification"):
 * out[rows][N] = A[rows][K] x W[N][K]^T through the library's weight-streaming GEMM kernel, on
 * the current device and the default stream.  W: N*K bf16 bit patterns (host); A: rows*K fp32
 * (host), rows a multiple of 8 and at most 128; K a multiple of 8.  plain: 0 = the stream-K
 * tensor-core kernel (steps of several sequences, prefill passes), 1 = the one-warp-per-feature
 * kernel it is cross-checked against, 2 = the row-range tensor-core kernel of single-sequence
 * steps (rows must be 8). */
anpd_status anpd_debug_gemm(const uint16_t* w_bf16, int N, int K, const float* a, int rows, float* out, int plain);

/* The same product as anpd_debug_gemm for callers that must not allocate device memory; the paper
 * has no counterpart for this call.  It exists for code that cannot afford a cudaMalloc inside the
 * library: a serving loop that an allocation's device-wide synchronisation would stall, or a process
 * whose device memory is wholly owned by another allocator, where a hidden allocation can fail.
 * All buffers are the caller's and live on the current DEVICE: w_bf16_dev N*K bf16 bit patterns
 * (row-major [N][K]), a_dev rows*K fp32, out_dev rows*N fp32 (written).  Work is issued on cuda_stream
 * and the call returns after it has completed.  Every temporary lives in one fixed array of about
 * 7 MiB that each GPU holds from the moment it loads the library until the process exits; the call
 * never calls cudaMalloc, cudaFree or any allocating routine.
 * Limits: rows a multiple of 8, at most 32; K a multiple of 8; ceil(N/128) * ceil(K/64) <= 128.
 * Larger sizes return ANPD_ERR_CAPACITY (and say so on stderr) without touching anything.
 * The array is shared by all calls on a device and keeps the previous call's contents; the call
 * clears what must start at zero itself.  Calls that overlap on the GPU (two streams, two threads)
 * race on it: issue them one after the other.  The first call on a device looks up the array's
 * device address; make that first call before any stream capture begins.  Every call waits for
 * its work on cuda_stream and reads a status word back before it returns. */
anpd_status anpd_gemm_static(const uint16_t* w_bf16_dev, int N, int K, const float* a_dev, int rows,
                             float* out_dev, void* cuda_stream);

const char* anpd_status_string(anpd_status s);

#ifdef __cplusplus
}
#endif
#endif /* ANPD_H */
