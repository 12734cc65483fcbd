/*
 * csd.h - C ABI of the review-step library for Cascade Speculative Drafting (arXiv 2312.11462).
 *
 * The library is hand-written CUDA for sm_100a.  It never allocates device memory: every device
 * buffer (weights, KV cache and activations inside a workspace, logits, token buffers) is
 * allocated by the caller and passed in as a plain pointer.  Handles (csd_model, csd_mag) are
 * small host objects owned by the library and released by the matching *_destroy call.
 *
 * Conventions
 *   - A pointer named *_dev is device memory, *_host is host memory.  Device buffers must stay
 *     valid until the stream has passed the call.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  All calls except
 *     csd_cascade_generate and csd_device_status only enqueue work; argument and shape errors
 *     are returned synchronously and nothing is enqueued in that case.
 *   - Errors found on the device (token id outside [0, vocab), a probe limit reached) never trap:
 *     the kernel records a code in a status word, substitutes a safe value and carries on;
 *     csd_device_status waits for the stream and returns-and-clears that word.
 *   - No call falls back to the CPU.  Without a CUDA device every compute call returns
 *     CSD_ERR_CUDA.
 */
#ifndef CSD_H
#define CSD_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    CSD_OK = 0,
    CSD_ERR_INVALID_ARG = 1, /* null pointer, negative size, value out of its documented range */
    CSD_ERR_SHAPE = 2,       /* a model dimension the kernels do not support                    */
    CSD_ERR_CAPACITY = 3,    /* kv_len + m > max_seq, workspace too small, block too long        */
    CSD_ERR_OOM = 4,         /* host allocation of a handle failed                              */
    CSD_ERR_CUDA = 5,        /* a CUDA runtime call failed (see csd_last_cuda_error)            */
    CSD_ERR_BAD_TOKEN = 6,   /* device status: a token id was outside [0, vocab)                */
    CSD_ERR_TIMEOUT = 7,     /* device status: a bounded probe loop reached its limit           */
    CSD_ERR_UNSUPPORTED = 8
} csd_status;

const char* csd_status_string(csd_status s);
/* Text of the last CUDA runtime error seen by this thread's calls ("" if none). */
const char* csd_last_cuda_error(void);
/* Waits for `stream`, stores the device status word (a csd_status) in *code_out, clears it. */
csd_status csd_device_status(void* stream, int* code_out);

/* ---------------------------------------------------------------------------------------------
 * Models.  The paper names the model families only (Section 5.1: a LLaMA-family 7B target with
 * a 68M draft; FLAN-T5 xxl with base and small drafts), so the architecture constants are the
 * public ones of those families:
 *   arch 0  decoder-only: pre-norm RMSNorm, rotary embedding on head-dim halves (i, i+Dh/2),
 *           scores scaled by 1/sqrt(Dh), SwiGLU feed-forward, untied output head, no biases.
 *   arch 1  encoder-decoder: RMS norm without mean-centring, unscaled scores plus a bucketed
 *           relative-position bias shared by all layers of a stack (bidirectional buckets in
 *           the encoder, causal in the decoder), cross-attention, gated-GELU (tanh form)
 *           feed-forward, untied output head, no biases.
 * Arithmetic: bf16 weights, fp32 activations and accumulation, K/V rounded to bf16
 * (nearest-even) when a position is appended to the cache.
 *
 * Weight blob (device, bf16, every tensor [out, in] row-major and starting on a 256-byte
 * boundary), in this order:
 *   embed [vocab, d_model]
 *   arch 1 only: enc_rel_bias [rel_buckets, n_heads];
 *                per encoder layer { norm1 [d], wq, wk, wv [d_inner, d], wo [d, d_inner],
 *                                    norm2 [d], wgate, wup [d_ff, d], wdown [d, d_ff] };
 *                enc_final_norm [d]; dec_rel_bias [rel_buckets, n_heads]
 *   per decoder layer { norm1, wq, wk, wv, wo,
 *                       arch 1 only: norm_x, xq, xk, xv, xo (cross-attention),
 *                       norm2, wgate, wup, wdown }
 *   final_norm [d]; lm_head [vocab, d_model]
 * with d_inner = n_heads * d_head.
 * ------------------------------------------------------------------------------------------- */
typedef struct csd_model csd_model;

typedef struct {
    int32_t arch;         /* 0 decoder-only, 1 encoder-decoder                              */
    int32_t n_layers;     /* decoder layers                                                  */
    int32_t n_enc_layers; /* encoder layers (arch 1)                                         */
    int32_t d_model;      /* multiple of 8                                                   */
    int32_t n_heads;
    int32_t d_head;       /* 32, 64 or 128                                                   */
    int32_t d_ff;         /* multiple of 8                                                   */
    int32_t vocab;
    int32_t max_seq;      /* decoder KV capacity in positions                                */
    int32_t max_rows;     /* most rows one review forward takes, <= 17                       */
    int32_t max_enc_len;  /* arch 1: most encoder positions                                  */
    int32_t rel_buckets;  /* arch 1: relative-position buckets (32)                          */
    int32_t rel_max_dist; /* arch 1: distance at which buckets saturate (128)                */
    float norm_eps;
    float rope_theta;     /* arch 0                                                          */
} csd_model_config;

#define CSD_MAX_ROWS 17

size_t csd_model_weight_bytes(const csd_model_config* cfg);
/* Workspace = KV cache (+ cross-attention K/V), activations, split partials, tables. */
size_t csd_model_workspace_bytes(const csd_model_config* cfg);

/* Binds a model to caller-owned weights and workspace (both device, 256-byte aligned, at least
 * the sizes above; the caller keeps them alive until csd_model_destroy).  Enqueues the
 * one-off table set-up (rotary cos/sin, relative-position bias by distance) on `stream`. */
csd_status csd_model_create(const csd_model_config* cfg, const void* weights_bf16_dev, size_t weight_bytes,
                            void* workspace_dev, size_t workspace_bytes, void* stream, csd_model** out);
csd_status csd_model_destroy(csd_model* m);

/* arch 1: runs the encoder over n tokens (1 <= n <= max_enc_len) and fills the static
 * cross-attention K/V of every decoder layer.  Must precede csd_review_forward. */
csd_status csd_encoder_forward(csd_model* m, const int32_t* enc_tokens_dev, int n, void* stream);

/* The review forward: the larger model scores all drafted positions of a block in one pass
 * (Sections 1-2).  One pass over m rows (1 <= m <= max_rows) at positions kv_len .. kv_len+m-1:
 * reads cache rows [0, kv_len), OVERWRITES rows [kv_len, kv_len+m), writes logits_out_dev
 * [m, vocab] fp32 row-major; row r is the model's next-token law after position kv_len+r, causal
 * inside the block.  The caller commits accepted positions by passing a larger kv_len next time;
 * rejected rows are simply overwritten (rollback is free).  logits_out_dev == NULL: the block is
 * only appended to the cache (prompt prefill, catching up) and the vocabulary projection is
 * skipped. */
csd_status csd_review_forward(csd_model* m, const int32_t* block_tokens_dev, int n_rows, int kv_len,
                              float* logits_out_dev, void* stream);

/* Batched review: the blocks of several sequences in one pass over the weights (the paper runs
 * batch 1; with k+1 <= 5 rows per sequence three sequences still fit the 17 rows one pass takes,
 * and the weights stream once for all of them).  models[0 .. n_seqs) are handles made from the SAME
 * weights and the same configuration, each with its own workspace, i.e. its own cache (for arch 1
 * each after its own csd_encoder_forward).  block_tokens_dev holds the sequences' rows one after
 * the other (n_rows_host[g] rows of sequence g at positions kv_len_host[g] ..), logits_out_dev
 * [sum of rows, vocab] in the same order (NULL: append only).  The contractions use the buffers of
 * models[0]; every sequence's attention reads and appends its own cache.  Sum of rows <= max_rows.
 * The host arrays are read before the call returns. */
csd_status csd_review_forward_batch(csd_model* const* models, int n_seqs, const int32_t* block_tokens_dev,
                                    const int32_t* n_rows_host, const int32_t* kv_len_host, float* logits_out_dev,
                                    void* stream);

/* Review of a TREE of drafted tokens in one pass (Section 5.1 and Appendix B combine the method
 * with tree attention: several candidate continuations hang off a node and the longest accepted
 * path wins).  Row 0 is the root (the newest token that is not in the cache yet, parent -1); row r
 * is a child of row parent_host[r] < r.  Row r sits at position kv_len + depth(r), attends to cache
 * rows [0, kv_len), to its ancestors and to itself, and logits row r is the model's next-token law
 * after the path from the root to r.  Cache rows [kv_len, kv_len + n_rows) are overwritten with the
 * rows in index order: only rows of a chain 0, 1, 2, .. (parent[r] = r - 1) leave valid cache entries,
 * so put the path most likely to be accepted first and re-feed what was accepted elsewhere.
 * parent_host is read before the call returns.  arch 0 only. */
csd_status csd_review_forward_tree(csd_model* m, const int32_t* block_tokens_dev, const int32_t* parent_host, int n_rows,
                                   int kv_len, float* logits_out_dev, void* stream);

/* Greedy acceptance along the tree reviewed by csd_review_forward_tree: starting at the root, the
 * target's arg-max at the current node is emitted; if a child of the node holds that token (the one
 * with the smallest row index if several do) the walk moves there, else it ends.  The emitted
 * tokens are the target's own greedy continuation (lossless).  out_dev holds 2 + 3 * n_rows int32:
 * [0] = number of tokens emitted (>= 1), [1] = number of leading rows of the accepted path that are
 * the chain 0, 1, 2, .. and therefore already sit in the cache at their positions (>= 1: the root),
 * [2 ..] the emitted tokens, [2 + n_rows ..] the rows of the accepted path (the rest is scratch). */
csd_status csd_tree_accept_greedy(const float* target_logits_dev, const int32_t* tokens_dev, const int32_t* parent_host,
                                  int n_rows, int vocab, int32_t* out_dev, void* stream);

/* Prompt prefill: the model takes the input tokens in one run (Section 2).  Appends n tokens
 * (any n >= 1 with kv_len + n <= max_seq) at positions kv_len .. kv_len+n-1 to the cache of every
 * layer and produces no logits.  Models whose layer matrices are large enough for the tensor-core
 * kernels go through the weights once per 128 tokens (wide blocks, two bf16 terms per fp32
 * activation); the rest, and a remainder of at most max_rows tokens, go through the review
 * kernels.  arch 1: decoder tokens, after csd_encoder_forward. */
csd_status csd_prefill(csd_model* m, const int32_t* tokens_dev, int n, int kv_len, void* stream);

/* Per-kernel-class timing of later forwards of this model (measurement aid; the paper's unit of
 * cost is "a single run" of a model, Section 4).  While enabled, every kernel launch of
 * csd_review_forward is bracketed by a CUDA event pair on the launching stream (a few
 * microseconds of overhead per launch).  csd_model_profile_read waits for the stream, sums the
 * pairs recorded since the last read per class and clears them. */
typedef struct {
    double gemm_ms;            /* weight-streaming GEMM launches                    */
    int64_t gemm_launches;
    double gemm_weight_bytes;  /* bf16 weight bytes those launches streamed         */
    double attn_ms;            /* block-attention launches                          */
    int64_t attn_launches;
    double other_ms;           /* embedding gather, rotary + K/V append             */
    int64_t other_launches;
} csd_profile;
csd_status csd_model_profile(csd_model* m, int enable);
csd_status csd_model_profile_read(csd_model* m, void* stream, csd_profile* out);

/* Y[m, N] = X[m, K] . W[N, K]^T, the weight-streaming contraction every layer of the review
 * forward is made of (W bf16 row-major, X and Y fp32 row-major, fp32 accumulation).  Exposed
 * for kernel-level tests and roofline measurements.  K multiple of 8; 1 <= m <= 17 runs the review
 * kernels, 18 <= m <= 128 the wide-block kernel of the prefill (two bf16 terms per fp32 value, relative
 * error about 1e-5; needs N * K >= 2^20 and K >= 64, CSD_ERR_UNSUPPORTED otherwise). */
size_t csd_linear_workspace_bytes(int m, int N, int K);
/* Which kernel the contraction uses, process-wide: 0 = automatic choice per shape, 1 = the
 * CUDA-core kernel (128-bit streaming loads, fp32 FMA), 2 = the tensor-core kernel (TMA-staged
 * weights, tcgen05.mma with fp32 accumulators in tensor memory) with equal shares of (tile, K block)
 * units per CTA wherever it applies (K >= 64), 3 = the tensor-core kernel in which every CTA owns
 * whole output columns over all of K (no partial sums between CTAs) wherever it applies, 2 elsewhere.
 * All give the same result up to fp32 summation order; the switch exists to measure them. */
csd_status csd_set_gemm_path(int path);
/* Which kernel the block attention uses, process-wide: 0 = automatic (tensor cores, mma.sync on
 * TMA-staged K/V tiles, for head dimensions 64 and 128; the CUDA-core kernel for 32), 1 = always
 * the CUDA-core kernel.  Same result up to fp32 summation order and the 2^-17 relative error of the
 * two-term bf16 form in which q and the softmax weights enter the MMAs. */
csd_status csd_set_attention_path(int path);
csd_status csd_linear(const void* W_bf16_dev, int N, int K, const float* X_dev, int m, float* Y_dev,
                      void* workspace_dev, size_t workspace_bytes, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Review rule (Section 2 "reviewing stage"; Section 3.1 for lenience and the greedy variant).
 * For each of `rows` independent rows: drafted tokens x_1..x_k with draft laws q_i and target
 * laws p_i = softmax(target_logits[i] / T):
 *   temperature > 0: x_i is accepted iff u_i * q_i(x_i) < lenience * p_i(x_i) with u_i uniform
 *     in [0,1); at the first rejection i the output token is drawn from norm(max(0, p_i - q_i))
 *     (from p_i if that is empty); if all k are accepted it is drawn from p_{k+1}.
 *   temperature == 0: greedy review: x_i is accepted iff it is the argmax of target_logits[i]
 *     (ties: smallest index); the output token is the argmax at the first mismatch (or at k).
 * q_i is softmax(draft_logits[i] / T), or the point mass on x_i where draft_logits_dev is NULL
 * or onehot_dev[row, i] != 0 (statistical drafter).  Lenience multiplies p_i only at positions
 * whose proposal carries a law; a point-mass position is tested with lenience 1 (Appendix B: no
 * lenience between the statistical drafter and its reviewer).
 * Uniforms: Philox4x32-10 with key (seed lo, seed hi) and counter (i, row, step lo, step hi);
 * word 0 -> u_i, word 1 -> the resampling uniform of position i; u = (word >> 8) * 2^-24.  The
 * resample is the inverse CDF in vocabulary order (smallest j with cumulative mass > u * total),
 * evaluated in fp64.
 * Layouts: target_logits_dev [rows, k+1, V] fp32, draft_logits_dev [rows, k, V] fp32 or NULL,
 * onehot_dev [rows, k] int32 or NULL, draft_tokens_dev [rows, k] int32; outputs n_accepted_dev
 * [rows], out_token_dev [rows] int32.  0 <= k <= 64.  A token id outside [0, V) is treated as
 * rejected and sets the device status.
 * ------------------------------------------------------------------------------------------- */
size_t csd_spec_accept_workspace_bytes(int rows, int k, int V);
csd_status csd_spec_accept(const float* target_logits_dev, const float* draft_logits_dev,
                           const int32_t* onehot_dev, const int32_t* draft_tokens_dev, int rows, int k, int V,
                           float temperature, float lenience, uint64_t seed, uint64_t step,
                           int32_t* n_accepted_dev, int32_t* out_token_dev, void* workspace_dev,
                           size_t workspace_bytes, void* stream);

/* The same review rule for callers that cannot allocate device memory (the paper has no
 * counterpart; this is a deployment convenience).  Some hosts of this library run where
 * cudaMalloc is off limits: inside a real-time serving loop that forbids allocator calls after
 * start-up, inside a process whose memory budget is fixed by another component, or from code
 * that only holds the buffers it was handed.  csd_spec_accept_static needs no workspace argument:
 * its scratch is a fixed 2 MiB array that is part of the library image (every GPU that loads the
 * library carries it until the process exits; csd_spec_accept_static_capacity returns the size).
 * The call allocates nothing, on the host or on the device, and takes the same inputs and gives
 * the same outputs as csd_spec_accept.  Differences:
 *   - problems whose scratch need (csd_spec_accept_workspace_bytes) exceeds the capacity are
 *     refused with CSD_ERR_CAPACITY; 64 rows x 16 drafted tokens x 128256 logits fits;
 *   - a token id outside [0, V) is still treated as rejected, but is not recorded in the device
 *     status word (recording would need that word to exist, and creating it allocates);
 *   - the first call on each device looks up the device address of the array (with that device
 *     current); make that first call outside any stream capture;
 *   - all calls share the one array, which keeps whatever the previous call left in it.  Nothing
 *     in it has to start at zero, but two calls that overlap on the GPU (different streams) would
 *     overwrite each other's intermediate results: issue them on one stream, or order them. */
size_t csd_spec_accept_static_capacity(void);
csd_status csd_spec_accept_static(const float* target_logits_dev, const float* draft_logits_dev,
                                  const int32_t* onehot_dev, const int32_t* draft_tokens_dev, int rows, int k, int V,
                                  float temperature, float lenience, uint64_t seed, uint64_t step,
                                  int32_t* n_accepted_dev, int32_t* out_token_dev, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Max-Gram statistical drafter (Section 3.3, Appendix A): the longest suffix of the sequence
 * (at most max_order tokens) that occurs in the haystack followed by at least one haystack
 * token, earliest occurrence; the proposal is the haystack tokens after it.  When the haystack
 * ends, or nothing matches (then one token comes from bigram_next[last token]), the search is
 * repeated on the extended sequence until n tokens exist.  Lookup goes through a hash table of
 * all n-grams of orders 1..max_order built once per haystack (exact under collisions: a slot
 * is verified against the haystack).
 * ------------------------------------------------------------------------------------------- */
typedef struct csd_mag csd_mag;
#define CSD_MAG_MAX_ORDER 32
size_t csd_mag_workspace_bytes(int L, int max_order, int table_slots);
/* haystack_dev [L] and bigram_next_dev [V] stay owned by the caller and must outlive the handle.
 * table_slots: 0 = default (power of two >= 2 * L * max_order), else a power of two >= the
 * number of n-grams (tests use small tables to force collisions). */
csd_status csd_mag_create(const int32_t* haystack_dev, int L, int V, const int32_t* bigram_next_dev,
                          int max_order, int table_slots, void* workspace_dev, size_t workspace_bytes,
                          void* stream, csd_mag** out);
csd_status csd_mag_destroy(csd_mag* g);
/* seq_dev [T] (T >= 1), 1 <= n <= 64; writes out_tokens_dev [n] (may alias seq_dev + T). */
csd_status csd_mag_draft(csd_mag* g, const int32_t* seq_dev, int T, int n, int32_t* out_tokens_dev,
                         void* stream);
/* The same search over a haystack that grows with the generation (Section 3.3 takes the match from
 * the input or from the existing generation): the handle's haystack followed by
 * seq_dev[gen_from .. T), 0 <= gen_from <= T.  A match must still be followed by a token of that
 * joined text, and the earliest occurrence wins, so the static part is preferred.  The generated
 * part is scanned directly on every call: it may shrink when a block is rejected. */
csd_status csd_mag_draft_dynamic(csd_mag* g, const int32_t* seq_dev, int T, int gen_from, int n,
                                 int32_t* out_tokens_dev, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Algorithm 1 (CascadeSpeculativeDraftingStep) driven until max_new tokens exist.
 * models[0] is the target, models[1 .. n_levels-1] the neural drafts, largest first; Max-Gram
 * sits below them.  K is n_levels x n_levels, row-major, upper-triangular: K[r][c] is the budget
 * of the slot that level c+1 drafts when level r reviews (level n_levels = Max-Gram, which
 * proposes the slot's remaining budget in one call).  The for-loop over c is the horizontal
 * cascade, the recursion into level c+1 the vertical cascade.  A review takes at most max_block
 * drafted tokens (surplus drafts are dropped, which keeps the output law).  Lenience applies
 * when a draft reviews, never when the target does.  Each level forwards every token it has not
 * cached yet, in chunks of at most the model's max_rows rows (this also serves as prompt prefill).
 * Decoder-only models: haystack = prompt, init_seq = prompt.  Encoder-decoder: haystack =
 * encoder input (the encoders are run here), init_seq = decoder start token(s).
 * dynamic_haystack != 0: Max-Gram also matches inside everything generated so far (the tokens after
 * init_seq, drafts that are still under review included), see csd_mag_draft_dynamic.
 * Host in, host out; the call returns after the stream has finished.
 * ------------------------------------------------------------------------------------------- */
typedef struct {
    int64_t tokens;      /* tokens generated                                           */
    int64_t reviews[8];  /* review calls per level (0 = target)                        */
    int64_t forwards[8]; /* forward passes per level, catch-up chunks included        */
    int64_t drafted[8];  /* drafted tokens presented to the level's reviews            */
    int64_t accepted[8]; /* of which accepted                                          */
    int64_t mag_calls;
    int64_t mag_tokens;
    int64_t kernel_launches; /* kernels this call enqueued                             */
    double prefill_ms;   /* device time until the first target review starts (events)  */
    double decode_ms;    /* device time from there to the last token (events)          */
    double total_ms;     /* host wall time of the whole call, copies included          */
} csd_cascade_stats;

size_t csd_cascade_workspace_bytes(int vocab, int max_block, int seq_capacity, int haystack_len, int max_order);
csd_status csd_cascade_generate(csd_model* const* models, int n_levels, const int32_t* K, int max_block,
                                float lenience, float temperature, uint64_t seed, int max_order,
                                int dynamic_haystack, const int32_t* haystack_host, int haystack_len,
                                const int32_t* bigram_next_dev, const int32_t* init_seq_host, int init_len,
                                int max_new, int32_t* out_tokens_host, int32_t* out_len,
                                csd_cascade_stats* stats,
                                void* workspace_dev, size_t workspace_bytes, void* stream);

/* Host helper, exposed for tests: relative-position bucket of arch 1 (rel = key - query). */
int csd_rel_bucket(int rel, int bidirectional, int n_buckets, int max_dist);

#ifdef __cplusplus
}
#endif
#endif /* CSD_H */
