/*
 * ssd.h -- C ABI of the speculative-sampling verification path on one sm_100a GPU.
 *
 * The library computes, entirely in its own CUDA kernels, what the paper's Section
 * "Autoregressive vs Speculative Sampling" and Section "Speculative Sampling" (Figure 2)
 * describe: the target model scores the pending token and K draft tokens in ONE decoder
 * forward against its key/value cache (Section "KV Caching", Figure 1), the draft tokens are
 * accepted or rejected left to right, one more token is drawn by the target, and both models'
 * caches are cut back to the accepted prefix (Section "So, what's the problem?").
 *
 * Conventions
 *  - Every function returns SSD_OK (0) or a negative ssd_status.  Argument errors are found on
 *    the host before anything is launched.  Nothing throws, aborts or exits.
 *  - "dev_" pointers are device memory, "host_" pointers are host memory.  The library never
 *    allocates or frees device memory: weights, cache slab, workspace and all in/out arrays
 *    belong to the caller and must stay valid until the work queued on the stream has run.
 *    Handles (ssd_model, ssd_kv) own small host structs only.
 *  - All calls queue work on the caller's stream (a cudaStream_t passed as void*) and return
 *    without waiting, except kv_lengths and ssd_device_status which synchronise that stream.
 *  - One stream per ssd_kv and per workspace at a time; calls that share either must be
 *    ordered on the same stream.
 *  - Everything runs on the current device.
 *
 * Tensors of a model (ssd_model_create), in this order; a tensor an architecture does not
 * have is passed as NULL:
 *     tok_emb [vocab, d], pos_emb [max_pos, d] (learned positions only),
 *     per layer: ln1_g [d], ln1_b [d], w_qkv [3d, d], b_qkv [3d], w_o [d, d], b_o [d],
 *                ln2_g [d], ln2_b [d], w_in [d_ff or 2*d_ff, d], b_in, w_out [d, d_ff], b_out [d],
 *     lnf_g [d], lnf_b [d], w_lm [vocab, d] (NULL when tie_lm_head).
 * Matrices are row-major [out_features, in_features] in the model dtype (fp32, or bf16);
 * vectors are fp32.  w_qkv rows are Q, then K, then V, each head-major.  For SwiGLU w_in rows
 * [0, d_ff) are the gate and [d_ff, 2 d_ff) the up projection.
 *
 * The KV cache slab (kv_init) is laid out [layer][sequence][K|V][head][position][head_dim] in the
 * model dtype behind a small header that holds the per-sequence lengths and a sticky status
 * word; a bf16 model stores keys (after rotary) and values rounded to bf16.
 */
#ifndef SSD_H_
#define SSD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ssd_model ssd_model; /* opaque */
typedef struct ssd_kv ssd_kv;       /* opaque */

typedef enum {
    SSD_OK = 0,
    SSD_E_ARG = -1,      /* NULL pointer, negative size, K out of range ... */
    SSD_E_SHAPE = -2,    /* architecture the kernels do not cover (see ssd_model_create) */
    SSD_E_CAPACITY = -3, /* rows would not fit the cache / workspace / position table */
    SSD_E_CUDA = -4,     /* a CUDA runtime or driver call failed */
    SSD_E_TIMEOUT = -5,  /* a bounded device-side wait gave up (reported by ssd_device_status) */
    SSD_E_UNIMPL = -6
} ssd_status;

typedef struct {
    int32_t n_layers, d_model, n_heads, head_dim, d_ff, vocab, max_pos;
    int32_t norm;              /* 0 LayerNorm, 1 RMSNorm */
    int32_t act;               /* 0 GELU (erf form), 1 SwiGLU */
    int32_t pos;               /* 0 learned absolute positions, 1 rotary (half-split pairing) */
    int32_t parallel_residual; /* 1: x + Attn(LN1 x) + MLP(LN2 x) */
    int32_t has_bias, tie_lm_head;
    int32_t dtype;             /* 0 fp32, 1 bf16 (matrices and KV cache) */
    int32_t rotary_dim;
    float rotary_base, norm_eps;
} ssd_arch;

enum { SSD_MAX_ROWS = 64,        /* rows (sequences x rows per sequence) of one forward */
       SSD_MAX_ROWS_PER_SEQ = 32 /* K + 1 <= 32 */ };

/*
 * Bind an architecture to caller-owned device tensors (order above, n_tensors = 2 + 12 L + 3).
 * Borrows the pointers; copies only the descriptor table into dev_desc (bf16 models; see
 * ssd_model_desc_bytes; NULL / 0 for fp32 models).  Covered: head_dim <= 128 and a multiple of 8,
 * n_heads * head_dim == d_model, rotary_dim even and <= head_dim; bf16 models additionally need
 * d_model, d_ff >= 128 and multiples of 8, vocab >= 128 (rows are fetched by tensor-map copies
 * of 128 x 64 elements).  Anything else: SSD_E_SHAPE.
 * (The decoder the target and draft models run: Eq. 1; block families named in Section
 * "Solution" / "Experiments": GPT-2, Dolly V2 = GPT-NeoX, Llama-2.)
 */
int ssd_model_create(const ssd_arch *arch, const void *const *dev_weights, int n_tensors, void *dev_desc,
                     size_t desc_bytes, ssd_model **out);

/* Bytes of the caller-owned device block a bf16 model needs for its descriptor table (tensor maps
 * of the matrices and pointers to the vectors, which the forward kernel walks on the device); 0 for
 * fp32 models.  Pass a 256-byte aligned block of at least this size to ssd_model_create, which
 * fills it once with a synchronous copy; it must outlive the model and its layer-skip drafts. */
size_t ssd_model_desc_bytes(const ssd_arch *arch);

/* Workspace bytes of the many-row prompt pass for `batch` sequences x rows_per_seq rows per pass
 * (rows_per_seq is cut to 8192 / batch); 0 when the model has no such pass (fp32 weights, a head
 * dimension that is not a multiple of 16, widths that are not multiples of 8). */
size_t ssd_prefill_workspace_bytes(const ssd_model *m, int batch, int rows_per_seq);

/* Which form kv_prefill takes: 0 (default) the many-row form from 256 rows per pass, 1 never,
 * 2 wherever the model and the workspace allow it (for tests on small shapes), 3 as 2 but with the
 * causal attention on warp-level MMAs also where the tcgen05 form (head dimension 128) applies.
 * SSD_E_ARG otherwise. */
int ssd_set_prefill_mode(int mode);

/* bf16 models run the whole forward as one cooperative kernel by default; 0 selects one launch per
 * step instead (same results up to fp32 summation order; kept for comparison). */
int ssd_set_persistent(int enable);

/* The single forward kernel has three forms of the K-query attention over the cache (Section "KV Caching":
 * the new rows attend to the stored keys / values): items on warp-level MMAs over 16-row tiles, 64 positions
 * per step; - head dimension 128 only - items on the tcgen05 tensor core with the scores in tensor memory,
 * 128 positions per step; and - passes of at most eight rows per sequence at head dimension 64 or 128 (draft
 * steps, decode steps, verification with K <= 7) - warp-level MMA items that carry the bf16 hi and lo parts of
 * the queries and of the probabilities in one 16-row tile, each warp on position blocks of its own.  mode 0
 * (default) picks per pass (the third form where it applies, else tensor-core items from 1024 positions per
 * split, else the first), 1 forces the first form, 2 the second wherever it applies, 3 the third where it
 * applies and the first elsewhere.  Same results up to fp32 summation order; for comparison and tests.
 * SSD_E_ARG for any other mode. */
int ssd_set_attention_mode(int mode);

/* A layer-skip draft: the first n_layers layers of `target` plus its final norm and LM head
 * (an early-exit style draft, cf. Section "Speculative Sampling").  Shares the target's tensors. */
int ssd_model_share_prefix(const ssd_model *target, int n_layers, ssd_model **draft_out);

void ssd_model_destroy(ssd_model *m);

/* Bytes of the cache slab for `batch` sequences of up to max_len positions (header included). */
size_t ssd_kv_bytes(const ssd_model *m, int batch, int max_len);

/* Bytes of workspace a forward over `batch` sequences with up to rows_per_seq rows each needs,
 * when the cache holds up to max_len positions.  batch * rows_per_seq <= SSD_MAX_ROWS. */
size_t ssd_workspace_bytes(const ssd_model *m, int batch, int rows_per_seq, int max_len);

/*
 * Wrap a caller-owned slab (256-byte aligned, >= ssd_kv_bytes) as the KV cache of `batch`
 * sequences; queues the zeroing of the whole slab on `stream`: header (all lengths 0, status
 * clear) and cache.  Attention reads whole position tiles and masks what lies beyond a sequence's
 * length, so those bytes must always be finite numbers: zeros at first, later only rows that earlier
 * passes wrote.
 * (Section "KV Caching": keys/values of past tokens are stored so later passes reuse them; one
 * cache per model, Section "So, what's the problem?".)
 */
int kv_init(const ssd_model *m, int batch, int max_len, void *dev_buf, size_t bytes, void *stream, ssd_kv **out);
void kv_destroy(ssd_kv *kv);

/*
 * Prompt pass: feeds dev_tokens[b, 0 .. n_tokens[b]) of every sequence (row stride max_tokens) and
 * commits them, so the cache holds n_tokens[b] more rows.  No logits are produced.
 * dev_n_tokens: int32 [batch] on the device, values <= max_tokens.
 * Two forms, chosen by the workspace the caller passes:
 *  - bf16 models whose workspace holds ssd_prefill_workspace_bytes(m, batch, c) for some c with
 *    batch * c >= 256 rows take the many-row form: equal passes of up to 8192 / batch rows per sequence
 *    (the largest the workspace fits), every linear layer as a tiled tcgen05 GEMM over 128 rows x 256
 *    weight rows per CTA with the activations as bf16 hi + lo, causal attention over 64-row tiles
 *    against the cache.  Compute-bound; the arithmetic is that of the few-row passes up to fp32
 *    summation order.
 *  - otherwise chunks through the few-row forward: as many rows per sequence as SSD_MAX_ROWS / batch,
 *    SSD_MAX_ROWS_PER_SEQ and the workspace allow (size it with ssd_workspace_bytes for that many rows
 *    to get the fewest passes); every pass streams all weights once.
 * Errors as the forward passes: SSD_E_CAPACITY when the prompt does not fit the cache or the workspace
 * holds not even a one-row pass; device-side conditions (a sequence that does not fit, a wait that ran
 * out) through the cache's status word.
 * (Section "KV Caching", Figure 1: the pass that fills the cache before sampling starts.)
 */
int kv_prefill(ssd_model *m, ssd_kv *kv, const int32_t *dev_tokens, const int32_t *dev_n_tokens, int max_tokens,
               void *dev_ws, size_t ws_bytes, void *stream);

/*
 * One draft step (Section "Speculative Sampling": the small model is called a few times in a row to
 * propose tokens).  Feeds n_in[b] (1..rows_in) rows per sequence -- the tokens the draft cache has
 * not seen yet -- commits them to the draft cache, turns the LAST fed row's logits into
 * q = softmax(logits / temperature), draws x~ = inverse-CDF(q, u[b]) and writes both.
 *   dev_tokens_in  int32, token j of sequence b at [b * tokens_stride + j], j < rows_in (1 or 2)
 *   dev_n_in       int32 [batch] or NULL (= rows_in for every sequence)
 *   dev_u          fp32, one uniform in [0,1) per sequence at [b * u_stride]
 *   dev_token_out  int32, written at [b * token_out_stride]
 *   dev_q_out      fp32 [vocab] per sequence at [b * q_stride] (element stride; the full row is
 *                  written: it is an input of target_verify)
 * temperature == 0 selects greedy: q is the one-hot at the argmax (lowest index on ties).
 */
int draft_step(ssd_model *draft, ssd_kv *dkv, const int32_t *dev_tokens_in, int tokens_stride, int rows_in,
               const int32_t *dev_n_in, float temperature, const float *dev_u, int u_stride,
               int32_t *dev_token_out, int token_out_stride, float *dev_q_out, size_t q_stride, void *dev_ws,
               size_t ws_bytes, void *stream);

/*
 * The draft loop of an iteration - n_steps draft steps - as one call (Section "Speculative Sampling": the draft
 * model proposes a short run of tokens before the target looks at them; Section "So, what's the problem?": the
 * draft keeps a cache of its own, which this call advances by every row it feeds).  Step 0 is draft_step's
 * (rows_in catch-up rows, n_in of them per sequence); step s > 0 feeds the token step s - 1 drew.  Step s reads
 * its uniform at dev_u[b * u_stride + s], writes its token to dev_tokens_out[b * token_out_stride + s] and its
 * q row to dev_q_out + b * q_stride + s * vocab (element strides; q_stride >= n_steps * vocab): with
 * token_out_stride = K + 1 and q_stride = K * vocab these are columns 1.. of target_verify's row block and its
 * q block.  bf16 models run all steps in ONE launch of the forward kernel, which ends every step itself (q, draw,
 * commit spread over the grid) and goes on without returning to the host, its weight stream running on across
 * the steps; other models, and any call made while a sampling restriction is set, run the same steps as
 * separate draft_step calls.  1 <= n_steps <= SSD_MAX_ROWS_PER_SEQ; results as n_steps calls of draft_step.
 */
int draft_steps(ssd_model *draft, ssd_kv *dkv, int n_steps, const int32_t *dev_tokens_in, int tokens_stride,
                int rows_in, const int32_t *dev_n_in, float temperature, const float *dev_u, int u_stride,
                int32_t *dev_tokens_out, int token_out_stride, float *dev_q_out, size_t q_stride, void *dev_ws,
                size_t ws_bytes, void *stream);

/*
 * The verification step (Section "Autoregressive vs Speculative Sampling": the target model scores
 * all K draft tokens in one pass; Figure 2).  One forward over K+1 rows per sequence
 *   dev_rows[b, 0..K] = pending token, x~_1 .. x~_K                 (int32, row stride K+1)
 * at positions len[b] .. len[b]+K against the cache, giving p_1 .. p_{K+1} = softmax(logits / T);
 * then per sequence, left to right: accept x~_i iff u_i * q_i(x~_i) < p_i(x~_i) (i.e. with
 * probability min(1, p/q)); at the first rejection draw the next token from
 * max(0, p_i - q_i) renormalised (from p_i if that residual is all zero); if all K are
 * accepted draw it from p_{K+1}; both draws by inverse CDF with u_{K+1}.
 *   dev_q           fp32 [batch, K, vocab] draft distributions (ignored when K == 0)
 *   dev_u           fp32 [batch, K+1]: K acceptance uniforms, then the resampling uniform
 *   dev_n_accepted  int32 [batch] out
 *   dev_next_token  int32 out at [b * next_token_stride]
 *   dev_p_debug     fp32 [batch, K+1, vocab] out or NULL: the p rows the decisions used
 * The K+1 key/value rows are written to the cache but NOT committed: the lengths stay as they
 * were until kv_commit.  K == 0 is the plain autoregressive decode step.  temperature == 0 is
 * greedy (one-hot distributions; the rule reduces to "x~_i equals the target argmax").
 */
int target_verify(ssd_model *target, ssd_kv *tkv, const int32_t *dev_rows, int K, const float *dev_q,
                  const float *dev_u, float temperature, int32_t *dev_n_accepted, int32_t *dev_next_token,
                  int next_token_stride, float *dev_p_debug, void *dev_ws, size_t ws_bytes, void *stream);

/*
 * Keep dev_n_keep[b] of the rows the last forward left uncommitted (length += n_keep).  NULL
 * keeps n_accepted + 1 as the last target_verify on this cache left it on the device.
 * Rejected rows are not erased: they lie beyond the length and are overwritten later
 * (Section "So, what's the problem?": no redundant calculation, no copy).
 * n_keep[b] is at most the number of rows of that forward.  A length that would exceed the cache's
 * capacity is clamped to it and SSD_E_CAPACITY is recorded in the sticky status word.  The host plans the
 * attention splits of a pass from an upper bound of the lengths, which the bookkeeping kernels keep close
 * to the real lengths and kv_lengths makes exact; a caller that makes a length jump in another way (a cache
 * it filled itself, then a large n_keep) calls kv_lengths before the next forward.
 */
int kv_commit(ssd_kv *kv, const int32_t *dev_n_keep, void *stream);

/* Cut sequences back: length[b] = min(length[b], dev_new_len[b]) (int32 [batch] on the device).  Rows beyond
 * the new length are not erased; later passes overwrite them.  This is how rejected draft rows leave a cache
 * and how a caller resynchronises a cache with a token sequence of its own choice: cut back, then feed the
 * other tokens.  After a cut and a re-feed the cache equals the cache of a fresh prompt pass over the same
 * tokens.  (Section "So, what's the problem?": the caches of both models are fixed up to the accepted
 * prefix, and nothing that is still valid is computed again.) */
int kv_rollback(ssd_kv *kv, const int32_t *dev_new_len, void *stream);

/*
 * Bookkeeping of one speculative iteration, on the device, after target_verify (K >= 0):
 *   target cache: length += a + 1;   draft cache (may be NULL): length = min(n + a, n + K - 1)
 *   with n = committed tokens before the iteration (= old target length + 1);
 *   emitted tokens x~_1..x~_a, y appended to dev_out_tokens[b, count[b]..] (row stride out_cap;
 *   tokens beyond out_cap are dropped, the count still advances); dev_rows[b, 0] = y (the next
 *   pending token); the draft's next catch-up rows: dev_draft_in[b] = {y}, n_in = 1, or
 *   {x~_K, y}, n_in = 2 when all K were accepted.  dev_out_*, dev_draft_* may be NULL.
 */
int spec_advance(ssd_kv *tkv, ssd_kv *dkv, int32_t *dev_rows, int K, const int32_t *dev_n_accepted,
                 const int32_t *dev_next_token, int next_token_stride, int32_t *dev_out_tokens, int out_cap,
                 int32_t *dev_out_count, int32_t *dev_draft_in, int32_t *dev_draft_n_in, void *stream);

/*
 * Restrict sampling to the most probable tokens (Section "Autoregressive vs Speculative Sampling" names
 * sampling "from top-p" beside the argmax; the paper gives no formula, the reading is): for every row of both
 * models, after softmax(logits / T), (1) top_k > 0: t = the top_k-th largest probability, tokens with p >= t
 * stay (ties with t all stay); (2) 0 < top_p < 1, on what (1) kept: t = the probability at which the running
 * sum over tokens of decreasing probability first reaches top_p x (mass kept by (1)), tokens with p >= t stay;
 * (3) the others get 0 and the kept ones are divided by their mass.  draft_step then exports and samples the
 * restricted q, target_verify / verify_from_logits apply the accept / resample rule to the restricted p (and
 * expect q restricted the same way), so the emitted tokens follow the restricted target distribution.
 * top_k = 0 and top_p = 1 (the default) switch it off; greedy rows (temperature 0) are unaffected.  Applies to
 * the calls queued afterwards; verify_from_logits_noalloc returns SSD_E_UNIMPL while a restriction is set.
 * SSD_E_ARG for top_k < 0 or top_p outside (0, 1].
 */
int ssd_set_sampling(int top_k, float top_p);

/* Copy the committed lengths to the host (synchronises the stream). */
int kv_lengths(ssd_kv *kv, int32_t *host_out, void *stream);

/* Read the cache's sticky device-side status word (0 or a negative ssd_status set by a kernel:
 * SSD_E_CAPACITY when rows did not fit, SSD_E_TIMEOUT when a bounded wait gave up).
 * Synchronises the stream. */
int ssd_device_status(ssd_kv *kv, int32_t *host_out, void *stream);

/* Stand-alone vocabulary-wide tail on caller-supplied logits (the accept / resample rule of
 * target_verify without the forward): dev_logits fp32 [batch, K+1, vocab].  Same outputs. */
int verify_from_logits(const float *dev_logits, int batch, int K, int vocab, const int32_t *dev_rows,
                       const float *dev_q, const float *dev_u, float temperature, int32_t *dev_n_accepted,
                       int32_t *dev_next_token, int next_token_stride, float *dev_p_debug, void *dev_scratch,
                       size_t scratch_bytes, void *stream);
size_t verify_scratch_bytes(int batch, int K);

/*
 * verify_from_logits without any scratch argument, for callers that must not allocate device
 * memory: code that runs inside someone else's memory plan (a serving runtime that hands out a
 * fixed arena and forbids cudaMalloc after start-up), inside a region where an allocation would
 * synchronise the device or fail (a latency-critical decode loop, a process whose memory is fully
 * committed to weights and KV cache), or from a language binding that can pass pointers through
 * but cannot own CUDA buffers.  The paper has no counterpart of this call; it is a packaging of the
 * same tail for such callers.
 *
 * The statistics that the two tail kernels pass to each other are kept in a fixed array inside
 * the library (SSD_NOALLOC_MAX_ROWS entries of 16 bytes = 64 KB, present on every GPU that loads
 * the library, for the life of the process).  Inputs and outputs are still the caller's.
 *   - batch * (K + 1) > SSD_NOALLOC_MAX_ROWS is refused with SSD_E_CAPACITY; nothing is launched.
 *   - The call never calls cudaMalloc / cudaFree or any allocating routine.
 *   - The first call on each device looks up the array's device address (a host-side query with
 *     that device current); make that first call outside any stream capture.
 *   - All calls on a device share the one array, and it keeps the previous call's contents.  Each
 *     call overwrites every entry it later reads, so stale contents are harmless; but two calls
 *     whose kernels overlap on the GPU (different streams, no ordering) race on it.  Order them.
 * Results are identical to verify_from_logits.
 */
enum { SSD_NOALLOC_MAX_ROWS = 4096 };
int verify_from_logits_noalloc(const float *dev_logits, int batch, int K, int vocab, const int32_t *dev_rows,
                               const float *dev_q, const float *dev_u, float temperature,
                               int32_t *dev_n_accepted, int32_t *dev_next_token, int next_token_stride,
                               float *dev_p_debug, void *stream);

/* Attention of one layer alone, for long-context checks: q fp32 [batch, rows, d] (already
 * position-encoded) against the cache of `layer`; row j of sequence b sees positions
 * 0 .. len[b] + j.  Output fp32 [batch, rows, d]. */
int attention_rows(ssd_model *m, ssd_kv *kv, int layer, const float *dev_q, int rows, float *dev_out,
                   void *dev_ws, size_t ws_bytes, void *stream);

/* Copy the logits the last forward left in the workspace (fp32 [batch, rows_per_seq, vocab]; the
 * conditional of Eq. 1 before the softmax) to dev_out, for inspection.  batch and rows_per_seq
 * must be those of that forward. */
int ssd_last_logits(const ssd_model *m, int batch, int rows_per_seq, const void *dev_ws, size_t ws_bytes,
                    float *dev_out, void *stream);

/* Profiling aid for the single-kernel forward, whose phases no external profiler can separate:
 * when enabled, one CTA stamps the GPU's nanosecond timer at kernel start, after every grid
 * barrier and at its end.  ssd_read_trace copies the stamps of the last forward that used this
 * workspace (same batch / rows_per_seq) to the host; consecutive differences are phase durations
 * in the order: set-up, embedding, then per layer [qkv(+MLP-in), attention, out-proj(+MLP-out),
 * statistics] (parallel residual) or [qkv, attention, out-proj, statistics, MLP-in, MLP-out,
 * statistics] (sequential), then the LM head.  Synchronises the stream.  Off by default. */
int ssd_set_trace(int enable);
int ssd_read_trace(const ssd_model *m, int batch, int rows_per_seq, const void *dev_ws, size_t ws_bytes,
                   uint64_t *host_out, int max_entries, int *n_out, void *stream);

/* Failure detection.  Every device-side wait is bounded: a wait that takes work (a weight tile, an operand,
 * a grid barrier, a count of finished attention items) gives up after `cycles` GPU clock cycles, records
 * SSD_E_TIMEOUT in the cache's sticky status word, and its kernel stops taking work, waits for its own
 * copies in flight (those drain waits keep the default bound), releases its tensor memory and returns, so
 * the context stays usable.  0 restores the default of about two seconds; negative: SSD_E_ARG.
 * ssd_wait_probe exercises that path without disturbing anything else: it queues a one-thread kernel that
 * waits, with the configured bound, on a barrier nobody ever arrives at; after it has run,
 * ssd_device_status(kv) reports SSD_E_TIMEOUT.  (No counterpart in the paper: housekeeping.) */
int ssd_set_wait_limit(long long cycles);
int ssd_wait_probe(ssd_kv *kv, void *stream);

/* Number of kernels this library has launched in this process so far. */
uint64_t ssd_launch_count(void);

/* Device time attributed to the kernel that streams the weights -- the single forward kernel of a
 * bf16 model, or every GEMM launch on the one-launch-per-step path: when enabled, each such launch
 * is bracketed by CUDA events on its stream; ssd_gemm_profile_read synchronises and returns the
 * launches and total milliseconds since the last reset.  Off by default. */
int ssd_gemm_profile(int enable);
int ssd_gemm_profile_read(uint64_t *launches, double *total_ms, int reset);

const char *ssd_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* SSD_H_ */
