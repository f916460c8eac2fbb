/*
 * knnssd - decode hot path of KNN-SSD self-speculative decoding on one NVIDIA B200.
 *
 * C ABI of libknnssd.so.  Plain pointers and sizes only; every pointer is marked
 * HOST or DEVICE below.  All functions return a knnssd_status (0 = OK); on a
 * non-OK status found before anything is enqueued (bad arguments, protocol order,
 * capacity) the session (context length, KV cache validity, active skip mask) is
 * left as it was before the call.  A failure found on the device while a pass ran
 * (KNNSSD_ERR_TIMEOUT, KNNSSD_ERR_CUDA, non-finite logits reported as
 * KNNSSD_ERR_DEGENERATE) leaves the cache in an unknown state: the context stays
 * usable but must be prefilled again (calls before that return KNNSSD_ERR_STATE).
 * Nothing aborts or throws across the boundary, and knnssd_last_error() gives a
 * one-line reason.  A context is bound to the CUDA
 * device that was current at knnssd_init and to the stream passed there; calls on
 * one context must not overlap (not thread-safe per context).
 *
 * Notation follows the paper: L decoder layers = 2L sublayers; a skip mask
 * z in {0,1}^{2L} with z[j] = 1 meaning "sublayer j is skipped while drafting"
 * (Sec. 3.1; Sec. 4.1), index 2l = attention sublayer of layer l, 2l+1 = its MLP
 * sublayer; A_i = {a_i1..a_ik} the anchors of domain i (Sec. 4.1, Eq. (2));
 * k = draft length.
 *
 * Session protocol:  init -> prefill -> (select_skipset | set_skipmask)
 *                    -> { draft -> verify }* ;  generate = all of it for one request.
 */
#ifndef KNNSSD_H
#define KNNSSD_H

#ifdef __cplusplus
extern "C" {
#endif

typedef struct knnssd_ctx knnssd_ctx; /* opaque: model view + session state */

typedef enum {
    KNNSSD_OK = 0,
    KNNSSD_ERR_INVALID_ARG = 1, /* NULL pointer, negative size, token id out of range, k > max_draft ... */
    KNNSSD_ERR_SHAPE = 2,       /* configuration the kernels do not support (see knnssd_init) */
    KNNSSD_ERR_CAPACITY = 3,    /* context would exceed max_seq */
    KNNSSD_ERR_STATE = 4,       /* call out of protocol order (e.g. draft before prefill / before a mask is set) */
    KNNSSD_ERR_DEGENERATE = 5,  /* zero or non-finite vector in the cosine search */
    KNNSSD_ERR_CUDA = 6,        /* a CUDA runtime call failed; text in knnssd_last_error */
    KNNSSD_ERR_TIMEOUT = 7      /* a bounded device-side wait gave up (every wait in the kernels has a poll limit) */
} knnssd_status;

typedef struct {
    int n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ff, vocab;
    int max_seq;            /* KV-cache capacity in positions */
    int max_draft;          /* largest k accepted by draft/verify/generate (1..15) */
    float rms_eps, rope_theta;
    int dtype;              /* 0: fp32 weights and KV cache; 1: bf16 weights and KV cache */
    int n_domains;          /* number of domains (may be 0: no anchors, masks set explicitly) */
    int anchors_per_domain; /* anchors per domain */
    int pool_mode;          /* 0: mean of the prompt's last-layer hidden states; 1: last position only */
} knnssd_config;

/* All DEVICE pointers, row-major [out][in], borrowed for the lifetime of the context
 * (the library makes no packed copy; the caller keeps them alive and unchanged).
 * Big matrices are fp32 or bf16 per knnssd_config.dtype; norm gains are always fp32.
 * The per-layer tables themselves are HOST arrays of n_layers DEVICE pointers. */
typedef struct {
    const void *tok_embed;         /* [vocab][d_model] */
    const float *final_norm;       /* [d_model] */
    const void *lm_head;           /* [vocab][d_model] */
    const float *const *attn_norm; /* [d_model] */
    const void *const *wq;         /* [n_heads*head_dim][d_model] */
    const void *const *wk;         /* [n_kv_heads*head_dim][d_model] */
    const void *const *wv;         /* [n_kv_heads*head_dim][d_model] */
    const void *const *wo;         /* [d_model][n_heads*head_dim] */
    const float *const *mlp_norm;  /* [d_model] */
    const void *const *w_gate;     /* [d_ff][d_model] */
    const void *const *w_up;       /* [d_ff][d_model] */
    const void *const *w_down;     /* [d_model][d_ff] */
} knnssd_weights;

typedef struct {
    int rounds;    /* draft+verify rounds run */
    int drafted;   /* draft steps taken (sum of k_eff) */
    int accepted;  /* draft tokens accepted */
    int tokens;    /* tokens emitted */
    float ms_prefill, ms_select, ms_draft, ms_verify; /* device time (CUDA events on the context's stream) */
} knnssd_stats;

/*
 * Create a context for one model and one request at a time.
 *   cfg, w            HOST structs (copied).  Supported: head_dim in {64, 128}, n_heads % n_kv_heads == 0,
 *                     d_model, d_ff, n_heads*head_dim multiples of 8; else KNNSSD_ERR_SHAPE.
 *   anchors_dev       DEVICE fp32 [n_domains*anchors_per_domain][d_model], borrowed; NULL iff n_domains == 0.
 *                     Anchors need not be normalised; a zero or non-finite anchor -> KNNSSD_ERR_DEGENERATE.
 *   skip_masks_host   HOST bytes [n_domains][2*n_layers], the stored per-domain masks z*_i (Sec. 4.1, Eq. (3)),
 *                     copied; NULL iff n_domains == 0.
 *   cuda_stream       a cudaStream_t (NULL = default stream); every kernel of this context runs on it.
 * The context owns the KV cache ([n_layers][n_kv_heads][max_seq][head_dim], K and V) and its work buffers.
 */
knnssd_status knnssd_init(const knnssd_config *cfg, const knnssd_weights *w, const float *anchors_dev,
                          const unsigned char *skip_masks_host, void *cuda_stream, knnssd_ctx **out);
void knnssd_destroy(knnssd_ctx *ctx);

/*
 * Run the full model over the prompt (Sec. 4.2: the new sample's last hidden vector comes from a pass of the
 * model over it): fills the KV cache for positions [0, n_tokens), keeps the pooled last-layer hidden state
 * (after the final RMSNorm) for select_skipset, and makes the greedy token after the prompt the pending token.
 *   tokens_host          HOST int32 [n_tokens], 1 <= n_tokens <= max_seq - 1
 *   pooled_dev_or_null   DEVICE fp32 [d_model]: receives the pooled vector; may be NULL
 *   first_token_or_null  HOST int: receives the pending token; may be NULL
 * Resets the session (length, statistics) first; the active mask is kept.
 */
knnssd_status knnssd_prefill(knnssd_ctx *ctx, const int *tokens_host, int n_tokens, float *pooled_dev_or_null,
                             int *first_token_or_null);

/*
 * Domain choice (Sec. 4.2, Eq. (4)): (i*, j*) = argmax_{i,j} cos(v, a_ij), lowest flat index on ties, then the
 * stored mask of domain i* becomes the active one.
 *   query_dev_or_null  DEVICE fp32 [d_model]; NULL = the pooled vector of the last prefill
 *   domain, anchor, cosine   HOST outputs (each may be NULL)
 * KNNSSD_ERR_DEGENERATE if the query has zero or non-finite norm; KNNSSD_ERR_STATE without anchors.
 */
knnssd_status knnssd_select_skipset(knnssd_ctx *ctx, const float *query_dev_or_null, int *domain, int *anchor,
                                    float *cosine);

/* Make an explicit mask z active (Sec. 3.1: z^(j) = 1 skips sublayer j while drafting; Sec. 4.1: a domain's stored
 * z*_i is such a mask).  mask_host: HOST bytes [2*n_layers], 1 = skipped while drafting. */
knnssd_status knnssd_set_skipmask(knnssd_ctx *ctx, const unsigned char *mask_host);

/*
 * Draft k tokens greedily with M(z), z the active mask (Sec. 4.2, drafting equation): step j feeds the pending
 * token (j = 0) or draft j-1 at position len+j through the retained sublayers only - skipped sublayers read no
 * weights and write no K/V - and takes the arg-max (lowest id on ties).
 *   k                  1 <= k <= max_draft, len + k + 1 <= max_seq
 *   draft_tokens_host  HOST int32 [k] output
 *   logits_dev_or_null DEVICE fp32 [k][vocab]: the draft model's logits per step; may be NULL
 * Does not change the committed length; K/V rows it writes are scratch until verify rewrites them.
 */
knnssd_status knnssd_draft(knnssd_ctx *ctx, int k, int *draft_tokens_host, float *logits_dev_or_null);

/*
 * Verify k drafted tokens with the full model in ONE pass over the k+1 rows [pending, d_0 .. d_{k-1}] at positions
 * len .. len+k (Sec. 4.2, verification paragraph), accept the longest prefix on which the full model's greedy
 * token equals the draft, emit the full model's own token after it, and commit len += n_accepted + 1 (rows beyond
 * are rolled back: dead and overwritten later).  k = 0 is a plain one-token step of the full model.
 *   draft_tokens_host   HOST int32 [k] (any tokens: need not come from knnssd_draft); may be NULL iff k == 0
 *   n_accepted, next_token   HOST outputs; next_token becomes the pending token
 *   logits_dev_or_null  DEVICE fp32 [k+1][vocab] full-model logits of the rows; may be NULL
 *   hidden_dev_or_null  DEVICE fp32 [k+1][d_model] last-layer hidden states after the final RMSNorm; may be NULL
 */
knnssd_status knnssd_verify(knnssd_ctx *ctx, const int *draft_tokens_host, int k, int *n_accepted, int *next_token,
                            float *logits_dev_or_null, float *hidden_dev_or_null);

/*
 * One request end to end: prefill, select_skipset (only if the context has anchors AND use_selection != 0;
 * otherwise the active mask is used and must have been set), then rounds of draft + verify until exactly max_new
 * tokens are out.  Each round drafts k_eff = min(k, remaining - 1) tokens, so the last round never overshoots.
 *   prompt_host HOST int32 [n_prompt];  out_tokens_host HOST int32 [max_new] output;  n_out HOST output
 *   accepts_host_or_null HOST int32 [max_new]: accepted count of each round (first stats.rounds entries)
 *   domain_or_null HOST output (-1 when no selection ran);  stats_or_null HOST output
 */
knnssd_status knnssd_generate(knnssd_ctx *ctx, const int *prompt_host, int n_prompt, int max_new, int k,
                              int use_selection, int *out_tokens_host, int *n_out, int *accepts_host_or_null,
                              int *domain_or_null, knnssd_stats *stats_or_null);

/*
 * The draft-and-verify loop of Sec. 4.2 (k tokens drafted with M(z), one verification pass of the full model, the
 * agreeing prefix kept, repeated), i.e. the decode part of knnssd_generate on an already prefilled session: optional select_skipset on the pooled vector
 * of the last prefill, then rounds of draft + verify until max_new tokens are out, the first of them being the
 * pending token.  Arguments as in knnssd_generate.  Statistics of rounds are restarted by this call.
 */
knnssd_status knnssd_decode(knnssd_ctx *ctx, int max_new, int k, int use_selection, int *out_tokens_host, int *n_out,
                            int *accepts_host_or_null, int *domain_or_null, knnssd_stats *stats_or_null);

/* Number of kernels this context has launched since it was created (-1 for a NULL context). */
long long knnssd_get_launch_count(const knnssd_ctx *ctx);

/* Committed context length (positions whose K/V are valid), and explicit rollback to a shorter length
 * (new_len <= current length; the pending token is unchanged, so this is meant for tests and benchmarks). */
int knnssd_get_length(const knnssd_ctx *ctx);
knnssd_status knnssd_set_length(knnssd_ctx *ctx, int new_len);

/* Replace the pending token (HOST value); lets a caller teacher-force a token stream. */
knnssd_status knnssd_set_pending(knnssd_ctx *ctx, int token);

/* Counters behind the paper's reported quantities (App. C.2): mean generated length M = tokens per verification
 * pass = (accepted + rounds) / rounds, acceptance rate alpha = accepted / drafted; plus device times per phase. */
knnssd_status knnssd_get_stats(const knnssd_ctx *ctx, knnssd_stats *out);
const char *knnssd_last_error(const knnssd_ctx *ctx);

/*
 * The objective of the mask search (Sec. 4.1, Eq. (3)): f(z) = the average inference time per verified token of
 * self-speculative decoding with the skip mask z on a domain's anchor samples.  The optimiser that proposes masks
 * (Bayesian optimisation in the paper) is the caller's; this call evaluates a batch of candidate masks.  For each
 * sample the prompt pass runs once (it does not depend on the mask); then every mask decodes max_new tokens (greedy,
 * k drafts per round) from the state the prompt pass left, and its draft + verification device time is added up.
 *   masks_host          HOST [n_masks][2 * n_layers], entries 0 / 1
 *   tokens_host         HOST int32: the samples' prompts one after the other; lens_host HOST int32 [n_samples]
 *   ms_per_token_host   HOST [n_masks]: sum over samples of (draft + verify ms, CUDA events) / tokens generated by
 *                       draft-and-verify rounds (max_new - 1 per sample: the first token comes from the prompt pass)
 *   accepted_host, drafted_host   HOST [n_masks] totals, or NULL
 * Leaves the session prefilled with the last sample and the last mask active.  Errors as knnssd_prefill / knnssd_decode.
 */
knnssd_status knnssd_mask_objective(knnssd_ctx *ctx, const unsigned char *masks_host, int n_masks,
                                    const int *tokens_host, const int *lens_host, int n_samples, int max_new, int k,
                                    float *ms_per_token_host, int *accepted_host, int *drafted_host);

/*
 * Device-time measurement of the two passes at the current length, for benchmarks: runs `iters` draft passes of one
 * step each (or verify passes over k+1 rows) without committing anything, bracketed by CUDA events on the context's
 * stream, and returns the mean milliseconds per pass.  which: 0 = draft step, 1 = verify pass over k+1 rows.
 * Also returns how many kernels one such pass launches and the mean device milliseconds spent per pass inside the
 * weight-streaming linear kernels alone (events around each of them in a separate, untimed replay).
 */
knnssd_status knnssd_time_pass(knnssd_ctx *ctx, int which, int k, int iters, float *ms_per_pass,
                               int *launches_per_pass, float *ms_linear_per_pass, int *linear_launches_per_pass);

/*
 * Per-operation timing inside the persistent pass kernel (bf16 models it serves; KNNSSD_ERR_SHAPE otherwise): runs
 * one pass as knnssd_time_pass does (which: 0 = draft step, 1 = verify pass over k+1 rows) with CTA 0 stamping the
 * device's nanosecond timer after each operation's work and after the grid barrier that follows it.
 *   cap          capacity of the four HOST output arrays
 *   op_types     0 embedding, 2 attention, 3 hidden-state output, 4 arg-max, 10 linear (store: QKV), 11 linear with
 *                residual add (O / down projection), 12 gate/up linear with SwiGLU, 14 LM head
 *   op_layers    decoder layer of the operation (0 for embedding / head / arg-max)
 *   us_work      microseconds from the previous operation's barrier to the end of this operation's work on CTA 0
 *   us_barrier   microseconds CTA 0 then waited at the barrier
 *   n_ops        operations reported
 */
knnssd_status knnssd_trace_pass(knnssd_ctx *ctx, int which, int k, int cap, int *op_types, int *op_layers, float *us_work,
                                float *us_barrier, int *n_ops);

/*
 * Test hook for the one device-side failure path (status enum above: KNNSSD_ERR_TIMEOUT).  Launches the persistent
 * pass kernel on an operation list that holds only the embedding, with a grid barrier that waits for more arrivals
 * than the launch has CTAs and a poll limit of spin_limit (1..1000000) instead of the kernel's own.  Every CTA's wait
 * runs out after spin_limit polls (well under a millisecond for a few thousand), the kernel returns normally, and the
 * call reports KNNSSD_ERR_TIMEOUT after bringing the barrier state back to idle.  Nothing faults or hangs.  The session
 * then needs a new prefill.  KNNSSD_ERR_SHAPE for models the persistent kernel does not serve.
 */
knnssd_status knnssd_debug_barrier_timeout(knnssd_ctx *ctx, unsigned spin_limit);

/* ---- stand-alone operators (same kernels the passes use; for per-kernel tests and measurements) ---- */

/*
 * y[m][o] = sum_i W[o][i] * x[m][i] for m < M <= 16: the weight-streaming linear kernel.
 *   W DEVICE [n_out][n_in] (dtype as above), x DEVICE fp32 [M][n_in], y DEVICE fp32 [M][n_out]; n_in % 8 == 0.
 */
knnssd_status knnssd_linear(const void *W_dev, int dtype, int n_out, int n_in, const float *x_dev, int M,
                            float *y_dev, void *cuda_stream);

/*
 * The contraction of the prompt pass (Sec. 4.2: the model's pass over the whole sample, T rows at once), on the
 * tensor cores: x is split into two bf16 terms (hi + lo) and multiplied with the bf16 weights, fp32 accumulation.
 *   mode 0   y[t][o]  = sum_i W0[o][i] x[t][i]
 *   mode 1   y[t][o] += sum_i W0[o][i] x[t][i]                      (residual add)
 *   mode 2   y[t][o]  = silu(sum_i W0[o][i] x[t][i]) * (sum_i W1[o][i] x[t][i]), rounded to hi + lo bf16 terms as
 *            the prompt pass hands it to the next map
 *   W0, W1 DEVICE bf16 [n_out][n_in], 16-byte aligned (W1 only for mode 2); x DEVICE fp32 [T][n_in];
 *   y DEVICE fp32 [T][n_out]; n_in % 64 == 0, n_out % 8 == 0, T >= 1.
 * Allocates and frees its temporary planes, and synchronises the stream before it returns.  KNNSSD_ERR_SHAPE for
 * sizes outside the rules above, KNNSSD_ERR_TIMEOUT if a device-side wait gave up.
 */
knnssd_status knnssd_gemm_split(const void *W0_dev, const void *W1_dev, int n_out, int n_in, const float *x_dev, int T,
                                int mode, float *y_dev, void *cuda_stream);

/*
 * The same linear map as knnssd_linear for M <= 16 rows, on the 5th-generation tensor cores: the weights are the
 * 128-row operand, the rows of x (two bf16 terms, hi + lo) the 16 columns, fp32 accumulation in tensor memory; the
 * input columns are split into chunks across CTAs and the chunks' partial sums added in chunk order.  Stand-alone:
 * the decode passes (Sec. 4.2) do not use it yet; it exists to measure what their linear phases would cost at 9..16
 * rows.
 *   W DEVICE bf16 [n_out][n_in], 16-byte aligned; x DEVICE fp32 [M][n_in]; y DEVICE fp32 [M][n_out]; n_in % 64 == 0;
 *   M > 16: KNNSSD_ERR_CAPACITY.  ms_kernels_host: HOST, device time of the contraction + the chunk sum (CUDA
 *   events), or NULL.  Allocates and frees its scratch; synchronises the stream.
 */
knnssd_status knnssd_linear_tc(const void *W_dev, int n_out, int n_in, const float *x_dev, int M, float *y_dev,
                               float *ms_kernels_host, void *cuda_stream);

/*
 * Anchor construction of the pre-inference stage (Sec. 4.1): K-means (Lloyd's iteration) over the sampled last
 * hidden vectors with as many clusters as domains, then, per cluster, the k members nearest to its centroid (Eq. (2)).
 * The paper does not say how K-means is started or stopped: the starting centroids are an argument, and the iteration
 * stops when a round changes no assignment or after max_rounds rounds.  A round = assign every point to its nearest
 * centroid (squared Euclidean distance, lowest index among equal distances), then move each centroid to the mean of
 * its members (a centroid without members stays).  Member sums and centroids are fp64; the assignment compares
 * distances formed from fp32 differences to the fp32-rounded centroid and accumulated to ~48 bits; Eq. (2) ranks the
 * members by distances computed entirely in fp64 against the fp64 centroid.
 *   x_dev               DEVICE fp32 [n_points][d], row-major, 16-byte aligned; borrowed
 *   init_centroids_dev  DEVICE fp32 [n_clusters][d]
 *   max_rounds >= 1, 1 <= k, 1 <= n_clusters <= 16 (more: KNNSSD_ERR_CAPACITY), n_points >= n_clusters
 *   labels_host         HOST int32 [n_points]: the cluster of each point (NULL: not wanted)
 *   centroids_out_dev   DEVICE fp64 [n_clusters][d] (NULL: not wanted)
 *   anchors_host        HOST int32 [n_clusters][k]: point indices, nearest first, lowest index first among equal
 *                       distances; -1 where a cluster has fewer than k members
 *   rounds_host         HOST: assignment rounds done (NULL: not wanted)
 *   ms_rounds_host      HOST: device time of all rounds' kernels, CUDA events on the stream (NULL: not wanted)
 * Allocates and frees its scratch; synchronises the stream.
 */
knnssd_status knnssd_build_anchors(const float *x_dev, int n_points, int d, int n_clusters,
                                   const float *init_centroids_dev, int max_rounds, int k, int *labels_host,
                                   double *centroids_out_dev, int *anchors_host, int *rounds_host, float *ms_rounds_host,
                                   void *cuda_stream);

/*
 * Sampled decoding (App. C.1 lists temperature 0.2 and top-p 0.85 in the decoding set-up; Sec. 1 and Sec. 3.1: the
 * method leaves the distribution of the generated tokens unchanged).  The paper prints no acceptance rule for the sampled
 * case; these three operators implement the rule of speculative sampling that has that property, on the logits that
 * knnssd_draft / knnssd_verify return.  Random numbers are INPUTS: one uniform in [0, 1) per draw.
 *
 * knnssd_filtered_probs: probs[r] = softmax(logits[r] / temperature) restricted to its nucleus and renormalised; a
 *   token is kept iff the probability of the tokens ranked before it (higher probability first, lower id first among
 *   equals) is below top_p, so at least one token is kept.  logits_dev, probs_dev DEVICE fp32 [rows][vocab] (may not
 *   overlap); temperature > 0, top_p > 0 (top_p > 1 keeps every token).  Asynchronous on the stream.
 */
knnssd_status knnssd_filtered_probs(const float *logits_dev, int rows, int vocab, float temperature, float top_p,
                                    float *probs_dev, void *cuda_stream);

/*
 * knnssd_sample_token: inverse CDF in token-id order - the smallest id x with w_0 + .. + w_x > u * sum(w).
 *   weights_dev DEVICE fp32 [vocab], non-negative, not necessarily normalised, with a positive sum; 0 <= u < 1;
 *   token_host HOST output.  Synchronises the stream.
 */
knnssd_status knnssd_sample_token(const float *weights_dev, int vocab, float u, int *token_host, void *cuda_stream);

/*
 * knnssd_spec_accept: one verification round.  p_dev DEVICE [k+1][vocab]: the full model's filtered distributions of
 *   the rows [pending, d_0 .. d_{k-1}]; q_dev DEVICE [k][vocab]: the draft model's filtered distributions the drafts
 *   were drawn from; drafts_host HOST int32 [k]; u_accept_host HOST [k] and u_final uniforms in [0, 1).
 *   Draft j is kept iff u_accept[j] * q_j(d_j) < p_j(d_j), i.e. with probability min(1, p_j(d_j) / q_j(d_j)); at the
 *   first rejected j the emitted token is drawn with u_final from max(0, p_j - q_j) (from p_j if that is zero
 *   everywhere); if all k are kept it is drawn from p_k.  k = 0 draws one token from p_0.
 *   n_accepted, next_token HOST outputs.  0 <= k <= 15.  Synchronises the stream.
 */
knnssd_status knnssd_spec_accept(const float *p_dev, const float *q_dev, const int *drafts_host, int k, int vocab,
                                 const float *u_accept_host, float u_final, int *n_accepted, int *next_token,
                                 void *cuda_stream);

/*
 * The draft-and-verify loop of Sec. 4.2 with sampled instead of greedy decoding, built from the three operators above
 * (App. C.1's temperature / top-p; the keep-or-resample rule described there), on an already prefilled session with an
 * active mask.  Emits exactly max_new tokens, the first being the pending token as it stands (the prompt pass leaves the
 * greedy one).  Each round drafts k_eff = min(k, remaining - 1) tokens: draft step j runs M(z), filters its logits into
 * q_j and draws d_j from q_j; one verification pass gives p_0 .. p_{k_eff}; the round keeps a prefix of the drafts and
 * emits one more token (knnssd_spec_accept's rule) and commits len += kept + 1.
 *   uniforms_host  HOST fp32 [n_uniforms], each in [0, 1); round r (0-based) uses entries r (2k + 1) + j for draw j of its
 *                  drafts (j < k), r (2k + 1) + k + j for the keep test of draft j, r (2k + 1) + 2k for its last draw;
 *                  n_uniforms >= (max_new - 1) (2k + 1) (a round emits at least one token)
 *   other arguments as knnssd_decode.  Errors as knnssd_decode; one host read-back per round.
 */
knnssd_status knnssd_decode_sampled(knnssd_ctx *ctx, int max_new, int k, float temperature, float top_p,
                                    const float *uniforms_host, int n_uniforms, int *out_tokens_host, int *n_out,
                                    int *accepts_host_or_null, knnssd_stats *stats_or_null);

/*
 * Cosine top-1 (Sec. 4.2, Eq. (4)) of one query against n anchors of dimension d, all DEVICE fp32; HOST outputs.
 * KNNSSD_ERR_DEGENERATE for a zero / non-finite query or anchor.
 */
knnssd_status knnssd_cosine_top1(const float *query_dev, const float *anchors_dev, int n, int d, int *best,
                                 float *cosine, void *cuda_stream);

/*
 * knnssd_cosine_top1 for callers that must not allocate device memory.  (No counterpart in the paper: this is a
 * deployment variant of the call above, same arithmetic, same results.)
 *
 * Who needs it: code that runs where cudaMalloc / cudaFree are off limits - inside a serving loop whose memory pool
 * was sized and handed out at start-up, in a process that shares the GPU under a fixed memory reservation, or in a
 * latency path where the implicit device synchronisation of cudaFree is not acceptable.  knnssd_cosine_top1 makes two
 * small cudaMalloc / cudaFree pairs per call for its per-anchor cosines and its result words; this variant keeps that
 * scratch in a fixed array inside the library's device image instead, and calls no allocating routine at all.
 *
 *   arguments   as knnssd_cosine_top1 (query_dev, anchors_dev DEVICE fp32; best, cosine HOST outputs)
 *   limit       n <= KNNSSD_STATIC_MAX_ANCHORS; a larger n returns KNNSSD_ERR_CAPACITY and touches nothing
 *   cost        every GPU that loads the library holds the array (about 16 KB) until the process exits
 *   first call  the first call on each device looks up the array's device address (once per device, with that device
 *               current).  Every call synchronises the stream and copies its two result words to the host, so it
 *               cannot run inside a stream capture at all
 *   sharing     all calls on a device use the same array, and it keeps what the previous call left there; the call
 *               clears the words that must start at zero itself.  Two calls that overlap on one GPU (different
 *               streams or host threads) race on it: serialise them
 */
#define KNNSSD_STATIC_MAX_ANCHORS 4096
knnssd_status knnssd_cosine_top1_static(const float *query_dev, const float *anchors_dev, int n, int d, int *best,
                                        float *cosine, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* KNNSSD_H */
