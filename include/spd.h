/*
 * spd.h -- C ABI of the speculative-decoding verification path for a multimodal target.
 *
 * The operations follow the paper's statement of the problem (letters: p = target,
 * q = draft; the paper uses the opposite letters):
 *   - the target generates conditioned on m projected image embeddings followed by the
 *     text, X_{n+1} ~ p(. | V_1..V_m, X_1..X_n)                      (Sec. 2.2, Eq. 1);
 *   - a small draft of the same architecture proposes gamma tokens auto-regressively from
 *     the text alone, x_j ~ q(. | X, x_1..x_{j-1})                    (Sec. 2.1, Sec. 3);
 *   - ONE target call scores all of them; token j is accepted with probability
 *     min{1, p_j(x_j)/q_j(x_j)}, the first rejected one is replaced by a draw from the
 *     normalised residual max(0, p_j - q_j), and if none is rejected one more token is
 *     drawn from the target's next row                                (Sec. 2.1, Sec. 3,
 *     Sec. 4 "Metrics": at most gamma + 1 tokens per target call);
 *   - with greedy decoding the output equals the target's own greedy continuation
 *                                                                     (Sec. 4 "Decoding").
 *
 * Conventions
 *   - Every function returns spd_status; none throws, aborts or traps the device.
 *     spd_last_error() gives a message for the last non-OK status of a context.
 *   - "device" pointers are CUDA device memory of the context's device; "host or device"
 *     pointers are classified with cudaPointerGetAttributes.  All work is enqueued on
 *     cfg.stream; a call that returns results into HOST memory synchronises that stream
 *     before returning, a call with only device outputs does not.
 *   - The caller owns every buffer it passes.  spd_create makes its own (repacked) device
 *     copy of the weights, so the caller may free them afterwards.
 *   - Matrices are row-major [out, in], in the model's dtype (0 = fp32, 1 = bfloat16);
 *     norm gains are fp32 [d_model]; there are no biases.
 *   - One sequence per context; spd_fork gives further sequences on the same weights and
 *     spd_batch_* runs several of them through one pass over the weights.
 *   - Call order: create -> prefill -> (draft -> verify)* ; anything else is SPD_ESTATE.
 */
#ifndef SPD_H_
#define SPD_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct spd_ctx spd_ctx;

typedef enum {
  SPD_OK = 0,
  SPD_EINVAL = 1,    /* bad argument or unsupported shape */
  SPD_ESTATE = 2,    /* call out of order */
  SPD_ENOMEM = 3,    /* device or host allocation failed */
  SPD_EOVERFLOW = 4, /* KV cache (max_seq) or gamma_max would be exceeded */
  SPD_ECUDA = 5,     /* a CUDA call failed */
  SPD_ETIMEOUT = 6,  /* a bounded device-side wait ran out; the context stays usable */
  SPD_ENOTIMPL = 7
} spd_status;

/* LLaMA-style decoder (Table 1: layers, heads, intermediate dim, hidden dim, SiLU). */
typedef struct {
  int n_layers, d_model, n_heads, d_ffn, vocab;
  int tied_embeddings; /* 1: LM head = token embedding table */
  float rms_eps;       /* RMSNorm epsilon (1e-5) */
  float rope_theta;    /* rotary base (10000); pairs are (i, i + d_head/2) */
  int dtype;           /* storage of matrices and KV cache: 0 = fp32, 1 = bf16 */
} spd_model_cfg;

typedef struct {
  spd_model_cfg target, draft;
  int max_seq;          /* KV rows per model (image rows + text + gamma_max + 1) */
  int gamma_max;        /* largest block size that will be used, 0..7 */
  float temperature;    /* both models' logits are divided by it before softmax */
  int greedy;           /* 1: argmax rule, probabilities and uniforms unused */
  int draft_adapter_in; /* 0: text-only draft (Sec. 3); else width of the image features
                           its linear adapter projects (Sec. 4 "Draft Model Candidates").
                           With draft_adapter_in == draft.d_model and no adapter matrix in the
                           draft's weights, spd_prefill's draft_image_feats are image rows
                           already in the draft's embedding space, e.g. the output of the
                           draft's own two-layer adapter (Appendix A.1) from spd_image_adapter */
  void* stream;         /* cudaStream_t, may be NULL (legacy default stream) */
  int grid_mode;        /* launch shape of the decode kernel.  0 or 1: one CTA per SM with a barrier in
                           global memory (the default and the measured best for both model sizes);
                           2: each model runs as one thread-block cluster of 16 CTAs (8 if 16 cannot be
                           placed) that synchronise through each other's shared memory -- cheaper
                           barriers, but only 16 SMs' worth of streaming (115M draft: 0.61 ms per step
                           against 0.31 ms).  Results do not depend on it beyond summation order. */
  int top_k;            /* sampling only: keep the k most probable tokens of every row (0: off) */
  float top_p;          /* sampling only: then the shortest most-probable prefix whose mass reaches top_p
                           times what is left (0 or >= 1: off).  Sec. 4 "Decoding" names sampling with
                           top-p / top-k as future work and defines neither; here BOTH the target's rows
                           and the draft's rows are truncated and renormalised (the exact definitions
                           are those of spd_truncate_probs), the draft tokens are drawn from the
                           truncated draft rows, draft_probs holds those rows, and the unchanged rule
                           of Sec. 2.1 runs on the truncated rows: the emitted tokens then follow the
                           truncated target distribution.  top_k = 1 reproduces greedy decoding. */
} spd_cfg;

/* Host or device pointers; per-layer entries are HOST arrays of n_layers pointers. */
typedef struct {
  const void* tok_embed;   /* [vocab, d_model] */
  const void* lm_head;     /* [vocab, d_model]; ignored when tied_embeddings */
  const float* final_norm; /* [d_model] */
  const void* adapter;     /* draft only: [d_model, draft_adapter_in], or NULL */
  const float* const* attn_norm;
  const void* const* wq;
  const void* const* wk;
  const void* const* wv;
  const void* const* wo;   /* each [d_model, d_model] */
  const float* const* ffn_norm;
  const void* const* w_gate;
  const void* const* w_up; /* each [d_ffn, d_model] */
  const void* const* w_down; /* [d_model, d_ffn] */
} spd_weights;

typedef struct {
  int blocks;          /* target calls made */
  int accepted;        /* draft tokens accepted in total */
  int tokens;          /* tokens written to out_ids */
  float tau;           /* block efficiency: tokens emitted per target call (Sec. 4) */
  float ms_total;      /* CUDA events around the whole loop */
  float ms_draft, ms_verify; /* sums of kernel times by the device clock (%globaltimer) */
  int graph_replays;   /* blocks issued by replaying the captured CUDA graph (0: plain launches) */
} spd_stats;

/* Validates cfg, copies and repacks the weights, allocates KV caches and workspaces,
 * builds the rotary table.  Shapes must satisfy: d_model <= 4096 and a multiple of 32,
 * d_head = d_model / n_heads in {32, 64, 128} (bf16 models: 64 or 128), d_ffn a multiple of 8, gamma_max <= 7, max_seq >= 16,
 * equal vocab for both models.  *out is NULL on failure. */
spd_status spd_create(const spd_weights* target_w, const spd_weights* draft_w,
                      const spd_cfg* cfg, spd_ctx** out);
void spd_destroy(spd_ctx* ctx);
const char* spd_last_error(const spd_ctx* ctx);

/* A second, independent sequence on the same models.  The method is stated for one sequence
 * (Sec. 2.1: one draft block, one target call, one accept/reject pass); serving several
 * sequences needs one KV cache pair, one device state and one set of work buffers per
 * sequence, while the repacked weights (13 GB for the 7B shape) exist once.  *out gets a
 * context with the same cfg and stream as `parent` that shares every weight buffer with it
 * and owns everything else; it starts un-prefilled.  Each sequence is then driven with the
 * calls below, in any interleaving on the shared stream (each call still streams the weights
 * once: sequences are not batched into one kernel), and rolled back on its own.  Destroy
 * order is free: the weights are released with the last context that uses them.  Errors:
 * SPD_EINVAL (NULL), SPD_ESTATE (parent already destroyed), SPD_ENOMEM / SPD_ECUDA with the
 * message left on `parent`.  Not thread-safe against other calls on `parent`. */
spd_status spd_fork(spd_ctx* parent, spd_ctx** out);

/* Prefill (Eq. 1): the target reads [image_embeds ; embed(prompt_ids)] at positions
 * 0..m+n-1 and fills its KV cache; its last row gives the first generated token (argmax,
 * or a draw with *u0).  The draft reads embed(prompt_ids) only, or, with an adapter,
 * [draft_image_feats W_a^T ; embed(prompt_ids)] (or [draft_image_feats ; embed(prompt_ids)]
 * when the rows are given in the draft's space, see spd_cfg.draft_adapter_in).
 *   image_embeds       fp32 [m, d_target], host or device; NULL iff m == 0
 *   draft_image_feats  fp32 [m, draft_adapter_in], host or device; NULL without adapter
 *   prompt_ids         int32 [n], host or device, n >= 1, each in [0, vocab): host ids are checked
 *                      before any work, device ids on the device (an offender is read as token 0,
 *                      the call returns SPD_EINVAL and the context stays un-prefilled)
 *   u0                 host, one uniform in [0,1); may be NULL when greedy
 *   first_token        host, out, may be NULL
 * Resets any earlier sequence. SPD_EOVERFLOW if m + n + gamma_max + 1 > max_seq. */
spd_status spd_prefill(spd_ctx* ctx, const float* image_embeds, int m,
                       const float* draft_image_feats, const int32_t* prompt_ids, int n,
                       const float* u0, int32_t* first_token);

/* Image adapter g_theta (Sec. 2.2: the image encodings H_1..H_m become the image embeddings
 * V_i = g_theta(H_i) that the target conditions on; Appendix A.1: an MLP of two linear layers,
 * 1024 -> 4096 -> 4096 for the 7B target, 1024 -> 1024 -> 1024 for a draft with its own
 * adapter).  Computes out = GELU(feats W1^T) W2^T on the tensor cores.  The paper names neither
 * the non-linearity nor biases: GELU in its exact form x * Phi(x) (LLaVA's projector) and no
 * biases are used.  The result is what spd_prefill takes as image_embeds.
 *   feats  fp32 [m, d_in], host or device (vision-encoder features; the encoder is not part
 *          of this library)
 *   w1     bf16 [d_hid, d_in], w2 bf16 [d_out, d_hid]: row-major, DEVICE, 16-byte aligned,
 *          owned by the caller and only read
 *   out    fp32 [m, d_out], DEVICE, 16-byte aligned
 * d_in and d_hid must be multiples of 8.  Activations are carried as bf16 hi + lo pairs with
 * fp32 accumulation, so the result matches an fp32 evaluation to ~1e-5 relative.  Uses the
 * context's stream and keeps its scratch in the context; synchronises the stream before
 * returning.  Errors: SPD_EINVAL (arguments, host weights), SPD_ENOMEM, SPD_ECUDA,
 * SPD_ETIMEOUT.  May be called before or after spd_prefill; it does not touch the sequence. */
spd_status spd_image_adapter(spd_ctx* ctx, const float* feats, int m, int d_in, const void* w1,
                             int d_hid, const void* w2, int d_out, float* out);

/* Draft step (Sec. 2.1): gamma tokens, one after the other, each drawn from the draft's
 * softmax(logits / T) with uniforms[j] (or argmax when greedy).
 *   uniforms     fp32 [gamma], host or device; may be NULL when greedy
 *   draft_ids    int32 [gamma], out, host or device; may be NULL (kept internally)
 *   draft_probs  fp32 [gamma, vocab], out, DEVICE; may be NULL (kept internally);
 *                not written when greedy */
spd_status spd_draft(spd_ctx* ctx, int gamma, const float* uniforms, int32_t* draft_ids,
                     float* draft_probs);

/* Verification (Sec. 2.1, Sec. 3): one target call on [pending, x_1..x_gamma] against
 * the KV cache, then the rejection rule; commits the accepted tokens and the next token
 * and rolls both KV caches back to the accepted length.
 *   draft_ids    int32 [gamma], host or device; NULL = the ids of the last spd_draft.
 *                They must be the tokens the draft was fed, or the draft's cache no
 *                longer matches the sequence (timing experiments may accept that).
 *   draft_probs  fp32 [gamma, vocab], DEVICE; NULL = those of the last spd_draft; unused
 *                when greedy
 *   uniforms     fp32 [gamma+1], host or device: gamma accept tests, then the one
 *                replacement / bonus draw; may be NULL when greedy
 *   n_accepted, next_token  int32, out, host or device (may be NULL)
 * gamma == 0 is a plain auto-regressive step of the target. */
spd_status spd_verify(spd_ctx* ctx, int gamma, const int32_t* draft_ids,
                      const float* draft_probs, const float* uniforms,
                      int32_t* n_accepted, int32_t* next_token);

/* ---- tree blocks (Sec. 5: "recent advancement in SPD algorithm to tree-based decoding can also be
 * used"; the paper defines no rule).  Built here: several candidates per position, verified in ONE
 * target call with a tree attention mask, by the multi-candidate rejection rule of the token-tree
 * systems the paper cites, which keeps Sec. 2.1's guarantee (emitted tokens follow the target's
 * distribution) when the candidates of a node are drawn independently from the draft's
 * distribution at that node.  Block rows: 0 = the pending token (root), 1..n = draft nodes,
 * parents before children; n <= gamma_max <= 7.  Every node gets its own K/V cache row while
 * siblings share a sequence position; a node attends the committed prefix, its ancestors and
 * itself.  Rule: starting at the root with cur = p_root, the children of the current node are
 * tried in row order; child c is accepted iff u[c-1] < min(1, cur(x_c) / q_node(x_c)); on
 * acceptance the walk descends (cur = p_c); on rejection cur <- max(0, cur - q_node) / sum and the
 * next child is tried; when no child is left the next token is drawn from cur with u[n].  Greedy:
 * a child is accepted iff it is the arg-max of p_node, else that arg-max is emitted.  A chain
 * (one child per node) is exactly spd_draft / spd_verify.  Afterwards the K/V rows of the
 * accepted nodes are moved to the positions they now hold, in both caches. */

/* Draft tree: every node at depth d-1 gets branching[d-1] children (d = 1..depth), drawn
 * independently from the draft's softmax(logits / T) at that node (greedy: its branching[d-1] most
 * probable tokens); the draft runs level by level, each level one tree-masked launch.
 *   branching    int32 [depth], HOST; the node count n = sum over levels must be <= gamma_max
 *   uniforms     fp32 [n], host or device: uniforms[i-1] draws node i; may be NULL when greedy
 *   node_ids     int32 [n], out, host or device, may be NULL (kept internally)
 *   parent_out   int32 [n+1], out, HOST, may be NULL: parent_out[0] = -1, rows level by level
 *   draft_probs  fp32 [n+1, vocab], out, DEVICE, may be NULL (kept internally): row r = the draft's
 *                distribution at block row r (rows of leaves unused); not written when greedy */
spd_status spd_draft_tree(spd_ctx* ctx, int depth, const int32_t* branching, const float* uniforms,
                          int32_t* node_ids, int32_t* parent_out, float* draft_probs);

/* Tree verification: one target call on [pending ; node_1..node_n] with the tree mask, the rule
 * above, commit of the accepted path and the next token, K/V compaction.
 *   parent       int32 [n+1], HOST, parent[0] = -1, parent[i] in 0..i-1
 *   node_ids     int32 [n], host or device; NULL = those of the last spd_draft_tree (same shape)
 *   draft_probs  fp32 [n+1, vocab], DEVICE; NULL = those of the last spd_draft_tree; unused when greedy
 *   uniforms     fp32 [n+1], host or device: n accept tests, then the one final draw; NULL when greedy
 *   n_accepted   int32, out: length of the accepted path
 *   path         int32 [depth of the tree], out: block rows of the accepted nodes, root downwards
 *   next_token   int32, out
 * Outputs may be host or device memory or NULL. */
spd_status spd_verify_tree(spd_ctx* ctx, int n_nodes, const int32_t* parent, const int32_t* node_ids,
                           const float* draft_probs, const float* uniforms, int32_t* n_accepted, int32_t* path,
                           int32_t* next_token);

/* Block loop (Fig. 1): repeats draft + verify until n_new tokens exist after the prompt;
 * the pending token (after spd_prefill: the token it produced) is the first of them.
 *   uniforms  fp32 [n_new, 2*gamma+1], host or device: per block gamma draft draws, then
 *             gamma+1 verification uniforms; may be NULL when greedy
 *   out_ids   int32 [n_new], HOST
 *   stats     host, may be NULL
 * gamma == 0 runs the target alone (the auto-regressive baseline). */
spd_status spd_generate(spd_ctx* ctx, int n_new, int gamma, const float* uniforms,
                        int32_t* out_ids, spd_stats* stats);

/* ---- several sequences, one pass over the weights ----
 * The method is stated for one sequence (Sec. 2.1), and its cost argument is that a target call
 * is bound by streaming the parameters (Sec. 1; Sec. 4 "Metrics": cost proportional to parameter
 * count).  When B sequences are decoded together the parameters should therefore be streamed
 * once for all of them.  A batch groups B contexts that share their weights (a context and its
 * spd_fork's, all on one stream).  A batched step runs the rows of all sequences -- B x (gamma+1)
 * for the verify step, B x 2 for a draft step, at most 128 -- through every projection as ONE
 * dense tensor-core GEMM, while rotary embedding, cache append, attention over each sequence's
 * own cache, the rejection rule and the commit stay per sequence: every sequence keeps its own
 * length, accepts its own number of tokens and can be rolled back on its own (spd_rollback on its
 * context).  Prefill stays per sequence (prompts have different lengths).  bf16 models only.
 * Batched and single-sequence calls may be mixed freely between blocks. */
typedef struct spd_batch spd_batch;

/* seqs: HOST array of B distinct contexts, all forks of one context (or that context itself);
 * B x (gamma_max + 1) <= 128.  The contexts must outlive the batch.  Errors are reported on
 * seqs[0] (spd_last_error(seqs[0])). */
spd_status spd_batch_create(spd_ctx* const* seqs, int B, spd_batch** out);
void spd_batch_destroy(spd_batch* batch);

/* gamma draft steps for every sequence (Sec. 2.1), each step one pass over the draft's weights.
 *   uniforms   fp32 [B, gamma], host or device; may be NULL when greedy
 *   draft_ids  int32 [B, gamma], out, host or device, may be NULL
 * The draft distributions are kept inside the batch for spd_batch_verify. */
spd_status spd_batch_draft(spd_batch* batch, int gamma, const float* uniforms, int32_t* draft_ids);

/* One target call on the B x (gamma+1) rows [pending_b, x_b1..x_b,gamma], then per sequence the
 * rejection rule (Sec. 2.1, Sec. 3), the commit and the roll-back of its caches to its accepted
 * length.  gamma must be that of the preceding spd_batch_draft; gamma == 0 is a plain
 * auto-regressive step of the target for every sequence.
 *   uniforms    fp32 [B, gamma+1], host or device; may be NULL when greedy
 *   n_accepted, next_token  int32 [B], out, host or device, may be NULL */
spd_status spd_batch_verify(spd_batch* batch, int gamma, const float* uniforms, int32_t* n_accepted,
                            int32_t* next_token);

/* Logits of the last batched call, fp32 [rows, vocab] (row b*(gamma+1)+m after a verify step,
 * b*2+m after a draft step), host or device.  Test support. */
spd_status spd_batch_get_logits(spd_batch* batch, float* logits, int rows);

/* Bytes one batched verify step must move: the target's weights once + every sequence's K/V rows
 * read and written (the figure its roofline is computed from). */
spd_status spd_batch_verify_bytes(spd_batch* batch, int gamma, double* bytes);

/* ---- test and benchmark support ---- */

/* Logits of the last spd_verify (rows <= gamma+1) / of the last spd_draft (rows <= gamma):
 * fp32 [rows, vocab] into host or device memory.  Prefill's last row: spd_get_logits with
 * rows = 1 directly after spd_prefill. */
spd_status spd_get_logits(spd_ctx* ctx, float* logits, int rows);
spd_status spd_get_draft_logits(spd_ctx* ctx, float* logits, int rows);

/* Rollback / resynchronisation: declares that the committed text is n_text tokens long
 * (prompt included, pending token excluded), that prev_token is its last token and
 * pending_token the token to feed next.  KV rows of positions >= the new length are
 * treated as stale; rows below it must belong to the same sequence.  O(1). */
spd_status spd_rollback(spd_ctx* ctx, int n_text, int32_t prev_token, int32_t pending_token);
spd_status spd_get_state(spd_ctx* ctx, int32_t* n_text, int32_t* pending_token);

/* Phase trace of spd_verify.  The first call switches tracing on (returns *n = 0).  Later
 * calls copy the trace of the last spd_verify into stamps[cap] (HOST).  Each entry is
 * (%globaltimer in ns << 8) | id, written by CTA 0: id 0 kernel start, 1 activation tile of
 * a projection built, 2 its last weight stage consumed, 3 phase finished, 4 grid barrier
 * passed.  Per layer the phases are QKV, attention, O-projection, gate/up, down; then LM
 * head, row statistics, sampling. */
spd_status spd_trace(spd_ctx* ctx, uint64_t* stamps, int cap, int* n);

/* The rejection rule alone (Sec. 2.1) on given probabilities, B independent sequences:
 *   p [B, gamma+1, V], q [B, gamma, V] fp32 DEVICE (q may be NULL when greedy)
 *   ids int32 [B, gamma], u fp32 [B, gamma+1] DEVICE (u may be NULL when greedy)
 *   n_acc, next int32 [B] DEVICE, out; both are -1 for a sequence with a draft id outside [0, V)
 *   (the ids live in device memory, so the host cannot check them before the launch)
 * Integer inverse-CDF sampling (weights truncated to 32 fractional bits, summed as
 * integers) makes the result independent of summation order. Asynchronous on stream. */
spd_status spd_reject_sample(const float* p, const float* q, const int32_t* ids,
                             const float* u, int B, int gamma, int V, int greedy,
                             int32_t* n_acc, int32_t* next, void* stream);

/* Top-k / top-p (nucleus) truncation of probability rows ahead of the rule (Sec. 4 "Decoding"
 * names sampling with top-p / top-k as future work; the paper itself decodes greedily).  Both
 * the target's rows p and the draft's rows q are truncated and renormalised, the draft tokens
 * are drawn from the truncated q, and spd_reject_sample is applied to the truncated rows; the
 * emitted tokens then follow the truncated target distribution.
 *   probs, out  fp32 [rows, V] DEVICE; out may be probs (in place)
 *   top_k       keep the k most probable tokens; <= 0 or >= V: off
 *   top_p       then keep the shortest most-probable prefix of what is left whose mass reaches
 *               top_p times the mass left; >= 1: off; must be > 0
 * Exact definitions: tokens are ordered by probability, equal probabilities by index (lower
 * first); masses are the integers trunc(w * 2^32) and are summed as integers; the target
 * mass is ceil(Z * trunc(top_p * 2^24) / 2^24), at least one token is kept; kept values are
 * divided by float(kept mass) * 2^-32, the others become 0.  The result is therefore
 * independent of any summation order.  Values <= 0 count as 0.
 * V is limited by the shared memory of one CTA (V <= ~56000).  Asynchronous on stream.
 * Errors: SPD_EINVAL (NULL, host pointers, sizes, top_p <= 0), SPD_ECUDA. */
spd_status spd_truncate_probs(const float* probs, float* out, int rows, int V, int top_k,
                              float top_p, void* stream);

/* Y[M,N] = X[M,K] W[N,K]^T with the weight-streaming kernel of the verify projections
 * (Eq. 1's linear maps at M = gamma+1 rows).  x, y fp32 DEVICE, w DEVICE in `dtype`;
 * 1 <= M <= 8, K a multiple of 8.  Asynchronous on stream. */
spd_status spd_skinny_gemm(const float* x, const void* w, int dtype, int M, int N, int K,
                           float* y, void* stream);

/* Status of the last spd_skinny_gemm (noalloc = 0) or spd_skinny_gemm_noalloc (noalloc = 1) on the
 * current device.  Both calls are asynchronous and have no context, so a bounded device-side
 * wait that ran out inside them (Conventions above) can only be seen afterwards: this call
 * synchronises `stream`, returns SPD_ETIMEOUT if the kernel's status word is set (y is then
 * garbage) and clears it, else SPD_OK; SPD_ESTATE before the first such call on this device.
 * spd_skinny_gemm_noalloc clears its status word at the start of every call, so ask before the
 * next call; spd_skinny_gemm's stays set (and its results garbage) until it is asked for. */
spd_status spd_skinny_gemm_status(int noalloc, void* stream);

/* Bounded waits, exercised (no counterpart in the paper; Conventions: no call may hang the
 * device).  Launches a small kernel on the context's stream that runs one of the forward
 * kernel's wait primitives on a condition that never becomes true, limited to `polls`
 * iterations (1 .. 2^20): which = 0 the shared-memory barrier wait of the weight ring, which = 1
 * the grid barrier with a target one arrival beyond the grid size.  The wait gives up, the
 * kernel returns normally and this call returns SPD_ETIMEOUT -- the status any call of this
 * library reports when one of its waits runs out.  The error word is cleared; the context and
 * its sequence are untouched and stay usable.  Synchronises the stream. */
spd_status spd_wait_selftest(spd_ctx* ctx, int which, unsigned polls);

/* The same product as spd_skinny_gemm for callers that must not allocate device memory.
 * (The paper has no counterpart for this entry point; it exists for integration reasons.)
 *
 * Who needs it: code that runs where cudaMalloc / cudaFree are off limits -- inside a
 * host program whose device memory is owned entirely by another allocator (a serving
 * engine or framework that hands out fixed arenas and forbids side allocations), inside
 * a latency-critical loop where the implicit device synchronisation of cudaMalloc/cudaFree
 * is unacceptable, or in a process whose memory budget was fixed at start-up.
 * spd_skinny_gemm keeps a growing device buffer for the repacked weights and allocates
 * it on demand; this variant instead uses a fixed scratch array compiled into the library
 * (SPD_NOALLOC_MAX_PACKED_BYTES plus a 512-byte header).  Every GPU that loads the library
 * holds that array until the process exits, whether or not this function is ever called.
 *
 *   - x, w, y, dtype, M, N, K, stream: exactly as spd_skinny_gemm (the caller still owns
 *     inputs and outputs).
 *   - Limit: the repacked weights, ceil(N/4)*4 * ceil(K*esz/512)*512 bytes with esz = 2
 *     (bf16) or 4 (fp32), must not exceed SPD_NOALLOC_MAX_PACKED_BYTES; otherwise the call
 *     does nothing, prints one line to stderr and returns SPD_EOVERFLOW.
 *   - It calls no cudaMalloc, cudaFree or other allocating routine.
 *   - The first call on each device (with that device current) looks up the device address
 *     of the scratch array and the device properties; make that first call before starting
 *     any stream capture.
 *   - All calls share the one array.  Its contents persist between calls; the words that
 *     must start at zero are cleared on the stream at the start of every call.  Two calls
 *     whose GPU work overlaps (different streams, or different host threads) race on it:
 *     serialise them.
 * Asynchronous on stream. */
#define SPD_NOALLOC_MAX_PACKED_BYTES (16u << 20)
spd_status spd_skinny_gemm_noalloc(const float* x, const void* w, int dtype, int M, int N,
                                   int K, float* y, void* stream);

/* Bytes that one verify step must move (weights + KV read + KV written) at the current
 * sequence length, the figure the roofline is computed from. */
spd_status spd_verify_bytes(spd_ctx* ctx, int gamma, double* bytes);

#ifdef __cplusplus
}
#endif
#endif /* SPD_H_ */
