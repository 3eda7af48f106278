/*
 * talon.h -- C ABI of the B200 (sm_100a) hot path of Talon, the confidence-aware,
 * budget-driven speculative-decoding method.
 *
 * The library builds a draft token tree layer by layer under a fixed node budget
 * (Algorithm 2 of the paper: Top-K at the root, Eq. 5; confidence gate p(u) >= mu * m_d
 * below it, Eq. 3-4; truncation to the remaining budget) and verifies it: tree attention
 * under the ancestor mask followed by the greedy longest-accepted-path walk (Appendix B).
 * The draft and target model forwards are the caller's: the caller hands in their logits
 * and the projected Q/K/V.
 *
 * Conventions that hold for every call unless a comment says otherwise:
 *  - Pointers named in a "device" comment are CUDA device pointers owned by the caller.
 *    The library never frees or reallocates them.  "host" pointers are ordinary memory.
 *  - A call only enqueues work on `stream` (a cudaStream_t passed as void*) and returns;
 *    it performs no synchronisation and no allocation after talon_create
 *    (talon_step_host and talon_poll_status are the two documented exceptions).
 *  - Errors that the host can see (null pointer, size out of range, misalignment) return
 *    a status at once with nothing enqueued.  Errors only the device can see (NaN or +inf
 *    logit, a row of only -inf) set a device status word that talon_poll_status reads;
 *    outputs stay defined (the layer adds no node for the affected sequence).
 *  - One context serves one stream at a time; calls on one context must not overlap.
 *  - Sequences of a batch are independent.  B is fixed by talon_reset until the next reset.
 *
 * Notation: B batch, V vocabulary, N node budget (root included, <= 128), K root top-k,
 * k per-parent candidate cap, D_max depth cap, W = ceil(N/64) mask words, Hq/Hkv query
 * and key/value heads, g = Hq/Hkv, Dh = 128 head dimension, L_b prefix length.
 */
#ifndef TALON_H_
#define TALON_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct talon_ctx talon_ctx;

typedef enum {
  TALON_OK = 0,
  TALON_ERR_INVALID_ARG = 1, /* null pointer, size out of range, misaligned row          */
  TALON_ERR_CAPACITY = 2,    /* request exceeds what the context was created for          */
  TALON_ERR_CUDA = 3,        /* a CUDA runtime call failed (see stderr for the message)   */
  TALON_ERR_TIMEOUT = 4,     /* a bounded device-side wait gave up: the tree arrays and   */
                             /* outputs of that step are undefined, call talon_reset     */
  TALON_ERR_NONFINITE = 5,   /* NaN / +inf logit, or a row holding only -inf              */
  TALON_ERR_UNSUPPORTED = 6  /* valid in the paper, not built (e.g. head_dim != 128)      */
} talon_status;

/* Hyper-parameters of Algorithm 2 ("Require" line: budget N, width K, threshold mu) plus the
 * shapes the verification step needs.  Defaults of the paper: N = 60, K = 10, mu = 0.03. */
typedef struct {
  int32_t batch_max;   /* largest B any later call may use (1..1024)                         */
  int32_t vocab;       /* V (2 .. 2^24-1)                                                    */
  int32_t budget;      /* N, root included (2..128)                                          */
  int32_t root_topk;   /* K of Eq. 5 (1..128)                                                */
  int32_t cand_topk;   /* k: candidates kept per parent before pooling (1..128); 0 = N-1,    *
                        * which reproduces Eq. 3's whole-vocabulary pool exactly, because a  *
                        * parent can never place more than N-|T| children                   */
  int32_t max_depth;   /* D_max: no node deeper than this (1..126)                           */
  int32_t init_layers; /* leading layers that use Top-K instead of the gate; paper: 1        */
  int32_t n_q_heads;   /* Hq                                                                 */
  int32_t n_kv_heads;  /* Hkv, divides Hq                                                    */
  int32_t head_dim;    /* Dh, must be 128                                                    */
  double  mu;          /* gate threshold of Eq. 4, in (0, 1]                                 */
} talon_params;

/* The draft tree T of Algorithm 2 as flat per-sequence arrays in caller-owned DEVICE memory.
 * Node 0 is the root x_t; nodes are stored layer by layer, each layer sorted by
 * (parent index, token id), so parent[i] < i.  Slots n_nodes[b]..N-1 hold sentinels after
 * talon_build_tree (token = parent = depth = position = -1, score = -inf, mask = own bit). */
typedef struct {
  int32_t  *n_nodes;   /* [B]              |T| per sequence                                  */
  int32_t  *token;     /* [B, N]           token id of each node                             */
  int32_t  *parent;    /* [B, N]           parent node index, -1 for the root                */
  int32_t  *depth;     /* [B, N]           root = 0                                          */
  int32_t  *position;  /* [B, N]           prefix_len + depth (written by talon_build_tree)  */
  int32_t  *layer_off; /* [B, D_max + 2]   nodes of depth d are layer_off[d]..layer_off[d+1]-1 */
  double   *score;     /* [B, N]           log of Eq. 2's path probability p(v)              */
  uint64_t *mask;      /* [B, N, W]        bit j of row i set iff node i attends to node j
                        *                  (itself and its ancestors; Fig. 2(b), Appendix B)  */
} talon_tree;

/* How talon_expand_layer finds the logit row of a frontier node. */
enum {
  TALON_ROWS_BY_NODE = 0,  /* row index = b * rows_per_seq + node index                       */
  TALON_ROWS_PACKED  = 1   /* row index = b * rows_per_seq + (node index - first frontier node) */
};

/* Creates a context on CUDA device `device` and allocates its workspace there (the only
 * allocation the library makes, apart from talon_step_host's staging buffers).
 * Returns INVALID_ARG / UNSUPPORTED for out-of-range parameters, CUDA on allocation failure. */
talon_status talon_create(talon_ctx **out_ctx, const talon_params *params, int device);

/* Frees the context's workspace.  Caller memory is untouched.  Null is accepted. */
talon_status talon_destroy(talon_ctx *ctx);

/* Initialisation of Algorithm 2: T <- {x_t}, P_0 <- {x_t}, p(x_t) <- 1, d <- 0, for B sequences.
 * root_tok   device [B]  last committed token x_t of each sequence
 * prefix_len device [B]  number of tokens before x_t, i.e. the KV-cache length L_b (>= 0)
 * Clears the device status word. */
talon_status talon_reset(talon_ctx *ctx, const talon_tree *tree, const int32_t *root_tok,
                         const int32_t *prefix_len, int32_t B, void *stream);

/* One pass of Algorithm 2's while-body for every sequence that still has budget: reads the
 * draft logits of the current frontier P_d (all nodes of depth d), forms the candidate pool
 * S_d with path scores p(u) = p(v) * softmax(logits_v)[w] (Eq. 3; per-parent top-k first),
 * applies Top-K (d < init_layers, Eq. 5) or the gate p(u) >= mu * max p (Eq. 4), truncates
 * to the remaining budget by score, and appends the survivors as depth d+1.
 * Ties: higher score first, then lower parent index, then lower token id.
 * logits       device fp32; row r starts at logits + r * row_stride; 16-byte aligned
 * row_stride   elements between rows, a multiple of 4 and >= V
 * rows_per_seq rows reserved per sequence in `logits` (N for BY_NODE)
 * layout       TALON_ROWS_BY_NODE or TALON_ROWS_PACKED
 * A sequence whose tree is full, whose frontier is empty, or whose depth reached D_max is
 * left unchanged; once d == D_max the call is a no-op.  -inf logits are legal (p = 0,
 * never selected).  The number of calls since talon_reset is the layer index d. */
talon_status talon_expand_layer(talon_ctx *ctx, const talon_tree *tree, const float *logits,
                                int64_t row_stride, int32_t rows_per_seq, int32_t layout,
                                void *stream);

/* Number of talon_expand_layer calls since the last talon_reset (host counter). */
int32_t talon_layers_run(const talon_ctx *ctx);

/* Closes the tree for verification (Fig. 2(b), Appendix B): position = prefix_len + depth,
 * sentinels in unused slots, remaining layer_off entries = n_nodes.
 * dense_mask  device [B, N, N] uint8 or null: if given, receives the mask as bytes
 *             (1 = row node attends to column node). */
talon_status talon_build_tree(talon_ctx *ctx, const talon_tree *tree, uint8_t *dense_mask,
                              void *stream);

/* The static tree the paper compares with (Algorithm 1, "Static Tree Construction") on the same
 * kernels.  Its depth loop is talon_expand_layer of a context created with
 *   budget = 1 + K * (D + 1), root_topk = cand_topk = K, max_depth = init_layers = D + 1:
 * every layer then takes each parent's Top-K tokens, pools the K x K proposals and keeps the K
 * best path probabilities as the next parents.  This call is the algorithm's last step,
 * T <- Top-N(T by p(u)): of every sequence's tree the `keep` nodes with the largest path scores
 * stay (equal scores: the lower node index, so parents outlive their children), in their old
 * order; parent links, ancestor-mask bits, layer offsets and n_nodes are renumbered in place.
 * Call talon_build_tree afterwards (positions, sentinels of the freed slots).
 *  keep  >= 1; a tree that is not larger is left as it is
 * Enqueues one kernel; no synchronisation. */
talon_status talon_prune_tree(talon_ctx *ctx, const talon_tree *tree, int32_t keep, void *stream);

/* Tree attention of the verification forward (Appendix B): query node i of sequence b and
 * query head h attends to all L_b prefix keys and to the tree keys j with mask bit (i, j)
 * set, softmax(sm_scale * q.k) in fp32, times V, accumulated in fp32, written as bf16.
 * All tensors bf16, device memory:
 *  q        [B, N, Hq, Dh] contiguous
 *  k_prefix, v_prefix  token t, head h of sequence b at
 *           base + (kv_start[b] + t) * kv_stride_t + h * kv_stride_h   (elements; Dh contiguous;
 *           strides multiples of 8)
 *  k_tree, v_tree      [B, N, Hkv, Dh] contiguous: keys/values of the tree tokens themselves
 *  kv_start device [B] int64 token offsets of each sequence's block (ragged or padded)
 *  kv_tokens           tokens allocated in k_prefix / v_prefix (host value): reads stop there, so
 *                      kv_start[b] + L_b <= kv_tokens must hold; memory between L_b and the next
 *                      multiple of 128 tokens may be read but never influences the result
 *  max_prefix_len      host upper bound of the prefix lengths given to talon_reset
 *  out      [B, N, Hq, Dh] contiguous; rows of unused node slots are written as zeros
 * Rotary embedding is the caller's business: Q/K arrive already rotated. */
talon_status talon_tree_attention(talon_ctx *ctx, const talon_tree *tree, const void *q,
                                  const void *k_prefix, const void *v_prefix,
                                  const void *k_tree, const void *v_tree,
                                  const int64_t *kv_start, int64_t kv_tokens, int64_t kv_stride_t,
                                  int64_t kv_stride_h, int32_t max_prefix_len, float sm_scale,
                                  void *out, void *stream);

/* Greedy verification (Appendix B steps 1-2 at temperature 0): t_i = argmax of the target
 * logits after node i (lowest id among equal maxima), then from the root follow the child
 * whose token equals t_cur until none does.  Call after talon_build_tree (the walk reads the closed
 * layer offsets).
 * target_logits device fp32, row of node i of sequence b at (b*N + i) * row_stride; 16-byte aligned rows
 * target_tok    device [B, N] or null: receives t_i (-1 for unused slots)
 * accept_len    device [B]: number of accepted draft tokens (root not counted)
 * accept_nodes  device [B, D_max + 1]: accepted node indices, root first, -1 padded
 * bonus_tok     device [B]: target token after the last accepted node */
talon_status talon_accept(talon_ctx *ctx, const talon_tree *tree, const float *target_logits,
                          int64_t row_stride, int32_t *target_tok, int32_t *accept_len,
                          int32_t *accept_nodes, int32_t *bonus_tok, void *stream);

/* talon_build_tree (without the dense mask) and talon_accept in one call, for the tail of a step:
 * the warp that walks a sequence's tree first writes that sequence's positions, sentinel slots and
 * closed layer offsets, so the closing kernel is not launched.  Nothing between the last expansion
 * layer and this call may need what talon_build_tree writes (talon_tree_attention does not: it
 * reads sizes and mask rows).  Arguments, results and errors as talon_accept; talon_step and
 * talon_loop end their steps with it. */
talon_status talon_close_and_accept(talon_ctx *ctx, const talon_tree *tree, const float *target_logits,
                                    int64_t row_stride, int32_t *target_tok, int32_t *accept_len,
                                    int32_t *accept_nodes, int32_t *bonus_tok, void *stream);

/* Sampling verification (Appendix B steps 1-3, the paper's temperature-1 setting; the appendix
 * names the steps and the property -- what is emitted is distributed exactly as the target
 * model's own samples -- and leaves the procedure to the literature it cites).  With p the
 * target's posterior softmax(target_logits / temperature) after the current node (the root
 * first), the children of that node are tried in storage order: child c with token w is
 * accepted when u_accept[c] * (mass not yet struck) < p(w), otherwise w is struck from p.  The
 * first accepted child becomes the current node; when none is accepted the correction token is
 * drawn from what is left of p by inverse CDF in token order with u_sample.  Call after
 * talon_build_tree (the walk reads the closed layer offsets).
 * target_logits device fp32, row of node i of sequence b at (b*N + i) * row_stride; 16-byte aligned rows
 * temperature   host value, > 0
 * u_accept      device [B, N] fp64 uniforms in [0, 1): node c consumes u_accept[b, c] if it is tried
 * u_sample      device [B] fp64 uniforms in [0, 1)
 * accept_len    device [B]; accept_nodes device [B, D_max + 1] (root first, -1 padded)
 * out_tok       device [B]: the correction token (the bonus token when a leaf was reached)
 * Vocabularies above 262144 return TALON_ERR_UNSUPPORTED.  A row without a softmax (NaN, +inf,
 * only -inf) sets the NONFINITE status; that sequence gets accept_len 0 and out_tok -1.
 * Decisions are taken in fp64 from fp32 row statistics: a uniform within about 1e-6 (relative) of
 * its threshold may fall on the other side than in exact arithmetic. */
talon_status talon_accept_sample(talon_ctx *ctx, const talon_tree *tree, const float *target_logits,
                                 int64_t row_stride, double temperature, const double *u_accept,
                                 const double *u_sample, int32_t *accept_len, int32_t *accept_nodes,
                                 int32_t *out_tok, void *stream);

/* What a verified step leaves for the next one (the generation loop of Section 5.3): for every
 * sequence b the key and value rows of the accepted nodes accept_nodes[b, 0 .. accept_len[b]]
 * (root first) are copied from k_tree / v_tree to the prefix cache at tokens prefix_len[b] ..
 * prefix_len[b] + accept_len[b] of the sequence's block, prefix_len[b] grows by accept_len[b] + 1,
 * root_tok[b] becomes next_tok[b] (talon_accept's bonus_tok or talon_accept_sample's out_tok), and
 * counters[b] advances by (1, draft passes, accept_len[b] + 1): the N_p, N_q and L of Section 5.3,
 * a draft pass being a layer Algorithm 2 expanded for this sequence.  Call after talon_build_tree and
 * one of the two verification calls.  The next step starts with talon_reset(root_tok, prefix_len).
 * All pointers device memory.  k_tree, v_tree [B, N, Hkv, Dh] bf16; k_prefix, v_prefix, kv_start,
 * kv_tokens, kv_stride_t, kv_stride_h as in talon_tree_attention (written here);
 * kv_limit  [B] int64 or null: first token offset past the block of sequence b (kv_tokens if null)
 * prefix_len [B] in/out; root_tok [B] out; counters [B, 3] int64 in/out or null.
 * A sequence whose block has no room is left as it is and the CAPACITY status is set. */
talon_status talon_commit(talon_ctx *ctx, const talon_tree *tree, const int32_t *accept_len,
                          const int32_t *accept_nodes, const int32_t *next_tok, const void *k_tree,
                          const void *v_tree, void *k_prefix, void *v_prefix, const int64_t *kv_start,
                          const int64_t *kv_limit, int64_t kv_tokens, int64_t kv_stride_t,
                          int64_t kv_stride_h, int32_t *prefix_len, int32_t *root_tok,
                          int64_t *counters, void *stream);

/* Synchronises `stream`, reads and returns the device status word (OK, NONFINITE, TIMEOUT,
 * CAPACITY).  The word stays set until the next talon_reset. */
talon_status talon_poll_status(talon_ctx *ctx, void *stream);

/* Host buffers in, host results out: one whole draft-and-verify step (reset, up to D_max
 * expansion layers, build, tree attention, accept) with the host-to-device and
 * device-to-host copies included.  All pointers are HOST memory (pinned memory makes the
 * copies asynchronous).  Layouts as in the device calls with rows BY_NODE and dense tensors:
 *  draft_logits  [B, N, V] fp32: row i holds the draft logits of node i (rows of nodes that
 *                are never expanded are not read)
 *  target_logits [B, N, V] fp32
 *  q [B,N,Hq,Dh], k_prefix/v_prefix [sum_b L_b, Hkv, Dh] (sequences back to back),
 *  k_tree/v_tree [B,N,Hkv,Dh], all bf16
 *  outputs: out_attn [B,N,Hq,Dh] bf16 (may be null), n_nodes [B], token/parent/depth/position
 *  [B,N] (each may be null), accept_len [B], accept_nodes [B, D_max+1], bonus_tok [B].
 * The first call allocates device staging buffers sized for batch_max inside the context
 * (a later call with a longer total prefix reallocates).  Synchronises `stream` before
 * returning and returns the device status. */
talon_status talon_step_host(talon_ctx *ctx, int32_t B, const int32_t *root_tok,
                             const int32_t *prefix_len, const float *draft_logits,
                             const float *target_logits, const void *q, const void *k_prefix,
                             const void *v_prefix, const void *k_tree, const void *v_tree,
                             float sm_scale, void *out_attn, int32_t *n_nodes, int32_t *token,
                             int32_t *parent, int32_t *depth, int32_t *position,
                             int32_t *accept_len, int32_t *accept_nodes, int32_t *bonus_tok,
                             void *stream);

/* Device buffers in, device results out: the same whole step as talon_step_host (Algorithm 2
 * until the budget or D_max is reached, then Appendix B's verification) as one call, so that a
 * caller pays for one library entry instead of D_max + 4.  Every pointer is DEVICE memory with
 * the layout of the call it is handed to: talon_reset (root_tok, prefix_len), talon_expand_layer
 * with rows BY_NODE (draft_logits, draft_row_stride, N rows per sequence), talon_tree_attention
 * (q .. out), talon_accept (target_logits .. bonus_tok; target_tok may be null).
 * n_layers  expansion layers to enqueue, 0..D_max (layers after the tree is full cost one
 *           frontier check each and read no logits)
 * Enqueues only; no synchronisation.
 * A step is a chain of small dependent kernels, so from the second call with exactly the same
 * arguments the library captures these launches into a CUDA graph once and replays it on later
 * calls (same kernels, same memory, one submission; up to 64 argument sets are kept, least
 * recently used first out).  The plain launch sequence is used on the legacy default stream, while
 * `stream` is being captured by the caller, while launches are timed (talon_timing_enable without
 * pause), and always when the environment has TALON_STEP_GRAPH=0. */
talon_status talon_step(talon_ctx *ctx, const talon_tree *tree, int32_t B, const int32_t *root_tok,
                        const int32_t *prefix_len, const float *draft_logits,
                        int64_t draft_row_stride, int32_t n_layers, const void *q,
                        const void *k_prefix, const void *v_prefix, const void *k_tree,
                        const void *v_tree, const int64_t *kv_start, int64_t kv_tokens,
                        int64_t kv_stride_t, int64_t kv_stride_h, int32_t max_prefix_len,
                        float sm_scale, void *out,
                        const float *target_logits, int64_t target_row_stride, int32_t *target_tok,
                        int32_t *accept_len, int32_t *accept_nodes, int32_t *bonus_tok,
                        void *stream);

/* Paged prefix cache (the layout serving systems keep for batches, which the paper's "Limitations"
 * name as the open case; Section 5.3's loop is the same).  The cache is a pool of pages of
 * TALON_PAGE_TOKENS tokens: token t of sequence b lives in page block_table[b, t / 128] at offset
 * t % 128, i.e. at cache token page * 128 + offset of a [n_pages * 128, Hkv, Dh] array with the
 * usual strides.  A page is one key tile of the attention kernel, so a tile never straddles pages.
 *  block_table   device [B, table_stride] int32 page numbers; a sequence needs
 *                ceil(prefix_len / 128) entries (talon_commit_paged: up to n_blocks[b])
 *  n_pages       pages in the pool (bounds the tensor map)
 * Otherwise as talon_tree_attention.  Query-group sizes that do not divide 128 return
 * TALON_ERR_UNSUPPORTED here (the warp-MMA kernel reads contiguous blocks only). */
#define TALON_PAGE_TOKENS 128
talon_status talon_tree_attention_paged(talon_ctx *ctx, const talon_tree *tree, const void *q,
                                        const void *k_pages, const void *v_pages, const void *k_tree,
                                        const void *v_tree, const int32_t *block_table,
                                        int32_t table_stride, int64_t n_pages, int64_t kv_stride_t,
                                        int64_t kv_stride_h, int32_t max_prefix_len, float sm_scale,
                                        void *out, void *stream);

/* talon_commit on a paged cache: the accepted path's K/V rows go to tokens prefix_len[b] + j of
 * sequence b through the page table.
 *  n_blocks  device [B]: pages the sequence owns (entries of its block_table row that are valid);
 *            a sequence whose accepted tokens do not fit in them is left untouched and
 *            TALON_ERR_CAPACITY is reported by talon_poll_status. */
talon_status talon_commit_paged(talon_ctx *ctx, const talon_tree *tree, const int32_t *accept_len,
                                const int32_t *accept_nodes, const int32_t *next_tok,
                                const void *k_tree, const void *v_tree, void *k_pages, void *v_pages,
                                const int32_t *block_table, int32_t table_stride,
                                const int32_t *n_blocks, int64_t n_pages, int64_t kv_stride_t,
                                int64_t kv_stride_h, int32_t *prefix_len, int32_t *root_tok,
                                int64_t *counters, void *stream);

/* Section 5.3's generation loop, n_steps draft-and-verify steps in one call: for every step the
 * launches of talon_step followed by talon_commit, so that the accepted tokens' K/V join the
 * prefix cache, prefix_len grows and the correction token is the next step's root, all on the
 * device (the call only enqueues; a caller may capture it into one CUDA graph).  The stand-ins for
 * the two model forwards are indexed by step: step s reads draft_logits + s * draft_step_stride,
 * target_logits + s * target_step_stride, q + s * q_step_stride and k_tree / v_tree +
 * s * kv_tree_step_stride (strides in elements), and writes accept_len / bonus_tok at
 * + s * result_step_stride and accept_nodes at + s * result_step_stride * (D_max + 1) (a stride of 0
 * keeps only the last step's).  root_tok, prefix_len, the cache and counters ([B, 3], as in
 * talon_commit; required) are read and advanced in place.
 *  max_prefix_len  bound on prefix_len[b] over ALL steps (the last step's prefix included) */
talon_status talon_loop(talon_ctx *ctx, const talon_tree *tree, int32_t B, int32_t n_steps,
                        int32_t *root_tok, int32_t *prefix_len, const float *draft_logits,
                        int64_t draft_row_stride, int64_t draft_step_stride, int32_t n_layers,
                        const void *q, int64_t q_step_stride, void *k_prefix, void *v_prefix,
                        const void *k_tree, const void *v_tree, int64_t kv_tree_step_stride,
                        const int64_t *kv_start, const int64_t *kv_limit, int64_t kv_tokens,
                        int64_t kv_stride_t, int64_t kv_stride_h, int32_t max_prefix_len,
                        float sm_scale, void *out, const float *target_logits,
                        int64_t target_row_stride, int64_t target_step_stride, int32_t *target_tok,
                        int32_t *accept_len, int32_t *accept_nodes, int32_t *bonus_tok,
                        int64_t result_step_stride, int64_t *counters, void *stream);

/* Section 5.3's figures from the counters talon_commit keeps (HOST copy of the [B, 3] array: N_p
 * verification passes, N_q draft passes, L tokens produced), summed over the sequences: draft
 * efficiency delta = N_q / N_p (Eq. 6), mean accepted tokens tau = L / N_p, and the wall-time
 * speed-up R = tau / (1 + c * delta) (Eq. 7) for a draft pass that costs cost_ratio = c target
 * passes.  Host arithmetic only; TALON_ERR_INVALID_ARG when no pass has been committed. */
talon_status talon_loop_metrics(const int64_t *counters, int32_t B, double cost_ratio, double *delta,
                                double *tau, double *speedup);

/* The paper has no counterpart for this call: it exists for callers that cannot allocate.
 * talon_accept needs a context, and talon_create calls cudaMalloc.  Code that runs inside a
 * fixed memory pool, or in a part of a serving loop where allocating is not allowed (it
 * synchronises the device and may fail when memory is tight), can use this call instead for the
 * first half of the greedy verification: t_i = argmax of target-logit row i, lowest id among
 * equal maxima.  A NaN never competes, wherever it sits in the row; a row that holds nothing but
 * NaN gives -1 (a row of -inf only gives token 0, like any other row of equal values).  It needs no context and calls no cudaMalloc,
 * cudaFree or any other allocating routine; its scratch (one 8-byte key per row) is a fixed
 * array inside the library image, TALON_NOALLOC_MAX_ROWS * 8 bytes on every GPU that loads the
 * library, held until the process exits.
 *  target_logits device fp32, row i at target_logits + i * row_stride; 16-byte aligned
 *  row_stride    elements between rows, a multiple of 4 and >= vocab
 *  n_rows        0 .. TALON_NOALLOC_MAX_ROWS; more returns TALON_ERR_CAPACITY, nothing enqueued
 *  target_tok    device [n_rows]
 * Runs on the current device; enqueues three kernels on `stream` and returns.  The first call on
 * a device looks up the array's device address (cudaGetSymbolAddress) and the SM count, under a
 * lock, so host threads may race to it; make that first call outside any stream capture.  Every call clears the rows it uses first, since
 * the array keeps the previous call's keys.  All calls share the one array: two calls that can
 * overlap on the GPU (different streams without an ordering between them) race. */
#define TALON_NOALLOC_MAX_ROWS 8192
talon_status talon_target_argmax_noalloc(const float *target_logits, int64_t row_stride, int32_t vocab,
                                         int32_t n_rows, int32_t *target_tok, void *stream);

/* Number of kernels the library has launched through this context since creation. */
int64_t talon_launch_count(const talon_ctx *ctx);

/* Kernel families of the library, for talon_timing_read. */
enum {
  TALON_K_RESET = 0,        /* tree initialisation of Algorithm 2                              */
  TALON_K_EXPAND_ROWS = 1,  /* softmax normaliser + per-parent top-k over the logit rows    */
  TALON_K_SELECT = 2,       /* Top-K / gate / budget truncation / append                    */
  TALON_K_BUILD = 3,        /* positions and sentinels                                      */
  TALON_K_ATTENTION = 4,    /* tree attention                                               */
  TALON_K_COMBINE = 5,      /* merge of split-KV partials                                   */
  TALON_K_ARGMAX = 6,       /* target argmax                                                */
  TALON_K_WALK = 7,         /* greedy accept walk                                           */
  TALON_K_ROWSTATS = 8,     /* softmax normaliser of the target rows (sampling verification) */
  TALON_K_SAMPLE = 9,       /* rejection walk and correction-token draw                     */
  TALON_K_COMMIT = 10,      /* accepted K/V rows into the prefix cache, counters            */
  TALON_N_KERNELS = 11
};

/* Per-kernel device timing.  With max_launches > 0 the context creates that many pairs of
 * CUDA events (an allocation; synchronises the device) and from then on brackets every launch
 * of the kernel families in kernel_mask (bit k = family k; 0 = all) with a pair recorded on the
 * launching stream, until the pairs run out.  max_launches = 0 switches timing off and destroys
 * the events.  Do not capture a stream into a CUDA graph while timing is on. */
talon_status talon_timing_enable(talon_ctx *ctx, int32_t max_launches, uint32_t kernel_mask);

/* Suspends (paused != 0) or resumes the bracketing without touching the events, so that a
 * caller can time a sample of its steps and leave the others undisturbed. */
talon_status talon_timing_pause(talon_ctx *ctx, int32_t paused);

/* Synchronises `stream`, adds up the elapsed time of the bracketed launches per kernel family
 * since the last read, and makes all pairs available again.
 * ms        host [TALON_N_KERNELS] summed milliseconds
 * launches  host [TALON_N_KERNELS] number of launches that were timed */
talon_status talon_timing_read(talon_ctx *ctx, void *stream, double *ms, int64_t *launches);

const char *talon_kernel_name(int32_t kernel);

const char *talon_status_string(talon_status s);

#ifdef __cplusplus
}
#endif
#endif /* TALON_H_ */
