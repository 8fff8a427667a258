/*
 * fspad.h - C ABI of the B200 (sm_100a) tree-verification library.
 *
 * One verify step of lossless speculative decoding, as the paper states it
 * (Section "Preliminaries"): the target model runs once over the flattened
 * draft tree under a mask that lets every token see only what it depends on,
 * its results are compared strictly with the tree, and mismatching tokens and
 * their descendants are discarded.  Three operations:
 *
 *   fspad_tree_attn    tree-masked verify attention of one layer
 *   fspad_tree_accept  lossless acceptance (greedy, or recursive rejection
 *                      sampling at temperature > 0; Section "Experiments"
 *                      evaluates T = 0 and T = 1 with unrelaxed acceptance)
 *   fspad_kv_compact   keep the accepted path's K/V rows, contiguous in the cache
 * and, one step earlier in the pipeline,
 *   fspad_draft_expand one draft step: per-row top-k, joint probabilities, next frontier
 *   fspad_tree_build   the draft phase's candidates -> the flattened token tree
 *
 * Conventions (shared by every call)
 *   - A tree has N <= 256 nodes (N <= 64 for fspad_tree_build) in topological order: parent[0] = -1 (node 0 is
 *     the root = the last token already emitted; it is always accepted) and
 *     0 <= parent[i] < i.  Children of a node are visited in increasing index.
 *   - "bf16" is a 16-bit brain-float bit pattern (typedef below).
 *   - Unless a parameter says "host", every pointer is a DEVICE pointer owned by
 *     the caller, 16-byte aligned, valid until the work queued on `stream` has
 *     finished.  The library never frees or reallocates caller memory.
 *   - Calls are asynchronous on `stream` (a cudaStream_t passed as void*; NULL =
 *     the default stream).  Calls that share a context must be queued on one
 *     stream at a time (the context owns scratch buffers).
 *   - Return value: 0 (FSPAD_OK) or a negative fspad_error.  Errors detectable
 *     on the host are returned before anything is launched.  Errors only the
 *     device can see (a malformed parent[] array, a prefix length that does not
 *     fit) are recorded in the context's status word, read by fspad_status();
 *     the outputs of that call are then unspecified but every access stays
 *     inside the caller's buffers.  Nothing traps, asserts or exits.
 */
#ifndef FSPAD_H
#define FSPAD_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef uint16_t fspad_bf16;
typedef struct fspad_ctx fspad_ctx;

typedef enum {
    FSPAD_OK = 0,
    FSPAD_ERR_NULL = -1,           /* a required pointer is NULL                       */
    FSPAD_ERR_ALIGN = -2,          /* a pointer is not 16-byte aligned                 */
    FSPAD_ERR_SHAPE = -3,          /* sizes inconsistent with the context              */
    FSPAD_ERR_TREE_TOO_LARGE = -4, /* n_nodes > 256 (tree builder: 64) or > max_nodes    */
    FSPAD_ERR_RANGE = -5,          /* prefix_len + n_nodes > max_len, T < 0 or NaN     */
    FSPAD_ERR_CUDA = -6,           /* a CUDA runtime call or launch failed             */
    FSPAD_ERR_TIMEOUT = -7,        /* a bounded device-side wait ran out               */
    FSPAD_ERR_BAD_TREE = -8,       /* parent[0] != -1 or parent[i] outside [0, i)      */
    FSPAD_ERR_NOMEM = -9,          /* device or host allocation failed at create time  */
    FSPAD_ERR_TOO_LARGE = -10      /* size beyond the fixed capacity of a no-allocation call */
} fspad_error;

typedef struct {
    int n_q_heads;        /* Hq                                                     */
    int n_kv_heads;       /* Hkv, divides Hq; query head h uses kv head h/(Hq/Hkv)   */
    int head_dim;         /* d, must be 128                                         */
    int max_nodes;        /* largest N any call will pass, 1..256                   */
    int vocab;            /* V                                                      */
    int n_layers;         /* layers in the cache handed to fspad_kv_compact          */
    int max_len;          /* rows per (sequence, kv head) of the cache               */
    int max_batch;        /* largest batch any call will pass                       */
    float softmax_scale;  /* 0 selects 1/sqrt(d)                                    */
} fspad_config;

/* Create a context on the CURRENT device: allocates the scratch buffers every
 * call needs (split-KV partials, per-node statistics), the second stream and
 * the events of fspad_verify_step, sized from `cfg`.  Synchronous.  *out is
 * NULL on failure.  (The device staging of fspad_verify_step_host is allocated
 * by that entry point's first call.) */
int fspad_create(const fspad_config *cfg, fspad_ctx **out);

/* Free everything the context owns.  Synchronises the device first. */
void fspad_destroy(fspad_ctx *ctx);

/* Synchronise `stream`, return the first device-recorded error since the last
 * call (FSPAD_OK if none) and clear it. */
int fspad_status(fspad_ctx *ctx, void *stream);

/* Static, human-readable name of an fspad_error. */
const char *fspad_strerror(int err);

/* Number of kernels the library has launched through this context so far
 * (host counter; lets a caller verify that work ran on the device). */
long long fspad_launch_count(const fspad_ctx *ctx);

/*
 * Self-test of the library's bounded device-side waits (error handling of the
 * library; no passage of the paper).  Every wait of a kernel on a barrier has
 * a poll limit; when it runs out the kernel records FSPAD_ERR_TIMEOUT in the
 * status word and returns.  This call queues one warp that waits, with a limit
 * of `polls` polls (1 .. 4096), on a barrier nothing ever arrives on: after it
 * fspad_status() returns FSPAD_ERR_TIMEOUT, and the context stays usable.
 */
int fspad_selftest_wait_timeout(fspad_ctx *ctx, int polls, void *stream);

/*
 * Tree-masked verify attention of one layer ("Preliminaries": the flattened
 * token tree is the target's input and the attention mask built from the tree
 * introduces the dependencies between its tokens).
 *
 * For sequence b, query node i and query head h (kv head g = h / (Hq/Hkv)):
 *   keys   = cache rows 0 .. L_b-1 of kv head g   (L_b = prefix_len[b])
 *          + tree row j for every j that is i itself or an ancestor of i
 *   out[b][i][h] = softmax(q[b][i][h] . k * softmax_scale) . v     over those keys
 * bf16 inputs, fp32 accumulation and softmax, bf16 output (round to nearest even).
 * q/k are used as given: no positional encoding is applied here.
 *
 *   q        [batch][n_nodes][Hq][d]
 *   k_cache, v_cache   [batch][Hkv][max_len][d]
 *   tree_k, tree_v     [batch][Hkv][n_nodes][d]; both may be NULL, in which case
 *            the tree rows are cache rows L_b .. L_b+n_nodes-1 of the same sequence
 *   parent   [batch][n_nodes] int32      prefix_len [batch] int32
 *   out      [batch][n_nodes][Hq][d]     (must not alias an input)
 * Requires 0 <= L_b and L_b + n_nodes <= max_len (device-checked: FSPAD_ERR_RANGE).
 */
int fspad_tree_attn(fspad_ctx *ctx, const fspad_bf16 *q, const fspad_bf16 *k_cache,
                    const fspad_bf16 *v_cache, const fspad_bf16 *tree_k, const fspad_bf16 *tree_v,
                    const int32_t *parent, const int32_t *prefix_len, int n_nodes, int batch,
                    fspad_bf16 *out, void *stream);

/*
 * Lossless tree acceptance ("Preliminaries": strict comparison of the tree with
 * the target's results, differing tokens and their descendants discarded;
 * "Experiments": greedy T = 0 and sampling T = 1, acceptance never relaxed).
 *
 * Per sequence b with T = temperature[b]:
 *   T == 0  walk from the root; at node cur accept the first child (index order)
 *           whose draft token equals argmax(target_logits[cur]) (lowest index on
 *           ties); stop when no child matches; bonus = argmax of the last node.
 *   T  > 0  recursive rejection sampling.  p = softmax(target_logits[cur]/T),
 *           q = draft_probs[cur].  For each child c (index order) with token x:
 *           accept iff uniforms[c] * q[x] < p[x]; on reject p <- normalise(
 *           max(p - q, 0)) (unchanged if that sum is 0), q[x] <- 0, q <- q/sum(q).
 *           When no child is accepted the bonus token is the inverse-CDF draw of
 *           the current p with uniforms[n_nodes]: the smallest token whose running
 *           sum (index order) exceeds u * sum; the largest positive-weight token
 *           if rounding leaves none.  Decisive scalars are evaluated in fp64.
 *   The rule at T > 0 is exactly lossless when the children of a node were drawn
 *   one after another without replacement from draft_probs[node].
 *
 *   target_logits [batch][n_nodes][V] fp32 (finite or -inf; NaN is a precondition violation)
 *   draft_probs   [batch][n_nodes][V] fp32 >= 0; may be NULL iff every temperature is 0
 *   draft_tokens, parent  [batch][n_nodes] int32, tokens in [0, V)
 *   temperature   [batch] fp32 >= 0
 *   uniforms      [batch][n_nodes+1] fp32 in [0,1); may be NULL iff draft_probs is NULL
 *   accepted_path [batch][max_nodes] int32: node ids from the root, -1 padded
 *   n_accepted    [batch] int32: nodes on the path, root included
 *   bonus_token   [batch] int32
 * Outputs stay on the device so fspad_kv_compact can consume them without a host sync.
 */
int fspad_tree_accept(fspad_ctx *ctx, const float *target_logits, const float *draft_probs,
                      const int32_t *draft_tokens, const int32_t *parent, const float *temperature,
                      const float *uniforms, int n_nodes, int batch, int32_t *accepted_path,
                      int32_t *n_accepted, int32_t *bonus_token, void *stream);

/*
 * The first stage of fspad_tree_accept on its own: one pass over every row of
 * logits [rows][V] giving row_max (fp32 maximum), row_arg (its lowest index)
 * and row_sum = sum_j exp((x_j - max)/T_row) accumulated from fp32 exponentials
 * (relative accuracy about 1e-6; the acceptance walk re-derives exact sums
 * where a decision is close).  temperature [rows / rows_per_seq] fp32, 0 -> 1.
 * With all three outputs NULL only the streaming pass over the logits runs (its per-CTA
 * partial results stay in the context's scratch): the HBM-bound kernel on its own, for
 * timing and profiling.
 */
int fspad_accept_stats(fspad_ctx *ctx, const float *logits, const float *temperature, int rows,
                       int rows_per_seq, float *row_max, double *row_sum, int32_t *row_arg,
                       void *stream);

/*
 * fspad_accept_stats without any allocation.  (The paper has no counterpart:
 * this entry point exists for the sake of the hosting program, not the method.)
 *
 * Who needs it: a caller that is not allowed to allocate device memory - for
 * instance a serving process whose own memory pool has claimed the whole GPU
 * and treats any outside cudaMalloc as an error, or code on a latency-critical
 * path where the implicit device synchronisation of an allocation is ruled out.
 * Such a caller cannot use fspad_create (it allocates the context's scratch),
 * so this call takes no context.  Its scratch (the per-CTA partial results of
 * each row) is a fixed array inside the library's device image:
 * about 0.5 MB that every GPU loading the library keeps until the process ends.
 *
 * Same inputs, outputs and results as fspad_accept_stats (vocab is passed
 * explicitly since there is no context), all DEVICE pointers owned by the caller.
 * Limits: rows <= 1024; larger calls return FSPAD_ERR_TOO_LARGE and launch nothing.
 * The call allocates and frees nothing, on the device or through any library.
 *
 * The first call on each device looks up the scratch array's device address
 * (a cudaGetSymbolAddress query, with that device current); make that first
 * call outside any stream capture.  All calls on a device share the one array:
 * a call rewrites every slot it later reads, so nothing needs clearing between
 * calls, but two calls whose GPU
 * work overlaps (different streams, or different host threads) race on it and
 * give undefined results - serialise them.
 */
int fspad_accept_stats_noalloc(const float *logits, const float *temperature, int rows,
                               int rows_per_seq, int vocab, float *row_max, double *row_sum,
                               int32_t *row_arg, void *stream);

/*
 * Target LM head with the per-node scan as its epilogue ("Preliminaries": the
 * target's one forward over the flattened tree yields, for every tree node, the
 * distribution the tree is compared with; the last step of that forward is the
 * product of the nodes' final hidden states with the vocabulary matrix).
 *
 *   logits[r][v] = sum_h hidden[r][h] * lm_head[v][h]     bf16 inputs, fp32 accumulation
 *   row_max / row_arg / row_sum of every row of logits as in fspad_accept_stats
 *
 * The tiles of the product are reduced to (maximum, lowest index, sum of
 * exponentials) as they leave the tensor cores; the logits themselves are
 * written only if logits_out is given.
 *
 *   hidden     [rows][hidden_dim] bf16        lm_head [vocab][hidden_dim] bf16 (vocab is the context's)
 *   hidden_dim a multiple of 8;  rows <= max_batch * max_nodes of the context
 *   temperature [rows / rows_per_seq] fp32 or NULL (0 -> 1), as in fspad_accept_stats
 *   logits_out [rows][vocab] fp32 or NULL;  row_max fp32, row_sum fp64, row_arg int32: [rows]
 * All pointers are device pointers, 16-byte aligned.  Rows are processed in slabs of 128; every slab
 * streams the vocabulary matrix once.  Accuracy: the products are exact, the fp32 accumulation over
 * hidden_dim terms leaves an absolute error of about 1e-5 (bounded by hidden_dim / 16 roundings of the
 * running sum) in every logit, so row_arg is the exact argmax wherever the maximum leads the runner-up
 * by more than that.
 */
int fspad_lm_head_stats(fspad_ctx *ctx, const fspad_bf16 *hidden, const fspad_bf16 *lm_head, int hidden_dim, int rows,
                        int rows_per_seq, const float *temperature, float *logits_out, float *row_max, double *row_sum,
                        int32_t *row_arg, void *stream);

/*
 * fspad_tree_accept fed by the LM head directly ("Preliminaries": forward, then strict comparison):
 * the logits of fspad_tree_accept are hidden . lm_head^T as in fspad_lm_head_stats, their scan happens
 * in the product's epilogue, and the acceptance walk follows.  Every other argument, the outputs and
 * the acceptance rule are those of fspad_tree_accept.
 *
 *   hidden [batch][n_nodes][hidden_dim] bf16;  lm_head [vocab][hidden_dim] bf16
 *   logits [batch][n_nodes][vocab] fp32, written by the call: required when draft_probs is given (the
 *          sampling walk reads the rows on its path), may be NULL when every temperature is 0, in
 *          which case no logit is ever written to memory.
 */
int fspad_lm_head_accept(fspad_ctx *ctx, const fspad_bf16 *hidden, const fspad_bf16 *lm_head, int hidden_dim,
                         const float *draft_probs, const int32_t *draft_tokens, const int32_t *parent,
                         const float *temperature, const float *uniforms, int n_nodes, int batch, float *logits,
                         int32_t *accepted_path, int32_t *n_accepted, int32_t *bonus_token, void *stream);

/*
 * Feature Sampler forward ("Feature Sampling": the Up projector maps the feature f and the Gate projector
 * the token embedding e to intermediate size; the embedding's image is activated by SiLU and multiplied,
 * element by element, with the feature's image; the Down projector maps the result back to hidden size,
 * where the residual connection adds the input feature):
 *
 *   eta[r] = W_down ( silu(W_gate e[r]) * (W_up f[r]) ) + f[r]
 *
 * bf16 inputs and weights, fp32 accumulation; the gated product is rounded to bf16 (it is the Down
 * projector's tensor-core operand) and so is eta.  This is the draft model's input synthesis, run once per
 * draft step on the frontier rows; no positional or normalisation step is applied here.
 *
 *   f, e     [rows][hidden_dim] bf16          rows <= 128
 *   w_up, w_gate [inter_dim][hidden_dim] bf16 w_down [hidden_dim][inter_dim] bf16
 *   inter    [rows][inter_dim] bf16, written: the gated product (kept: it is the second product's operand)
 *   eta      [rows][hidden_dim] bf16, written
 *   workspace  device memory of at least fspad_feature_sampler_workspace_bytes(rows, hidden_dim, inter_dim)
 *            bytes, owned by the caller (fp32 partial sums of the split products); contents are scratch
 * hidden_dim and inter_dim multiples of 8; all pointers device, 16-byte aligned.  Errors: FSPAD_ERR_SHAPE
 * for sizes outside these ranges, FSPAD_ERR_RANGE for a workspace that is too small.
 */
size_t fspad_feature_sampler_workspace_bytes(int rows, int hidden_dim, int inter_dim);
int fspad_feature_sampler(fspad_ctx *ctx, const fspad_bf16 *f, const fspad_bf16 *e, const fspad_bf16 *w_up,
                          const fspad_bf16 *w_gate, const fspad_bf16 *w_down, int rows, int hidden_dim, int inter_dim,
                          fspad_bf16 *inter, fspad_bf16 *eta, void *workspace, size_t workspace_bytes, void *stream);

/*
 * Dynamic token tree, one draft step ("Preliminaries", last paragraph: the
 * output of each draft step is truncated to its top-k, and every token carries
 * the joint probability of its path).  Called once per level of the draft
 * phase; fspad_tree_build then turns the accumulated candidates into the tree.
 *
 *   logprobs      [batch][n_frontier][vocab] float, device: the draft model's
 *                 log-probabilities of the next token after each frontier node
 *                 (vocab is the context's); NaN not allowed.
 *   frontier_logp [batch][n_frontier] float, device: joint log-probability of
 *                 each frontier node (0 for the root at the first level).
 *   frontier_cand [batch][n_frontier] int32, device: candidate index of each
 *                 frontier node (-1 for the root).
 *   n_frontier, top_k: 1 .. 16 (top_k <= vocab); width: 1 .. n_frontier * top_k.
 *   base, n_cand_cap: the new candidates get the indices base .. base +
 *                 n_frontier * top_k - 1 of arrays that hold n_cand_cap entries
 *                 per sequence; the caller advances base from level to level.
 *
 * For frontier node f the top_k largest entries of its row (equal values: the
 * lower token first) become the candidates base + f * top_k + r, r = 0 for the
 * most probable: cand_parent = frontier_cand[f], cand_token = the token,
 * cand_logp = frontier_logp[f] + value (one single-precision addition).  The
 * `width` new candidates with the largest joint value (equal values: the lower
 * candidate index first) are returned, in that order, as next_cand / next_logp
 * [batch][width]: the frontier of the next level.  cand_* are [batch][n_cand_cap],
 * device, owned by the caller; only the new entries are written.  Per-piece
 * lists live in the context's scratch (allocated by fspad_create): one call per
 * context at a time.  Asynchronous on `stream`.  Errors: FSPAD_ERR_SHAPE for
 * sizes outside the ranges above, FSPAD_ERR_TOO_LARGE when ceil(vocab / 4096) *
 * top_k exceeds 1024.
 */
int fspad_draft_expand(fspad_ctx *ctx, const float *logprobs, const float *frontier_logp,
                       const int32_t *frontier_cand, int n_frontier, int top_k, int width, int base, int n_cand_cap,
                       int batch, int32_t *cand_parent, int32_t *cand_token, float *cand_logp, int32_t *next_cand,
                       float *next_logp, void *stream);

/*
 * Dynamic token tree, final stage ("Preliminaries", last paragraph: each draft
 * step is truncated to its top-k, every token carries the joint probability of
 * its path, and one top-k over all tokens after the draft phase gives a valid
 * tree of bounded size; "Performance on Fewer Candidate Tokens" halves both
 * budgets).  Turns the candidates a draft phase left behind into the flattened
 * tree that fspad_tree_attn / fspad_tree_accept take.
 *
 *   cand_parent [batch][n_cand] int32, device: index of the candidate's parent
 *               candidate, -1 for a child of the root.  Candidates are listed
 *               level by level: a parent has a lower index than its children.
 *   cand_token  [batch][n_cand] int32, device.
 *   cand_logp   [batch][n_cand] float, device: joint log-probability of the path
 *               from the root; never larger than the parent's; -inf allowed, NaN
 *               not.
 *   root_token  [batch] int32, device: token of node 0.
 *   n_cand      1 .. 1024;  n_nodes 1 .. min(64, max_nodes of the context).
 *
 * Kept: the n_nodes - 1 candidates with the largest joint probability; among
 * equal values the lower index first (so a parent is never displaced by a child
 * of equal probability).  Output, all [batch][n_nodes] int32, device, written
 * by the call: node 0 is the root (parent -1, token root_token, candidate -1);
 * the kept candidates follow ordered by depth and, inside a depth, by candidate
 * index, so parent_out[i] < i.  cand_out[i] is the candidate a node came from.
 * n_out[b] = 1 + min(n_nodes - 1, n_cand); entries from n_out[b] on are -1.
 * anc_out [batch][n_nodes] uint64, device, may be NULL: bit j of anc_out[i] is
 * set iff node j is node i or one of its ancestors - the attention mask the
 * target verifies the tree under ("Preliminaries": the mask is updated from the
 * token tree); 0 from n_out[b] on.
 * Nothing is allocated; the caller owns every array.  A parent index out of
 * order, or joint probabilities that grow along a path (a kept candidate whose
 * parent was not kept), set FSPAD_ERR_BAD_TREE in the status word; all writes
 * stay in bounds.
 */
int fspad_tree_build(fspad_ctx *ctx, const int32_t *cand_parent, const int32_t *cand_token,
                     const float *cand_logp, const int32_t *root_token, int n_cand, int n_nodes, int batch,
                     int32_t *parent_out, int32_t *token_out, int32_t *cand_out, uint64_t *anc_out,
                     int32_t *n_out, void *stream);

/*
 * Accepted-path KV compaction ("Preliminaries": the discarded tokens leave the
 * sequence; only the accepted path continues it).  For every layer, K and V,
 * sequence b and kv head: row L_b + accepted_path[b][j] moves to row L_b + j for
 * j = 0 .. n_accepted[b]-1, as if all moves happened at once (a destination may
 * be another move's source).  Rows >= L_b + n_accepted[b] keep their old
 * contents and are dead.  new_len[b] = L_b + n_accepted[b] (may be NULL).
 *
 *   cache [n_layers][2][batch][Hkv][max_len][d] bf16, updated in place
 *   accepted_path [batch][max_nodes], n_accepted [batch], prefix_len [batch], new_len [batch]: int32
 */
int fspad_kv_compact(fspad_ctx *ctx, fspad_bf16 *cache, const int32_t *accepted_path,
                     const int32_t *n_accepted, const int32_t *prefix_len, int batch,
                     int32_t *new_len, void *stream);

/*
 * Cache append of the accepted path: compaction for a caller that keeps the tree's K/V rows of the verify
 * forward outside the cache ("Preliminaries": the accepted tokens continue the sequence, the others and
 * their descendants are discarded - here the discarded rows never reach the cache at all).  For every layer,
 * K and V, sequence b and kv head:
 *   cache[..][L_b + j][:] = tree_kv[..][accepted_path[b][j]][:],  j = 0 .. n_accepted[b]-1;
 * nothing else in the cache changes.  new_len[b] = L_b + n_accepted[b] (may be NULL).
 *
 *   cache   [n_layers][2][batch][Hkv][max_len][d] bf16 (device), updated in place
 *   tree_kv [n_layers][2][batch][Hkv][n_nodes][d] bf16 (device), read only; must not overlap cache
 *   accepted_path [batch][max_nodes], n_accepted [batch], prefix_len [batch], new_len [batch]: int32 (device)
 * Both arrays stay the caller's.  Errors: NULL / misaligned pointers and sizes beyond the context are
 * refused on the host; a path entry outside [0, n_nodes), n_accepted outside [0, n_nodes] or
 * L_b + n_accepted[b] > max_len set FSPAD_ERR_RANGE in the status word and the offending rows are skipped.
 */
int fspad_kv_append(fspad_ctx *ctx, fspad_bf16 *cache, const fspad_bf16 *tree_kv, const int32_t *accepted_path,
                    const int32_t *n_accepted, const int32_t *prefix_len, int n_nodes, int batch, int32_t *new_len,
                    void *stream);

/*
 * The same two operations on a cache that is not contiguous (the paper's remark on practical frameworks in
 * "Performance on Fewer Candidate Tokens" is the only place it touches deployment; serving systems keep the
 * cache in fixed-size blocks).  The cache is a pool of blocks of 128 rows and a per-sequence block table:
 * cache row r of sequence b is row r % 128 of block block_table[b][r / 128].
 *
 *   k_pool, v_pool [n_blocks][Hkv][128][d] bf16          (fspad_tree_attn_paged: one layer's K and V pools)
 *   pool   [n_layers][2][n_blocks][Hkv][128][d] bf16     (fspad_kv_compact_paged: all layers, updated in place)
 *   block_table [batch][blocks_per_seq] int32, entries in [0, n_blocks); the blocks of the rows a call touches
 *               (rows 0 .. L_b + n_nodes - 1) must be distinct within a sequence and not shared between sequences
 * Everything else - the other arguments, the results, the error reporting - is as in fspad_tree_attn and
 * fspad_kv_compact with max_len = 128 * blocks_per_seq; a table entry out of range is reported as
 * FSPAD_ERR_RANGE (device-checked, accesses stay inside the pool).  FSPAD_ERR_TOO_LARGE: more than 128
 * blocks would fall to one CTA (blocks_per_seq above 128 times the number of key ranges the call uses).
 * Trees of up to 256 nodes, as in the contiguous calls.
 */
int fspad_tree_attn_paged(fspad_ctx *ctx, const fspad_bf16 *q, const fspad_bf16 *k_pool, const fspad_bf16 *v_pool,
                          const int32_t *block_table, int blocks_per_seq, int n_blocks, const fspad_bf16 *tree_k,
                          const fspad_bf16 *tree_v, const int32_t *parent, const int32_t *prefix_len, int n_nodes,
                          int batch, fspad_bf16 *out, void *stream);
int fspad_kv_compact_paged(fspad_ctx *ctx, fspad_bf16 *pool, const int32_t *block_table, int blocks_per_seq, int n_blocks,
                           const int32_t *accepted_path, const int32_t *n_accepted, const int32_t *prefix_len, int batch,
                           int32_t *new_len, void *stream);

/*
 * One whole verify step on DEVICE buffers ("Preliminaries": the target's single
 * forward over the flattened tree, the strict comparison of its results with the
 * tree, and the removal of the rejected tokens are one step of the decoding
 * loop).  Equivalent to fspad_tree_attn (over the K and V planes of layer
 * `attn_layer` of `cache`), fspad_tree_accept and fspad_kv_compact queued one
 * after the other on `stream`, with the same arguments, outputs and errors, but
 * the attention runs on a second stream owned by the context, forked from and
 * joined back into `stream` with events: attention and acceptance share no
 * data, so their kernels overlap on the device.  Compaction follows the
 * acceptance directly when tree_k / tree_v are given (attention then never
 * reads the cache rows compaction rewrites); when they are NULL (tree rows
 * taken from cache rows L_b ..) compaction waits for the attention as well.
 * In the first case, when draft_probs is given and a sequence has at most 64
 * (layer, K/V, kv head) slices, the kernel that walks the tree makes the
 * compaction's moves itself (same result; an invalid prefix length is then
 * reported by that kernel).
 * Work queued on `stream` after the call sees every output.  The call only
 * enqueues work and records / waits on events, so it may be captured into a
 * CUDA graph.  One call per context at a time.
 *
 *   cache  [n_layers][2][batch][Hkv][max_len][d] bf16, updated in place by the compaction
 *   attn_layer  0 .. n_layers-1
 *   every other argument as in the three calls it replaces
 */
int fspad_verify_step(fspad_ctx *ctx, fspad_bf16 *cache, int attn_layer, const fspad_bf16 *q,
                      const fspad_bf16 *tree_k, const fspad_bf16 *tree_v, const int32_t *parent,
                      const int32_t *prefix_len, const float *target_logits, const float *draft_probs,
                      const int32_t *draft_tokens, const float *temperature, const float *uniforms,
                      int n_nodes, int batch, fspad_bf16 *attn_out, int32_t *accepted_path,
                      int32_t *n_accepted, int32_t *bonus_token, int32_t *new_len, void *stream);

/*
 * One whole verify step from HOST buffers: copies the step's inputs to device
 * staging owned by the context (allocated by the first call, which therefore
 * must not be made inside a stream capture), writes the tree rows into cache
 * rows L_b.. of layer 0, runs fspad_verify_step (attention over layer 0) on
 * `stream`, copies the results back and synchronises the stream.  The KV cache
 * is device-resident state that persists between steps (the caller's device
 * pointer `cache`, layout as in fspad_kv_compact); everything else is host
 * memory (pinned memory makes the copies asynchronous).  Host outputs:
 * attn_out [batch][n_nodes][Hq][d] bf16, accepted_path [batch][max_nodes],
 * n_accepted, bonus_token, new_len [batch].  draft_probs/uniforms may be NULL
 * when every temperature is 0.  Returns the first host- or device-detected error.
 */
int fspad_verify_step_host(fspad_ctx *ctx, fspad_bf16 *cache /* device */,
                           const fspad_bf16 *q, const fspad_bf16 *tree_k, const fspad_bf16 *tree_v,
                           const int32_t *parent, const int32_t *prefix_len,
                           const float *target_logits, const float *draft_probs,
                           const int32_t *draft_tokens, const float *temperature,
                           const float *uniforms, int n_nodes, int batch, fspad_bf16 *attn_out,
                           int32_t *accepted_path, int32_t *n_accepted, int32_t *bonus_token,
                           int32_t *new_len, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* FSPAD_H */
