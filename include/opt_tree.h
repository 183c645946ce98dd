/*
 * opt_tree.h — C ABI of the B200 (sm_100a) OPT-Tree draft-tree library.
 *
 * One decoding step of speculative decoding with an adaptive draft tree (Algorithm 2 of
 * the OPT-Tree paper) is: construct the tree (Algorithm 1), compute its tree attention
 * mask, run the target model on it, verify.  This library implements everything in that
 * step except the two model forwards, which are replaced by bf16 logit tables:
 *
 *   draft "model"  L_d [H][V] bf16, target "model" L_t [H][V] bf16, row-major; the next-token
 *   logits of a node holding token t at depth d (root: d = 0) are row (t*31 + d) mod H.
 *
 * Conventions
 *   - Every pointer marked (dev) is device memory on the context's device, owned by the
 *     caller; (host) is host memory.  build / mask / verify / row_softmax_topk only enqueue
 *     work on `stream` (a cudaStream_t passed as void*, NULL = default stream); they never
 *     allocate, free or synchronise.
 *   - Return value: OPT_TREE_OK (0) or a negative opt_tree_status.  Nothing throws, aborts
 *     or traps.  Errors detected on the device (a bounded wait that expired, an index that
 *     failed its bounds check) are recorded in a device status word, read back with
 *     opt_tree_last_device_status().
 *   - Logits must be finite or -inf (no NaN, no +inf); a row must hold at least one finite
 *     value.  Behaviour on other inputs is unspecified but never faults.
 *   - The root is not a node of the output, is not counted in n and has no mask bit
 *     (Section 3, definition of E_sub: the root is left out of the node count).
 */
#ifndef OPT_TREE_H_
#define OPT_TREE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    OPT_TREE_OK = 0,
    OPT_TREE_ERR_INVALID_ARG = -1,   /* null pointer, non-positive size, B > max_batch ... */
    OPT_TREE_ERR_UNSUPPORTED = -2,   /* n > 1024, k > 32, k > V, more than 510 layers ... */
    OPT_TREE_ERR_CUDA = -3,          /* a CUDA runtime call failed */
    OPT_TREE_ERR_TIMEOUT = -4,       /* a bounded device-side wait expired */
    OPT_TREE_ERR_INTERNAL = -5       /* a device-side bounds check failed */
} opt_tree_status;

#define OPT_TREE_MAX_N 1024
#define OPT_TREE_MAX_K 32

typedef struct opt_tree_ctx opt_tree_ctx;   /* opaque; owns only its workspace */

/* Problem sizes fixed for the lifetime of a context.
 *   V          vocabulary size (columns of the tables), V >= 1
 *   H          rows of the tables, H >= 1
 *   n          node budget of the tree (Algorithm 1 input n), 1 <= n <= OPT_TREE_MAX_N
 *   k          at most k children per node (the k most probable next tokens), 1 <= k <= OPT_TREE_MAX_K
 *   max_depth  cap on the number of drafted layers; Algorithm 1 also caps the depth by n;
 *              min(max_depth, n) <= 510
 *   max_batch  largest B any call will pass */
typedef struct {
    int32_t V, H, n, k, max_depth, max_batch;
} opt_tree_config;

/* One batch of built trees, structure of arrays (all dev).  Nodes of a tree are packed in
 * the order (depth ascending, parent's packed index ascending, sibling rank ascending), so a
 * parent always precedes its children.  Unused tail slots i >= n_sel hold token -1,
 * parent -1, depth 0, phat 0. */
typedef struct {
    int32_t *token;          /* [B][n]  token id of node i */
    int32_t *parent;         /* [B][n]  packed index of the parent, -1 = child of the root */
    int32_t *depth;          /* [B][n]  1-based depth */
    double  *phat;           /* [B][n]  path value, Eq. 2: product of draft probabilities along the path */
    int32_t *n_sel;          /* [B]     nodes kept, min(n, nodes drafted) */
    int32_t *depth_reached;  /* [B]     layers drafted before the loop of Algorithm 1 stopped */
    double  *expected_len;   /* [B]     E(A), Eq. 3: sum of the kept path values */
    double  *esub_trace;     /* [B][max_depth] or NULL: E_sub(T, n) after each drafted layer, 0 beyond */
} opt_tree_out;

/* Workspace bytes a context allocates for cfg (0 if cfg is invalid). */
size_t opt_tree_workspace_bytes(const opt_tree_config *cfg);

/* Creates a context on the current CUDA device and allocates its workspace once
 * (cudaMalloc).  *ctx is set to NULL on failure. */
int opt_tree_create(opt_tree_ctx **ctx, const opt_tree_config *cfg);
int opt_tree_destroy(opt_tree_ctx *ctx);

/* Algorithm 1 (construction of an OPT-Tree) for B independent sequences.
 *   draft_logits_bf16 (dev) [H][V]   16-byte aligned base
 *   root_token        (dev) [B]      last token x_l of each input sequence, 0 <= token < V
 *   delta                            threshold of the loop test (E_sub(T,n) - E > delta); pass
 *                                    -INFINITY to draft min(max_depth, n) layers unconditionally
 *   out                              filled as described at opt_tree_out
 * Per layer, every node of the last layer is expanded (fused row softmax + top-k over V), the
 * candidates' path values are parent value x child probability (Eq. 2), the next layer is the n
 * candidates of largest path value (ties: lower candidate index), E_sub(T,n) is the sum of the n
 * largest path values drafted so far, and the final tree is those n nodes (last line of
 * Algorithm 1).  The layer whose gain did not exceed delta stays in T. */
int opt_tree_build(opt_tree_ctx *ctx, const void *draft_logits_bf16, const int32_t *root_token,
                   int32_t B, float delta, const opt_tree_out *out, void *stream);

/* Tree attention mask and position ids (Algorithm 2, second line; Figure 1 caption: nodes of
 * one layer share a position index).
 *   tree          a batch written by opt_tree_build (parent, depth, n_sel are read)
 *   base_pos      (dev) [B] or NULL (= 0): position of the root token
 *   mask          (dev) [B][n][W], W = ceil(n/64): bit (j % 64) of word j/64 of row i is set iff
 *                 node j is node i or an ancestor of node i; rows i >= n_sel are zero.  The root
 *                 and the prefix are visible to every node and are not stored.
 *   position_ids  (dev) [B][n]: base_pos + depth for kept nodes, 0 for unused slots */
int opt_tree_mask(opt_tree_ctx *ctx, const opt_tree_out *tree, int32_t B, const int32_t *base_pos,
                  uint64_t *mask, int32_t *position_ids, void *stream);

/* Greedy verification (Preliminaries, greedy sampling; Algorithm 2, Verify): the target's
 * most probable token after the root and after every kept node (ties: lowest token id), then
 * the longest root branch that follows those tokens, plus the token after the last hit.
 *   target_logits_bf16 (dev) [H][V]
 *   accept_len    (dev) [B]               A = matched nodes + 1  (1 <= A <= depth_reached + 1)
 *   accept_tokens (dev) [B][max_depth+1]  the A accepted tokens, then -1
 *   accept_nodes  (dev) [B][max_depth]    packed indices of the A-1 matched nodes, then -1
 *   next_root     (dev) [B]               last accepted token = root of the next step */
int opt_tree_verify(opt_tree_ctx *ctx, const opt_tree_out *tree, const void *target_logits_bf16,
                    const int32_t *root_token, int32_t B, int32_t *accept_len, int32_t *accept_tokens,
                    int32_t *accept_nodes, int32_t *next_root, void *stream);

/* Greedy verification for callers that must not allocate (the paper has no counterpart; this is a
 * packaging variant of opt_tree_verify, same kernel, same results).
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a serving engine that owns
 * the whole device heap through its own pool and forbids driver allocations after start-up, or in a
 * latency-critical loop where an allocation's implicit device synchronisation is unacceptable.  Such
 * a caller cannot make an opt_tree_ctx (opt_tree_create allocates the workspace), so this entry
 * point takes the problem sizes directly and keeps the kernel's scratch (the target's best token
 * per node, one arrival counter per sequence, a status word) in a fixed array that is part of the
 * library image: about 65 KB on every GPU that loads the library, held until the process exits.
 *
 * Limits: B <= OPT_TREE_STATIC_MAX_BATCH and cfg->n <= OPT_TREE_STATIC_MAX_N, otherwise
 * OPT_TREE_ERR_UNSUPPORTED and nothing is launched.  cfg->max_batch is ignored.
 * It calls no cudaMalloc / cudaFree and no allocating library routine; it enqueues one small
 * memset, the kernel and (if device_status is given) one 4-byte device-to-device copy on `stream`.
 * The first call on each device asks the runtime for the array's device address (with that device
 * current); make that first call outside any stream capture.
 * Every call on a device shares the one array: two calls whose kernels may overlap on the GPU
 * (different streams, no dependency between them) race on it -- order them.  The array keeps what
 * the last call wrote; each call clears the counters and the status word before its kernel.
 *   tree, target_logits_bf16, root_token, accept_*, next_root: as for opt_tree_verify
 *   device_status (dev) [1] or NULL: receives OPT_TREE_OK or the first device-side error of this call */
#define OPT_TREE_STATIC_MAX_BATCH 64
#define OPT_TREE_STATIC_MAX_N 256
int opt_tree_verify_static(const opt_tree_config *cfg, const opt_tree_out *tree, const void *target_logits_bf16,
                           const int32_t *root_token, int32_t B, int32_t *accept_len, int32_t *accept_tokens,
                           int32_t *accept_nodes, int32_t *next_root, int32_t *device_status, void *stream);

/* The row step of Algorithm 1 on its own (children rule after Eq. 2): for each listed row,
 * the min(k, V) most probable tokens (logit descending, token id ascending) and their softmax
 * probabilities.
 *   logits_bf16 (dev) [H][V];  rows (dev) [nrows] row indices in [0, H)
 *   tok_out (dev) [nrows][k] int32, prob_out (dev) [nrows][k] double (entries >= min(k,V): -1 / 0) */
int opt_tree_row_softmax_topk(opt_tree_ctx *ctx, const void *logits_bf16, const int32_t *rows,
                              int32_t nrows, int32_t *tok_out, double *prob_out, void *stream);

/* opt_tree_build with frontier pruning: of every new layer only the nodes that are among the n
 * largest of T at that moment are drafted from (their rows of the draft table are the only ones
 * read).  By Theorem 1 a node's descendants have smaller path values than the node, so what is
 * left out can never reach the n largest: the outputs (tree, E(A), E_sub trace, depth_reached)
 * are those of opt_tree_build, for fewer rows.  Algorithm 1 as printed drafts from the whole last
 * layer; this variant is the one Section 3 has in mind when it notes that the input of a
 * drafting step is at most n tokens.
 *   rows_read (dev) [B] int32 or NULL: draft rows each sequence read (the root's included)
 * Arguments, ownership and errors otherwise as opt_tree_build. */
int opt_tree_build_pruned(opt_tree_ctx *ctx, const void *draft_logits_bf16, const int32_t *root_token,
                          int32_t B, float delta, const opt_tree_out *out, int32_t *rows_read, void *stream);

/* Layer-by-layer build, for a caller that runs a real draft model: Algorithm 1 with the draft step
 * (the next-token distributions of the last layer's nodes) left to the caller.
 * opt_tree_layers_begin starts B trees; every opt_tree_layers_step takes the logits of the nodes
 * that are to be expanded (first the root's, then each returned layer's), grows every tree by one
 * layer exactly as opt_tree_build does (row softmax + top-k, Eq. 2, the n best candidates, E_sub,
 * the loop test with `delta`) and returns the next layer; a tree whose growth stops is packed into
 * `out` in that call.  The trees are those of opt_tree_build for the same logits.
 *   frontier_logits (dev) bf16 [B][frontier_stride][V]: row f of sequence b belongs to node f of the
 *                   layer returned by the previous step (the root for the first step); rows at or
 *                   beyond a sequence's count are read but ignored.  1 <= frontier_stride <= n
 *   out             as in opt_tree_build; written for a sequence when it stops
 *   next_tokens     (dev) [B][n] int32  tokens of the new layer's nodes (to be expanded next)
 *   next_parent     (dev) [B][n] int32  for each, the index of its parent in the previous layer
 *   next_count      (dev) [B]   int32  nodes in the new layer; 0: this tree is finished
 * One context builds one batch of trees at a time this way (the state lives in its workspace).
 * Both calls only enqueue work on `stream`; errors as opt_tree_build. */
int opt_tree_layers_begin(opt_tree_ctx *ctx, int32_t B, void *stream);
int opt_tree_layers_step(opt_tree_ctx *ctx, const void *frontier_logits_bf16, int32_t frontier_stride, int32_t B,
                         float delta, const opt_tree_out *out, int32_t *next_tokens, int32_t *next_parent,
                         int32_t *next_count, void *stream);

/* Verification with sampling at temperature tau > 0.  The paper evaluates a temperature of 1 and says
 * only that the acceptable tokens change; this library's rule: at every position of the walk the next
 * token is drawn from the target's distribution softmax(x / tau) and accepted, and the walk goes on
 * while the current node has a child that carries the drawn token.  The emitted tokens are thus a
 * sample of the target model; outputs are those of opt_tree_verify.
 * Randomness is reproducible: one uniform per (sequence b, position j; 0 = root, i+1 = node i) from the
 * counter-based generator Philox4x32-10 (Salmon et al., 2011) with key = seed and counter =
 * (j, b, step low word, step high word), u = top 53 bits of the first two output words * 2^-53; the
 * draw is by inverse CDF in token order on e_v = exp((x_v - max x) / tau): the first token whose running
 * sum exceeds u * sum (the last token with e_v > 0 if rounding leaves none).  The row is read once: the
 * running sum is formed per segment of 512 logits in single precision (exponent arithmetic exact for
 * bf16 logits), and in double precision inside the segment where u * sum falls, so the token is that of
 * a double-precision inverse CDF unless u * sum lies within about 1e-6 * sum of a running sum.
 * `step` is the caller's decoding step number, so that successive steps use fresh uniforms.
 * Errors as opt_tree_verify; tau <= 0 or NaN is OPT_TREE_ERR_INVALID_ARG. */
int opt_tree_verify_sampled(opt_tree_ctx *ctx, const opt_tree_out *tree, const void *target_logits_bf16,
                            const int32_t *root_token, int32_t B, double tau, uint64_t seed, uint64_t step,
                            int32_t *accept_len, int32_t *accept_tokens, int32_t *accept_nodes,
                            int32_t *next_root, void *stream);

/* Bookkeeping after verification (Algorithm 2: the mask that M(T_opt, mask) consumes, in dense
 * form; Section 3, last paragraph: both models keep key and value caches, so after Verify only
 * the accepted tokens' entries stay).  The paper fixes neither format; this library's are:
 * the target sees n+1 tokens per step, position 0 the root (the last accepted token), position
 * i+1 packed node i.
 *   mask        (dev) [B][n][W]      bitmask written by opt_tree_mask
 *   accept_len, accept_nodes (dev)   as written by opt_tree_verify
 *   dense_mask  (dev) [B][n+1][n+1] uint8: 1 iff the row's token may attend to the column's token
 *               inside the step (itself; for a kept node also the root and its ancestors); unused
 *               positions attend to themselves only
 *   kv_gather   (dev) [B][max_depth+1] int32: step positions whose keys and values stay cached, in
 *               path order (0 = root, then 1 + accept_nodes[j]); -1 beyond kv_keep
 *   kv_keep     (dev) [B] int32: entries kept = accept_len (the last accepted token is the next
 *               step's root and has no entry yet)
 * Enqueues one kernel on `stream`; returns OPT_TREE_ERR_INVALID_ARG for null pointers or B out of
 * range.  Reads and writes only the caller's arrays and the context's status word. */
int opt_tree_post_verify(opt_tree_ctx *ctx, const opt_tree_out *tree, const uint64_t *mask,
                         const int32_t *accept_len, const int32_t *accept_nodes, int32_t B,
                         uint8_t *dense_mask, int32_t *kv_gather, int32_t *kv_keep, void *stream);

/* One whole decoding step (build, mask, verify) with HOST buffers: copies root_token and
 * base_pos to the device, runs the three stages, copies every output back and synchronises the
 * stream before returning.  The logit tables stay on the device (they stand in for the models).
 * The inputs and the outputs cross the bus in one copy each, through pinned staging memory the
 * context owns (so the caller's buffers need not be pinned); the staging is reused by every call,
 * hence one call at a time per context.  Any output pointer may be NULL to skip it; shapes are
 * those of opt_tree_out / opt_tree_mask / opt_tree_verify. */
typedef struct {
    int32_t *token, *parent, *depth; double *phat;                 /* (host) [B][n] */
    int32_t *n_sel, *depth_reached; double *expected_len;          /* (host) [B] */
    uint64_t *mask; int32_t *position_ids;                         /* (host) [B][n][W], [B][n] */
    int32_t *accept_len, *accept_tokens, *accept_nodes, *next_root;/* (host) [B], [B][D+1], [B][D], [B] */
} opt_tree_host_out;

int opt_tree_step_host(opt_tree_ctx *ctx, const void *draft_logits_bf16, const void *target_logits_bf16,
                       const int32_t *root_token_host, const int32_t *base_pos_host, int32_t B, float delta,
                       const opt_tree_host_out *out, void *stream);

/* Self-test of the library's bounded device-side waits (not a step of the paper's method; the
 * persistent build waits on mailboxes, counters and shared-memory barriers, each wait with a limit
 * after which it records OPT_TREE_ERR_TIMEOUT and returns instead of hanging).  Launches one small
 * kernel in which each kind of wait is entered on something nobody completes, with a limit of
 * about 2^16 clock cycles (or 2^10 polls): a shared-memory barrier awaited by a whole warp, one
 * awaited by a single thread, a candidate path-value word, a candidate token word, and the row
 * fetcher's mailbox poll loop.
 *   result (dev) [OPT_TREE_SELFTEST_WAITS] int32: one status word per wait, in that order; each must
 *                read OPT_TREE_ERR_TIMEOUT once the stream has been synchronised
 * The context's own status word is not touched.  Enqueues two small memsets and the kernel. */
#define OPT_TREE_SELFTEST_WAITS 5
int opt_tree_selftest_waits(opt_tree_ctx *ctx, int32_t *result, void *stream);

/* Reads (and clears) the device status word; synchronises the device.  *status_host is
 * OPT_TREE_OK or the first device-side error recorded since the last call. */
int opt_tree_last_device_status(opt_tree_ctx *ctx, int32_t *status_host);

/* Number of kernels the library has launched through this context since it was created. */
int64_t opt_tree_launch_count(const opt_tree_ctx *ctx);

const char *opt_tree_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* OPT_TREE_H_ */
