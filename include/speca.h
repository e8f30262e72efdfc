/*
 * speca.h -- C ABI of libspeca: speculative verification, greedy acceptance and
 * commit over the recurrent state of a gated-delta-rule (GDN) linear-attention
 * layer, plus the single-token decode step, as CUDA kernels for NVIDIA B200
 * (sm_100a).
 *
 * Notation.  L layers, B sequences, H heads, d_k key width, d_v value width,
 * T = node_offsets[B] draft nodes packed over the batch.  A "unit" is one
 * (layer, sequence, head); units never interact.
 *
 * The rule applied by every entry point (GDN layer, Section 2.2; Eq. 1 is its
 * un-gated, erase-free special case):
 *
 *        S' = S * alpha (I - beta k k^T) + beta v k^T          o = scale * S' q
 *
 * with S in R^{d_v x d_k}.  Equivalently  S' = alpha S + u k^T  with the
 * corrected value  u = beta (v - alpha S k).
 *
 * Layouts (row-major, last index contiguous), identical in every call:
 *      S, S0       float   [L][B][H][d_v][d_k]
 *      q, k        bf16    [L][T][H][d_k]      (16-bit storage, uint16_t here)
 *      v           bf16    [L][T][H][d_v]
 *      alpha, beta float   [L][T][H]
 *      o, u        float   [L][T][H][d_v]
 *      node_offsets int32  [B+1]   sequence b owns nodes node_offsets[b] .. node_offsets[b+1]-1
 *      parent, depth, draft_tok, target_tok   int32 [T]
 * For speca_decode_step there is exactly one token per sequence (T == B).
 *
 * Topology contract (parent-pointer array, Section 4.2 and Section 7).  parent[]
 * holds indices LOCAL to the sequence; -1 means "child of the committed state".
 * Nodes are in a topological order: parent[i] < i.  Several -1 nodes (a forest)
 * are legal.  depth[i] = 1 for children of the committed state, else
 * depth[parent[i]] + 1; it is optional (NULL) and only cross-checked.
 *
 * Memory and ownership.  Every pointer except `dims` is a CUDA DEVICE pointer
 * owned by the caller; `dims` is host memory read during the call only.  No
 * entry point allocates or frees device memory, synchronises, or keeps state
 * between calls.  All work is
 * enqueued on `stream` (a cudaStream_t passed as void*; NULL = default stream)
 * and the call returns immediately.  Every tensor base must be 16-byte aligned.
 * Outputs must not alias inputs; speca_decode_step and speca_commit update S in
 * place; the verify calls never write S0.
 *
 * Errors.  The return value is SPECA_OK or a negative SPECA_ERR_* for anything
 * the host can see (NULL pointer, unsupported shape, misalignment, bad size,
 * CUDA launch failure); nothing is launched in that case.  Faults that live in
 * device memory (bad parent pointer, offsets that decrease, a sequence larger
 * than dims.max_nodes or deeper than dims.max_depth, an accepted path that is
 * not a parent chain, a bounded wait that expired) make the kernels skip the
 * affected sequence -- its outputs and its state stay untouched (one exception: an expired wait inside the
 * one-pass speca_commit_verify_tree, see there) -- and OR a
 * SPECA_STATUS_* bit into *status_word, a device int32 the caller zeroes
 * beforehand and reads back when it wants to know.  No kernel traps.
 */
#ifndef SPECA_H
#define SPECA_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SPECA_VERSION 100

/* return codes */
#define SPECA_OK                0
#define SPECA_ERR_NULL         -1   /* a required pointer is NULL                        */
#define SPECA_ERR_UNSUPPORTED  -2   /* shape outside the supported set (see speca_dims)  */
#define SPECA_ERR_ALIGN        -3   /* a tensor base is not 16-byte aligned              */
#define SPECA_ERR_RANGE        -4   /* a count is negative or too large                  */
#define SPECA_ERR_CUDA         -5   /* the CUDA runtime reported an error at launch      */
#define SPECA_ERR_WORKSPACE    -6   /* workspace NULL or smaller than required           */
#define SPECA_ERR_TOO_LARGE    -7   /* problem exceeds the built-in scratch of a _noalloc entry point */

/* bits of *status_word */
#define SPECA_STATUS_BAD_PARENT   1   /* parent[i] < -1 or parent[i] >= i                          */
#define SPECA_STATUS_BAD_OFFSETS  2   /* node_offsets not non-decreasing / not ending at T         */
#define SPECA_STATUS_BAD_PATH     4   /* accepted path is not a chain of parent links from a root  */
#define SPECA_STATUS_TOO_DEEP     8   /* a node deeper than max_depth / path_len > max_depth       */
#define SPECA_STATUS_TOO_MANY    16   /* a sequence has more than dims.max_nodes nodes             */
#define SPECA_STATUS_TIMEOUT     32   /* a bounded device-side wait gave up                        */
#define SPECA_STATUS_BAD_DEPTH   64   /* depth[] given and inconsistent with parent[]              */

/* verification routes (dims.route) */
#define SPECA_ROUTE_AUTO        0   /* library picks                                              */
#define SPECA_ROUTE_SERIAL      1   /* state-resident walk, one rank-1 update per node (Section 4.1) */
#define SPECA_ROUTE_FACTORIZED  2   /* tree-masked factorised form on tensor cores (Section 4.2), fp32-grade */
#define SPECA_ROUTE_TF32        3   /* the same factorisation with the state read once as TF32 (single pass)  */
#define SPECA_ROUTE_EFFECTIVE   4   /* effective-query form of the factorisation, fp32-grade (trees up to 16 levels) */
/* SPECA_ROUTE_FACTORIZED takes d_v in {128, 256}, max_depth <= 16 and max_nodes <= 64 (d_k = 128) or <= 32
 * (d_k = 256).  Both tensor-core operands are split into a TF32 head and its exact remainder, so outputs
 * carry fp32 accuracy whatever the magnitude of the state.  AUTO uses it whenever it applies and the serial
 * route otherwise; asking for it explicitly outside these shapes is SPECA_ERR_UNSUPPORTED.
 * SPECA_ROUTE_TF32 is never picked by AUTO: it reads the fp32 state through a single TF32 pass (10 mantissa
 * bits, truncated), which leaves errors of about 2^-11 of the output's scale, growing with the state; it takes
 * max_depth <= 8 with max_nodes <= 64 (d_k = 128) or <= 32 (d_k = 256), or max_depth <= 16 with max_nodes <=
 * 32, and is the only route on which speca_commit_verify_tree runs as ONE pass over the state. */

/* recurrences (dims.rule; Section 5.1, remark on other layer types).  A DeltaNet layer (k, v, beta, no
 * decay) is the gated delta rule with alpha = 1 and needs no value of its own. */
#define SPECA_RULE_GATED_DELTA     0   /* S' = S alpha (I - beta k k^T) + beta v k^T   (GDN)                   */
#define SPECA_RULE_GATED_NO_ERASE  1   /* S' = alpha S + beta v k^T   (GLA-style: key, value, gate; no read-out) */

typedef struct speca_dims {
    int32_t n_layers;    /* L >= 1                                                     */
    int32_t batch;       /* B >= 1                                                     */
    int32_t heads;       /* H >= 1                                                     */
    int32_t d_k;         /* 64, 128 or 256                                             */
    int32_t d_v;         /* multiple of 32, <= 1024                                    */
    float   scale;       /* o = scale * S q  (1.0f reproduces the paper's minimal form) */
    int32_t max_depth;   /* longest root path in nodes, 1..16; width of path_idx rows  */
    int32_t max_nodes;   /* node budget per sequence (Section 6.1), 1..1024            */
    int32_t route;       /* SPECA_ROUTE_*                                              */
    int32_t rule;        /* SPECA_RULE_*: which recurrence the layer applies           */
} speca_dims;

int         speca_version(void);
const char *speca_strerror(int code);

/* Bytes of caller-provided device scratch the verify calls need for `total_nodes`
 * packed nodes (topology plan shared by all layers and heads).  Positive for valid arguments; 0 if dims is NULL,
 * dims->batch < 1 or total_nodes < 0. */
size_t speca_workspace_bytes(const speca_dims *dims, int32_t total_nodes);

/* Single-token decode step, the autoregressive baseline (Section 2.2: every step
 * reads the previous state and writes the updated one).  For every unit:
 * S <- rule(S; k, v, alpha, beta) in place, o = scale * S_new q.  T == B. */
int speca_decode_step(const speca_dims *dims, float *S,
                      const uint16_t *q, const uint16_t *k, const uint16_t *v,
                      const float *alpha, const float *beta, float *o, void *stream);

/* Chain verification (Section 4.1, state-resident serial verification; the
 * p_j = j-1 special case of Section 7).  Node j of a sequence sees the state after
 * nodes 0..j of that sequence were applied to S0.  Writes o for every node and,
 * if u_or_null != NULL, the corrected values u (a WY-style factor record that,
 * with k and alpha, rebuilds any node's state).  S0 is read once per unit. */
int speca_verify_chain(const speca_dims *dims, const float *S0,
                       const uint16_t *q, const uint16_t *k, const uint16_t *v,
                       const float *alpha, const float *beta,
                       const int32_t *node_offsets, int32_t total_nodes,
                       float *o, float *u_or_null,
                       void *workspace, size_t workspace_bytes,
                       int32_t *status_word, void *stream);

/* Tree verification (Sections 4.2-4.3).  Node t sees the state obtained by applying
 * the rule along its own ancestor path root..t starting from S0; siblings never
 * influence each other and shared prefixes are computed once.  Same outputs as
 * speca_verify_chain; `depth_or_null` is optional. */
int speca_verify_tree(const speca_dims *dims, const float *S0,
                      const uint16_t *q, const uint16_t *k, const uint16_t *v,
                      const float *alpha, const float *beta,
                      const int32_t *node_offsets, int32_t total_nodes,
                      const int32_t *parent, const int32_t *depth_or_null,
                      float *o, float *u_or_null,
                      void *workspace, size_t workspace_bytes,
                      int32_t *status_word, void *stream);

/* Greedy posterior selection (Section 2.1; all end-to-end runs of Section 8 decode
 * greedily).  With pred(-1) = root_target_tok[b] and pred(i) = target_tok[i], node t is
 * matched iff draft_tok[t] == pred(parent[t]) and its parent is matched.  Writes the
 * root path of the deepest matched node (lowest index on ties) to path_idx[b][0..len),
 * pads the row with -1, path_len[b] = len (0 if the first token already misses), and
 * next_tok[b] = pred(last accepted node).  Integer-exact. */
int speca_greedy_accept(int32_t batch, int32_t max_depth,
                        const int32_t *node_offsets, const int32_t *parent,
                        const int32_t *draft_tok, const int32_t *target_tok,
                        const int32_t *root_target_tok,
                        int32_t *path_idx, int32_t *path_len, int32_t *next_tok,
                        int32_t *status_word, void *stream);

/* Stochastic posterior selection (the rejection-sampling-style rule of Section 2.1), for callers that
 * sample instead of decoding greedily.  p_target, p_draft, uniform: float [T], device, packed like the
 * nodes.  p_draft[t] is the probability the drafter gave node t's token, p_target[t] the probability the
 * target gives it at t's parent -- for a node with lower-index siblings: in the residual distribution
 * that remains once those siblings have been rejected, which the caller computes from its logits --
 * and uniform[t] a number in [0, 1) drawn by the caller.  Node t passes iff
 * uniform[t] * p_draft[t] < p_target[t] (fp32 product, then comparison; i.e. uniform < min(1, p/q)).
 * Starting at the committed state the walk moves to the first child, in ascending index, that passes,
 * and stops when none does; the nodes visited are written to path_idx[b][0..len) (rest -1) and
 * path_len[b] = len.  For a chain this is the acceptance rule of speculative sampling verbatim.  The
 * token that follows the accepted path (drawn from the residual at the stopping node, or from the
 * target distribution if a leaf was reached) needs vocabulary-sized distributions and stays with the
 * caller.  Integer-exact given the three arrays; bad topology is reported and accepts nothing. */
int speca_stochastic_accept(int32_t batch, int32_t max_depth,
                            const int32_t *node_offsets, const int32_t *parent,
                            const float *p_target, const float *p_draft, const float *uniform,
                            int32_t *path_idx, int32_t *path_len,
                            int32_t *status_word, void *stream);

/* Commit (Section 5.1 factor buffering, Eq. 3; Section 5.2 immediate update): gathers
 * the factor records (k, v, alpha, beta) on the accepted path path_idx[b][0..path_len[b])
 * and advances S over them in place, in fp32.  path_len[b] == 0 leaves
 * the sequence's state bitwise untouched (it is neither read nor written).  If
 * parent_or_null is given the path is checked to be a chain of parent links starting at
 * a child of the committed state; an invalid path skips the sequence.
 * The state is advanced token by token; in large batches (d_k <= 128) paths of four to
 * eight nodes are advanced in the unrolled form of Section 4.2 instead (one product of the
 * state tile with all keys of the path, the recurrence per row, one rank-A update, on
 * tensor cores with every fp32 operand split into a TF32 head and its exact remainder).
 * Both forms carry fp32 accuracy; they differ in rounding order, so the state of a
 * sequence is reproducible for a given batch shape, not across batch shapes.  The call
 * launches one or two kernels on `stream`. */
int speca_commit(const speca_dims *dims, float *S,
                 const uint16_t *k, const uint16_t *v,
                 const float *alpha, const float *beta,
                 const int32_t *node_offsets, int32_t total_nodes,
                 const int32_t *parent_or_null,
                 const int32_t *path_idx, const int32_t *path_len,
                 int32_t *status_word, void *stream);

/* Fused commit-and-verify: the delayed state update of Section 5.2 ("update fused into
 * the next verification", Eq. 3 applied while the state tile is on chip).  Equivalent to
 *     speca_commit(S, previous draft's records, path_idx, path_len)   followed by
 *     speca_verify_tree(S, new draft)
 * but the state crosses HBM twice (one read, one write) instead of three times.
 *
 * Pending commit: k_prev, v_prev, alpha_prev, beta_prev are the previous draft's records
 * (layouts as in speca_verify_tree, packed by node_offsets_prev, total_nodes_prev nodes),
 * path_idx / path_len its accepted paths as written by speca_greedy_accept, and
 * u_prev_or_null the `u` the previous verification wrote for that draft ([L,Tp,H,d_v]).
 * Each path must be a root path of the previous draft's tree (a node's u embeds its
 * ancestors, so u of nodes that do not form such a path cannot be combined); pass
 * parent_prev_or_null to have that checked.  A
 * sequence with an invalid path gets STATUS_BAD_PATH / TOO_DEEP, its state is not
 * advanced, and its new draft is verified from the state as it stands (exactly what the
 * two separate calls do).  A sequence whose new tree is empty or rejected still gets its
 * commit.  total_nodes_prev == 0 means nothing is pending (plain verification, S is not
 * written); total_nodes == 0 means nothing to verify (plain commit).
 *
 * New draft and outputs: as speca_verify_tree, except that S is read and written.  Pass
 * u_or_null to be able to fuse the next round; it must not be the buffer u_prev_or_null
 * points to, and o / u must not alias any input.
 *
 * One pass or two.  With dims.route = SPECA_ROUTE_TF32, a shape that route takes with max_depth <= 8 (d_v in
 * {128, 256}; d_k = 128 with max_nodes <= 64 or d_k = 256 with max_nodes <= 32) and u_prev_or_null given, ONE
 * kernel does both: the pending update is then S <- gamma_A S + sum_i (gamma_A / gamma_i) u_i k_i^T, which needs
 * only u, k and alpha of the accepted nodes (v_prev and beta_prev are not read); outputs and the committed state
 * carry the accuracy of that route (2e-3-grade, not fp32-grade).  On every other route -- AUTO included -- the
 * commit and verify kernels are launched back to back on `stream`: same results at fp32 accuracy, the state
 * crossing HBM three times.  workspace_bytes must be at least speca_workspace_bytes().
 * After SPECA_STATUS_TIMEOUT from the one-pass kernel the state of the affected units is undefined (slices
 * already sent back have been advanced, the others not): reload it from the caller's copy. */
int speca_commit_verify_tree(const speca_dims *dims, float *S,
                             const uint16_t *k_prev, const uint16_t *v_prev,
                             const float *alpha_prev, const float *beta_prev,
                             const float *u_prev_or_null,
                             const int32_t *node_offsets_prev, int32_t total_nodes_prev,
                             const int32_t *parent_prev_or_null,
                             const int32_t *path_idx, const int32_t *path_len,
                             const uint16_t *q, const uint16_t *k, const uint16_t *v,
                             const float *alpha, const float *beta,
                             const int32_t *node_offsets, int32_t total_nodes,
                             const int32_t *parent, const int32_t *depth_or_null,
                             float *o, float *u_or_null,
                             void *workspace, size_t workspace_bytes,
                             int32_t *status_word, void *stream);

/* Draft-side utilities (integer work in front of the verification; Sections 6.1 and 7).
 *
 * speca_tree_mask_to_parent: the proposal converter.  mask uint8 [B][max_nodes][max_nodes]; for sequence b
 * with n = node_offsets[b+1] - node_offsets[b] nodes, mask[b][i][j] != 0 (i, j < n) iff node j is node i
 * or one of its ancestors (a drafter's tree attention mask).  Writes parent[node_offsets[b] + i] = the
 * deepest strict ancestor of i (local index), -1 if it has none.  A mask that is not the mask of a tree in
 * topological order sets STATUS_BAD_PARENT and leaves the sequence's parents untouched.
 *
 * speca_prune_tree: confidence-guided pruning.  logp float [T] are the drafter's step log-probabilities;
 * q(v) is their sum over the root path of v (fp32, root first), q* its maximum over the sequence.  Kept are
 * the nodes with q(v) >= q* - tau, of those the `budget` best by q (ties: lower index), and of those only
 * nodes whose parent is kept -- with log-probabilities (<= 0) q never increases along a path and the last
 * rule changes nothing.  The kept nodes of all sequences are written packed, in their original order:
 * out_offsets [B+1], out_parent [.] (re-indexed, local), out_index [.] (original local index); out_parent
 * and out_index need room for T entries.  A sequence with bad topology is reported and contributes nothing.
 *
 * speca_chain_decompose: the heavy-light chain decomposition of Section 4.3 (the scheduling unit of the
 * paper's hybrid route: node-disjoint chains that together cover the tree, each verifiable as a chain from
 * the boundary state of the node it hangs off).  The heavy child of a node is its child with the largest
 * subtree (lowest index on ties); a node continues its parent's chain iff it is that heavy child, every
 * other node -- and every child of the committed state -- heads a chain.  Writes chain_head[node_offsets[b]
 * + i] = local index of the first node of i's chain and n_chains[b] = the number of chains.  On any root
 * path at most floor(log2(n)) chains are entered below the first.  A sequence with bad topology is
 * reported, gets n_chains[b] = 0 and its chain_head entries are left untouched.  No kernel of this library
 * consumes the result: its own tree routes keep branch states on chip (the serial walk only borrows the
 * heavy-path order), so the decomposition is a utility for callers that schedule chains themselves. */
int speca_tree_mask_to_parent(int32_t batch, int32_t max_nodes, const uint8_t *mask,
                              const int32_t *node_offsets, int32_t *parent,
                              int32_t *status_word, void *stream);
int speca_chain_decompose(int32_t batch, int32_t max_nodes,
                          const int32_t *node_offsets, const int32_t *parent,
                          int32_t *chain_head, int32_t *n_chains,
                          int32_t *status_word, void *stream);
int speca_prune_tree(int32_t batch, int32_t max_nodes, float tau, int32_t budget,
                     const int32_t *node_offsets, const int32_t *parent, const float *logp,
                     int32_t *out_offsets, int32_t *out_parent, int32_t *out_index,
                     int32_t *status_word, void *stream);

/* Commit of the convolution state (Section 7: the state holder keeps (S, C); Section 8.4 checks that C
 * is reproduced exactly).  The GDN layer is preceded by a causal depthwise convolution whose state is the
 * last W = kernel_size - 1 inputs of every channel:
 *      C   bf16 [L][B][W][channels]   oldest input first, updated in place
 *      x   bf16 [L][T][channels]      inputs of the draft nodes (same packing as q, k, v)
 * For every sequence the inputs of the accepted nodes path_idx[b][0..path_len[b]) are shifted into the
 * register in path order: C becomes the last W rows of (old C rows, then the accepted rows).  16-bit
 * patterns are copied, so the result is exact.  path_len[b] == 0 leaves the sequence's C untouched; a path
 * with an index outside the sequence or longer than max_depth sets STATUS_BAD_PATH / TOO_DEEP and skips it.
 * channels must be a multiple of 8, 1 <= W <= 8; C and x 16-byte aligned. */
int speca_commit_conv(int32_t n_layers, int32_t batch, int32_t channels, int32_t width, int32_t max_depth,
                      uint16_t *C, const uint16_t *x,
                      const int32_t *node_offsets, int32_t total_nodes,
                      const int32_t *path_idx, const int32_t *path_len,
                      int32_t *status_word, void *stream);

/* ---------------------------------------------------------------------------
 * Variant of speca_verify_tree for callers that cannot provide scratch memory.
 * (The paper has no counterpart: this is a property of the library, not of the method.)
 *
 * Who needs it: code that runs where device allocation is off limits -- a serving loop
 * whose memory pool is frozen after start-up, a plug-in that is handed tensors but no
 * allocator, a latency-critical path where cudaMalloc (which synchronises the device)
 * would stall every other stream.  Such a caller still owns the inputs and outputs, but
 * has nowhere to take the verify workspace from.
 *
 * This entry point is speca_verify_tree with the workspace argument removed: the scratch
 * (topology plan shared by all layers and heads) lives in a fixed array inside the library
 * image, SPECA_NOALLOC_SCRATCH_BYTES per GPU that loads the library, held until the process
 * exits.  It neither allocates nor frees device memory and calls nothing that does.
 *
 * Limits: dims->batch <= SPECA_NOALLOC_MAX_BATCH and total_nodes <= SPECA_NOALLOC_MAX_NODES,
 * otherwise SPECA_ERR_TOO_LARGE and nothing is launched.
 *
 * The first call on each device looks up the device address of the array.  That query makes
 * no allocation of its own, but with lazy module loading it can be the moment the CUDA runtime
 * loads this library's device code onto that GPU (which is when the array comes to exist there):
 * make that first call once per device during start-up, outside any stream capture and outside
 * the latency-critical path.  The lookup may be raced by several host threads.  Every call on
 * a device uses the same array and finds in it whatever the previous call left; the
 * kernels rewrite all of it they read, so nothing needs clearing by the caller -- but two
 * calls whose kernels overlap on the GPU (different streams, no ordering between them)
 * race on the array and must be serialised by the caller.
 */
#define SPECA_NOALLOC_MAX_BATCH   256
#define SPECA_NOALLOC_MAX_NODES   16384
#define SPECA_NOALLOC_SCRATCH_BYTES (2048 + 1024 + 16 * 65536 + 12288)

int speca_verify_tree_noalloc(const speca_dims *dims, const float *S0,
                              const uint16_t *q, const uint16_t *k, const uint16_t *v,
                              const float *alpha, const float *beta,
                              const int32_t *node_offsets, int32_t total_nodes,
                              const int32_t *parent, const int32_t *depth_or_null,
                              float *o, float *u_or_null,
                              int32_t *status_word, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* SPECA_H */
