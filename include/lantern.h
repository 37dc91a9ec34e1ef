/*
 * lantern.h -- C ABI of the relaxed tree-verification hot path (LANTERN++).
 *
 * Notation follows the paper (Sec. 2 "Notations"): p is the DRAFTER
 * distribution, q is the TARGET distribution; a draft token x is accepted with
 * probability min(1, sum_{a in A(x)} q(a) / p(x)).
 *
 * Conventions for every entry point
 *  - Pointers are DEVICE pointers owned by the caller unless marked "host".
 *  - Work is enqueued on `stream` (a cudaStream_t passed as void*; NULL is the
 *    default stream).  Nothing synchronises; outputs are valid once the stream
 *    has reached the end of the call.  Outputs are fully overwritten.
 *  - Errors come back as a lantern_status.  Invalid arguments are detected on the
 *    host before anything is launched.  Problems that only the device can see
 *    (a table index out of range, a copy that did not complete in time) are
 *    OR-ed into *device_status as LANTERN_DEV_* bits; the kernels never trap.
 *  - Same inputs and same uniforms / seed give the same bytes.
 *  - Only lantern_tree_create and lantern_forest_create allocate (a few hundred bytes per tree).
 *  - Entry points may be called from several host threads at once as long as the calls do not
 *    share output buffers or a workspace; lantern_set_cluster_size is the exception (see there).
 *  - The neighbour table must not list a token among its own neighbours and a row's entries
 *    must be distinct (lantern_build_neighbors guarantees both).
 */
#ifndef LANTERN_H_
#define LANTERN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  LANTERN_OK = 0,
  LANTERN_ERR_INVALID_ARG = 1,  /* NULL required pointer, bad range, misaligned rows, bad tree  */
  LANTERN_ERR_UNSUPPORTED = 2,  /* size beyond what the kernels are built for                   */
  LANTERN_ERR_WORKSPACE = 3,    /* workspace missing or smaller than *_workspace() reports      */
  LANTERN_ERR_CUDA = 4          /* a CUDA runtime call failed (launch, copy, allocation)        */
} lantern_status;

typedef enum { LANTERN_F32 = 0, LANTERN_BF16 = 1 } lantern_dtype;

/* bits of *device_status */
enum {
  LANTERN_DEV_BAD_INDEX = 1,    /* a token or neighbour index fell outside the vocabulary; it was
                                   treated as probability 0                                     */
  LANTERN_DEV_TIMEOUT = 2,      /* a bounded on-chip wait expired; the data was re-read with
                                   plain loads and the CTA made no further asynchronous copies.
                                   Never observed; treat the call's results as suspect          */
  LANTERN_DEV_EMPTY_ROW = 4,    /* a row had no finite logit                                    */
  LANTERN_DEV_KEY_TIES = 8      /* draft sampling: more Gumbel keys than the kernel ranks exactly
                                   lay within 2.5e-4 of the last child's key; the children are
                                   distinct draws, their order may differ from an exact ranking */
};

const char* lantern_status_string(lantern_status s);

/* ---- static draft tree (Sec. 2.1 "Tree Drafting and Verification") -------------------------
 * Node 0 stands for the last committed token; every other node carries one draft token.
 * Nodes are numbered breadth first: parent[0] = -1, 0 <= parent[i] < i, parent[] non-decreasing,
 * so the children of a node are contiguous and stored in the order they were drawn (rank order).
 * At most LANTERN_MAX_CHILDREN children per node, at most LANTERN_MAX_NODES nodes.
 * `parent` is a HOST array; it is copied, the caller keeps ownership. */
#define LANTERN_MAX_CHILDREN 8
#define LANTERN_MAX_NODES 1024
typedef struct lantern_tree lantern_tree;
lantern_status lantern_tree_create(const int32_t* parent /* host [n_nodes] */, int32_t n_nodes,
                                   lantern_tree** out);
lantern_status lantern_tree_destroy(lantern_tree* tree);
int32_t lantern_tree_max_depth(const lantern_tree* tree);  /* depth of the deepest node */
/* A forest: one tree per sequence (Sec. 2.1, dynamic tree drafting: the shape of the draft tree
 * depends on the sequence), each numbered as above and padded to max_nodes.  parent is a HOST
 * array [batch][max_nodes] of which row b uses its first n_nodes[b] entries (host [batch]).  The
 * handle is used like a tree with max_nodes nodes by lantern_verify_tree (and _static) for exactly
 * `batch` sequences: per-node arrays are [batch][max_nodes], entries of padding nodes are ignored
 * on input and -1 on output.  Served by the streaming kernels' eager launch only: rows that a
 * top-k truncates, lazy_walk = 1 and kernels = 2 return LANTERN_ERR_UNSUPPORTED, and so does
 * lantern_sample_draft_tree (such trees are drafted deterministically; verify them with
 * draft_deterministic = 1).  Destroyed with lantern_tree_destroy.                               */
lantern_status lantern_forest_create(const int32_t* parent /* host */, const int32_t* n_nodes /* host */,
                                     int32_t batch, int32_t max_nodes, lantern_tree** out);

/* ---- parameters (App. B "Models": guidance, temperature, top-k; Sec. 4: k, lambda) ---------
 * Row post-processing, identical for target rows (-> q) and drafter rows (-> p):
 *   z_j = fma(cfg_scale, cond_j - uncond_j, uncond_j) * (1/temperature)      (float32 ops)
 *   z_j = cond_j * (1/temperature)                         when the uncond pointer is NULL
 *   tokens outside [allowed_begin, allowed_end) get -inf
 *   top_k > 0: every z_j below the top_k-th largest value becomes -inf (ties at it are kept)
 *   distribution = softmax(z)                                                                  */
typedef struct {
  float cfg_scale;
  float temperature;       /* > 0 */
  int32_t top_k_target;    /* 0 = off */
  int32_t top_k_draft;     /* 0 = off */
  float lambda;            /* multiplicative bound of Sec. 4, >= 1; 1 = no relaxation */
  int32_t k;               /* neighbours considered per draft token, 0..k_table; 0 = standard
                              speculative sampling                                              */
  int32_t vocab;           /* V, logits per row */
  int32_t code_offset;     /* token t has latent code t - code_offset ...                       */
  int32_t n_codes;         /* ... iff 0 <= t - code_offset < n_codes (the table's row count L)  */
  int32_t allowed_begin;   /* tokens outside [allowed_begin, allowed_end) are masked            */
  int32_t allowed_end;     /* 0 means V                                                         */
  uint64_t seed;           /* Philox-4x32-10 key; used only where uniforms are not supplied     */
  uint64_t step;           /* counter base, < 2^62: change it every decode step                 */
  float delta;             /* 0: multiplicative bound lambda (Sec. 4).  > 0: additive bound of
                              Sec. 2.2 instead (lambda unused): neighbours join A while their own
                              running sum of q stays < delta, i.e. TVD(q, q~) < delta            */
  int32_t lazy_walk;       /* lantern_verify_tree only.  0: every node of the tree is verified
                              (one launch over B*N nodes), then the walk.  1: path walk (Sec. 2.1):
                              one thread-block cluster per sequence verifies the root, moves to
                              the accepted child and so on, reading only the rows on the accepted
                              path; accept_len / out_tokens / out_nodes are the same, the per-node
                              outputs are written for the nodes on the path only                */
  int32_t subset_rule;     /* which subset of the neighbour list forms A (Sec. 4 states only the
                              inequality).  0: the longest prefix of the distance-ordered list that
                              keeps the bound.  1: greedy skip: a neighbour that would break the
                              bound is passed over and the search goes on down the list           */
  int32_t draft_deterministic; /* lantern_verify_tree only.  1: the draft tokens were chosen
                              deterministically (Sec. 3: what dynamic-tree drafting does), i.e.
                              p(x) = 1 for each of them: a child is accepted with probability
                              min(1, m), the residual after a rejection is q~ without x, and the
                              drafter rows are never read (draft_* may be NULL)                   */
  int32_t kernels;         /* 0: the library chooses between its kernels by size (see "which kernels a
                              call launches").  1: streaming kernels wherever they apply, whatever
                              the size.  2: never the streaming kernels.  Results are the same     */
} lantern_params;
/* subset_rule = 1 and draft_deterministic = 1 are served by the streaming kernels only: rows that a
 * top-k truncates return LANTERN_ERR_UNSUPPORTED with either of them.                              */

/* ---- (1) latent-neighbour table -------------------------------------------------------------
 * Sec. 2.2 / Sec. 4: B_k(x) = the k nearest neighbours of codebook vector c_x (App. A.1:
 * C = {c_1..c_L}, c_i in R^d).  Metric: squared Euclidean distance on the raw rows.  For every
 * row i the k rows j != i with the smallest (distance, j), ascending; exact (distances are
 * evaluated in double precision before ranking), so duplicate rows tie by index.
 *   codebook  [L][d] row-major, dt = F32 or BF16            nbr_idx  [L][k] int32
 *   nbr_dist  [L][k] float32 squared distances, or NULL
 *   workspace device scratch of at least lantern_build_neighbors_workspace() bytes, 256-B aligned
 *             (row norms, and for the tcgen05 kernel the candidate lists of its CTAs: up to
 *             160 * 128 * (k + 128 + max(k, 192)) * 8 bytes; 0 bytes for the brute-force kernel)
 * bfloat16 codebooks with k <= 320 take a tensor-core path: approximate distances from bf16 MMAs
 * select a superset of the neighbours (with a proven error margin), which is then ranked exactly.
 * L >= 8192 and d a multiple of 8 up to 256: tcgen05 MMAs with accumulators in tensor memory; the
 * codebook must be 16-byte aligned.  Smaller L with d a multiple of 16 in [32, 256]: mma.sync.
 * Everything else takes an exact brute-force kernel.  The table is the same whichever kernel
 * builds it.  Every wait inside the tcgen05 kernel is bounded; should one run out, the rows of the
 * affected query tiles are written as -1 (never observed; callers may check nbr_idx[i][0] >= 0).
 * Requires 1 <= k <= min(L-1, 1024), 1 <= d <= 4096.                                            */
size_t lantern_build_neighbors_workspace(lantern_dtype dt, int32_t L, int32_t d, int32_t k);
lantern_status lantern_build_neighbors(const void* codebook, lantern_dtype dt, int32_t L, int32_t d,
                                       int32_t k, int32_t* nbr_idx, float* nbr_dist,
                                       void* workspace, size_t workspace_bytes, void* stream);

/* ---- (3) stochastic static-tree drafting ----------------------------------------------------
 * Sec. 2.1: at a node with s children the drafter samples s tokens from p(. | path).  Drawn
 * without replacement by Gumbel-top-s: key_j = log p_j - log(-log U_j); the s largest keys in
 * descending order (ties: lower token id) become the children's tokens, in stored order.
 * Expands the parents with node id in [parent_begin, parent_end) (one tree level, or 0..N for the
 * whole tree when all drafter rows are known).
 *   draft_cond / draft_uncond  [B][N][V] logits, row n = drafter output at node n; uncond NULL =
 *                              no guidance.  Element (b, n, j) at  b*seq_stride + n*row_stride + j
 *                              (strides in elements; rows must start 16-byte aligned).
 *   gumbel_uniforms            [B][N][V] float32 in (0,1) indexed like the rows (contiguous), or
 *                              NULL: Philox stream 0, U = ((x >> 9) + 0.5) * 2^-23
 *   tokens                     [B][N] int32, entries of the expanded parents' children are
 *                              written (-1 where fewer than s tokens have positive probability)
 *   draft_prob                 [B][N] float32 p(token) under the parent's row, or NULL           */
lantern_status lantern_sample_draft_tree(const lantern_params* params, const lantern_tree* tree,
                                         const void* draft_cond, const void* draft_uncond,
                                         lantern_dtype dt, int64_t row_stride, int64_t seq_stride,
                                         int32_t batch, int32_t parent_begin, int32_t parent_end,
                                         const float* gumbel_uniforms, int32_t* tokens,
                                         float* draft_prob, int32_t* device_status, void* stream);

/* ---- (2) relaxed verification of the tree ---------------------------------------------------
 * Sec. 4 and App. A.2 (Eq. 1-2), per node n with children c_1..c_s in stored order:
 *   q_cur = q(n), p_cur = p(n)
 *   for each child c with token x:
 *     A = {x} + longest prefix of x's neighbour list (first k entries of the table row) whose
 *         running sum of q_cur, q_cur(x) included, stays < lambda * q_cur(x);   m = sum_A q_cur
 *         (params->delta > 0, Sec. 2.2: ... whose own running sum stays < delta instead)
 *     accept c iff u_accept[c] < min(1, m / p_cur(x))
 *     on rejection: move A's mass onto x, q_cur = normalise([q~ - p_cur]_+), drop x from p_cur
 *   if no child was accepted (or n is a leaf): node_token[n] = inverse-CDF sample of q_cur with
 *   u_resample[n], in token-id order.
 * Then the walk (Sec. 2.1): from the root follow accepted children; out_tokens holds the accepted
 * draft tokens followed by the token sampled where the walk stops.
 *   nbr_idx        [n_codes][k_table] table of (1); may be NULL when params->k == 0
 *   target_* / draft_*  [B][N][V] logits as in (3); draft rows of leaves are never read
 *   tokens         [B][N] draft tokens (entry 0 unused; negative = no draft, skipped)
 *   u_accept, u_resample  [B][N] float32 in [0,1), or NULL: Philox streams 1 / 2,
 *                  u = (x >> 8) * 2^-24
 *   accept_len     [B]            number of accepted draft tokens
 *   out_tokens, out_nodes  [B][max_depth+1]; entries beyond accept_len+1 are set to -1
 *   node_next, node_token  [B][N] or NULL (then they live in the workspace)
 *   node_mass, node_thresh [B][N] float32 m and accept probability per tested child, -1 where
 *                  a node was not tested; or NULL
 *   device_status  one int32, OR-ed with LANTERN_DEV_* bits; or NULL
 *   workspace      device scratch >= lantern_verify_tree_workspace() bytes (12 bytes per node:
 *                  node_next, node_token and one repair flag; plus 256 bytes), 256-byte aligned.  It may be
 *                  NULL when node_next and node_token are both given; rows truncated by top-k
 *                  then take the dense kernel instead of the faster list-based one, which needs
 *                  the flags.                                                                    */
size_t lantern_verify_tree_workspace(const lantern_tree* tree, int32_t batch);
lantern_status lantern_verify_tree(const lantern_params* params, const lantern_tree* tree,
                                   const int32_t* nbr_idx, int32_t k_table,
                                   const void* target_cond, const void* target_uncond,
                                   const void* draft_cond, const void* draft_uncond,
                                   lantern_dtype dt, int64_t row_stride, int64_t seq_stride,
                                   int32_t batch, const int32_t* tokens,
                                   const float* u_accept, const float* u_resample,
                                   int32_t* accept_len, int32_t* out_tokens, int32_t* out_nodes,
                                   int32_t* node_next, int32_t* node_token,
                                   float* node_mass, float* node_thresh,
                                   int32_t* device_status, void* workspace, size_t workspace_bytes,
                                   void* stream);

/* ---- which kernels a call launches ---------------------------------------------------------------
 * Rows that no top-k truncates are handled by streaming kernels (LANTERN_PATH_STREAM): every row is
 * read from HBM once and never held on chip; a rejection is one more read-only pass over the
 * node's two rows, served by L2.  Rows that App. B's top-k truncation cuts to at most 1280 entries,
 * in vocabularies of at most 16384 tokens, are handled by list-based kernels (LANTERN_PATH_LISTS:
 * the row is compacted to its survivors; everything after works on those), followed by a launch of
 * the dense kernels that redoes the nodes whose rows did not fit the lists' fixed buffers (massive
 * ties; usually none).  All other calls (top-k on wide vocabularies, the path walk) run the dense
 * kernels alone (LANTERN_PATH_DENSE: rows held in shared memory).  So do small calls without top-k
 * (fewer than 128 tree nodes, or fewer than both 256 and 4 Mi / vocab expanded parents, in the whole
 * batch) whose rows fit the dense
 * kernels: a handful of nodes is a chain of dependent steps, which shared-memory rows shorten.
 * params->kernels overrides the choice by size.  Results are the same either way; these queries
 * only tell which it will be for a batch of `batch` sequences (lantern_verify_tree additionally
 * needs its full workspace for the list path).
 * Launches per call: lantern_sample_draft_tree 1 (streaming, dense) or 2 (lists + repair);
 * lantern_verify_tree 2 (streaming + walk, dense + walk, or lists + repair launch that also
 * walks), or 1 with params->lazy_walk (the path-walk kernel walks as it goes).  Returns -1 on NULL
 * arguments.                                                                                      */
#define LANTERN_PATH_DENSE 0
#define LANTERN_PATH_LISTS 1
#define LANTERN_PATH_STREAM 2
int32_t lantern_verify_tree_path(const lantern_params* params, const lantern_tree* tree, int32_t batch);
int32_t lantern_sample_draft_tree_path(const lantern_params* params, const lantern_tree* tree, int32_t batch);

/* ---- relaxed verification without any allocation ---------------------------------------------
 * The paper has no counterpart to this entry point; it exists for callers that must not, or
 * cannot, allocate device memory around the call: code running inside a memory pool that is
 * already fully handed out, a serving loop that forbids cudaMalloc because it synchronises the
 * device, or a host that only passes buffers it was given.  It is lantern_verify_tree with the
 * per-node scratch (accepted child, drawn token and repair flag of every node, 12 bytes per node)
 * taken from a fixed array inside the library instead of a caller workspace.  The array holds
 * lantern_verify_tree_static_max_nodes() = 65536 nodes (768 KB), so batch * n_nodes must not
 * exceed that: larger calls return LANTERN_ERR_UNSUPPORTED and launch nothing.  Every GPU that
 * loads the library keeps the array until the process exits.
 *  - Nothing is allocated or freed, by this call or by anything it calls.
 *  - The first call on a device looks up the array's device address (a one-time query with that
 *    device current); make that first call outside any stream capture.
 *  - All calls on a device share the one array and it keeps the previous call's contents.  The
 *    kernel writes every entry it later reads, so nothing needs clearing, but two calls that
 *    overlap on the GPU (different streams, no ordering between them) race on it and give
 *    wrong results.  Order such calls, or give the overlapping ones a workspace through
 *    lantern_verify_tree.
 * Arguments and results are those of lantern_verify_tree; node_next / node_token are not
 * returned.                                                                                      */
int32_t lantern_verify_tree_static_max_nodes(void);
lantern_status lantern_verify_tree_static(const lantern_params* params, const lantern_tree* tree,
                                          const int32_t* nbr_idx, int32_t k_table,
                                          const void* target_cond, const void* target_uncond,
                                          const void* draft_cond, const void* draft_uncond,
                                          lantern_dtype dt, int64_t row_stride, int64_t seq_stride,
                                          int32_t batch, const int32_t* tokens,
                                          const float* u_accept, const float* u_resample,
                                          int32_t* accept_len, int32_t* out_tokens, int32_t* out_nodes,
                                          float* node_mass, float* node_thresh,
                                          int32_t* device_status, void* stream);

/* ---- (5) dynamic-tree drafting -------------------------------------------------------------
 * Sec. 2.1, the dynamic variant of tree drafting: every draft node t_i carries the global accept
 * value V_i = product of the drafter's confidences c_j along the path from the root (the
 * confidence of a token is its probability in the drafter's post-processed row); a depth of
 * drafting gives every frontier node its n_children most confident tokens and keeps the n_expand
 * candidates with the largest V as the next frontier; at the end the nodes are trimmed by V
 * (Sec. 3: with low confidences the product decays fast and the tree stays shallow).  The tokens
 * are chosen deterministically, so such a tree is verified with draft_deterministic = 1.
 *
 * A sequence's candidates live in a pool of pool_size entries (entry 0 = the root: the caller sets
 * pool_parent = -1, pool_token = -1, pool_logv = 0, pool_depth = 0).  Values are kept as log V in
 * double.  Equal values rank by lower index: tokens of a row by (z descending, token ascending),
 * candidates by (log V descending, pool index ascending), so a parent ranks before its children.
 *
 * lantern_expand_frontier, one depth:
 *   draft_cond / draft_uncond  drafter rows of the frontier nodes: row of slot f of sequence b at
 *             b * seq_stride + f * row_stride (elements); uncond NULL = no guidance.  Post-processing
 *             as for every other entry point (guidance, temperature, allowed range); top_k_draft
 *             must be 0 (LANTERN_ERR_UNSUPPORTED otherwise)
 *   frontier  [batch][n_frontier] pool index of the node in each slot, -1 = empty slot
 *   pool_*    [batch][pool_size]; the n_frontier * n_children candidates of this depth are written
 *             at pool_offset + f * n_children + rank (parent = the slot's node, depth = `depth`,
 *             log V = the parent's + ln c); candidates of empty slots get log V = -inf
 *   next_frontier  [batch][n_expand] pool indices of the chosen candidates in rank order, -1 beyond
 *             the number of candidates
 * 1 <= n_children <= LANTERN_MAX_CHILDREN, n_frontier * n_children <= 2048, pool_size <= 2048.
 *
 * lantern_trim_tree: of the first pool_used entries keep the root and the max_nodes - 1 others with
 * the largest log V, renumbered breadth first as lantern_tree_create wants them.
 *   n_nodes [batch]; parent / token / pool_index / logv [batch][max_nodes] (unused tail: -1, -inf)
 *   max_depth  the largest value in pool_depth (the number of depths drafted)                     */
lantern_status lantern_expand_frontier(const lantern_params* params, const void* draft_cond,
                                       const void* draft_uncond, lantern_dtype dt, int64_t row_stride,
                                       int64_t seq_stride, int32_t batch, int32_t n_frontier,
                                       int32_t n_children, int32_t n_expand, const int32_t* frontier,
                                       int32_t pool_size, int32_t pool_offset, int32_t depth,
                                       int32_t* pool_parent, int32_t* pool_token, double* pool_logv,
                                       int32_t* pool_depth, int32_t* next_frontier, void* stream);
lantern_status lantern_trim_tree(int32_t batch, int32_t pool_size, int32_t pool_used, int32_t max_depth,
                                 const int32_t* pool_parent, const int32_t* pool_token,
                                 const double* pool_logv, const int32_t* pool_depth, int32_t max_nodes,
                                 int32_t* n_nodes, int32_t* parent, int32_t* token, int32_t* pool_index,
                                 double* logv, void* stream);

/* Raw Philox-4x32-10 words (Salmon et al., SC 2011) for counters (first + i, c1, c2, c3), i in
 * [0, n): out[i][0..3].  Exists so that the generator can be checked against other
 * implementations.  out is a device pointer to n*4 uint32.                                      */
lantern_status lantern_philox_raw(uint64_t seed, uint32_t first, uint32_t c1, uint32_t c2,
                                  uint32_t c3, int32_t n, uint32_t* out, void* stream);

/* Tuning knob: number of CTAs a logit row is split over (a thread-block cluster), 0 = choose
 * automatically; any value other than 0, 1, 2, 4, 8, 16 is ignored.  Returns the previous value.
 * Results do not depend on it beyond float32 summation order.  The setting is one unsynchronised
 * process-wide variable: it is not thread-safe, it applies to every later call of every thread on
 * every device, and a non-zero value also makes top-k rows take the dense kernels.  Set it once at
 * start-up, or not at all.                                                                       */
int32_t lantern_set_cluster_size(int32_t ctas_per_row);
int32_t lantern_get_cluster_size(void);      /* the current setting */

#ifdef __cplusplus
}
#endif
#endif /* LANTERN_H_ */
