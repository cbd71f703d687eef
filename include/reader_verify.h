/*
 * reader_verify.h -- C ABI of the batched tree-verification step of READER-style lossless
 * speculative decoding, implemented as hand-written CUDA for sm_100a (NVIDIA B200).
 *
 * One decoding step of the method (Algorithm 1: the Verify call and the cache maintenance that
 * follows it) hands a draft tree per sequence to the target model, which scores every node in one
 * pass (Sec. 3.2), keeps the longest root path the model agrees with (Algorithm 5; Appendix C,
 * invariants 1-3) and appends the accepted entries to the KV cache without gaps (Sec. 4.3,
 * Algorithm 4).  This library is the attention, acceptance and cache part of that step:
 *
 *     reader_tree_encode   parent array  ->  per-node ancestor bitmask           (Sec. 3.2 mask)
 *     reader_verify_attn   tree-masked attention over paged cache + tree K/V     (Sec. 3.2)
 *     reader_accept        target argmax + longest consistent root path          (Algorithm 5)
 *     reader_kv_commit     accepted K/V rows -> cache tail, seq_lens += n_acc    (Algorithm 4)
 *   and, beside these: reader_sample_targets (the sampling policies of Appendix C in place of the
 *   argmax), reader_verify_prepare / reader_verify_attn_prepared (the per-step part of the attention call
 *   done once for all layers), reader_accept_commit (acceptance and commit in one launch), reader_kv_commit_layers (all
 *   layers of a model in one launch), reader_kv_rearrange
 *   (Algorithm 4 on the paper's padded cache layout), reader_verify_attn_padded /
 *   reader_padded_append / reader_padded_rearrange (the padded cache of Sec. 4.3 run as a cache, to be
 *   measured against the paged one), reader_accept_noalloc.
 *
 * Conventions common to every call
 *   - Every pointer named below is a DEVICE pointer owned by the caller unless it says "host".
 *     The library allocates no device memory; scratch comes from the caller's workspace.
 *   - `stream` is a cudaStream_t passed as void*.  Calls only enqueue work on it: none of them
 *     synchronises or reads device data on the host.
 *   - Tensors are dense, row-major, last index fastest.  bf16 tensors are raw 16-bit patterns.
 *     Pointers to bf16/f32/u64 tensors must be 16-byte aligned.
 *   - Errors have two channels.  (1) The return value reports what the host can check (null or
 *     misaligned pointers, unsupported shapes, workspace too small, a CUDA launch error); on
 *     such an error nothing has been launched.  (2) `status_out[b]` (device, one word per
 *     sequence) reports what only the data can tell: a malformed parent array, a page id
 *     outside the pool, a length beyond the page table.  A sequence with a non-zero status gets
 *     defined outputs (attention rows and lse zero; n_acc 0, path -1, bonus -1; nothing
 *     committed) and does not disturb the others.  No kernel traps, asserts or waits unbounded.
 *   - A context is bound to one device and is not thread-safe: it caches the TMA descriptors of the
 *     tensors it saw last, so calls on one context come from one host thread at a time (use one
 *     context per thread or serialise).  Calls on different contexts are independent.
 *   - An empty batch (batch = 0) is legal everywhere: the call returns READER_OK, launches nothing
 *     and looks at no tensor pointer.
 *   - Tree convention: node 0 is the root = the last token already chosen by the target model
 *     (its K/V is part of the tree tensors, not yet of the cache); parent[0] = -1 and
 *     0 <= parent[j] < j.  At most READER_MAX_NODES nodes.
 */
#ifndef READER_VERIFY_H
#define READER_VERIFY_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define READER_MAX_NODES 128
#define READER_PAGE_SIZE 64
#define READER_NOALLOC_MAX_ROWS 4096 /* batch * n_nodes limit of reader_accept_noalloc */

typedef struct reader_ctx reader_ctx; /* opaque: device id, SM count, driver entry points */

typedef enum {
    READER_OK = 0,
    READER_ERR_INVALID_ARG = 1, /* null/misaligned pointer, size out of range */
    READER_ERR_BAD_TREE = 2,    /* status word: parent array breaks the tree convention */
    READER_ERR_CAPACITY = 3,    /* status word: length beyond the page table / commit has no room */
    READER_ERR_WORKSPACE = 4,   /* workspace smaller than reader_workspace_bytes() */
    READER_ERR_UNSUPPORTED = 5, /* shape the kernels are not built for */
    READER_ERR_TIMEOUT = 6,     /* status word: a bounded device-side wait gave up */
    READER_ERR_CUDA = 7,        /* a CUDA runtime/driver call failed */
    READER_ERR_BAD_PAGE = 8,    /* status word: page-table entry outside [0, num_pages) */
    READER_ERR_TOO_LARGE = 9    /* more rows than reader_accept_noalloc's built-in scratch holds */
} reader_status;

/*
 * One layer's paged KV cache (Sec. 4.3: per-sample cache without internal padding).
 *   k_pool, v_pool   bf16 [num_pages][n_kv_heads][page_size][head_dim]
 *   page_table       i32  [batch][max_pages_per_seq]; entry p of row b is the pool page that
 *                    holds logical positions p*page_size .. p*page_size+page_size-1 of sequence b
 *   seq_lens         i32  [batch] committed tokens per sequence; read by reader_verify_attn,
 *                    updated by reader_kv_commit
 *   shared_prefix_len  tokens (multiple of page_size, 0 = none) whose pages are the same pool
 *                    pages in every row of page_table (stored once); commits never write there
 * page_size must be READER_PAGE_SIZE; head_dim 64 or 128.
 */
typedef struct {
    void *k_pool;
    void *v_pool;
    int32_t num_pages, page_size, n_kv_heads, head_dim;
    const int32_t *page_table;
    int32_t max_pages_per_seq;
    int32_t *seq_lens;
    int32_t shared_prefix_len;
} reader_kv_cache;

/*
 * The draft trees of one step (Sec. 3.2; built by the drafting side of Algorithm 1).
 *   parent     i32 [batch][n_nodes]
 *   anc_mask   u64 [batch][n_nodes][2]  bit i of the 128-bit word of node j is set iff node i is
 *              j itself or an ancestor of j (from reader_tree_encode); NULL = encode internally
 */
typedef struct {
    int32_t batch, n_nodes;
    const int32_t *parent;
    const uint64_t *anc_mask;
} reader_tree;

/* Creates a context for CUDA device `device` (host call; may initialise the CUDA context).
 * *out is host memory owned by the library until reader_destroy.  READER_ERR_UNSUPPORTED when the
 * device is not of compute capability 10.x or the tensor-core attention kernel cannot be set up on it
 * (no tensor-map encoder in the driver, too little shared memory): the library never serves calls
 * from a slower path on its own. */
reader_status reader_create(reader_ctx **out, int device);
void reader_destroy(reader_ctx *ctx);
const char *reader_status_string(reader_status s);

/* Chooses the attention kernel: 0 = automatic (the tensor-core kernel, as a single launch for calls with
 * few units and as preparation + attention + combine otherwise; the CUDA-core kernel only for the shapes
 * the former is not built for: a GQA group that does not divide 128, a non-positive scale), 1 = always
 * the CUDA-core kernel, 2 = the tensor-core kernel on the three-launch path or READER_ERR_UNSUPPORTED,
 * 3 = the tensor-core kernel as a single launch or READER_ERR_UNSUPPORTED (batch * n_kv_heads * M tiles
 * must fit the GPU in one wave).  All compute Sec. 3.2's attention; this is a testing aid. Host call. */
reader_status reader_set_attn_kernel(reader_ctx *ctx, int32_t which);

/* Chooses how reader_verify_attn divides its work among thread blocks: 0 = automatic, 1 = always equal
 * ranges of the flattened tile list (best balance), 2 = the aligned partition whenever a prefix is
 * shared (every KV stream cut at the same relative positions, so that the sequences sharing a prefix
 * walk it in step and a prefix larger than the L2 cache is fetched from HBM once; automatic above 48 MB
 * of shared K and V).  Results do not depend on the choice beyond rounding; this is a testing and
 * measuring aid.  Host call. */
reader_status reader_set_partition(reader_ctx *ctx, int32_t which);

/* Profiling aid (host call): when both are non-NULL cudaEvent_t handles, the next calls of
 * reader_verify_attn (and of its prepared and padded forms) record `start` on the stream right before the main attention kernel and
 * `stop` right after it (the preparation and combine kernels lie outside).  NULL, NULL turns it off. */
reader_status reader_set_timing_events(reader_ctx *ctx, void *start, void *stop);

/* The same for reader_accept and reader_accept_commit called with logits: the events bracket the argmax
 * kernel (the acceptance walk that follows lies outside).  NULL, NULL turns it off. */
reader_status reader_set_accept_timing_events(reader_ctx *ctx, void *start, void *stop);

/* Bytes of device scratch that reader_verify_attn / reader_accept need for at most `max_batch`
 * sequences of at most `max_nodes` nodes.  Host call, no CUDA work.  Returns 0 on bad arguments. */
size_t reader_workspace_bytes(const reader_ctx *ctx, int32_t max_batch, int32_t max_nodes,
                              int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim);

/*
 * Sec. 3.2 decoding mask.  For every sequence b and node j writes the 128-bit ancestor-or-self
 * set anc_mask_out[b][j][0..1] and level_out[b][j] = number of nodes on the path root..j (nullable).
 * status_out[b] = READER_ERR_BAD_TREE when parent[b] breaks the tree convention (its masks are
 * then zero).  1 <= n_nodes <= READER_MAX_NODES.
 */
reader_status reader_tree_encode(reader_ctx *ctx, const int32_t *parent, int32_t batch, int32_t n_nodes,
                                 uint64_t *anc_mask_out, int32_t *level_out, int32_t *status_out,
                                 void *stream);

/*
 * Sec. 3.2 verification attention.  For sequence b, node j and query head h (KV head h / G,
 * G = n_q_heads / n_kv_heads) the query q[b][j][h] attends, with scores scaled by
 * softmax_scale, to the committed keys 0 .. seq_lens[b]-1 of the paged cache and to the tree
 * keys k_tree[b][i] of the nodes i that are j or an ancestor of j.
 *   q, out          bf16 [batch][n_nodes][n_q_heads][head_dim]
 *   k_tree, v_tree  bf16 [batch][n_nodes][n_kv_heads][head_dim]
 *   lse_out         f32  [batch][n_nodes][n_q_heads], natural log of the softmax denominator; nullable
 *   workspace       at least reader_workspace_bytes(...) bytes, 256-byte aligned; contents are
 *                   scratch, calls that share it must not overlap on the GPU
 *   status_out      i32 [batch]
 * Arithmetic: bf16 inputs, fp32 accumulation and softmax, probabilities rounded to bf16 before the
 * value product where tensor cores are used, bf16 (nearest-even) output.
 */
reader_status reader_verify_attn(reader_ctx *ctx, const void *q, int32_t n_q_heads,
                                 const void *k_tree, const void *v_tree,
                                 const reader_kv_cache *cache, const reader_tree *tree,
                                 float softmax_scale, void *out, float *lse_out,
                                 void *workspace, size_t workspace_bytes, int32_t *status_out,
                                 void *stream);

/*
 * Algorithm 5 (the comparison with the base model's choice) with the greedy policy of Appendix C.  If `logits` (f32
 * [batch][n_nodes][vocab]) is given, target_ids[b][j] is first set to the lowest index of the
 * row maximum (a NaN never wins; a NaN in slot 0 counts as -inf); otherwise target_ids is read
 * as given (any policy's per-node choice, e.g. a sampler driven by coupled uniforms).
 * A node is accepted when it is the root or its parent is accepted and
 * node_tokens[node] == target_ids[parent].  Returns the longest accepted root path with at most
 * max_path nodes (lowest end node among equals; equal sibling tokens are all followed):
 *   path_out   i32 [batch][max_path] node ids from the root, padded with -1
 *   n_acc_out  i32 [batch] nodes on the path, root counted (>= 1 for a valid tree)
 *   bonus_out  i32 [batch] target_ids at the end node: the token to emit after the path
 * The tokens appended to the output this step are node_tokens[path[1..n_acc-1]] then bonus.
 * workspace: as for reader_verify_attn (used only when logits is given).
 */
reader_status reader_accept(reader_ctx *ctx, const reader_tree *tree, const int32_t *node_tokens,
                            const float *logits, int32_t vocab, int32_t *target_ids,
                            int32_t max_path, int32_t *path_out, int32_t *n_acc_out,
                            int32_t *bonus_out, void *workspace, size_t workspace_bytes,
                            int32_t *status_out, void *stream);

/*
 * Appendix C, randomized decoding: the per-node target of a sampling policy, x* = F(P, U_t), for
 * use as `target_ids` of reader_accept(logits = NULL).  F is temperature sampling through the
 * inverse CDF.  One uniform serves one output position: every node of tree level lv (root = 1)
 * uses uniforms[b][lv - 1], and the caller passes the same uniforms the plain (non-speculative) run
 * would use for those positions -- that coupling is what makes the decoded text identical.
 *   logits      f32 [batch][n_nodes][vocab], 16-byte aligned
 *   uniforms    f32 [batch][n_nodes], values in [0, 1) (clamped into it)
 *   temperature > 0
 *   top_k       0 = no filtering; k >= 1 keeps only the logits that are at least the k-th largest of
 *               their row (NaN counts as -inf; logits equal to that value are all kept)
 *   top_p       >= 1 = no filtering; 0 < p < 1 keeps, of what top_k left, the smallest set of highest
 *               logits whose weight reaches the share p (logits equal to the last admitted one are
 *               admitted with it)
 *   target_ids  i32 [batch][n_nodes] out
 * The CDF is integer arithmetic (fp32 weights from a fixed fused-multiply-add polynomial for
 * 2^x, truncated to 40 fractional bits; exact 64-bit sums; threshold (S * trunc(u 2^24)) >> 24;
 * first token whose inclusive prefix sum exceeds it), so the result does not depend on how the
 * sum is parallelised.  NaN and -inf logits are never drawn; a row without any weight gives 0.
 * vocab <= 2 Mi.  No workspace.
 */
reader_status reader_sample_targets(reader_ctx *ctx, const reader_tree *tree, const float *logits, int32_t vocab,
                                    const float *uniforms, float temperature, int32_t top_k, float top_p,
                                    int32_t *target_ids, void *stream);

/*
 * Sec. 4.3 / Algorithm 4 in per-step form.  For k < n_acc[b] the K/V rows of node path[b][k]
 * (all KV heads) are copied to logical position seq_lens[b] + k of sequence b, i.e. pool slot
 * page_table[b][(L+k)/page_size]*page_size + (L+k)%page_size, which is also written to
 * slots_out[b][k] (i32 [batch][max_path], -1 padded).  If update_seq_lens != 0, seq_lens[b] +=
 * n_acc[b] afterwards (pass 0 for all but the last layer that shares seq_lens).  A sequence
 * whose page table cannot hold the new positions, or that would write below
 * shared_prefix_len, gets READER_ERR_CAPACITY and is left untouched.
 */
reader_status reader_kv_commit(reader_ctx *ctx, reader_kv_cache *cache, const void *k_tree,
                               const void *v_tree, int32_t batch, int32_t n_nodes,
                               const int32_t *path, const int32_t *n_acc, int32_t max_path,
                               int32_t update_seq_lens, int32_t *slots_out, int32_t *status_out,
                               void *stream);

/*
 * reader_accept followed by reader_kv_commit for one layer, with the acceptance walk and the commit
 * in a single launch (Algorithm 5, then Sec. 4.3 / Algorithm 4 in per-step form): one dependent
 * launch fewer per decoding step.  Arguments and results are those of the two calls: status_out is
 * reader_accept's status word, commit_status_out reader_kv_commit's; path_out and n_acc_out are both
 * outputs of the walk and what is committed.
 */
reader_status reader_accept_commit(reader_ctx *ctx, const reader_tree *tree, const int32_t *node_tokens,
                                   const float *logits, int32_t vocab, int32_t *target_ids, int32_t max_path,
                                   reader_kv_cache *cache, const void *k_tree, const void *v_tree,
                                   int32_t update_seq_lens, int32_t *path_out, int32_t *n_acc_out,
                                   int32_t *bonus_out, int32_t *slots_out, void *workspace,
                                   size_t workspace_bytes, int32_t *status_out, int32_t *commit_status_out,
                                   void *stream);

/*
 * reader_kv_commit for every layer of a model in one launch (the accepted path is the same in all
 * layers; a 32-layer model would otherwise issue 32 small kernels per step).
 *   caches     HOST array [n_layers] of reader_kv_cache: each layer's own k_pool / v_pool; all layers
 *              must share page_table, seq_lens, num_pages, n_kv_heads, head_dim, max_pages_per_seq and
 *              shared_prefix_len (one block table for the whole model), else READER_ERR_INVALID_ARG
 *   k_trees, v_trees  HOST arrays [n_layers] of device pointers, bf16 [batch][n_nodes][n_kv_heads][head_dim]
 * slots_out, status_out and the seq_lens update are those of reader_kv_commit (the check has the
 * same outcome in every layer).  n_layers >= 1.
 */
reader_status reader_kv_commit_layers(reader_ctx *ctx, const reader_kv_cache *caches, const void *const *k_trees,
                                      const void *const *v_trees, int32_t n_layers, int32_t batch, int32_t n_nodes,
                                      const int32_t *path, const int32_t *n_acc, int32_t max_path,
                                      int32_t update_seq_lens, int32_t *slots_out, int32_t *status_out, void *stream);

/*
 * Sec. 4.3 / Algorithm 4 on the paper's own cache layout (not the paged cache of the calls above):
 * a rectangular batch cache whose per-sample rows hold real entries and internal padding.
 *   k, v         bf16 [batch][n_kv_heads][capacity][head_dim], compacted in place
 *   valid        u8   [batch][capacity]: non-zero marks a real entry (a mask; values are not tested
 *                for zero); rewritten to 1..10..0
 *   lengths_out  i32  [batch]: real entries per sample
 * Per sample the real entries move to the front in order (RemoveInternalZeroPadding +
 * TightConcatenate) and the vacated tail is zeroed.  head_dim a multiple of 8; k, v 16-byte aligned.
 */
reader_status reader_kv_rearrange(reader_ctx *ctx, void *k, void *v, int32_t batch, int32_t n_kv_heads,
                                  int32_t capacity, int32_t head_dim, uint8_t *valid, int32_t *lengths_out,
                                  void *stream);

/*
 * reader_verify_attn in two parts, for a model with several layers: all layers of a step see the same
 * trees, lengths and block table, so the checks, the masks and the work partition are made once
 * (reader_verify_prepare) and every layer then runs only its attention and combine kernels
 * (reader_verify_attn_prepared) -- one launch and several microseconds fewer per layer.
 *
 * reader_verify_prepare: cache->page_table / seq_lens / shapes and tree are read (k_pool, v_pool are
 * not); status_out (i32 [batch]) receives the status words of reader_verify_attn and stays in use by
 * the prepared calls.  The result lives in `workspace`.
 * reader_verify_attn_prepared: same arguments as reader_verify_attn, with this layer's q, k_tree,
 * v_tree, pools and out; workspace, batch, tree (parent and anc_mask pointers), n_q_heads and the
 * cache's page_table, seq_lens and shapes must be the ones given to the last reader_verify_prepare on
 * this context, else READER_ERR_INVALID_ARG.  Between the two nothing may change seq_lens, the page
 * table or the trees, and no other reader_verify_attn* call may use the workspace (reader_accept* may).
 * Rows of a rejected sequence are zeroed in every layer's out.  A bounded wait that gives up in one
 * layer marks all later layers of the step as well (READER_ERR_TIMEOUT in status_out, zero rows).
 */
reader_status reader_verify_prepare(reader_ctx *ctx, const reader_kv_cache *cache, const reader_tree *tree,
                                    int32_t n_q_heads, void *workspace, size_t workspace_bytes,
                                    int32_t *status_out, void *stream);
reader_status reader_verify_attn_prepared(reader_ctx *ctx, const void *q, int32_t n_q_heads, const void *k_tree,
                                          const void *v_tree, const reader_kv_cache *cache,
                                          const reader_tree *tree, float softmax_scale, void *out,
                                          float *lse_out, void *workspace, size_t workspace_bytes,
                                          void *stream);

/*
 * The padded batch cache of Sec. 4.3 as a cache in its own right: the layout the paper starts from,
 * kept here beside the paged cache so that the two designs can be run and measured against each
 * other.  Every sample owns one row of `capacity` positions; all rows are in use up to the common
 * length *extent; within a row real entries and padding alternate as the steps left them.
 *   k, v      bf16 [batch][n_kv_heads][capacity][head_dim]
 *   valid     u8   [batch][capacity]: non-zero marks a real entry; zero at and beyond *extent
 *             (the two calls that move *extent keep it so; the attention ignores bytes there anyway)
 *   extent    i32  [1] DEVICE scalar: rows at or beyond it are unused in every sample
 * Padding rows may hold anything (the calls below write zeros there, as the paper does): no
 * query ever sees them.
 */
typedef struct {
    void *k;
    void *v;
    uint8_t *valid;
    int32_t *extent;
    int32_t capacity, n_kv_heads, head_dim;
} reader_padded_cache;

/* Workspace for reader_verify_attn_padded: that of reader_workspace_bytes plus the packed mask. */
size_t reader_padded_workspace_bytes(const reader_ctx *ctx, int32_t max_batch, int32_t max_nodes,
                                     int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim,
                                     int32_t capacity);

/*
 * reader_verify_attn (Sec. 3.2) over a padded batch cache: node j of sample b attends over the
 * real entries of row b below *extent, in position order, and over the tree nodes on its root
 * path.  Arguments, outputs, kernels and error channels are those of reader_verify_attn; there is
 * no page table, and status_out[b] = READER_ERR_CAPACITY for every sample when *extent is outside
 * [0, capacity].  Every sample costs the common length, padding included: that is the overhead
 * Sec. 4.3 describes.  head_dim 64 or 128; k, v 16-byte aligned.
 */
reader_status reader_verify_attn_padded(reader_ctx *ctx, const void *q, int32_t n_q_heads, const void *k_tree,
                                        const void *v_tree, const reader_padded_cache *cache,
                                        const reader_tree *tree, float softmax_scale, void *out, float *lse_out,
                                        void *workspace, size_t workspace_bytes, int32_t *status_out,
                                        void *stream);

/*
 * One step's growth of a padded batch cache (Sec. 4.3: a long accepted span in one sample makes
 * every other sample pad up to the new maximum length).  The K/V rows of path[b][0 .. n_acc[b]-1]
 * are written at positions *extent .. *extent + n_acc[b] - 1 of row b and marked real; zero rows
 * marked padding fill row b up to *extent + max_b n_acc[b], which becomes the new *extent.
 *   k_tree, v_tree  bf16 [batch][n_nodes][n_kv_heads][head_dim];  path i32 [batch][max_path];
 *   n_acc i32 [batch] (the outputs of reader_accept)
 * All or nothing: when the new length exceeds capacity, an n_acc is outside [0, max_path] or a path
 * entry is not a node, every status_out[b] is READER_ERR_CAPACITY and nothing is changed.
 * head_dim a multiple of 8.
 */
reader_status reader_padded_append(reader_ctx *ctx, reader_padded_cache *cache, const void *k_tree,
                                   const void *v_tree, int32_t batch, int32_t n_nodes, const int32_t *path,
                                   const int32_t *n_acc, int32_t max_path, int32_t *status_out, void *stream);

/*
 * reader_kv_rearrange (Algorithm 4) on a reader_padded_cache, all `capacity` positions of it:
 * afterwards every row is compact, lengths_out[b] (i32 [batch]) holds its entries and *extent is
 * the longest of them.
 */
reader_status reader_padded_rearrange(reader_ctx *ctx, reader_padded_cache *cache, int32_t batch,
                                      int32_t *lengths_out, void *stream);

/*
 * reader_accept with target logits, for callers that cannot provide a workspace.  (The paper has
 * no counterpart: this exists only because of how the library is deployed.)  Think of a serving
 * process that gave all device memory to its own pool at start-up, or a decode loop that may not
 * make an allocating call between steps: neither can cudaMalloc the scratch reader_accept wants.
 * Here the per-block (maximum, index) pairs of the logits scan live in a 2 MiB array inside the
 * library's device image instead; every GPU that loads the library holds it until the process
 * exits.  Inputs, outputs and results are exactly those of reader_accept(logits != NULL).
 *   - batch * n_nodes must not exceed READER_NOALLOC_MAX_ROWS, else READER_ERR_TOO_LARGE is
 *     returned and nothing is launched.
 *   - The call allocates nothing.  Its first use on a device looks up the array's device address
 *     (once per device; the context's device must be current): make that first call before any
 *     stream capture begins.
 *   - All calls share the array and leave their pairs in it.  Nothing in it needs clearing, every
 *     slot read is written earlier in the same call; but calls that can overlap on the GPU (two
 *     streams, two host threads) race on it -- issue them on one stream or order them.
 *   - The events of reader_set_accept_timing_events are not recorded by this call.
 */
reader_status reader_accept_noalloc(reader_ctx *ctx, const reader_tree *tree, const int32_t *node_tokens,
                                    const float *logits, int32_t vocab, int32_t *target_ids,
                                    int32_t max_path, int32_t *path_out, int32_t *n_acc_out,
                                    int32_t *bonus_out, int32_t *status_out, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* READER_VERIFY_H */
