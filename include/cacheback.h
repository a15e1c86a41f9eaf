/*
 * cacheback.h — C ABI of the Cacheback draft-and-verify step on one NVIDIA B200 (sm_100a).
 *
 * One decoding step of Cacheback speculative decoding (paper Section 3) is, per sequence of a batch:
 *   cb_update      slide a window over the newly accepted tokens and insert every leader->follower pair
 *                  into the sequence's LRU cache table                       (Section 3.1; 3.2 last par.)
 *   cb_draft_tree  grow a draft token tree by recursive table queries, breadth first, and emit parent
 *                  indices, depths and the ancestor ("tree attention") mask  (Section 3.2)
 *   cb_tree_attn   let every tree token attend to the sequence's paged KV cache plus its tree ancestors
 *                  (the attention of the single verification forward pass)    (Section 3.2)
 *   cb_accept      take the target's greedy choice after every node and keep the longest verified
 *                  branch plus one more token                                 (Section 3.2)
 *
 * Conventions
 *   - Every tensor pointer is a DEVICE pointer owned by the caller unless a parameter says "host".
 *     The library never allocates or frees device memory: all of its state and scratch lives in the
 *     workspace handed to cb_create.
 *   - `stream` is a cudaStream_t passed as void*. The four step calls and cb_reset only enqueue work
 *     on it; they never synchronise.  Calls on one context must be ordered (same stream, or events).
 *   - Host-detectable argument errors are returned at once and nothing is enqueued.  Conditions only
 *     the device can see (a probe limit, a bounded wait that ran out) are recorded in a device status
 *     word; the kernel finishes cleanly and cb_poll_status reports the first such code.
 *   - Token ids are int32 >= 0; -1 is "no token".  Rows of per-node outputs beyond a sequence's node
 *     count are padded: tokens / parents / depths / accepted nodes / emitted tokens with -1, mask and
 *     attention rows with 0.
 *   - bf16 tensors are passed as void* (16-bit brain floats, row-major, last index fastest).
 */
#ifndef CACHEBACK_H_
#define CACHEBACK_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct cb_ctx cb_ctx; /* opaque */

typedef enum {
    CB_OK = 0,
    CB_ERR_INVALID_ARG = 1,
    CB_ERR_WORKSPACE_TOO_SMALL = 2,
    CB_ERR_CUDA = 3,
    CB_ERR_PROBE_LIMIT = 4, /* device: a hash probe visited every bucket without finding a free slot  */
    CB_ERR_TIMEOUT = 5,     /* device: a bounded wait (mbarrier / flag) ran out                        */
    CB_ERR_UNSUPPORTED = 6,
    CB_ERR_STATIC_LIMIT = 7, /* cb_accept_static: the problem does not fit the built-in scratch array       */
    CB_ERR_KV_FULL = 8,      /* device: cb_kv_commit found a sequence whose pages cannot hold the new tokens   */
    CB_ERR_CANARY = 9        /* checking build only: a guard word beside a workspace region was overwritten    */
} cb_status;

enum { CB_DTYPE_F32 = 0, CB_DTYPE_BF16 = 1 };

/* cb_config.flags */
enum {
    CB_FLAG_NO_FOLLOWER_REFRESH = 1u, /* re-inserting a stored follower leaves its recency unchanged     */
    CB_FLAG_ATTN_CUDA_CORES = 2u,     /* run tree attention on the plain CUDA-core kernel (debug aid)    */
    CB_FLAG_ATTN_CTA_PAIRS = 4u       /* tree attention of multi-row-tile launches (head_dim 128) as pairs of
                                         CTAs issuing 2-CTA tensor-core products; measured slower than the
                                         default on the configurations benchmarked, kept as an alternative */
};

/*
 * Shape of one context. Table parameters follow Section 3.1 / 3.2:
 *   LL, FL  leader / follower length in tokens          (1..4, 1..8)
 *   LC, FC  leader capacity per sequence, follower capacity per leader   (1..2^20, 1..128)
 *   max_nodes  tree-size cap, root included: the paper's total draft length (TDL)   (1..128)
 *   crt        nodes reserved for query levels >= 2: level 1 fills at most max(1, max_nodes - crt)
 *   max_depth  deepest node depth allowed (root = 0)
 * Attention shape: n_q_heads % n_kv_heads == 0, head_dim in {64, 128}, page_size == 16.
 * vocab is the logits row length for cb_accept.
 */
typedef struct {
    int32_t batch;
    int32_t LL, FL, LC, FC;
    int32_t max_nodes, crt, max_depth;
    int32_t vocab;
    int32_t n_q_heads, n_kv_heads, head_dim, page_size;
    uint32_t flags;
} cb_config;

/* Bytes of device workspace cb_create needs for this shape (tables + scratch). Host call. */
cb_status cb_workspace_bytes(const cb_config* cfg, size_t* bytes);

/*
 * Creates a context over caller-owned device memory `dev_workspace` (256-byte aligned, `bytes` long,
 * on the current device) and empties every table.  Synchronises the device once.  *out is a small
 * host object; the workspace must outlive it and belongs to the library until cb_destroy.
 */
cb_status cb_create(const cb_config* cfg, void* dev_workspace, size_t bytes, cb_ctx** out);

/* Frees the host object only; never touches caller memory. NULL is allowed. */
void cb_destroy(cb_ctx* ctx);

/*
 * Empties the tables of the sequences whose entry in dev_seq_mask ([batch] int32, non-zero = reset) is
 * set, or of all sequences when dev_seq_mask is NULL (the per-task state reset of Section 4).
 */
cb_status cb_reset(cb_ctx* ctx, const int32_t* dev_seq_mask, void* stream);

/*
 * Table update (Section 3.1 insertion rules; Section 3.2, last paragraph: every leader-follower window that the newly
 * accepted tokens complete is inserted; Section 3.3 prompt initialisation = the same call with n_old = 0).
 *   tokens   int32 [batch, row_stride]  token history of every sequence
 *   n_old    int32 [batch]  tokens already ingested by earlier calls
 *   n_new    int32 [batch]  tokens valid now (n_new >= n_old; n_new <= row_stride)
 * For sequence b every complete window i (leader = tokens[i .. i+LL), follower = tokens[i+LL ..
 * i+LL+FL)) whose last token is new (i+LL+FL-1 in [n_old, n_new)) is inserted in increasing i:
 * the leader is created (evicting the least recently used leader with its followers when LC are
 * stored) or refreshed; the follower is appended (evicting the leader's least recently inserted
 * follower when FC are stored) or, if already stored, refreshed.
 */
cb_status cb_update(cb_ctx* ctx, const int32_t* tokens, int64_t row_stride, const int32_t* n_old,
                    const int32_t* n_new, void* stream);

/*
 * cb_update for long runs of new tokens (Section 3.3: the dynamic table is initialised with a sliding window over the
 * prompt).  Same arguments, same resulting tables, clocks and counters as cb_update; the work of one sequence is spread
 * over many warps where that cannot change the result (no leader can be evicted during the run: leaders stored + windows
 * <= LC, and at least 64 windows), and done by one warp in order otherwise.  Two launches (seven with scratch attached,
 * see below).  CB_CNT_FOLLOWER_EVICTIONS counts the followers this call displaced from the lists; on the order-free path
 * a follower that the run itself would have stored and displaced again is never stored and so is not counted.
 */
cb_status cb_update_bulk(cb_ctx* ctx, const int32_t* tokens, int64_t row_stride, const int32_t* n_old,
                         const int32_t* n_new, void* stream);

/*
 * Scratch memory for the order-free path of cb_update_bulk.  After a run in which no leader can be evicted, and under the
 * reading that re-inserting a stored follower refreshes it (the default), a leader's stamp is that of its last window and its
 * followers are the FC distinct ones touched last (Section 3.1: both lists are least-recently-used lists), whatever the
 * order of the windows.  With scratch attached, the sequences of a call whose runs qualify (as above) and fit the scratch,
 * taken in batch order, are reduced that way: one thread per window, then one warp per distinct leader.  The resulting
 * tables and clocks are those of cb_update; which place a follower or an entry takes inside the table may differ, which no
 * call reports.
 *   cb_bulk_scratch_bytes    HOST out: bytes for calls whose qualifying runs hold up to max_windows windows in total
 *                            (about 84 to 164 bytes per window: two hash tables of the next power of two >= 2 * max_windows
 *                            slots); cfg->batch sizes a small per-sequence array.
 *   cb_bulk_scratch_attach   dev_scratch: DEVICE, 256-byte aligned, `bytes` long, owned by the caller and to be kept while
 *                            attached; its content need not be initialised and is overwritten by every cb_update_bulk call.
 *                            NULL detaches.  Calls on one context that use it must not overlap.
 * Errors: CB_ERR_INVALID_ARG (null, misaligned, too small for any table).
 */
cb_status cb_bulk_scratch_bytes(const cb_config* cfg, int64_t max_windows, size_t* bytes);
cb_status cb_bulk_scratch_attach(cb_ctx* ctx, void* dev_scratch, size_t bytes);

/*
 * Draft-tree growth (Section 3.2).
 *   tokens, row_stride  as in cb_update;  seq_len int32 [batch] = tokens valid per sequence
 * Node 0 is the last token of the sequence (the one token whose K/V is not cached yet).  Level 1
 * queries the table with the last LL tokens of the sequence; every later level queries, for each leaf
 * that ends a complete follower, the last LL tokens of sequence ++ path-to-leaf.  Followers are
 * attached most recently inserted first, each as a chain of FL nodes; growth is breadth first and stops
 * at max_nodes (level 1 at max_nodes - crt), at max_depth, or when no leaf has a follower.  A chain
 * that does not fit is cut short and not grown further.  Every issued query refreshes its leader.
 * Outputs (all device):
 *   tree_tokens, tree_parent, tree_depth  int32 [batch, max_nodes]   parent of node 0 is -1
 *   tree_mask   uint32 [batch, max_nodes, W], W = ceil(max_nodes / 32): bit j of row i is set iff
 *               node j is node i or an ancestor of it
 *   n_nodes     int32 [batch]
 * A sequence with seq_len < 1 gets n_nodes = 0; with fewer than LL tokens, the root only.
 */
cb_status cb_draft_tree(cb_ctx* ctx, const int32_t* tokens, int64_t row_stride, const int32_t* seq_len,
                        int32_t* tree_tokens, int32_t* tree_parent, int32_t* tree_depth,
                        uint32_t* tree_mask, int32_t* n_nodes, void* stream);

/*
 * cb_update followed by cb_draft_tree on the grown sequences, in one launch (Section 3.2: the table is brought up to
 * date with the newly accepted tokens before the next draft is made from it).  Same arguments, results, table state
 * and errors as cb_update(tokens, row_stride, n_old, n_new) followed by cb_draft_tree(tokens, row_stride, n_new, ...);
 * at small batch the step saves a kernel boundary.
 */
cb_status cb_update_draft_tree(cb_ctx* ctx, const int32_t* tokens, int64_t row_stride, const int32_t* n_old,
                               const int32_t* n_new, int32_t* tree_tokens, int32_t* tree_parent, int32_t* tree_depth,
                               uint32_t* tree_mask, int32_t* n_nodes, void* stream);

/*
 * Extra branches from another drafter (Conclusion: because the drafts form a tree, the predicted drafts of other
 * speculative-decoding methods can be inserted as additional branches).  Call it between cb_draft_tree and the
 * verification pass.
 *   branches    int32 [batch, n_branches, max_len]   each row a run of tokens continuing the sequence after its last token
 *   branch_len  int32 [batch, n_branches]            tokens valid in each row (<= 0: none)
 *   n_branches <= 64
 * The tree arrays are those cb_draft_tree wrote and are extended in place.  For every sequence with a root, the branches
 * are taken in order; each becomes a chain of new nodes below the root (node 0), cut where the tree would exceed max_nodes
 * or a node max_depth, and ended by a negative token.  Branches are not compared with nodes already present.  The mask
 * rows of the new nodes and n_nodes are updated.  The tables are not touched.
 */
cb_status cb_tree_add_branches(cb_ctx* ctx, const int32_t* branches, const int32_t* branch_len, int32_t n_branches,
                               int32_t max_len, int32_t* tree_tokens, int32_t* tree_parent, int32_t* tree_depth,
                               uint32_t* tree_mask, int32_t* n_nodes, void* stream);

/*
 * Tree-masked attention over the paged KV cache (Section 3.2, "tree attention": a token attends only
 * to its ancestors in the draft tree; the cached context is fully visible).
 * With T = max_nodes, Hq / Hkv = n_q_heads / n_kv_heads, D = head_dim, P = page_size:
 *   q            bf16 [batch, T, Hq, D]
 *   k_pool,v_pool bf16 [num_pages, P, Hkv, D]   cached keys / values, paged
 *   block_table  int32 [batch, max_pages]       page id of the j-th page of each sequence
 *   ctx_len      int32 [batch]                  cached tokens per sequence (<= max_pages * P)
 *   k_tree,v_tree bf16 [batch, T, Hkv, D]       keys / values of the tree tokens themselves
 *   tree_mask    uint32 [batch, T, W], n_nodes int32 [batch]   as written by cb_draft_tree
 *   out          bf16 [batch, T, Hq, D]         rows >= n_nodes are written as zero
 *   lse          float [batch, Hq, T] or NULL   natural-log sum of exponentials per row (0 for padding)
 *   max_ctx      host upper bound on every ctx_len (0 = max_pages * P); used only to size the grid
 *   scale        softmax scale; 0 selects 1/sqrt(D)
 * Row (b, i, h) = softmax_j(scale * q.k_j) v_j over j in {cached tokens of kv head h / (Hq/Hkv)}
 * U {tree nodes in mask row i}; fp32 accumulation and softmax, output rounded to bf16.
 * All base pointers must be 16-byte aligned.
 * Keys and values are fetched a tile at a time and what lies outside a row's key set is given probability 0, not skipped,
 * so everything a tile covers must be finite (0 x NaN would reach the output): all T rows of k_tree / v_tree of every
 * sequence, including rows >= n_nodes, and the slots of a sequence's last, partly filled page beyond ctx_len.  Pages past
 * the last one are never read.  Buffers from an allocator that does not clear them must be zeroed once.
 */
typedef struct {
    const void* q;
    const void* k_pool;
    const void* v_pool;
    const int32_t* block_table;
    const int32_t* ctx_len;
    const void* k_tree;
    const void* v_tree;
    const uint32_t* tree_mask;
    const int32_t* n_nodes;
    void* out;
    float* lse;
    int32_t max_pages;
    int32_t num_pages;
    int32_t max_ctx;
    float scale;
} cb_attn_args;

cb_status cb_tree_attn(cb_ctx* ctx, const cb_attn_args* args, void* stream);

/*
 * Greedy acceptance (Section 3.2: the forward pass yields one more token than the accepted draft
 * tokens, so a step emits between 1 and 1 + longest-branch tokens).
 *   tree_tokens, tree_parent, tree_depth, n_nodes   as written by cb_draft_tree
 *   logits        [batch, max_nodes, vocab] of logits_dtype (CB_DTYPE_F32 / CB_DTYPE_BF16), node rows
 *                 logits_row_stride elements apart (sequence stride = max_nodes * logits_row_stride);
 *                 finite values only.  target[i] = index of the first maximum of row i.
 *   target_ids_in int32 [batch, max_nodes]: targets given directly.  Exactly one of logits /
 *                 target_ids_in is non-NULL.
 * Node i > 0 is verified iff its parent is verified and tree_tokens[i] == target[parent]; the root is
 * verified.  The deepest verified node wins (lowest index among equally deep ones).  With m its depth:
 *   n_accept       int32 [batch]               = m
 *   accept_nodes   int32 [batch, max_depth]    the m nodes below the root on the winning path
 *   out_tokens     int32 [batch, max_depth+1]  their tokens followed by target[winner]  (m+1 tokens)
 *   target_ids_out int32 [batch, max_nodes] or NULL: the argmax of every valid row (-1 for padding)
 */
cb_status cb_accept(cb_ctx* ctx, const int32_t* tree_tokens, const int32_t* tree_parent,
                    const int32_t* tree_depth, const int32_t* n_nodes, const void* logits,
                    int32_t logits_dtype, int64_t logits_row_stride, const int32_t* target_ids_in,
                    int32_t* n_accept, int32_t* accept_nodes, int32_t* out_tokens,
                    int32_t* target_ids_out, void* stream);

/*
 * One step's acceptance and the next step's update and draft in one launch (Fig. 2: per sequence the three follow one
 * another — the emitted tokens extend the sequence, their windows go into the table, the next tree is drafted from it).
 * Same results, table state, counters and errors as
 *   cb_accept(tree_*, n_nodes, logits, ..., NULL, n_accept, accept_nodes, out_tokens, target_ids_out);
 *   tokens[b][seq_len[b] .. seq_len[b] + n_accept[b] + 1) = out_tokens[b][0 .. n_accept[b] + 1);   old = seq_len;   seq_len += n_accept + 1;
 *   cb_update(tokens, row_stride, old, seq_len);   cb_draft_tree(tokens, row_stride, seq_len, next_*);
 * At small batch the step saves two kernel boundaries.
 *   logits .. target_ids_out   as in cb_accept (logits only)
 *   tokens      int32 [batch, row_stride]  DEVICE, read and written: the emitted tokens are appended
 *   seq_len     int32 [batch]              DEVICE, read and written: tokens valid per sequence
 *   next_tokens, next_parent, next_depth, next_mask, next_n_nodes   the next tree, as written by cb_draft_tree; they may be the
 *               arrays of the verified tree (a sequence's acceptance has read them before its draft writes them)
 * A sequence whose history has no room for the emitted tokens (seq_len + n_accept + 1 > row_stride) keeps its length, nothing
 * is appended, the draft is made from the sequence as it is, and CB_ERR_INVALID_ARG is recorded in the device status.  A
 * sequence with an empty tree (n_nodes = 0) emits nothing.
 */
typedef struct cb_accept_draft_args {
    const void* logits;
    int32_t logits_dtype;
    int64_t logits_row_stride;
    const int32_t* tree_tokens;
    const int32_t* tree_parent;
    const int32_t* tree_depth;
    const int32_t* n_nodes;
    int32_t* n_accept;
    int32_t* accept_nodes;
    int32_t* out_tokens;
    int32_t* target_ids_out;
    int32_t* tokens;
    int64_t row_stride;
    int32_t* seq_len;
    int32_t* next_tokens;
    int32_t* next_parent;
    int32_t* next_depth;
    uint32_t* next_mask;
    int32_t* next_n_nodes;
} cb_accept_draft_args;

cb_status cb_accept_update_draft_tree(cb_ctx* ctx, const cb_accept_draft_args* args, void* stream);

/*
 * KV commit of the accepted path (Section 3.2: the draft tokens and the pending token are the tokens of the
 * verification pass that have no cached K/V; once a branch is accepted its tokens are ordinary context for the next
 * step).  For every sequence b with m = n_accept[b], the tree root (node 0) and the accepted nodes accept_nodes[b, 0..m),
 * in that order, become context tokens ctx_len[b] .. ctx_len[b] + m: their rows of k_tree / v_tree are copied into the
 * paged cache (page block_table[b, pos / P], slot pos % P) and ctx_len[b] grows by m + 1.  The bonus token of cb_accept
 * has no K/V yet: it is the next step's root.
 *   k_pool, v_pool  bf16 [num_pages, P, Hkv, D]   written
 *   block_table     int32 [batch, max_pages]      must already name pages for the new positions
 *   ctx_len         int32 [batch]                 read and updated in place
 *   k_tree, v_tree  bf16 [batch, T, Hkv, D]
 *   n_accept        int32 [batch], accept_nodes int32 [batch, max_depth]   as written by cb_accept
 * A sequence with ctx_len + m + 1 > max_pages * P is left untouched and CB_ERR_KV_FULL is recorded in the device status;
 * a node or page index outside its tensor is skipped and recorded as CB_ERR_INVALID_ARG.  Only enqueues work.
 */
typedef struct {
    void* k_pool;
    void* v_pool;
    const int32_t* block_table;
    int32_t* ctx_len;
    const void* k_tree;
    const void* v_tree;
    const int32_t* n_accept;
    const int32_t* accept_nodes;
    int32_t max_pages;
    int32_t num_pages;
} cb_kv_commit_args;

cb_status cb_kv_commit(cb_ctx* ctx, const cb_kv_commit_args* args, void* stream);

/*
 * Frozen table (Section 3.3): a second, read-only table built offline from the most frequent leader-follower pairs of a
 * corpus.  A step drafts from the dynamic table first and then lets the frozen table add branches while the tree is below
 * its size cap; insertions never reach it.
 *
 * A frozen table is one device buffer owned by the caller, of cb_frozen_bytes() bytes, 256-byte aligned, shared by every
 * sequence and every context that attaches it, and only read by the step calls.  LL and FL must equal the context's;
 * LC (1..2^20) and FC (1..128) are its own.
 *
 *   cb_frozen_load    fills the buffer from HOST arrays: leaders int32 [n_leaders, LL], n_followers int32 [n_leaders]
 *                     (1..FC each), followers int32 [n_leaders, FC, FL], each leader's followers most frequent first,
 *                     leaders most frequent first.  Synchronises the device.
 *   cb_frozen_dump    the reverse, into HOST arrays sized for LC leaders (any may be NULL; unused follower places -1):
 *                     leaders by falling corpus count, equal counts by rising tokens.  Synchronises the device.
 *   cb_frozen_attach  makes cb_draft_tree of this context run the second pass; dev_table = NULL detaches.  Host call, no
 *                     device work; order it against draft calls in flight yourself.
 *
 * With a frozen table attached, cb_draft_tree continues after the dynamic pass while the tree has fewer than max_nodes
 * nodes: it visits, first in first out, every node that can carry a follower list (the root and the last node of every
 * complete follower, in creation order; the ends of the complete followers the frozen pass adds join the queue), looks
 * the node's key up in the frozen table and attaches the stored followers, most frequent first, under the same rules as
 * the dynamic pass (a query at the root only while fewer than max(1, max_nodes - crt) nodes exist, any other while fewer
 * than max_nodes; max_depth; a follower that does not fit is cut short).  Frozen followers are not compared with the
 * branches already present.  Frozen queries touch no recency and are counted in CB_CNT_FROZEN_QUERIES / _HITS.
 *
 * Offline construction (Section 4: from a corpus sample, the LC most frequent n-grams of length LL become the leaders,
 * and each leader keeps the FC most frequent n-grams of length FL that follow it).
 *   cb_frozen_build   counts on the GPU.  dev_corpus int32 [n_tokens] (device, ids >= 0, one token stream,
 *                     n_tokens <= 2^30); an occurrence is counted where LL + FL tokens are available, so every leader
 *                     has at least one follower; equal counts are ordered by the tokens, smallest first.  dev_scratch:
 *                     cb_frozen_build_bytes() bytes of device memory, 256-byte aligned, free again after the call.
 *                     Overwrites dev_table.  Enqueues on `stream` and waits for it; returns CB_ERR_INVALID_ARG if a
 *                     negative token was met (its windows are left out).
 */
typedef struct {
    int32_t LL, FL, LC, FC;
} cb_frozen_config;

cb_status cb_frozen_bytes(const cb_frozen_config* cfg, size_t* bytes);
cb_status cb_frozen_load(const cb_frozen_config* cfg, void* dev_table, size_t bytes, int32_t n_leaders,
                         const int32_t* leaders, const int32_t* n_followers, const int32_t* followers);
cb_status cb_frozen_dump(const cb_frozen_config* cfg, const void* dev_table, size_t bytes, int32_t* n_leaders,
                         int32_t* leaders, int32_t* n_followers, int32_t* followers);
cb_status cb_frozen_attach(cb_ctx* ctx, const cb_frozen_config* cfg, const void* dev_table, size_t bytes);
cb_status cb_frozen_build_bytes(const cb_frozen_config* cfg, int64_t n_tokens, size_t* scratch_bytes);
cb_status cb_frozen_build(const cb_frozen_config* cfg, const int32_t* dev_corpus, int64_t n_tokens, void* dev_table,
                          size_t table_bytes, void* dev_scratch, size_t scratch_bytes, void* stream);

/*
 * cb_accept_static — cb_accept (logits form) for callers that must not allocate device memory.
 * (The paper has no counterpart; this is a packaging variant of the call above.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits — inside a framework's memory pool whose
 * owner forbids side allocations, in a plugin that is handed buffers but no allocator, or under a
 * memory budget that is fixed before the library is loaded.  Such a caller cannot provide the workspace
 * cb_create wants, so this entry point needs no context at all: the scratch that the arg-max reduction
 * uses (one packed maximum per logits row and one arrival counter per sequence) lives in a fixed array
 * that is part of the library image.  Every GPU that loads the library carries that array
 * (CB_STATIC_MAX_ROWS * 8 + CB_STATIC_MAX_BATCH * 4 bytes = 68 KiB) until the process exits.
 *
 * Shape arguments replace the context: batch, max_nodes (1..128), max_depth (>= 0), vocab (>= 1).
 * All other arguments, the result and the tie rules are exactly those of cb_accept with logits given;
 * target_ids_out may be NULL.
 *
 * Limits: batch <= CB_STATIC_MAX_BATCH and batch * max_nodes <= CB_STATIC_MAX_ROWS; anything larger
 * returns CB_ERR_STATIC_LIMIT and enqueues nothing.
 *
 * The call never allocates or frees (no cudaMalloc / cudaFree, no allocating library routine).  The first
 * call on each device looks up the array's device address once, with that device current; make that
 * first call outside any stream capture.  Before each launch the part of the array in use is cleared
 * on `stream`.  All calls on a device share the one array: two calls that may overlap on the GPU
 * (different streams without an ordering between them) race on it and give wrong results; order them.
 */
enum { CB_STATIC_MAX_BATCH = 1024, CB_STATIC_MAX_ROWS = 8192 };
cb_status cb_accept_static(int32_t batch, int32_t max_nodes, int32_t max_depth, int32_t vocab,
                           const int32_t* tree_tokens, const int32_t* tree_parent, const int32_t* tree_depth,
                           const int32_t* n_nodes, const void* logits, int32_t logits_dtype,
                           int64_t logits_row_stride, int32_t* n_accept, int32_t* accept_nodes,
                           int32_t* out_tokens, int32_t* target_ids_out, void* stream);

/*
 * Canonical view of one sequence's table, for checkpointing and for comparing table contents:
 * leaders least recently used first, each leader's followers least recently inserted first.
 * HOST buffers: leaders int32 [LC, LL], n_followers int32 [LC], followers int32 [LC, FC, FL]
 * (unused follower slots -1); any of them may be NULL.  *n_leaders receives the count.  Synchronises.
 */
cb_status cb_table_dump(cb_ctx* ctx, int32_t seq, int32_t* n_leaders, int32_t* leaders,
                        int32_t* n_followers, int32_t* followers);

/* Replaces one sequence's table by the given canonical content (same HOST layouts as cb_table_dump;
 * recency = position). Synchronises. */
cb_status cb_table_load(cb_ctx* ctx, int32_t seq, int32_t n_leaders, const int32_t* leaders,
                        const int32_t* n_followers, const int32_t* followers);

/*
 * Reads (and clears) the device status word and copies the counters to the HOST array `counters`
 * (CB_NUM_COUNTERS entries, may be NULL).  Synchronises.
 */
enum {
    CB_CNT_INSERTS = 0,
    CB_CNT_LEADER_EVICTIONS = 1,
    CB_CNT_FOLLOWER_EVICTIONS = 2,
    CB_CNT_QUERIES = 3,
    CB_CNT_QUERY_HITS = 4,
    CB_CNT_MAX_PROBE = 5,
    CB_CNT_FROZEN_QUERIES = 6,
    CB_CNT_FROZEN_HITS = 7,
    CB_NUM_COUNTERS = 8
};
cb_status cb_poll_status(cb_ctx* ctx, cb_status* device_status, uint64_t* counters);

/*
 * 1 if this library is the checking build (compiled with -DCB_DEBUG), else 0.  No counterpart in the paper: the checking
 * build is the stand-in for a memory checker.  In it every table slot, entry id, page id and node index that a kernel takes
 * from memory is range-checked before use (a value out of range records CB_ERR_INVALID_ARG in the device status and the
 * access is skipped; nothing traps), and every workspace region is followed by 256 guard bytes that cb_poll_status verifies
 * (CB_ERR_CANARY if one changed).  cb_workspace_bytes is larger in that build.  Results are identical to the regular build.
 */
int cb_debug_build(void);

/* Kernels launched by this library since the process started (host-side count). */
uint64_t cb_launch_count(void);

const char* cb_status_str(cb_status s);

#ifdef __cplusplus
}
#endif
#endif /* CACHEBACK_H_ */
