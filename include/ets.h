/*
 * ets.h - C ABI of the tree-decode attention library for prefix-shared paged KV.
 *
 * Problem statement (paper: "ETS: Efficient Tree Search for Inference-Time Scaling",
 * arXiv 2502.13575).  A PRM-guided search keeps a tree of reasoning-step nodes; a
 * trajectory is a root-to-leaf path, and trajectories that pass through the same node
 * share that node's KV cache (Section 4.1; Appendix B, the node/leaf formulation of
 * Eq. 5).  Decoding is memory-bandwidth bound and its cost is the KV that must be loaded
 * per step (Sections 1 and 3); turning KV sharing into fewer loads needs an attention
 * kernel that reads each shared segment once (Section 3, item 1).  This library is that
 * step: every live leaf issues one grouped-query decode query, and its attention spans
 * the concatenated K/V of its root-to-leaf path,
 *
 *     out[l,a,:] = sum_t softmax_t( sm_scale * <q[l,a,:], K_l[t, a/G, :]> ) * V_l[t, a/G, :]
 *     lse[l,a]   = log sum_t exp( sm_scale * <q[l,a,:], K_l[t, a/G, :]> )
 *
 * with G = num_q_heads / num_kv_heads, no mask and no positional transform, while the
 * tree's unique K/V is streamed from device memory once per (node, kv head), not once
 * per leaf.  The paper itself ships no kernel and prints no attention formula; the
 * formula above is textbook softmax attention.
 *
 * Conventions
 *   - Every function returns an int32 status: ETS_OK or a negative ETS_ERR_* code.
 *     Nothing throws, aborts or traps the device.  ets_last_error() gives a message.
 *   - A failed call leaves the context as it was before the call.
 *   - "HOST" / "DEVICE" below says where a pointer must point.  The library never takes
 *     ownership of caller memory and never allocates device memory after ets_create.
 *   - All device work is enqueued on the cuda_stream argument (a cudaStream_t passed as
 *     void*; NULL = the legacy default stream).  Calls on one context must be issued from
 *     one host thread at a time and, if several streams are used, ordered by the caller.
 *   - bf16 tensors are dense, row-major, innermost index last.
 */
#ifndef ETS_H_
#define ETS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ETS_OK                   0
#define ETS_ERR_INVALID_ARG     -1  /* null pointer, negative size, index out of range      */
#define ETS_ERR_BAD_TREE        -2  /* parent/leaf arrays do not describe a valid forest    */
#define ETS_ERR_POOL_EXHAUSTED  -3  /* not enough pages, or a workspace bound was exceeded  */
#define ETS_ERR_UNSUPPORTED     -4  /* geometry the kernels do not cover                    */
#define ETS_ERR_STATE           -5  /* call order: no tree yet, host-only context, ...      */
#define ETS_ERR_CUDA            -6  /* a CUDA runtime call failed                           */
#define ETS_ERR_DEVICE_TIMEOUT  -7  /* a bounded device-side wait ran out                   */

typedef struct ets_ctx ets_ctx; /* opaque, library-owned */

/* Geometry and capacity bounds, fixed for the life of a context. */
typedef struct ets_config {
    int32_t num_q_heads;        /* Hq; multiple of num_kv_heads; Hq/Hkv in {1,2,4,8,16}     */
    int32_t num_kv_heads;       /* Hkv                                                       */
    int32_t head_dim;           /* d: 64 or 128                                              */
    int32_t page_size;          /* tokens per page: 16                                       */
    int32_t num_layers;         /* independent K/V pools sharing one set of tables           */
    int32_t max_nodes;          /* bound on n_nodes of any tree                              */
    int32_t max_leaves;         /* bound on n_leaves of any tree                             */
    int32_t max_path_tokens;    /* bound on the token capacity summed along one path         */
    int64_t max_path_entries;   /* bound on the sum over leaves of nodes on their path       */
    int64_t pages_per_layer;    /* pool capacity in pages (same for every layer)             */
    int32_t max_append_tokens;  /* bound on tokens per ets_kv_append*_host call (0: leaves)  */
    int32_t device;             /* CUDA device ordinal; -1 = host-only context (tables only) */
    float   sm_scale;           /* 0 -> 1/sqrt(head_dim)                                     */
    int32_t flags;              /* reserved, must be 0                                       */
} ets_config;

/*
 * Byte sizes of the three caller-provided DEVICE buffers for a configuration: the two pool
 * buffers (called K pool and V pool for their sizes' sake; together they hold num_layers *
 * pages_per_layer pages of page_size tokens for all KV heads, bf16, in a layout private to the
 * library, which spreads the pages over both buffers and keeps a page's K and V next to each
 * other) and the workspace (tables, partial results, staging).  All three must be 1024-byte
 * aligned (cudaMalloc blocks are; a caching allocator may hand out small blocks on 512-byte
 * boundaries).  Pool contents need no initialisation.
 */
int32_t ets_pool_bytes(const ets_config* cfg, size_t* k_bytes, size_t* v_bytes,
                       size_t* workspace_bytes);

/*
 * Create a context over caller-owned DEVICE buffers that must outlive it.  With
 * cfg->device == -1 the three pointers may be NULL and only the host-side calls
 * (ets_tree_build, ets_tree_export, ets_work_export, ets_get_stats) are usable.
 */
int32_t ets_create(const ets_config* cfg, void* k_pool, void* v_pool, void* workspace,
                   ets_ctx** out);
int32_t ets_destroy(ets_ctx* ctx);

/*
 * Tree flatten (host).  Section 4.1: the tree of step nodes, whose shared nodes mean shared
 * KV; Section 2.2: shared KV segments are stored once and referenced.  Replaces the current
 * topology.
 *   parent[n_nodes]      HOST  parent index in [-1, i): -1 = a root, parents precede children
 *   cap_tokens[n_nodes]  HOST  tokens the node holds or will hold; it reserves
 *                              ceil(cap/page_size) pages
 *   keep_pages_of        HOST  nullable; keep_pages_of[i] = node index of the PREVIOUS build whose
 *                              pages, contents and length node i inherits (clipped to its new
 *                              capacity), or -1.  An old node may be named once.
 *   leaf_node[n_leaves]  HOST  node each live leaf sits at; may repeat, may be internal
 * Page rule (bit-exact, see ets_tree_export): free pages form a min-heap of ids; pages of
 * old nodes that nobody keeps are freed first; then nodes in index order take their kept pages
 * and pop the lowest free ids.  Every layer uses the same ids.
 * The tables are uploaded asynchronously on cuda_stream; decode/append calls that should see
 * the new tree must be ordered after it on that stream.
 * Errors: ETS_ERR_BAD_TREE, ETS_ERR_POOL_EXHAUSTED (pages or a config bound), ETS_ERR_INVALID_ARG.
 */
int32_t ets_tree_build(ets_ctx* ctx, int32_t n_nodes, const int32_t* parent,
                       const int32_t* cap_tokens, const int32_t* keep_pages_of,
                       int32_t n_leaves, const int32_t* leaf_node, void* cuda_stream);

/*
 * Flattened tables, for bit-exact checks.  Counts are always written; each non-NULL HOST
 * pointer receives the table (the caller sizes them from a first call with NULL pointers).
 *   node_page_off[n_nodes+1], page_ids[n_pages]         pages of each node, in token order
 *   node_leaf_off[n_nodes+1], node_leaves[n_group]      leaves below each node, ascending
 *   leaf_path_off[n_leaves+1], leaf_path[n_path]        path of each leaf, root first
 *   leaf_path_pos[n_path]                               leaf's position in that node's group
 *   node_depth[n_nodes], node_len[n_nodes]              depth (root 0), current token count
 */
typedef struct ets_tables_host {
    int32_t n_nodes, n_leaves;
    int64_t n_pages, n_group, n_path;
    int32_t *node_page_off, *page_ids, *node_leaf_off, *node_leaves;
    int32_t *leaf_path_off, *leaf_path, *leaf_path_pos, *node_depth, *node_len;
} ets_tables_host;
int32_t ets_tree_export(const ets_ctx* ctx, ets_tables_host* out);

/*
 * The private work decomposition, exported for invariant checks only (its content is an
 * implementation choice and may change): runs of chained nodes with one query group are
 * fused into segments; the page slots of a segment are cut into pieces, and a work item is one
 * (piece, kv head, leaf tile).  Items of narrow query groups (at most 16 rows) come first and form a
 * queue ordered longest piece first: resident warp w of the attention kernel takes item w and then
 * claims the following items one at a time.  Items of wide groups follow, one CTA each.
 *   unit[n_units*4]     per page slot: page id, node, first token index within the node, 0
 *   item[n_items*8]     unit_begin, unit_count, kv_head, leaf_list_begin (into node_leaves),
 *                       n_leaves_in_tile, partial_slot_of_first_leaf, segment id, flags
 *   leaf_slot_off[n_leaves*num_kv_heads+1], leaf_slots[n_leaf_slots]
 *                       partial slots to merge per (leaf, kv head)
 *   worker_off[n_workers+1]   first item of resident warp w: [worker_off[w], worker_off[w+1]), one
 *                       item or none; worker_off[n_workers] is also the number of narrow items
 *                       when that is below n_workers
 */
typedef struct ets_work_host {
    int64_t n_units, n_items, n_leaf_slots, n_partial_slots, n_workers;
    int32_t *unit, *item, *leaf_slot_off, *leaf_slots, *worker_off;
} ets_work_host;
int32_t ets_work_export(const ets_ctx* ctx, ets_work_host* out);

/*
 * KV append.  Section 1: each trajectory needs KV state for every token it has generated;
 * Section 3, item 3: KV of earlier steps is reused by later ones.  Appends n_new[i] tokens to
 * node node_id[i] of one layer (distinct nodes per call), growing its length there; fails with
 * ETS_ERR_POOL_EXHAUSTED if a node would exceed its cap_tokens.
 *   node_id[n_items], n_new[n_items]  HOST
 *   k_new, v_new   bf16 [sum(n_new), num_kv_heads, head_dim], items packed in order.
 *                  DEVICE for ets_kv_append; HOST for ets_kv_append_host (copied through a
 *                  staging area of max_append_tokens tokens; pinned memory makes the copy async)
 * Asynchronous on cuda_stream; host arrays may be reused when the call returns, k_new/v_new
 * after the stream has passed the call.
 */
int32_t ets_kv_append(ets_ctx* ctx, int32_t layer, int32_t n_items, const int32_t* node_id,
                      const int32_t* n_new, const void* k_new, const void* v_new,
                      void* cuda_stream);
int32_t ets_kv_append_host(ets_ctx* ctx, int32_t layer, int32_t n_items, const int32_t* node_id,
                           const int32_t* n_new, const void* k_new, const void* v_new,
                           void* cuda_stream);
/*
 * Token lengths are tracked per (layer, node): within one decode step layer l has already
 * received the new token while deeper layers have not, and each layer's attention must see
 * exactly its own tokens.  ets_tree_export reports layer 0; this reads any layer's lengths
 * into node_len[n_nodes] (HOST).
 */
int32_t ets_get_node_len(const ets_ctx* ctx, int32_t layer, int32_t* node_len);

/*
 * Tree-decode attention: node-partial attention over every (segment chunk, kv head, leaf tile)
 * followed by the log-sum-exp merge along each leaf's path (the formula at the top of this
 * file).
 *   q    bf16 [n_leaves, num_q_heads, head_dim]
 *   out  bf16 [n_leaves, num_q_heads, head_dim]   (fp32 result rounded to nearest even)
 *   lse  fp32 [n_leaves, num_q_heads], natural log; nullable
 * DEVICE pointers for ets_tree_attn_decode; HOST pointers for ets_tree_attn_decode_host, which
 * copies q in and out/lse back on library streams ordered after cuda_stream's work so far (the
 * results are valid once cuda_stream has passed the call; see ETS_OPT_HOST_PIPELINE for the relaxed form).  A leaf whose path holds no token yields zeros and lse = -inf.
 * Errors: ETS_ERR_STATE (no tree), ETS_ERR_INVALID_ARG, ETS_ERR_CUDA.
 */
int32_t ets_tree_attn_decode(ets_ctx* ctx, int32_t layer, const void* q, void* out, float* lse,
                             void* cuda_stream);
int32_t ets_tree_attn_decode_host(ets_ctx* ctx, int32_t layer, const void* q, void* out,
                                  float* lse, void* cuda_stream);

/*
 * One decode iteration of one layer in a single call (Section 1: every generated token adds KV state to
 * its trajectory; Section 3, item 3: later steps reuse it): the new token of live leaf l (row l of
 * k_new / v_new, bf16 [n_leaves, num_kv_heads, head_dim], DEVICE) is appended to the node the leaf
 * sits at, then tree-decode attention runs with q / out / lse as in ets_tree_attn_decode, so that
 * every query sees its own new token.  Lengths grow inside the capacity reserved by
 * ets_tree_build; no rebuild is needed between iterations.  Same as ets_kv_append with
 * (leaf_node, all ones) followed by ets_tree_attn_decode.
 * Errors: those of the two calls; in particular ETS_ERR_INVALID_ARG when two leaves sit at the
 * same node and ETS_ERR_POOL_EXHAUSTED when a node is full (nothing is appended then).
 */
int32_t ets_decode_step(ets_ctx* ctx, int32_t layer, const void* k_new, const void* v_new,
                        const void* q, void* out, float* lse, void* cuda_stream);
/*
 * For callers that capture ets_decode_step into a CUDA graph and replay it: a replay appends on the device
 * (the captured append reads the node lengths there), but the library's host-side record of the lengths,
 * which the capacity checks and the next ets_tree_build use, only saw the captured call.  Tell it that
 * `times` further decode steps of `layer` have run (host only, no launch).  Capture after one ordinary call
 * of the same step (the first call uploads the append's descriptor list), with ETS_OPT_OVERLAP_APPEND and
 * ETS_OPT_TIMING off; the caller keeps the replays inside cap_tokens (the device-side append refuses and
 * raises the status word otherwise).  Errors: ETS_ERR_POOL_EXHAUSTED if the count cannot have fitted.
 */
int32_t ets_note_decode_steps(ets_ctx* ctx, int32_t layer, int32_t times);

/* The same with HOST buffers (k_new, v_new, q in; out, lse back), copied through the workspace's staging
 * areas on the library's streams like ets_kv_append_host + ets_tree_attn_decode_host, in one call and
 * with one event for the three inputs.  With ETS_OPT_PACKED_INPUTS set, k_new, v_new and q that are
 * adjacent in host memory in this order (the output of a fused projection) travel in one copy.  Follows ETS_OPT_HOST_PIPELINE. */
int32_t ets_decode_step_host(ets_ctx* ctx, int32_t layer, const void* k_new, const void* v_new,
                             const void* q, void* out, float* lse, void* cuda_stream);

/*
 * The same for n_layers consecutive layers in one call, for callers that hold all layers' inputs of a decode
 * iteration in host memory (a host-to-device copy of tens of MiB runs at about twice the rate of one of a few MiB):
 *   inputs  HOST bf16, ONE allocation: n_layers records, record j = [k_new | v_new | q] of layer first_layer + j,
 *           each part shaped as in ets_decode_step, the parts and the records packed without gaps
 *   out     HOST bf16 [n_layers, n_leaves, num_q_heads, head_dim];  lse  HOST fp32 [n_layers, n_leaves, num_q_heads], nullable
 * The inputs of up to four layers travel in one copy, their kernels run back to back, their outputs return in one
 * copy, and groups of layers alternate between two staging areas.  Follows ETS_OPT_HOST_PIPELINE like the other
 * *_host calls.  All capacity checks are made before anything is launched.
 */
int32_t ets_decode_step_host_layers(ets_ctx* ctx, int32_t first_layer, int32_t n_layers, const void* inputs,
                                    void* out, float* lse, void* cuda_stream);

/*
 * Attention of the tokens of newly generated steps: what prefilling a step, or scoring it with the
 * reward model, computes (Section 5.1: every new step is scored by a PRM; Section 4.1: the steps of a
 * trajectory share their ancestors' KV).  Every query token is a "leaf" sitting at its step's node
 * (ets_tree_build accepts many leaves on one node): it attends to all tokens of the node's ancestors
 * and to the first leaf_limit[l] tokens of its own node, i.e. causally inside the step.  For the j-th of
 * T new tokens of a node that now holds len tokens, leaf_limit = len - T + j + 1; with leaf_limit =
 * len the call equals ets_tree_attn_decode.  The step's K/V must have been appended before.
 *   q, out, lse   as in ets_tree_attn_decode, one row per leaf (DEVICE)
 *   leaf_limit    DEVICE int32 [n_leaves]; values are clipped to [0, current length of the node]
 * Query groups of more than 16 rows (leaves * Hq/Hkv) that the last build classed as wide run on the
 * tcgen05 kernel, the rest on the scalar kernel: build the tree with ETS_OPT_WIDE set to 17 so that every
 * dense group takes the tensor cores, or with ETS_OPT_PATH_ITEMS (faster: one item per tile and path).  A query that sees no token yields zeros and lse = -inf.
 * Errors: as ets_tree_attn_decode.
 */
int32_t ets_tree_attn_prefill(ets_ctx* ctx, int32_t layer, const void* q, const int32_t* leaf_limit,
                              void* out, float* lse, void* cuda_stream);

/*
 * Tree-decode attention for callers that cannot allocate device memory (the paper has no
 * counterpart: this is a packaging convenience, not a step of the method).  Same arguments,
 * result and errors as ets_tree_attn_decode (DEVICE pointers), but the partial results between
 * the attention and merge kernels live in an 8 MiB array built into the library instead of the
 * caller's workspace.  Meant for embedders whose host application owns the memory budget or
 * forbids allocation calls on its hot path (a cudaMalloc may synchronise the device).
 *   - Limit: with rows = partial_slots * (Hq/Hkv) (see ets_get_stats), rows * 8 bytes rounded up to a
 *     multiple of 256, plus rows * head_dim * 4 bytes, must fit in 8 MiB; larger trees are refused
 *     with ETS_ERR_POOL_EXHAUSTED and a message.  ETS_OPT_TIMING is ignored by this call.
 *   - The first call on each device looks up the array's device address; make it before starting
 *     any stream capture.  The call itself makes no allocation of any kind.
 *   - One array per GPU, shared by every call and context: calls that overlap in time on the
 *     same GPU corrupt each other.  The array keeps old contents between calls; none of it needs
 *     clearing, because each call rewrites every slot it later reads.
 */
int32_t ets_tree_attn_decode_static(ets_ctx* ctx, int32_t layer, const void* q, void* out, float* lse,
                                    void* cuda_stream);

/*
 * Read one node's current K and V rows of one layer back in token order:
 * bf16 [node_len, num_kv_heads, head_dim] each, DEVICE pointers (either may be NULL).
 */
int32_t ets_kv_read_debug(ets_ctx* ctx, int32_t layer, int32_t node, void* k_out, void* v_out,
                          void* cuda_stream);

/*
 * Selection step of the search (host only, no context needed).  Section 4 and Appendix B: from the
 * rewards of the live trajectories compute the REBASE weights W_i (Eq. 1: highest reward first,
 * W_i = ceil(N_i exp(R_i / T_R) / sum over the trajectories not served yet), N_1 = width and
 * N_{i+1} = N_i - W_i), then keep the set S of trajectories that maximises Eq. 4,
 *     sum_{i in S} W_i / sum_i W_i  -  lambda_b |V_S| / |V_A|  +  lambda_d |C_S| / |C_A|,    |S| >= 1,
 * where V_S are the nodes with a kept trajectory at or below them, V_A all n_nodes nodes, C_S the
 * clusters with a kept member and C_A all clusters (a cluster counts once any member is kept, as the
 * text of Appendix B.2 says), and finally hand the width out again over the kept trajectories
 * (Eq. 3).  The maximiser is found exactly by branch and bound over the tree (the paper calls a
 * general ILP solver); among equal optima the choice is unspecified.
 *   parent[n_nodes], leaf_node[n_leaves]   HOST, as in ets_tree_build: trajectory i ends at leaf_node[i]
 *   reward[n_leaves]                       HOST fp64, finite
 *   cluster[n_leaves]                      HOST, nullable: cluster label of each trajectory, negative = none
 *   weight, keep, continuations [n_leaves], node_kept [n_nodes]   HOST outputs, each nullable:
 *                                          W_i, 0/1, W'_i (0 where pruned), 0/1 per node of the tree
 *   result->proven_optimal                 0 when params->node_limit (0 = 2^20 search nodes) ran out:
 *                                          `keep` is then the best set found
 * Errors: ETS_ERR_INVALID_ARG (null array, width <= 0, temperature <= 0, negative lambda, non-finite
 * reward), ETS_ERR_BAD_TREE.
 */
typedef struct ets_select_params {
    double temperature, lambda_b, lambda_d;
    int32_t width, reserved;
    int64_t node_limit;
    const int32_t* node_tokens;   /* HOST, nullable: tokens held by each node, for the KV-size figures below */
} ets_select_params;
typedef struct ets_select_result {
    double objective;
    int64_t nodes_explored;
    int32_t proven_optimal, n_kept, n_nodes_kept, reserved;
    /* "KV size" of Section 3 for this step, when params->node_tokens is given (else 0): tokens held by the    */
    /* nodes of the retained tree V_S, and by all nodes that have a trajectory at or below them                */
    int64_t kv_tokens_kept, kv_tokens_all;
} ets_select_result;
int32_t ets_select(int32_t n_nodes, const int32_t* parent, int32_t n_leaves, const int32_t* leaf_node,
                   const double* reward, const int32_t* cluster, const ets_select_params* params,
                   int32_t* weight, int32_t* keep, int32_t* continuations, int32_t* node_kept,
                   ets_select_result* result);

/* Counters of the current tree.  "KV size" follows Section 3: the unique KV state of the tree. */
typedef struct ets_stats {
    int64_t n_nodes, n_leaves;
    int64_t unique_tokens;      /* sum over nodes of current length (layer 0)                */
    int64_t unique_kv_bytes;    /* unique_tokens * 2 * Hkv * d * 2, one layer                */
    int64_t path_tokens;        /* sum over leaves of tokens on their path: what a kernel    */
                                /* without prefix sharing would read                         */
    int64_t pages_used, pages_free;
    int64_t n_segments, n_chunks, n_items, n_units, n_partial_slots;
    int64_t attended_tokens;    /* current tokens of nodes that have a leaf below them       */
    int64_t n_narrow_items;     /* items of narrow query groups (the first ones in the list) */
} ets_stats;
int32_t ets_get_stats(const ets_ctx* ctx, ets_stats* out);

/* Tuning and instrumentation knobs; unknown keys give ETS_ERR_INVALID_ARG. */
#define ETS_OPT_CHUNK_PAGES   1  /* longest page run per work item (0 = no limit); next build    */
#define ETS_OPT_KERNEL        2  /* 0 tensor-core attention kernels (default), 1 scalar-FMA kernel;  */
                                 /* rebuild the tree after changing it                             */
#define ETS_OPT_WIDE          4  /* smallest query group, in rows (leaves * Hq/Hkv, at least 17), that */
                                 /* goes to the tcgen05 kernel (default 33); 0: none.  Next build.      */
                                 /* While the option is untouched, a tree so small that a warp of the    */
                                 /* streaming kernel would read four page slots or fewer gets no such    */
                                 /* items (the second kernel's launch costs more than it saves there),   */
                                 /* and a tree on which the tcgen05 kernel would end after the streaming */
                                 /* kernel (most of its K/V under large query groups) is built with 49.  */
#define ETS_OPT_PATH_ITEMS    7  /* 1: the next builds serve ets_tree_attn_prefill only: a work item is one   */
                                 /* (node that leaves sit at, kv head, tile of its leaves) and walks the node's */
                                 /* whole path, so a dense tile keeps its accumulator resident and leaves one  */
                                 /* partial per row; the decode entry points then return ETS_ERR_STATE         */
#define ETS_OPT_OVERLAP_APPEND 8 /* 1: ets_kv_append / ets_decode_step may start their append while the kernel    */
                                 /* before it in the stream is still running, if that kernel signals early    */
                                 /* (programmatic dependent launch; the library's merge kernel does, so in a   */
                                 /* loop over layers the append runs under the previous call's merge).  Only   */
                                 /* for callers whose k_new / v_new are complete when the call is made: not    */
                                 /* when the kernel that writes them is the one before the call in the stream   */
                                 /* and signals early itself.  Default 0.                                      */
#define ETS_OPT_PACKED_INPUTS 9  /* 1: the caller promises that whenever k_new, v_new and q of ets_decode_step_host  */
                                 /* are adjacent in this order they lie in ONE host allocation, so one copy may  */
                                 /* span them (two pinned allocations that merely touch must not be copied as    */
                                 /* one).  Default 0: three copies.                                             */
#define ETS_OPT_HOST_PIPELINE 6  /* 1: the *_host calls return without making cuda_stream wait for   */
                                 /* them, so the copies of one call overlap the kernels of the next;   */
                                 /* results are valid after ets_host_join + synchronising that stream;  */
                                 /* the calls are ordered after cuda_stream's work only as of the first */
                                 /* *_host call following a join                                        */
#define ETS_OPT_TIMING        3  /* 1: bracket the attention and merge kernels with events (ets_timing_read);   */
                                 /* 2: the kernels record device time stamps instead (ets_stamps_read), which  */
                                 /* leaves the launches chained as they are; 0: neither                        */
#define ETS_OPT_LAUNCH_CHAIN 10  /* 1 (default): the kernels of a call go to cuda_stream as a chain of programmatic  */
                                 /* dependent launches: each may become resident and run its set-up (barriers,      */
                                 /* table reads) under the tail of the one before, and waits for it before it       */
                                 /* touches anything that kernel writes; the tcgen05 kernel runs beside the          */
                                 /* streaming kernel on the same stream.  Every kernel waits for its predecessor     */
                                 /* before it ends, so work queued behind a call is ordered behind all of it.        */
                                 /* 0: ordinary launches, the tcgen05 kernel on a library stream forked from and     */
                                 /* joined into cuda_stream.                                                         */
#define ETS_OPT_TEST_FIRST_WAIT_POLLS 11 /* for tests of the time-out path: number of polls after which the FIRST   */
                                 /* wait for data of every worker of the attention kernels gives up (0: at once);   */
                                 /* the worker then raises ETS_ERR_DEVICE_TIMEOUT (ets_poll_status), starts nothing  */
                                 /* new, waits with the ordinary bound for the copies it had started, and returns;   */
                                 /* that call's outputs are undefined.  Negative: the ordinary bound (default).      */
int32_t ets_set_option(ets_ctx* ctx, int32_t key, int64_t value);

/*
 * With ETS_OPT_HOST_PIPELINE on: makes cuda_stream wait for every ets_kv_append_host /
 * ets_tree_attn_decode_host call issued so far (their kernels and their copies back to the host).
 * Any other device-side call on the context (tree build, device-pointer append/decode, status poll)
 * joins implicitly first.  Without the option every *_host call joins by itself.
 */
int32_t ets_host_join(ets_ctx* ctx, void* cuda_stream);

/* With ETS_OPT_TIMING on: waits for the recorded events, returns and clears the sums. */
int32_t ets_timing_read(ets_ctx* ctx, double* attn_ms, double* merge_ms, int64_t* n_calls);

/*
 * With ETS_OPT_TIMING = 2: per kind of kernel (0 append, 1 streaming attention, 2 tcgen05 attention, 3 merge, 4 the
 * moment the streaming kernel's wait for the kernel ahead of it returned) and launch since the last read, the
 * earliest start and the latest end over the kernel's CTAs on the GPU's global nanosecond timer.  count[k] launches
 * of kind k were recorded (at most ETS_STAMP_LAUNCHES; further ones are dropped).  Synchronises the device, copies
 * the table to `out` (HOST) and clears it.  Launches captured into a CUDA graph record stamps if the option was on
 * at capture time.  A measurement aid: the paper has no counterpart.
 */
#define ETS_STAMP_KINDS 5
#define ETS_STAMP_LAUNCHES 4096
typedef struct ets_stamps_host {
    uint32_t count[8];
    uint32_t reserved[8];
    uint64_t start_ns[ETS_STAMP_KINDS][ETS_STAMP_LAUNCHES];
    uint64_t end_ns[ETS_STAMP_KINDS][ETS_STAMP_LAUNCHES];
} ets_stamps_host;
int32_t ets_stamps_read(ets_ctx* ctx, ets_stamps_host* out);

/*
 * Synchronise cuda_stream and report the device-side status word: ETS_OK, or
 * ETS_ERR_DEVICE_TIMEOUT / ETS_ERR_INVALID_ARG if a kernel gave up on a bounded wait or
 * skipped an out-of-range table entry.  Clears the word.
 */
int32_t ets_poll_status(ets_ctx* ctx, void* cuda_stream);

/*
 * Measurement probes (the paper has no counterpart; bench.py reports them beside the attention numbers).
 * ets_probe_stream_read: a persistent kernel with the streaming attention kernel's data path and no
 * arithmetic reads `bytes` of `buf` (DEVICE, 1024-byte aligned) once: n_ctas CTAs of 8 warps, every warp
 * keeping `depth` (1..8) linear bulk copies of chunk_bytes (a multiple of 1024) in flight into shared
 * memory (8 * depth * chunk_bytes must fit in 227 KiB).  Timed by the caller with events on cuda_stream.
 * ets_probe_empty_launch: a kernel that does nothing, n_ctas CTAs of 256 threads with smem_bytes of
 * dynamic shared memory: what a launch of that shape costs.
 *   scratch   DEVICE, 8 KiB, 16-byte aligned, zeroed by the caller; the int32 at byte 4096 is set to
 *             ETS_ERR_DEVICE_TIMEOUT if a bounded wait of the probe ran out
 * Asynchronous.  Errors: ETS_ERR_INVALID_ARG, ETS_ERR_CUDA.
 */
int32_t ets_probe_stream_read(const void* buf, size_t bytes, int32_t chunk_bytes, int32_t depth,
                              int32_t n_ctas, void* scratch, void* cuda_stream);
int32_t ets_probe_empty_launch(int32_t n_ctas, size_t smem_bytes, void* scratch, void* cuda_stream);

const char* ets_last_error(const ets_ctx* ctx);
const char* ets_version(void);

#ifdef __cplusplus
}
#endif
#endif /* ETS_H_ */
