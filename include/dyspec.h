/*
 * dyspec.h -- C ABI of the B200 (sm_100a) tree-verify attention library.
 *
 * The library implements the hot path of one DySpec decoding step: the target model's
 * verification pass over a draft token tree (paper Sec. 2, "Speculative Decoding" and
 * "Tree Attention"; App. C "Efficiency of Optimized Tree Attention").  Every tree node is a
 * query; it attends to the whole prefix KV cache plus the tree rows of its ancestors and itself.
 *
 * Conventions shared by all calls
 *   - Every function returns an int: DYSPEC_OK (0) or a negative DYSPEC_ERR_* code.  Nothing
 *     throws, aborts or traps.  Errors the host can see (NULL pointers, unsupported shapes, small
 *     workspace, misaligned pointers) are returned before anything is launched.
 *   - Pointers marked "dev" are CUDA device pointers of the current device; pointers marked
 *     "host" are ordinary host pointers that are only read during the call.
 *   - The caller owns every buffer.  Attention and mask calls enqueue kernels on `stream` and
 *     return without synchronising; the caller's buffers must stay alive until the stream reaches
 *     them.  Plan creation/destruction are the only calls that allocate or free device memory.
 *   - Conditions only the device can see (a parent index that is not in {-1} U [0, i); a bounded
 *     wait that ran out) store a non-zero DYSPEC_ERR_* code into the optional `status` word (dev
 *     int32, the caller zeroes it) and the kernel still completes normally.
 *   - bf16 tensors are passed as `const void*`; layouts are row-major with the last index fastest.
 *   - Stream order.  Kernels are launched with programmatic stream serialisation: a kernel may start
 *     while the kernel before it in the stream is finishing, and it reads and processes its pure
 *     inputs (parents, q, k_cache, v_cache, page_table: the attention kernels work through the prefix
 *     keys) before it waits for that kernel; everything it writes, and the mask and tile sets it reads,
 *     it touches only after the wait.  Inputs written by ordinary kernels or copies earlier in
 *     the stream are safe (without an early-launch signal the stream serialises fully, as always),
 *     and so is every sequence of this library's own calls.  The one thing to avoid is producing
 *     those inputs with a foreign kernel that itself signals early launch of its dependents
 *     (griddepcontrol.launch_dependents) directly before a call of this library.
 *
 * Packed rows: ancestor_bits[i][w], w < words_per_row, has bit b (LSB = bit 0) set iff tree node
 * 32*w + b is node i itself or an ancestor of node i (Sec. 2, the mask(A) equation, plus the self
 * bit of causal attention).  Unused bits are zero.  words_per_row is a multiple of 4 (16-byte rows).
 */
#ifndef DYSPEC_H_
#define DYSPEC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct CUstream_st* dyspec_stream_t; /* a cudaStream_t */

enum {
  DYSPEC_OK = 0,
  DYSPEC_ERR_INVALID_ARG = -1, /* NULL / negative / inconsistent argument */
  DYSPEC_ERR_UNSUPPORTED = -2, /* shape outside the supported set (see dyspec_plan_create) */
  DYSPEC_ERR_WORKSPACE = -3,   /* workspace smaller than dyspec_plan_workspace_bytes, or misaligned */
  DYSPEC_ERR_CUDA = -4,        /* a CUDA runtime / driver call failed (launch, tensor-map encode, alloc) */
  DYSPEC_ERR_BAD_TREE = -5,    /* device-detected: some parents[i] outside {-1} U [0, i) */
  DYSPEC_ERR_TIMEOUT = -6      /* device-detected: a bounded in-kernel wait ran out */
};

#define DYSPEC_MAX_NODES 2048 /* largest tree per request (the paper's largest real tree is 768, Sec. 5 / App. B;
                                 its random-tree experiment goes up to 2048, App. C.1, Table 5) */

/* Static, never-freed description of an error code. */
const char* dyspec_error_string(int code);

/* Library version, major*10000 + minor*100 + patch. */
int dyspec_version(void);

/* Smallest legal words_per_row for trees of up to max_nodes nodes: 4*ceil(max_nodes/128); <0 on bad input. */
int dyspec_words_per_row(int max_nodes);

/*
 * (1) Mask builder, single request (Sec. 2, mask(A): "i is ancestor of j").
 *   parents        dev  int32 [n_nodes]   parents[i] = -1 (a root) or an index < i
 *   ancestor_bits  dev  uint32 [n_nodes][words_per_row]  (written; 16-byte aligned)
 *   depths         dev  int32 [n_nodes] or NULL           (written: number of ancestors)
 *   status         dev  int32 [1] or NULL                 (DYSPEC_ERR_BAD_TREE stored on a bad parent;
 *                                                          such a node is treated as a root)
 * n_nodes = 0 is a no-op.  n_nodes > DYSPEC_MAX_NODES or 32*words_per_row < n_nodes is rejected.
 */
int dyspec_build_tree_mask(const int32_t* parents, int n_nodes, uint32_t* ancestor_bits, int32_t* depths,
                           int words_per_row, int32_t* status, dyspec_stream_t stream);

/*
 * (1a) The same for a ragged batch without a plan: node_offsets is a HOST array [n_req + 1] (prefix sums
 * of the tree sizes), parents are request-local indices, concatenated; request r's mask rows and depths
 * start at node_offsets[r]; every row uses the same words_per_row.  status: dev int32 [n_req] or NULL (one
 * word per request).  The request list travels with the launch (kernel parameters): one launch per 768
 * requests, nothing allocated, no host pointer kept.
 */
int dyspec_build_tree_mask_batched(const int32_t* parents, const int32_t* node_offsets_host, int n_req,
                                   uint32_t* ancestor_bits, int32_t* depths, int words_per_row, int32_t* status,
                                   dyspec_stream_t stream);

/*
 * (2) Plans.  A plan fixes the static shape and the ragged batch structure, runs the host-side
 * scheduler (work list of (request, kv-head, query-tile, kv-split) items balanced over the SMs)
 * and owns a small device copy of that list.  Create it once per batch structure; reuse it for
 * every layer and step with the same (prefix_len, n_nodes).  A plan belongs to the CUDA device that
 * is current when it is created: the attention calls return DYSPEC_ERR_INVALID_ARG when another
 * device is current.
 *
 *   n_q_heads, n_kv_heads  H_q, H_kv; group g = H_q / H_kv must be 1, 2, 4 or 8
 *   head_dim               64 or 128
 *   n_req                  number of requests (>= 0)
 *   prefix_len   host int32 [n_req]   L_r >= 0
 *   n_nodes      host int32 [n_req]   0 <= n_r <= DYSPEC_MAX_NODES
 *   kv_row_offset host int64 [n_req]  row of request r's token 0 in k_cache / v_cache; request r
 *                                     occupies rows off_r .. off_r + L_r + n_r - 1: prefix rows first,
 *                                     then one row per tree node in node order
 *   kv_total_rows          number of rows of k_cache / v_cache (>= every off_r + L_r + n_r)
 *   words_per_row          row stride of ancestor_bits, a multiple of 4 with 32*W >= max n_r and
 *                          W <= DYSPEC_MAX_NODES / 32
 *   scale                  softmax scale; <= 0 selects 1/sqrt(head_dim)
 * Query/output rows of request r start at node_offset_r = n_0 + ... + n_{r-1}; so do its mask rows
 * and parents.
 */
typedef struct dyspec_plan dyspec_plan_t;

int dyspec_plan_create(dyspec_plan_t** plan, int n_q_heads, int n_kv_heads, int head_dim, int n_req,
                       const int32_t* prefix_len, const int32_t* n_nodes, const int64_t* kv_row_offset,
                       int64_t kv_total_rows, int words_per_row, float scale);
int dyspec_plan_destroy(dyspec_plan_t* plan);

/* Bytes of scratch the attention call needs (split-KV partials, the words of the shared work queue); may
 * be 0.  The caller zeroes the workspace once, before its first use. */
size_t dyspec_plan_workspace_bytes(const dyspec_plan_t* plan);

/* Scheduler introspection (for tests and benchmarks): field 0 = work items, 1 = CTAs launched,
 * 2 = query-tile groups, 3 = groups that are split, 4 = max splits of a group, 5 = kernel regime
 * (0 = 64-row tiles for small trees, 1 = 2 x 128-row tcgen05 tiles), 6 = total key tiles, 7 = query rows per tile,
 * 8 = thread-block cluster size (1 = no clusters), 9 = 1 when the CTAs take whole groups from a shared
 * queue on the device instead of fixed lists (the item list then shows the nominal assignment), 10 = 1 when
 * split groups are merged by a separate combine launch (0: no split groups, or they are merged on chip or
 * inside the attention kernel). */
int64_t dyspec_plan_info(const dyspec_plan_t* plan, int field);

/* Host-only view of the scheduler, for tests and tools: validates the arguments and schedules exactly
 * as dyspec_plan_create does (requests packed back to back in the cache) but makes no CUDA call.
 * Copies up to max_items work items into items_out (host, 8 int32 each: request, kv head, first
 * packed query row, first key tile, one-past-last key tile, partial slot or -1, group id, number of
 * splits of the group), the per-CTA item ranges into cta_begin_out (host, n_ctas + 1 entries, at most
 * max_ctas) and, into info_out (host int64 [12]), dyspec_plan_info fields 0-7 followed by keys per
 * tile, workspace bytes, the cluster size and dyspec_plan_info field 10.  Any output pointer may be NULL.  Returns the item count or an error. */
int dyspec_schedule_dry_run(int n_q_heads, int n_kv_heads, int head_dim, int n_req, const int32_t* prefix_len,
                            const int32_t* n_nodes, int words_per_row, int32_t* items_out, int max_items,
                            int32_t* cta_begin_out, int max_ctas, int64_t* info_out);

/* Testing knobs, process-wide; a plan keeps the values it was created with: force the regime (-1 = automatic), the number of
 * CTAs the scheduler balances over (0 = automatic; a negative value -c instead sets the scheduler's
 * per-item cost to c key tiles), and combine_mode = m + 16 k.  m says how split-KV partials are merged:
 * 0 = by the separate combine kernel, 2 (default) = without a combine launch where the plan allows: inside a
 * thread-block cluster per group when the plan is uniform enough (few groups of similar length; small-tile
 * regime: through distributed shared memory, no workspace; tcgen05 regime: the partials travel through the
 * workspace and the cluster's hardware barrier stands in for counters and polling), else in the tcgen05
 * regime by the split items themselves inside the attention kernel, with arrival counters in the workspace,
 * when the grid is one wave; else as 0.  1 = as 2, but the tcgen05 regime never uses clusters.  (Items that
 * wait for arrival counters do so inside the kernel, bounded to one second: this assumes that the process may
 * use every SM of the device it counted.  Where it may not -- a reduced SM share under MPS, a green context --
 * create the plans with m = 0.  The CTAs of a cluster are scheduled together by the hardware: no such
 * assumption there; where the device cannot hold even one cluster of the planned size, the plan falls back
 * to the counters.)  k says whether the scheduler may deal whole
 * (unsplit) groups to the CTAs instead of cutting them to equal budgets: 0 (default) = when its cost
 * model says that is quicker (and force_ctas is 0), 1 = never, 2 = always. */
int dyspec_set_tuning(int force_regime, int force_ctas, int combine_mode);

/* Developer aid: event trace of the attention kernels.  The hooks are compiled out of the ordinary
 * library (even never-taken checks in the MMA-issuing and softmax loops cost the tensor-core kernel
 * 8 - 10 %): build with DYSPEC_NVCC_FLAGS="-DDYSPEC_TRACE" (event trace) and / or "-DDYSPEC_CTA_STAMPS"
 * (per-CTA wall-clock stamps); in an ordinary build a non-NULL buffer is refused with
 * DYSPEC_ERR_UNSUPPORTED.  trace_buffer is a dev uint64 array of capacity_entries entries that the
 * caller zeroes; while set, CTA 0 of every tensor-core attention launch writes (tag << 44 | SM clock)
 * entries into three equal regions (MMA issuer, softmax half A, softmax half B; tags are listed in
 * csrc/attn_tc.cu; zero entries are unused).  When capacity_entries > 4096 the last 2048 entries are
 * not part of those regions: there each of the first 256 CTAs of an attention launch leaves 8
 * wall-clock stamps (globaltimer, ns) of its phases, listed where the kernels take them.  Pass
 * (NULL, 0) to switch it off (the default). */
int dyspec_set_trace(void* trace_buffer, int capacity_entries);

/*
 * (1b) Mask builder for the whole ragged batch of a plan: request r's parents (request-local
 * indices) start at node_offset_r, its mask rows and depths likewise.
 *   parents dev int32 [sum n_r]; ancestor_bits dev uint32 [sum n_r][W]; depths dev int32 [sum n_r] or NULL;
 *   status dev int32 [1] or NULL.
 */
int dyspec_plan_build_tree_mask(const dyspec_plan_t* plan, const int32_t* parents, uint32_t* ancestor_bits,
                                int32_t* depths, int32_t* status, dyspec_stream_t stream);

/*
 * (3) Tree-verify attention over a ragged batch (Sec. 2 "Tree Attention"; App. C: the prompt is
 * part of the mask, so prefix keys are visible to every node).  For request r, query head h,
 * node i:  out[i,h,:] = softmax_t(scale * <q[i,h,:], k[t,h/g,:]>) . v[t,h/g,:]  over
 * t in {prefix rows} U {tree rows of the nodes whose bit is set in ancestor_bits[i]}.
 * bf16 inputs, fp32 scores / softmax / accumulation, bf16 (round-to-nearest-even) output.
 *   q              dev bf16 [sum n_r][H_q][D]            (16-byte aligned)
 *   k_cache,v_cache dev bf16 [kv_total_rows][H_kv][D]    (16-byte aligned)
 *   ancestor_bits  dev uint32 [sum n_r][W]               (from the mask builder)
 *   out            dev bf16 [sum n_r][H_q][D]            (written)
 *   workspace      dev, >= dyspec_plan_workspace_bytes(plan), 256-byte aligned; it must be zero before the
 *                  first call (the caller zeroes it once; the kernels leave its counters zero).  Two
 *                  calls that overlap on the GPU need two workspaces (a workspace holds the split-KV
 *                  partials and words that a launch uses and clears: the arrival counters of the split
 *                  groups, the head of the plan's shared work queue); calls that follow each other on one stream may share one, and a
 *                  plan may be shared by any number of calls.
 *   status         dev int32 [1] or NULL
 */
int dyspec_tree_attention_ragged(const dyspec_plan_t* plan, const void* q, const void* k_cache, const void* v_cache,
                                 const uint32_t* ancestor_bits, void* out, void* workspace, size_t workspace_bytes,
                                 int32_t* status, dyspec_stream_t stream);

/*
 * (3b) Single-request convenience form.  The static shape comes from dyspec_set_default_shape.  The
 * library keeps, per device and static shape, a small bounded cache: the plans of the last 8
 * (prefix_len, n_nodes) pairs seen (all layers of a decoding step share one pair, so a step costs one
 * miss), their device tables in buffers that are reused when a plan is replaced, and one workspace sized
 * for the worst case of the shape (about 40 MB at head_dim 128).  The first eight misses of a shape
 * allocate those; after that a miss only runs the host scheduler and sends its tables down `stream` in kernel
 * parameters -- no allocation, no synchronisation -- unless a tree is large enough to outgrow a table
 * buffer (64 KB to start with), which replaces that buffer once.  dyspec_release_cache frees everything
 * (call it with no library work in flight).  k_cache / v_cache hold exactly prefix_len + n_nodes rows.
 * All calls of one shape share the workspace and the table buffers, so they must follow each other on
 * the GPU (one stream, or streams ordered by events); use the ragged form with workspaces of your own
 * for calls that may overlap.
 */
int dyspec_set_default_shape(int n_q_heads, int n_kv_heads, int head_dim, int words_per_row, float scale);
int dyspec_tree_attention(const void* q, const void* k_cache, const void* v_cache, int prefix_len,
                          const uint32_t* ancestor_bits, int n_nodes, void* out, dyspec_stream_t stream);
int dyspec_release_cache(void);

/*
 * (3c) Single-request attention that allocates nothing.  (The paper has no counterpart: this is an
 * integration aid, not part of the method.)
 *
 * Who needs it: code that may not call cudaMalloc / cudaFree at the point where it wants attention --
 * for instance an inference server whose device memory was handed, all of it, to its own pool at
 * start-up, a plug-in that runs under a host framework's "no allocation in the step function" rule,
 * or a process running so close to the memory limit that a late cudaMalloc could fail.  Such a
 * caller can build neither a plan (plan creation allocates its device work list) nor a workspace.
 *
 * Here the scheduled work list and the split-KV partials live in one fixed device array of
 * DYSPEC_STATIC_SCRATCH_BYTES that is part of the library image: every GPU that loads the library
 * holds those bytes until the process exits, whether or not this call is ever used.  The call runs
 * the host scheduler, writes the work list into the array on `stream` (the tables travel in kernel
 * parameters, so no host memory of the call is referred to after it returns and the stream is not
 * synchronised), and launches the same kernels as dyspec_tree_attention_ragged; it calls no cudaMalloc,
 * cudaFree or allocating routine.
 * Arguments are those of dyspec_tree_attention plus the static shape (see dyspec_plan_create) and an
 * optional status word; k_cache / v_cache hold exactly prefix_len + n_nodes rows.
 *
 *   - A batch whose work list plus partials exceed the array is refused with DYSPEC_ERR_WORKSPACE
 *     before anything is launched (as a guide: Llama2-70B shape, prefix 1500, 40 nodes needs 12.2 MiB;
 *     small uniform batches that merge their splits on chip need only a few KiB).
 *   - The first call on each device looks up the array's device address (with that device current), a
 *     synchronous call of the CUDA runtime; later calls on that device do not.
 *   - All calls share the one array, which keeps the previous call's contents; each call rewrites the
 *     tables and clears the counters it needs.  Calls on the same stream are ordered and safe.  Two
 *     calls that overlap on the GPU (different streams, or different host threads without ordering)
 *     race on the array and give wrong results.
 */
#define DYSPEC_STATIC_SCRATCH_BYTES (16u << 20)
int dyspec_tree_attention_static(const void* q, const void* k_cache, const void* v_cache, int prefix_len,
                                 const uint32_t* ancestor_bits, int n_nodes, void* out, int n_q_heads, int n_kv_heads,
                                 int head_dim, int words_per_row, float scale, int32_t* status, dyspec_stream_t stream);

/*
 * (4) Block-sparsity friendly token order (App. C; Table 5).  The paper renumbers the tree tokens in
 * depth-first order (an approximation of heavy-path order) so that the tree part of the attention
 * mask touches few b x b blocks, and lets the attention kernel skip the empty blocks.
 *
 * dyspec_dfs_reorder / dyspec_plan_dfs_reorder: pre-order numbering that visits roots, and the
 * children of every node, in increasing old index.
 *   parents      dev int32 [n]          as for the mask builder (ragged form: all requests, node order)
 *   order        dev int32 [n] or NULL  (written) order[k] = old index of the node whose new index is k
 *   new_of_old   dev int32 [n] or NULL  (written) inverse permutation
 *   new_parents  dev int32 [n] or NULL  (written) parent array in the new numbering; again
 *                                        new_parents[k] < k.  Must not alias parents.
 *   status       dev int32 [1] or NULL  DYSPEC_ERR_BAD_TREE on a bad parent (node treated as a root)
 * Indices are local to the request; request r's entries start at node_offset_r in every array.
 * The caller feeds the tree tokens to the model in the new order (token k = old token order[k]), so
 * Q rows and tree K/V rows arrive in that order, and builds the mask from new_parents.
 *
 * dyspec_build_tree_mask_tiles / dyspec_plan_build_tree_mask_tiles: the mask builder, which also
 * writes for every node which 64-column tiles of the tree its row touches:
 *   node_tiles   dev uint32 [n]  (written) bit t set iff the node or one of its ancestors has an
 *                                 index in [64 t, 64 t + 64)
 * dyspec_tree_attention_ragged_sparse: dyspec_tree_attention_ragged that skips the tree key tiles no
 * row of a query tile touches (node_tiles must come from the same parents as ancestor_bits; NULL
 * gives dyspec_tree_attention_ragged).  Results are those of the dense call up to the order of the
 * fp32 additions.  Only the tcgen05 regime skips tiles, and only for a query tile with at least three
 * tree key tiles besides the ones that hold its own nodes (those, which every row sees, run first, before
 * the tile sets are read); the small-tree regime, whose tree part is one or two key tiles, ignores
 * node_tiles.
 */
int dyspec_dfs_reorder(const int32_t* parents, int n_nodes, int32_t* order, int32_t* new_of_old, int32_t* new_parents,
                       int32_t* status, dyspec_stream_t stream);
int dyspec_plan_dfs_reorder(const dyspec_plan_t* plan, const int32_t* parents, int32_t* order, int32_t* new_of_old,
                            int32_t* new_parents, int32_t* status, dyspec_stream_t stream);
int dyspec_build_tree_mask_tiles(const int32_t* parents, int n_nodes, uint32_t* ancestor_bits, int32_t* depths,
                                 uint32_t* node_tiles, int words_per_row, int32_t* status, dyspec_stream_t stream);
int dyspec_plan_build_tree_mask_tiles(const dyspec_plan_t* plan, const int32_t* parents, uint32_t* ancestor_bits,
                                      int32_t* depths, uint32_t* node_tiles, int32_t* status, dyspec_stream_t stream);
/* The paper's workload measure for this optimisation (App. C.1, Table 5, "Block Count"): the number of
 * block x block tiles of one request's packed mask that hold a visible pair.  block = 32, 64 or 128;
 * count: dev uint64 [1] (written; cleared first, on `stream`). */
int dyspec_mask_block_count(const uint32_t* ancestor_bits, int n_nodes, int words_per_row, int block, uint64_t* count,
                            dyspec_stream_t stream);
int dyspec_tree_attention_ragged_sparse(const dyspec_plan_t* plan, const void* q, const void* k_cache,
                                        const void* v_cache, const uint32_t* ancestor_bits, const uint32_t* node_tiles,
                                        void* out, void* workspace, size_t workspace_bytes, int32_t* status,
                                        dyspec_stream_t stream);

/*
 * (5) Verification of the token tree (Algorithm 3: multi-branch rejection sampling along the tree), the
 * step that follows the tree attention.  For each request the walk starts at node 0; at a node it tries
 * the node's children in increasing index: child with token y is accepted when u <= R[y] / D[y]
 * (R starts as the target distribution at the node, D as the draft distribution there); after a
 * rejection R <- norm(max(R - D, 0)), D[y] <- 0, and the node is given up when D has become all zero,
 * else D <- norm(D).  When no child is accepted a token is drawn from R and the walk ends.  As the
 * paper prints it, a walk that reaches a leaf ends without a further token; bonus_at_leaf != 0 draws
 * the usual extra token from the target distribution at the leaf.  The paper prints the acceptance
 * number as N(0,1); it is read as U(0,1).  Random numbers are inputs.
 *
 *   parents, tokens   dev int32 [N]        N = node_offsets[n_req]; token carried by each node (root's unused)
 *   draft_probs       dev float [N][vocab] Draft(node, .): what the node's children were drawn from
 *   target_probs      dev float [N][vocab] Target(node, .)          (rows 16-byte aligned: vocab % 4 == 0)
 *   accept_u          dev float [N]        U(0,1) number used when that node is tried
 *   sample_u          dev float [N]        U(0,1) number used when a token is drawn at that node (inverse
 *                                          CDF in token order: first v with cumsum(R)[v] > u * sum(R))
 *   node_offsets      dev int32 [n_req+1]  request r owns nodes node_offsets[r] .. node_offsets[r+1]-1
 *   max_nodes         upper bound of the requests' node counts (<= DYSPEC_MAX_NODES); a request with more
 *                     nodes emits nothing (n_accepted = 0) and sets status DYSPEC_ERR_INVALID_ARG
 *   vocab             <= DYSPEC_MAX_VOCAB
 *   accepted_tokens   dev int32 [n_req][max_out]  (written) the emitted tokens, in order
 *   accepted_nodes    dev int32 [n_req][max_out]  (written) the accepted node of each, -1 for a drawn token
 *   n_accepted        dev int32 [n_req]           (written) how many (entries past max_out are dropped)
 *   status            DYSPEC_ERR_BAD_TREE on a bad parent, DYSPEC_ERR_INVALID_ARG on a token outside the vocabulary
 * Probabilities are fp32; decisions are taken in fp32 with sums in a different order from a
 * sequential implementation, so a decision whose deciding number lies within rounding of its
 * threshold may differ from another implementation's.
 */
#define DYSPEC_MAX_VOCAB 32768
int dyspec_verify_tree(const int32_t* parents, const int32_t* tokens, const float* draft_probs, const float* target_probs,
                       const float* accept_u, const float* sample_u, const int32_t* node_offsets, int n_req,
                       int max_nodes, int vocab, int bonus_at_leaf, int32_t* accepted_tokens, int32_t* accepted_nodes,
                       int32_t* n_accepted, int max_out, int32_t* status, dyspec_stream_t stream);

/*
 * (6) Construction of the draft token tree (Sec. 4.1-4.3, Algorithm 1; App. B, Algorithm 2), the step
 * before the tree attention.  The paper runs it on the CPU between draft-model calls; here the draft
 * model is represented by a table so that the whole loop runs in one launch: the distribution that
 * follows a tree position is row  (row(parent) * 2654435761 + (token + 1) * 40503  mod 2^32) mod n_rows
 * of draft_table (the root's row is root_row[r]), and the uniform number of the j-th sampling at a
 * position is uniforms[(row * 7919 + j * 104729 + 17  mod 2^32) mod n_uniforms].  A real draft model
 * replaces the table by its own calls; the arithmetic per node is the same.
 *
 * greedy (Algorithm 1): repeat m times: take the expandable slot with the largest estimated
 * acceptance rate v (ties: the one opened first), draw a token y from the residual distribution R at
 * that position (inverse CDF in token order), add the node, open the slots (v (1 - R[y]), same
 * position, next attempt) and (v R[y], first sampling under the new node).  (The printed listing
 * adds the node one line before it samples the token: read in the order that makes sense.)
 * threshold (Algorithm 2): layer by layer, every position keeps drawing while v >= threshold (the
 * listing prints `v < t`; the text says the guesses above the threshold are the ones kept), until
 * max_nodes guesses exist.  With threshold = values[m] of the greedy tree it builds the same tree.
 *
 *   draft_table   dev float [n_rows][vocab]   (rows 16-byte aligned: vocab % 4 == 0, vocab <= DYSPEC_MAX_VOCAB)
 *   uniforms      dev float [n_uniforms]      U(0,1) numbers
 *   root_row      dev int32 [n_req]           (taken modulo n_rows, non-negative remainder)
 *   outputs, stride S = m + 1 (greedy) or max_nodes + 1 (threshold) per request, node 0 = the root:
 *   parents, tokens, rows  dev int32 [n_req][S];  values, child_values  dev float [n_req][S]
 *                 values[k] = the estimated acceptance rate node k was created with, child_values[k] =
 *                 that of the first sampling under it;  n_nodes dev int32 [n_req] = nodes incl. the root
 * m, max_nodes <= DYSPEC_MAX_NODES - 1.  Values are fp32; as for dyspec_verify_tree, a choice between
 * numbers closer than rounding may fall differently from another implementation's.
 */
int dyspec_build_tree_greedy(const float* draft_table, int n_rows, int vocab, const float* uniforms, int n_uniforms,
                             const int32_t* root_row, int n_req, int m, int32_t* parents, int32_t* tokens, float* values,
                             float* child_values, int32_t* rows, int32_t* n_nodes, dyspec_stream_t stream);
int dyspec_build_tree_threshold(const float* draft_table, int n_rows, int vocab, const float* uniforms, int n_uniforms,
                                const int32_t* root_row, int n_req, float threshold, int max_nodes, int32_t* parents,
                                int32_t* tokens, float* values, float* child_values, int32_t* rows, int32_t* n_nodes,
                                dyspec_stream_t stream);

/*
 * (7) Keeping the accepted path in the KV cache (after dyspec_verify_tree; the paper only says that the
 * accepted tokens extend the prefix).  For request r with kept nodes k_0 < k_1 < ... row off_r + L_r + i
 * of k_cache and v_cache takes the content of row off_r + L_r + k_i, in place, and new_prefix_len[r] =
 * L_r + their number.  The kept nodes are the entries >= 0 of accepted_nodes (entries < 0 are emitted
 * tokens without a tree node) and, when keep_root != 0 and the request's walk emitted anything
 * (n_accepted[r] > 0), node 0 in front of them: dyspec_verify_tree walks from node 0 and lists only the
 * accepted children, but node 0 is the last token decoded before the step, a query row of the
 * verification pass whose own K/V row (tree row 0) was computed in that pass, so the sequence the next
 * step attends to is old prefix + node 0 + accepted path.  Pass keep_root = 1 when accepted_nodes comes
 * from dyspec_verify_tree; keep_root = 0 makes the call a plain gather of the listed rows.
 * Rows past the new prefix keep their old content.  One call per layer (per pair of caches).
 *   k_cache, v_cache  dev bf16 [rows][n_kv_heads][head_dim] (16-byte aligned; row bytes a multiple of 16)
 *   kv_row_offset     dev int64 [n_req];  prefix_len  dev int32 [n_req]
 *   accepted_nodes    dev int32 [n_req][max_out], n_accepted dev int32 [n_req]  (as written by dyspec_verify_tree;
 *                     node indices increase along a request's list)
 *   new_prefix_len    dev int32 [n_req] or NULL (written)
 */
int dyspec_compact_kv(void* k_cache, void* v_cache, const int64_t* kv_row_offset, const int32_t* prefix_len,
                      const int32_t* accepted_nodes, const int32_t* n_accepted, int n_req, int max_out, int n_kv_heads,
                      int head_dim, int keep_root, int32_t* new_prefix_len, dyspec_stream_t stream);

/*
 * (8) Paged KV cache (the paper does not fix the cache's memory layout; this is the layout of a serving
 * stack).  k_cache / v_cache are a pool of pages of page_size rows (a power of two, >= 128, so that no
 * key tile straddles two pages).  Prefix token t of request r lies at pool row
 *     page_table[r * pages_per_req + t / page_size] * page_size + t % page_size
 * and the request's tree rows (one per node, in node order) are the contiguous pool rows
 * tree_row_offset[r] .. tree_row_offset[r] + n_r - 1, outside the prefix pages (scratch rows of the
 * speculation step; dyspec_compact_kv_paged moves the accepted ones into the prefix pages).
 * Alternatively (tree_row_offset == NULL) the tree rows are part of the paged sequence: node j of
 * request r is token L_r + j, addressed by the rule above like a prefix token (the draft tokens' K/V were
 * appended to the sequence's pages).  Key tiles then follow the sequence, whatever L_r modulo the tile
 * size is: a row's mask slice for a tile is its bit row shifted by that remainder.  The per-node tile sets
 * (node_tiles) are ignored by such a plan.
 * Rows of a mapped page past the request's last token are read and masked: they must hold finite values
 * (zero a page when it is allocated).  A page number that is negative or beyond the pool reads as zeros,
 * it does not fault; the result for that request is then meaningless.
 *
 * dyspec_plan_create_paged: as dyspec_plan_create, with tree_row_offset (host int64 [n_req], or NULL: tree
 * rows inside the pages) in place of kv_row_offset, kv_total_rows = rows of the pool, and the page size.
 * The plan works with
 * dyspec_tree_attention_paged only (the contiguous calls return DYSPEC_ERR_INVALID_ARG for it, and this
 * call for a contiguous plan); the mask builder and reorder calls take either kind.
 *   page_table   dev int32 [n_req][pages_per_req]; entries past a request's last prefix page (last page of
 *                prefix + tree when the tree rows are inside the pages, which pages_per_req must cover:
 *                DYSPEC_ERR_INVALID_ARG otherwise) are not read.
 *                Like q and the caches it is read before the preceding kernel of the stream is known to
 *                have finished, so it must not be written by the kernel launched just before this call.
 *   node_tiles   as in dyspec_tree_attention_ragged_sparse, or NULL
 * Everything else as in dyspec_tree_attention_ragged.
 */
int dyspec_plan_create_paged(dyspec_plan_t** plan, int n_q_heads, int n_kv_heads, int head_dim, int n_req,
                             const int32_t* prefix_len, const int32_t* n_nodes, const int64_t* tree_row_offset,
                             int64_t kv_total_rows, int page_size, int words_per_row, float scale);
int dyspec_tree_attention_paged(const dyspec_plan_t* plan, const void* q, const void* k_cache, const void* v_cache,
                                const int32_t* page_table, int pages_per_req, const uint32_t* ancestor_bits,
                                const uint32_t* node_tiles, void* out, void* workspace, size_t workspace_bytes,
                                int32_t* status, dyspec_stream_t stream);

/*
 * (8b) Accepted-path compaction for the paged cache: for request r with kept nodes k_0 < k_1 < ...
 * (as in dyspec_compact_kv, keep_root included) the pool row of prefix token L_r + i takes the content of
 * tree row tree_row_offset[r] + k_i, for K and V, and new_prefix_len[r] = L_r + their number.  The page table must
 * already hold a page for every new token; a token without one (entry < 0 or past pages_per_req) stops
 * that request's copy there, new_prefix_len[r] counts what was kept, and *status = DYSPEC_ERR_INVALID_ARG.
 * tree_row_offset == NULL: the tree rows are tokens L_r .. of the paged sequence (node k = token L_r + k);
 * the rows then move in place, inside the request's pages (a kept node whose token has no page stops the
 * copy in the same way).
 * page_size: a power of two (any).  Other arguments as in dyspec_compact_kv; all arrays dev.
 */
int dyspec_compact_kv_paged(void* k_cache, void* v_cache, const int64_t* tree_row_offset, const int32_t* page_table,
                            int pages_per_req, int page_size, const int32_t* prefix_len, const int32_t* accepted_nodes,
                            const int32_t* n_accepted, int n_req, int max_out, int n_kv_heads, int head_dim,
                            int keep_root, int32_t* new_prefix_len, int32_t* status, dyspec_stream_t stream);

#ifdef __cplusplus
}
#endif
#endif /* DYSPEC_H_ */
