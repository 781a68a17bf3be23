/*
 * dg4 -- fused sparse attention over And-Inverter Graphs for NVIDIA B200 (sm_100a).
 *
 * C ABI of libdg4.so.  One GPU per handle.  The caller owns every tensor and the
 * stream; the library owns only what hangs off a dg4_graph.  Forward calls enqueue
 * work on the given stream and return; they never allocate, never synchronise and
 * never block without bound.  Argument errors are returned synchronously; nothing
 * throws, aborts or traps.
 *
 * Paper: DeepGate4 (arXiv 2502.01681).  Passages are cited by section / equation.
 *
 * Conventions
 *   - "host" / "device" in a comment says where a pointer must live.
 *   - Tensors are row-major [rows, d] with a leading dimension `ld*` in ELEMENTS.
 *     Base pointers must be 16-byte aligned and ld * sizeof(element) a multiple
 *     of 16 bytes, otherwise DG4_ERR_INVALID_ARG.
 *   - Every forward call must be made with the handle's device current (DG4_ERR_INVALID_ARG otherwise).
 *   - d = 128 only.  heads a power of two: 1 .. 16 for bf16 storage, 1 .. 32 for fp32 storage
 *     (a head must span whole 16-byte pieces of a row).  Attention: fp32 or bf16 storage,
 *     fp32 arithmetic.  Projections: bf16 storage, fp32 accumulation.
 *     Anything else returns DG4_ERR_UNSUPPORTED (there is no fallback path).
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 */
#ifndef DG4_H
#define DG4_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    DG4_OK = 0,
    DG4_ERR_INVALID_ARG = -1,  /* null pointer, bad size, bad alignment                      */
    DG4_ERR_NOT_SORTED  = -2,  /* row_ptr not starting at 0 / not non-decreasing              */
    DG4_ERR_BAD_DEGREE  = -3,  /* a node with more than two fan-ins                           */
    DG4_ERR_BAD_LEVEL   = -4,  /* an edge (u, v) with level[u] >= level[v], or a source id
                                  out of range, or a negative level                           */
    DG4_ERR_UNSUPPORTED = -5,  /* d, heads, dtype or hops outside the supported set           */
    DG4_ERR_ALLOC       = -6,  /* device or host allocation failed                            */
    DG4_ERR_CUDA        = -7,  /* a CUDA runtime call failed; see dg4_last_error()            */
    DG4_ERR_TIMEOUT     = -8   /* a bounded device-side wait ran out                          */
} dg4_status;

typedef enum { DG4_F32 = 0, DG4_BF16 = 1 } dg4_dtype;

enum {
    DG4_FLAG_RESIDUAL = 1,     /* output projection adds the layer's input row                */
    DG4_FLAG_LEVEL_LAUNCHES = 2, /* levelised layer: one group of kernel launches per level instead of the
                                  single persistent kernel (same results; kept for comparison)   */
    DG4_FLAG_FUSED_LAYER = 4   /* all-parallel layer: the K|V projection followed by ONE kernel (queries from
                                  the X tiles, attention, output projection, residual; Q and O never reach
                                  memory) instead of three kernels.  Same results bit for bit; measured a
                                  little slower to equal, so it is not the default.  bf16, two hops at most */
};

/* Per-call description of the attention layer. */
typedef struct {
    int32_t d;                 /* model width; 128                                            */
    int32_t heads;             /* number of heads; d_head = d / heads                         */
    int32_t dtype;             /* dg4_dtype of Q, K, V, O (and of X, H, weights)              */
    int32_t flags;             /* DG4_FLAG_*                                                  */
    float   scale;             /* multiplies every dot-product score, e.g. 1/sqrt(d_head)     */
} dg4_desc;

typedef struct dg4_graph dg4_graph;   /* opaque; device-resident index arrays of one circuit */

typedef struct {
    int64_t n_nodes;
    int64_t n_edges;
    int64_t n_nbr;             /* total neighbourhood entries, sum over v of |N(v)|           */
    int32_t n_levels;          /* 1 + max level                                               */
    int32_t max_class;         /* 2^(hops+1) - 1: upper bound of |N(v)|                       */
    int32_t hops;
    int32_t perm_chunk;        /* chunk length of the degree-class permutation (0 = global)   */
    int32_t n_chunks;
    int32_t device;
} dg4_graph_info_t;

/* Index arrays a graph handle holds (all int32), for dg4_graph_export. */
typedef enum {
    DG4_ARR_NBR_PTR = 0,        /* [n+1]                 start of N(v) in NBR_IDX                        */
    DG4_ARR_NBR_IDX = 1,        /* [n_nbr]               members of N(v): v first, the rest ascending    */
    DG4_ARR_LEVEL_PTR = 2,      /* [n_levels+1]          start of level l in LEVEL_NODES                 */
    DG4_ARR_LEVEL_NODES = 3,    /* [n]                   node ids ordered by (level, id)                 */
    DG4_ARR_PERM = 4,           /* [n]                   ids ordered by (chunk, |N(v)|, id)              */
    DG4_ARR_CLASS_PTR = 5,      /* [n_chunks, max_class+1]  start of class c+1 of a chunk in PERM;
                                                         last entry of a row = end of the chunk        */
    DG4_ARR_LEVEL_PERM = 6,     /* [n]                   ids ordered by (level, |N(v)|, id)              */
    DG4_ARR_LEVEL_CLASS_PTR = 7,/* [n_levels, max_class+1]  same as CLASS_PTR with levels as segments    */
    DG4_ARR_NBR_PAD = 8         /* [n, max_class+1]      fixed-width neighbour table read by the kernels:
                                                         |N(v)|, then the members other than v ascending,
                                                         then v repeated as filler                       */
} dg4_array_id;

const char* dg4_status_string(dg4_status s);
/* Detail of the last error on the calling thread ("" if none).  Valid until the next failing call. */
const char* dg4_last_error(void);

/* Number of GPU kernels this library has launched in the calling process so far (monotone; for the
 * accounting of benchmarks -- the paper has no counterpart). */
int64_t dg4_launch_count(void);

/*
 * Graph prep.  Sec. 3.2: node kinds are told apart by in-degree (0 primary input, 1 NOT, 2 AND); Eq. 1
 * defines the logic level; cone_k(v) = { u : a path u -> v of length <= k } with v included, at most
 * 2^(k+1)-1 members.  Sec. 3.5 restricts attention to that set (the "virtual edges").
 *
 * Validates the circuit on the host, uploads it, and builds on the device:
 *   the neighbourhood lists N(v) = cone_hops(v) as a CSR (v first, then ascending id, duplicates
 *   collapsed), the level buckets, and the degree-class orderings (stable by (segment, |N(v)|, id),
 *   segments = consecutive id chunks of perm_chunk nodes, and = levels).
 *
 *   n_nodes     >= 1
 *   row_ptr     host, [n_nodes+1], destination-sorted CSR of DIRECT fan-ins (no self entry)
 *   col_idx     host, [row_ptr[n_nodes]], source ids; any order inside a row; a repeated source is allowed
 *   level       host, [n_nodes]; any layering with level[u] < level[v] on every edge is accepted
 *   hops        1 (fan-ins + self), 2 (2-hop fan-in cone + self), or 3 .. 8 (wider cones, the paper uses k = 8:
 *               up to 2^(hops+1)-1 members).  For hops > 2 only the neighbourhood CSR and the level buckets are
 *               built (no fixed-width table, no class orderings: exporting those returns DG4_ERR_UNSUPPORTED),
 *               the lists must stay below 2^31 entries and dg4_graph_rebuild is not available.
 *   perm_chunk  0 (one chunk) or a positive multiple of 1024
 *   device      CUDA ordinal; made current for the duration of the call and restored
 *   out         receives the handle; untouched on error
 *
 * Allocates device memory and returns when the handle is complete; not for use inside a captured region.  Its
 * uploads and kernels run on a stream of their own: the call neither waits for nor delays work the caller has in
 * flight on other streams (cones of more than two hops are the exception: that path synchronises the device).  The
 * two small results it needs on the host (the size of the lists, the level offsets) are written by a kernel into
 * pinned, mapped host memory owned by the library, so they do not queue behind a large device-to-host copy
 * either.
 * Errors: INVALID_ARG, NOT_SORTED, BAD_DEGREE, BAD_LEVEL, UNSUPPORTED, ALLOC, CUDA.
 */
dg4_status dg4_graph_create(int32_t n_nodes, const int32_t* row_ptr, const int32_t* col_idx,
                            const int32_t* level, int32_t hops, int32_t perm_chunk, int32_t device,
                            dg4_graph** out);

/* Re-runs the device part of graph prep (neighbourhoods, buckets, class orderings) from the circuit the
 * handle already holds, on `stream`, reusing the handle's buffers.  Asynchronous; allocates nothing.
 * The arrays are unchanged in content; this entry exists so the device pass can be timed on its own. */
dg4_status dg4_graph_rebuild(dg4_graph* g, void* stream);

/* Frees the handle and its device memory; waits for the device (kernels still using the handle finish first).
 * NULL is accepted. */
dg4_status dg4_graph_destroy(dg4_graph* g);

/* The same without waiting (the paper has no counterpart): the handle's device memory is released in the order
 * of `stream`, i.e. after the work enqueued there so far, and goes back to the library's pool, from which later
 * dg4_graph_create calls are served without a call into the driver that would wait for running kernels.  The
 * caller guarantees that no other stream still uses the handle.  Handles of cones of more than two hops are freed
 * as by dg4_graph_destroy.  NULL is accepted. */
dg4_status dg4_graph_destroy_async(dg4_graph* g, void* stream);

/* Gives the unused part of the library's memory pool on `device` back to the driver (freed handles leave their
 * memory in the pool for later dg4_graph_create calls).  Waits for the device.  The paper has no counterpart. */
dg4_status dg4_memory_trim(int32_t device);
dg4_status dg4_graph_info(const dg4_graph* g, dg4_graph_info_t* out);

/* Copies one index array to the host (synchronises the device).  host_dst may be NULL to query the
 * length only.  capacity and *n_written count int32 elements.  INVALID_ARG if capacity is too small. */
dg4_status dg4_graph_export(const dg4_graph* g, dg4_array_id which, int32_t* host_dst, int64_t capacity,
                            int64_t* n_written);

/*
 * Algorithm 1 (graph partition): the roots whose cones the partition collects, for cone depth k = the hops the
 * handle was created with and stride delta.  Roots are the nodes on levels k, k + delta, ... and the nodes
 * without fan-out (added to the group of their own level; a node that qualifies both ways appears once),
 * grouped by level and ordered by id inside a level.  The cone of a root r is its list in DG4_ARR_NBR_IDX.
 *   roots      device, capacity n_nodes int32; receives the root ids
 *   group_ptr  device, n_levels + 1 int32; group_ptr[l] = number of roots on levels below l
 *   n_roots    host; receives the number of roots
 * The graph's device must be current.  Allocates scratch and synchronises (a graph-prep call, not a forward call).
 */
dg4_status dg4_graph_partition(const dg4_graph* g, int32_t delta, int32_t* roots, int32_t* group_ptr,
                               int64_t* n_roots);

/*
 * The updating strategy of Sec. 3.4 (intra- and inter-level updating) over the partition of Algorithm 1, for a
 * stack of attention layers, with the table of historical embeddings on the device.  Cone depth k = the hops the
 * handle was created with; stride delta; mini-batches of `batch` consecutive cones (ascending root id) inside a
 * level group.  For each mini-batch, in the order of Algorithm 2's loop (groups l = k, k + delta, ... and the
 * groups that only hold cones of fan-out-free gates, ascending):
 *   - the sub-graph is the union S of the mini-batch's cones;
 *   - a gate of S that an earlier mini-batch has updated (same group: intra-level; earlier group: inter-level)
 *     enters with its row of the table, attends to itself only (its in-edges are removed) and is not stored again;
 *   - every other gate v of S enters with its row of the table (its input row: it was never stored), and attends
 *     to itself and to the members of cone_k(v) present in S;
 *   - all gates of S go through the n_layers layers together (QKV projection, attention over those lists, output
 *     projection (+ residual if desc->flags has DG4_FLAG_RESIDUAL)); then the rows of the gates that were not
 *     frozen are stored in the table and every gate of S is marked as updated.
 * A gate no cone covers keeps its input row.
 *   H           device, [n, d] bf16: on entry the input rows, on return the table of historical embeddings
 *   W_qkv, W_o  host arrays of n_layers device pointers ([3d, d] and [d, d] bf16 each); n_layers 1 .. 64
 *   delta       >= 1 (the paper uses delta < k so that consecutive groups overlap; not enforced)
 *   batch       1 .. 65536 cones per mini-batch (the paper uses 128)
 *   workspace   device, dg4_cone_update_workspace_bytes() bytes, 256-byte aligned: three int32 per gate plus
 *               buffers sized by the mini-batch (at most batch * (2^(k+1)-1) gates), not by the circuit
 *   stored      device, [n] int32 or NULL: receives how many times each gate's row was stored (0 or 1)
 *   n_batches   host or NULL: receives the number of mini-batches
 * Unlike the other forward calls this one is a host-driven loop: it runs Algorithm 1 (dg4_graph_partition, which
 * allocates its scratch and synchronises the device) and then reads the size of each mini-batch's sub-graph back
 * from the device, so it waits on `stream` between mini-batches and must not be captured.  On return all work has
 * been enqueued on `stream`.  Errors: INVALID_ARG, UNSUPPORTED (dtype other than bf16, heads > 16), ALLOC, CUDA.
 */
size_t dg4_cone_update_workspace_bytes(const dg4_graph* g, const dg4_desc* desc, int32_t batch);
dg4_status dg4_cone_update_fwd(const dg4_graph* g, const dg4_desc* desc, void* H, int64_t ldh, int32_t n_layers,
                               const void* const* W_qkv, const void* const* W_o, int32_t delta, int32_t batch,
                               void* workspace, size_t workspace_bytes, int32_t* stored, int64_t* n_batches,
                               void* stream);

/* Waits for the device to go idle and reads the handle's status word: DG4_OK, or DG4_ERR_TIMEOUT if a bounded
 * device-side wait of an earlier forward call ran out (that call's output is then incomplete). */
dg4_status dg4_graph_poll_status(const dg4_graph* g, int32_t* out);

/* Device pointer to one index array (owned by the handle, valid until destroy); NULL on bad arguments. */
const int32_t* dg4_graph_device_array(const dg4_graph* g, dg4_array_id which);

/*
 * QKV projection: [Q | K | V] = X * W_qkv^T for every node (Sec. 3.5: the Transformer block is kept and
 * only its attention is restricted, so the block's dense projections stay).
 *   X      device, [n, d] bf16, leading dimension ldx
 *   W_qkv  device, [3d, d] bf16 row-major (output-major): rows 0..d-1 give Q, d..2d-1 K, 2d..3d-1 V
 *   Q,K,V  device, [n, d] bf16 each.  K and V may interleave in one [n, 2d] buffer (V = K + d, ldk = ldv = 2d).
 * fp32 accumulation, one rounding to bf16 per stored element.  UNSUPPORTED unless desc->dtype is bf16.
 */
dg4_status dg4_qkv_project(const dg4_graph* g, const dg4_desc* desc,
                           const void* X, int64_t ldx, const void* W_qkv,
                           void* Q, int64_t ldq, void* K, int64_t ldk, void* V, int64_t ldv, void* stream);

/*
 * Fused sparse attention (Sec. 3.5; kernel mapping informed by Sec. 3.7's remarks on low in-degree):
 * for every node v and head h,
 *     s_u = scale * <Q[v,h,:], K[u,h,:]>  for u in N(v),   alpha = softmax_u(s),   O[v,h,:] = sum_u alpha_u V[u,h,:]
 * Scores live in registers only; no per-edge tensor is written.  fp32 arithmetic; O rounded once on store.
 *   Q, K, V  device, [n, d] of desc->dtype;   O  device, [n, d], must not alias K or V.
 */
dg4_status dg4_sparse_attn_fwd(const dg4_graph* g, const dg4_desc* desc,
                               const void* Q, int64_t ldq, const void* K, int64_t ldk,
                               const void* V, int64_t ldv, void* O, int64_t ldo, void* stream);

/*
 * The same fused attention with the additive score of graph-attention layers (the form the fused GAT kernels
 * discussed in Sec. 2 and Sec. 3.7 aggregate with; the paper does not restate the formula): per head h
 *     e_u = LeakyReLU(S_src[u,h] + S_dst[v,h]),  alpha = softmax over u in N(v),  O[v,h,:] = sum_u alpha_u V[u,h,:]
 * with node-level scalars instead of key rows (a neighbour then costs one value row plus 4 bytes per head).
 *   S_dst, S_src    device, [n, heads] fp32, contiguous
 *   negative_slope  of the LeakyReLU (0.2 in the usual definition)
 *   V, O            device, [n, d] of desc->dtype; O must not alias V.  desc->scale is not used.
 */
dg4_status dg4_sparse_attn_additive_fwd(const dg4_graph* g, const dg4_desc* desc,
                                        const float* S_dst, const float* S_src, float negative_slope,
                                        const void* V, int64_t ldv, void* O, int64_t ldo, void* stream);

/*
 * Output projection of the attention sub-layer (Sec. 3.5: the Transformer block around the restricted attention is
 * kept, and with it the block's output projection and residual connection):
 * H_out = O * W_o^T (+ H_res if desc->flags has DG4_FLAG_RESIDUAL and H_res != NULL).
 *   O device [n, d] bf16;  W_o device [d, d] bf16 (output-major);  H_res device [n, d] bf16 or NULL;
 *   H_out device [n, d] bf16; may alias H_res (each row is read before it is written by the same thread).
 */
dg4_status dg4_out_project(const dg4_graph* g, const dg4_desc* desc,
                           const void* O, int64_t ldo, const void* W_o,
                           const void* H_res, int64_t ldh, void* H_out, int64_t ldho, void* stream);

/* Bytes of caller-provided device workspace the two layer calls need for this graph (256-byte aligned base). */
size_t dg4_layer_workspace_bytes(const dg4_graph* g, const dg4_desc* desc);

/*
 * One layer for all nodes at once (Sec. 3.5: the attention sub-layer of the Transformer block with its attention
 * restricted to cone_k(v)): QKV projection -> sparse attention -> output projection (+ residual),
 * every node reading the same input H_in.   H_in, H_out: device [n, d] bf16; they may be the same buffer
 * only if ldh == ldho (rows are then updated in place after all reads of the layer's input are done).
 * With DG4_FLAG_FUSED_LAYER (bf16, heads a power of two up to 16, cones of two hops at most; ignored otherwise) the
 * layer runs as the K|V projection followed by one kernel that never writes Q or O to memory; the rows it
 * produces are the same bit for bit.
 */
dg4_status dg4_layer_fwd_parallel(const dg4_graph* g, const dg4_desc* desc,
                                  const void* H_in, int64_t ldh, const void* W_qkv, const void* W_o,
                                  void* H_out, int64_t ldho, void* workspace, size_t workspace_bytes,
                                  void* stream);

/*
 * The all-nodes-parallel layer for callers that cannot allocate device memory.  (The paper has no
 * counterpart; this is a deployment aid.)
 *
 * Who needs it: programs in which nobody may call cudaMalloc (or a framework allocator) by the time the layer
 * runs -- a service that divided up the GPU at start-up and locked the pool, a plug-in inside a host
 * application that owns the device heap, a latency-critical loop that cannot take the device-wide
 * synchronisation cudaMalloc / cudaFree imply.  Same computation and same arguments as
 * dg4_layer_fwd_parallel, minus the workspace: the intermediates (Q, K|V, O) live in a fixed 32 MiB array
 * that is part of the library image and is held on every GPU that loads the library until the process exits.
 *
 *   - Capacity: graphs of at most dg4_static_max_nodes() = 32 768 nodes (1 KiB of scratch per node);
 *     larger graphs are rejected with DG4_ERR_INVALID_ARG and a message naming the limit.
 *   - The graph's device must be current.  The first call on a device looks up the array's device address
 *     (once per device), and the driver may instantiate the library's image on that device -- and with it reserve
 *     the 32 MiB -- only at that moment rather than when the library was loaded.  So make one call per device
 *     at start-up, before device memory is divided up and outside any stream capture; it can fail with
 *     DG4_ERR_CUDA if the 32 MiB cannot be had.
 *   - After that first call, a call takes nothing from the device heap and nothing from the host heap, and
 *     frees nothing.
 *   - All calls share the one array.  It is never cleared and needs no clearing (a call writes every scratch
 *     row before reading it), but calls that overlap on the GPU -- different streams, or several host
 *     threads -- race on it: run them one after another.
 */
dg4_status dg4_layer_fwd_parallel_static(const dg4_graph* g, const dg4_desc* desc,
                                         const void* H_in, int64_t ldh, const void* W_qkv, const void* W_o,
                                         void* H_out, int64_t ldho, void* stream);
int64_t dg4_static_max_nodes(void);

/*
 * One layer in the paper's level-by-level order (Sec. 1 and Sec. 3.4: gates are encoded in strict
 * topological order and each gate is computed once).  Levels 0, 1, ... are processed in turn; a node
 * takes its query and its own key/value from its row as it was when the call started, and the key/value
 * of every other member of N(v) (all on lower levels) from that node's row as already updated by this
 * call.  H is updated in place.
 *   H              device, [n, d] bf16, leading dimension ldh
 *   workspace      device, at least dg4_layer_workspace_bytes() bytes
 *   device_status  device int32 or NULL; receives a dg4_status (0, or DG4_ERR_TIMEOUT if a bounded
 *                  device-side wait ran out; the call still returns and the context stays usable)
 */
dg4_status dg4_layer_fwd_levelised(const dg4_graph* g, const dg4_desc* desc,
                                   void* H, int64_t ldh, const void* W_qkv, const void* W_o,
                                   void* workspace, size_t workspace_bytes,
                                   int32_t* device_status, void* stream);

/*
 * Several levelised layers in one call, run as a wavefront (Sec. 3.4's level order, applied to a stack of
 * layers): the result is exactly that of n_layers successive dg4_layer_fwd_levelised calls with W_qkv[k], W_o[k],
 * but layer k+1 starts on a level as soon as layer k has finished that level, so the chain of dependent steps is
 * n_levels + n_layers - 1 long instead of n_layers * n_levels.
 *   n_layers     1 .. 8
 *   W_qkv, W_o   host arrays of n_layers device pointers ([3d, d] and [d, d] bf16 each)
 *   workspace    device, at least dg4_layers_workspace_bytes() bytes, 256-byte aligned
 * Other arguments as for dg4_layer_fwd_levelised.
 */
size_t dg4_layers_workspace_bytes(const dg4_graph* g, const dg4_desc* desc, int32_t n_layers);
dg4_status dg4_layers_fwd_levelised(const dg4_graph* g, const dg4_desc* desc, void* H, int64_t ldh,
                                    int32_t n_layers, const void* const* W_qkv, const void* const* W_o,
                                    void* workspace, size_t workspace_bytes, int32_t* device_status, void* stream);

/*
 * The rest of the Transformer block around the attention (Sec. 3.5: only the multi-head attention module is
 * replaced, the structure of the original Transformer layer is kept; that layer is post-norm with a two-matrix
 * ReLU feed-forward sub-layer; the paper's figure of the block is not part of its text, so this reading is the
 * library's stated choice).  bf16 rows, fp32 arithmetic, d = 128.  All pointers are device pointers; rows have
 * 128 valid elements and leading dimensions ldx / ldy in elements (multiples of 8); gamma, beta, b1, b2 are fp32
 * vectors, 16-byte aligned.  eps >= 0 enters under the square root.  Asynchronous on `stream`; the number of rows
 * is the handle's node count.  Errors: DG4_ERR_INVALID_ARG (null, misaligned, bad eps), DG4_ERR_UNSUPPORTED
 * (d != 128, dtype != bf16, d_ff != 512), DG4_ERR_CUDA; a device-side wait that runs out records DG4_ERR_TIMEOUT
 * in the handle's status word (dg4_graph_poll_status).
 *
 * dg4_layernorm_fwd: Y[i,:] = (X[i,:] - mean_i) / sqrt(var_i + eps) * gamma + beta, mean and biased variance over
 * the 128 features of row i.  Y may be X.
 *
 * dg4_ffn_fwd: Y = LayerNorm(X + max(0, X W1^T + b1) W2^T + b2) with W1 [d_ff, 128] and W2 [128, d_ff] row-major
 * bf16 (out x in), d_ff = 512.  The hidden activations are rounded to bf16 between the two products and are never
 * written to global memory.  Y may be X.
 *
 * dg4_block_fwd_parallel: one whole block on all nodes at once:
 *     H1 = LayerNorm_1(H_in + Attention(H_in) W_o^T),   H_out = LayerNorm_2(H1 + FFN(H1)),
 * Attention being dg4_qkv_project + dg4_sparse_attn_fwd on the handle's neighbourhoods (desc gives heads and
 * scale; the residual connections are always on).  workspace: dg4_layer_workspace_bytes() bytes, 256-byte aligned,
 * owned by the caller; the library allocates nothing.  H_out may be H_in.
 *
 * dg4_block_fwd_levelised: the same block in the paper's level-by-level order (Sec. 1 and Sec. 3.4 for the order,
 * Sec. 3.5 for the block), in place on H: levels 0, 1, ... in turn; a node takes its query and its own key / value
 * from its row as it was when the call started, and the key / value of every other member of N(v) from that node's
 * row as already replaced by this call, i.e. from its BLOCK output.  The block runs
 * as ONE persistent cooperative kernel: half of its CTAs take the attention sub-layer of each level, the other half
 * the LayerNorm, feed-forward sub-layer, LayerNorm and the K | V refresh from the block's output rows, and the two
 * hand the levels to one another through per-level counters (every wait bounded; DG4_ERR_TIMEOUT in the handle's
 * status word if one runs out).  With DG4_FLAG_LEVEL_LAUNCHES: one group of kernel launches
 * per level (the level's rows are taken through the handle's level buckets).  Same results either way.
 * The persistent kernel is launched cooperatively in clusters of two CTAs (a tile's rows go from its attention-stage
 * CTA to its feed-forward-stage CTA through distributed shared memory); if the device cannot hold all pairs at once,
 * if the environment variable DG4_NO_CLUSTER_PAIRS is set, or if a tool has injected itself into the process
 * (CUDA_INJECTION64_PATH / NV_COMPUTE_PROFILER_PERFWORKS_DIR set: profilers that cannot replay such a launch), it is
 * launched plainly cooperatively and the rows go through global memory.
 */
dg4_status dg4_layernorm_fwd(const dg4_graph* g, const dg4_desc* desc, const void* X, int64_t ldx,
                             const float* gamma, const float* beta, float eps, void* Y, int64_t ldy, void* stream);
dg4_status dg4_ffn_fwd(const dg4_graph* g, const dg4_desc* desc, const void* X, int64_t ldx, const void* W1,
                       const float* b1, const void* W2, const float* b2, const float* gamma, const float* beta,
                       float eps, int32_t d_ff, void* Y, int64_t ldy, void* stream);
dg4_status dg4_block_fwd_parallel(const dg4_graph* g, const dg4_desc* desc, const void* H_in, int64_t ldh,
                                  const void* W_qkv, const void* W_o, const float* ln1_gamma, const float* ln1_beta,
                                  const void* W1, const float* b1, const void* W2, const float* b2,
                                  const float* ln2_gamma, const float* ln2_beta, float eps, int32_t d_ff,
                                  void* H_out, int64_t ldho, void* workspace, size_t workspace_bytes, void* stream);
dg4_status dg4_block_fwd_levelised(const dg4_graph* g, const dg4_desc* desc, void* H, int64_t ldh,
                                   const void* W_qkv, const void* W_o, const float* ln1_gamma, const float* ln1_beta,
                                   const void* W1, const float* b1, const void* W2, const float* b2,
                                   const float* ln2_gamma, const float* ln2_beta, float eps, int32_t d_ff,
                                   void* workspace, size_t workspace_bytes, void* stream);
/* Several blocks in level-by-level order in one call, as ONE wavefront (block k+1 takes a level as soon as block k
 * has finished it): the same result as n_blocks successive dg4_block_fwd_levelised calls, bit for bit, with a
 * dependent chain n_levels + 2 n_blocks - 1 stage steps long instead of n_blocks * 2 * n_levels.  Every parameter
 * of the single-block call becomes a host array of n_blocks device pointers (1 .. 8 blocks); eps and d_ff are
 * shared.  workspace: at least dg4_blocks_workspace_bytes() bytes, 256-byte aligned.  Always the persistent kernel. */
size_t dg4_blocks_workspace_bytes(const dg4_graph* g, const dg4_desc* desc, int32_t n_blocks);
dg4_status dg4_blocks_fwd_levelised(const dg4_graph* g, const dg4_desc* desc, void* H, int64_t ldh, int32_t n_blocks,
                                    const void* const* W_qkv, const void* const* W_o,
                                    const float* const* ln1_gamma, const float* const* ln1_beta,
                                    const void* const* W1, const float* const* b1, const void* const* W2,
                                    const float* const* b2, const float* const* ln2_gamma,
                                    const float* const* ln2_beta, float eps, int32_t d_ff, void* workspace,
                                    size_t workspace_bytes, void* stream);

/*
 * Diagnostic (the paper has no counterpart): launches one small CTA that waits, with the same bounded wait the
 * pipelines of this library use, on a barrier nothing ever arrives on.  The wait gives up after its poll limit
 * (about a second) and the kernel writes DG4_ERR_TIMEOUT to *device_status (device int32) and returns normally:
 * nothing traps, the context stays usable.  Asynchronous on `stream`.
 */
dg4_status dg4_selftest_bounded_wait(int32_t* device_status, void* stream);

/*
 * Diagnostics for the error paths (the paper has no counterpart).
 *
 * dg4_debug_set_poll_limit: every device-side wait of the pipelined kernels (projection, feed-forward, levelised)
 * polls a bounded number of times before it gives up, records DG4_ERR_TIMEOUT in the status word and lets the
 * kernel wind down (copies and MMAs already started are still waited for, tensor memory is freed, the kernel
 * returns).  This sets that number for the launches that follow, process-wide; 0 restores the default (about a
 * second).  A tiny value makes the waits run out at once, which is how the wind-down is exercised without anything
 * actually being stuck; results of such launches are incomplete by design.
 *
 * dg4_debug_override_current_device: every forward call checks that the handle's device is the calling thread's
 * current CUDA device and returns DG4_ERR_INVALID_ARG otherwise (its kernels would dereference another GPU's
 * arrays).  This makes that check, on the calling thread, behave as if `device` were current (-1 = off), so the
 * refusal can be tested on a machine with one GPU.
 */
void dg4_debug_set_poll_limit(uint32_t polls);
void dg4_debug_override_current_device(int32_t device);

#ifdef __cplusplus
}
#endif
#endif /* DG4_H */
