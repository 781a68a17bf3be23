// Internal declarations shared by the translation units of libdg4.so (not part of the public ABI).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stdio.h>
#include <stdarg.h>

#include "dg4.h"

// ---- error plumbing -------------------------------------------------------------------------
void dg4_set_error(const char* fmt, ...);

#define DG4_CUDA_TRY(expr)                                                                   \
    do {                                                                                     \
        cudaError_t _e = (expr);                                                             \
        if (_e != cudaSuccess) {                                                             \
            dg4_set_error("%s failed: %s (%s:%d)", #expr, cudaGetErrorString(_e), __FILE__, __LINE__); \
            return (_e == cudaErrorMemoryAllocation) ? DG4_ERR_ALLOC : DG4_ERR_CUDA;         \
        }                                                                                    \
    } while (0)

#define DG4_FAIL(code, ...)          \
    do {                             \
        dg4_set_error(__VA_ARGS__);  \
        return (code);               \
    } while (0)

// ---- argument checks shared by the forward entry points (dg4_layer.cu) -----------------------------
// INVALID_ARG unless the graph's device is the calling thread's current device: every forward call dereferences
// the handle's device arrays in its kernels, so a call made with another device current must be refused on the host.
dg4_status dg4i_check_device(const dg4_graph* g);
dg4_status dg4i_check_desc(const dg4_desc* d, bool need_bf16);
dg4_status dg4i_check_tensor(const char* name, const void* p, int64_t ld, int elem_size, int min_ld);
// Poll limit of the bounded device-side waits (mbarrier phases, level counters) handed to every kernel launch:
// the built-in default unless dg4_debug_set_poll_limit changed it.
uint32_t dg4i_poll_limit();
#define DG4I_DEFAULT_POLL_LIMIT (1u << 24)

// ---- tensor maps -----------------------------------------------------------------------------------
// Tensor map over a [rows, 128] bf16 row-major matrix with leading dimension ld (elements): box = 64 columns x
// box_rows rows, 128-byte swizzle, rows past the end read as zero and are clipped on store (dg4_project.cu).
struct CUtensorMap_st;
dg4_status dg4i_make_row_map(CUtensorMap_st* map, const void* base, int64_t rows, int64_t ld, int box_rows);

// ---- launch accounting (every kernel launch of the library bumps this counter) ------------------
void dg4i_count_launch(int n = 1);

// ---- the graph handle -----------------------------------------------------------------------
struct dg4_graph {
    int32_t device = 0;
    int32_t n = 0;            // nodes
    int64_t e = 0;            // direct fan-in edges
    int64_t n_nbr = 0;        // neighbourhood entries
    int32_t n_levels = 0;
    int32_t hops = 0;
    int32_t max_class = 0;
    int32_t perm_chunk = 0;   // 0 = one chunk
    int32_t n_chunks = 1;

    // circuit as uploaded
    int32_t* row_ptr = nullptr;   // [n+1]
    int32_t* col_idx = nullptr;   // [e]
    int32_t* level = nullptr;     // [n]
    // built by graph prep
    int32_t* nbr_ptr = nullptr;          // [n+1]
    int32_t* nbr_idx = nullptr;          // [n_nbr]
    int32_t* nbr_pad = nullptr;          // [n, pad_width]: |N(v)|, then the members other than v (filler: v)
    int32_t pad_width = 0;               // max_class + 1 (0 for cones wider than two hops: no table)
    bool wide = false;                   // hops > 2: CSR lists only, no fixed-width table, no class orderings
    bool pooled = false;                 // device buffers come from the library's stream-ordered pool
    int32_t* level_ptr = nullptr;        // [n_levels+1]
    int32_t* level_nodes = nullptr;      // [n]
    int32_t* perm = nullptr;             // [n]
    int32_t* class_ptr = nullptr;        // [n_chunks*(max_class+1)]
    int32_t* level_perm = nullptr;       // [n]
    int32_t* level_class_ptr = nullptr;  // [n_levels*(max_class+1)]
    // scratch of graph prep (kept so that a rebuild allocates nothing)
    int32_t* seq_a = nullptr;            // [n]
    int32_t* seq_b = nullptr;            // [n]
    int32_t* hist = nullptr;             // [hist_len]
    int32_t* block_sums = nullptr;       // [block_sums_len]
    int64_t hist_len = 0;
    int64_t block_sums_len = 0;
    // host copy of the level boundaries (the levelised driver launches per level)
    int32_t* h_level_ptr = nullptr;      // [n_levels+1]
    // device status word written by kernels whose bounded waits ran out (0 = ok)
    int32_t* dev_status = nullptr;
};

// ---- kernels' host launchers (each enqueues on `st` and returns) -----------------------------
dg4_status dg4i_graph_device_pass(dg4_graph* g, cudaStream_t st, bool sizes_only);
// exclusive prefix sum of n int32 values (in place allowed); block_sums: scratch of the graph handle
dg4_status dg4i_exclusive_scan(const int32_t* in, int32_t* out, int64_t n, int32_t* block_sums, cudaStream_t st);
// cones wider than two hops (graphs created with hops 3..8): fills nbr_ptr, allocates and fills nbr_idx
dg4_status dg4i_build_wide_cones(dg4_graph* g);

struct dg4i_attn_args {
    const void* Q; int64_t ldq;
    const void* K; int64_t ldk;
    const void* V; int64_t ldv;
    void* O; int64_t ldo;
    const int32_t* nbr_pad;     // [n, max_nbr + 1] fixed-width neighbour table (cones of at most two hops)
    const int32_t* node_list;   // nullable: node ids to process; else ids first..first+count-1
    int32_t first;
    int32_t count;
    int32_t heads;
    int32_t max_nbr;            // 3 or 7; larger for cones wider than two hops
    int32_t dtype;
    float scale;
};
// What the less common kernels need on top (kept out of the struct above: the main kernel compiles to fewer
// registers and instructions with the smaller parameter block).
struct dg4i_attn_more {
    const int32_t* nbr_ptr = nullptr;   // CSR lists, used for wider cones
    const int32_t* nbr_idx = nullptr;
    const float* s_dst = nullptr;       // additive-score variant: node-level scalars [n, heads] fp32
    const float* s_src = nullptr;
    float slope = 0.f;
};
// `more` may be null for graphs with cones of at most two hops
dg4_status dg4i_attn_launch(const dg4i_attn_args& a, const dg4i_attn_more* more, cudaStream_t st);
dg4_status dg4i_attn_additive_launch(const dg4i_attn_args& a, const dg4i_attn_more& more, cudaStream_t st);

// Y[r, 0:n_out] = A[r, 0:128] * W[0:n_out, 0:128]^T (+ R[r, :]) for rows r of a list (or 0..rows-1).
// Output column block j (of 128) goes to out[j] with leading dimension ldo[j].
struct dg4i_proj_args {
    const __nv_bfloat16* A; int64_t lda;
    const __nv_bfloat16* W;            // [n_out, 128] row-major
    int32_t n_out;                     // 128, 256 or 384
    __nv_bfloat16* out[3]; int64_t ldo[3];
    const __nv_bfloat16* R; int64_t ldr;   // nullable residual, added to column block 0 only
    const int32_t* row_list;           // nullable
    int32_t first;                     // offset into row_list (or first row id)
    int32_t rows;
    int32_t* status = nullptr;         // device status word: receives DG4_ERR_TIMEOUT if a bounded wait runs out
};
dg4_status dg4i_proj_launch(const dg4i_proj_args& a, cudaStream_t st);

// The all-nodes-parallel layer behind its K | V projection as one kernel (dg4_fused.cu): Q from the X tiles,
// attention, output projection (+ residual) per 128-node tile.  Supported for bf16, heads a power of two up to
// 16, and graphs with the fixed-width neighbour table (two hops at most).
bool dg4i_fused_layer_supported(const dg4_graph* g, const dg4_desc* desc);
dg4_status dg4i_fused_layer_launch(const dg4_graph* g, const dg4_desc* desc, const __nv_bfloat16* X, int64_t ldx,
                                   const __nv_bfloat16* KV, const __nv_bfloat16* W_q, const __nv_bfloat16* W_o,
                                   __nv_bfloat16* H_out, int64_t ldho, int32_t* status, cudaStream_t st);

// Persistent levelised kernel over n_layers layers run as a wavefront.  KV[k] ([n, 256] bf16, contents irrelevant on
// entry) receives layer k's K | V rows of the nodes as they are updated.  H is updated in place.  `sync` is zeroed
// by the call and must hold dg4i_levelised_sync_bytes() bytes.
#define DG4I_MAX_LAYERS 8
size_t dg4i_levelised_sync_bytes(const dg4_graph* g, int n_layers);
// With `block` (an array of n_layers entries): whole Transformer blocks level by level -- for every block one group
// of CTAs runs the attention sub-layer of each level, another its LayerNorm, feed-forward sub-layer, LayerNorm
// and the K | V refresh from the block's output rows; the stages of all blocks form one wavefront.  `sync` then
// holds dg4i_levelised_sync_bytes(g, 2 * n_layers) bytes.
struct dg4i_block_tail {
    const float* ln1_gamma; const float* ln1_beta;
    const __nv_bfloat16* W1; const float* b1;          // [512, 128], [512]
    const __nv_bfloat16* W2; const float* b2;          // [128, 512], [128]
    const float* ln2_gamma; const float* ln2_beta;
    float eps;
};
dg4_status dg4i_levelised_launch(const dg4_graph* g, const dg4_desc* desc, int n_layers,
                                 __nv_bfloat16* const* KV, __nv_bfloat16* H, int64_t ldh,
                                 const __nv_bfloat16* const* W_qkv, const __nv_bfloat16* const* W_o, int32_t* sync,
                                 int32_t* status, cudaStream_t st, const dg4i_block_tail* block = nullptr);
