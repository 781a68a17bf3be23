// Public forward entry points: argument checks, then launches on the caller's stream.
// The all-parallel layer is QKV projection -> sparse attention -> output projection over all nodes.
// The levelised layer (Sec. 1 / Sec. 3.4: strict topological order, each gate computed once) projects
// Q|K|V of every node from the layer's input once -- a node's own query, key and value always come from
// its row as it was at the start of the layer -- and then, level by level, runs the attention for that
// level's nodes, writes their new rows, and refreshes their K|V rows so that higher levels gather the
// updated ones.  By default that walk is one persistent kernel (dg4_levelised.cu), which can also run several
// layers as a wavefront; with DG4_FLAG_LEVEL_LAUNCHES it is one group of launches per level (kept for
// comparison, and the only levelised driver for cones wider than two hops).

#include "dg4_internal.h"

#include <string.h>
#include <atomic>

namespace {

thread_local char g_err[512] = "";
thread_local int g_device_override = -1;      // dg4_debug_override_current_device
std::atomic<long long> g_launches{0};
std::atomic<uint32_t> g_poll_limit{DG4I_DEFAULT_POLL_LIMIT};

bool aligned16(const void* p) { return (((uintptr_t)p) & 15u) == 0; }

}  // namespace

dg4_status dg4i_check_device(const dg4_graph* g) {
    if (!g) DG4_FAIL(DG4_ERR_INVALID_ARG, "null graph");
    int cur = g_device_override;
    if (cur < 0) DG4_CUDA_TRY(cudaGetDevice(&cur));
    if (cur != g->device)
        DG4_FAIL(DG4_ERR_INVALID_ARG, "the graph lives on device %d but device %d is current", g->device, cur);
    return DG4_OK;
}

uint32_t dg4i_poll_limit() { return g_poll_limit.load(std::memory_order_relaxed); }

extern "C" void dg4_debug_override_current_device(int32_t device) { g_device_override = device; }

extern "C" void dg4_debug_set_poll_limit(uint32_t polls) {
    g_poll_limit.store(polls ? polls : DG4I_DEFAULT_POLL_LIMIT, std::memory_order_relaxed);
}

dg4_status dg4i_check_desc(const dg4_desc* d, bool need_bf16) {
    if (!d) DG4_FAIL(DG4_ERR_INVALID_ARG, "null descriptor");
    if (d->d != 128) DG4_FAIL(DG4_ERR_UNSUPPORTED, "d = %d: only d = 128 is supported", d->d);
    if (d->dtype != DG4_F32 && d->dtype != DG4_BF16) DG4_FAIL(DG4_ERR_UNSUPPORTED, "unknown dtype %d", d->dtype);
    if (need_bf16 && d->dtype != DG4_BF16) DG4_FAIL(DG4_ERR_UNSUPPORTED, "projections are bf16 only");
    const int lanes = d->dtype == DG4_BF16 ? 16 : 32;
    if (d->heads < 1 || d->heads > lanes || (lanes % d->heads) != 0)
        DG4_FAIL(DG4_ERR_UNSUPPORTED, "heads = %d: must be a power of two up to %d", d->heads, lanes);
    if (!(d->scale == d->scale) || d->scale > 3.0e38f || d->scale < -3.0e38f)
        DG4_FAIL(DG4_ERR_INVALID_ARG, "scale is not finite");
    return DG4_OK;
}

dg4_status dg4i_check_tensor(const char* name, const void* p, int64_t ld, int elem_size, int min_ld) {
    if (!p) DG4_FAIL(DG4_ERR_INVALID_ARG, "%s is null", name);
    if (!aligned16(p)) DG4_FAIL(DG4_ERR_INVALID_ARG, "%s is not 16-byte aligned", name);
    if (ld < min_ld) DG4_FAIL(DG4_ERR_INVALID_ARG, "leading dimension of %s (%lld) is below %d", name, (long long)ld, min_ld);
    if ((ld * elem_size) % 16 != 0)
        DG4_FAIL(DG4_ERR_INVALID_ARG, "leading dimension of %s (%lld elements) is not a multiple of 16 bytes", name, (long long)ld);
    return DG4_OK;
}

namespace {

#define CHECK(expr) do { dg4_status _s = (expr); if (_s != DG4_OK) return _s; } while (0)
#define check_desc dg4i_check_desc
#define check_tensor dg4i_check_tensor

struct Workspace {
    __nv_bfloat16* Q;    // [n, 128]
    __nv_bfloat16* KV;   // [n, 256]: K | V interleaved per node (one 512-byte stretch per neighbour)
    __nv_bfloat16* O;    // [n, 128]
};

size_t tensors_bytes(int64_t n) { return ((size_t)n * 128 * 2 * 4 + 255) & ~(size_t)255; }
size_t sync_bytes(const dg4_graph* g, int n_layers) { return (dg4i_levelised_sync_bytes(g, n_layers) + 255) & ~(size_t)255; }
size_t workspace_bytes(const dg4_graph* g) { return tensors_bytes(g->n) + sync_bytes(g, 1); }
// several levelised layers in one call: per layer a K|V table [n,256], then the counters
size_t layer_tables_bytes(int64_t n) { return ((size_t)n * 512 + 255) & ~(size_t)255; }
size_t layers_workspace_bytes(const dg4_graph* g, int n_layers) {
    size_t multi = layer_tables_bytes(g->n) * (size_t)n_layers + sync_bytes(g, n_layers);
    size_t single = workspace_bytes(g);          // the per-level-launch driver reuses one layer's workspace
    return multi > single ? multi : single;
}

Workspace carve(void* ws, int64_t n) {
    Workspace w;
    char* p = (char*)ws;
    w.Q = (__nv_bfloat16*)p;
    w.KV = (__nv_bfloat16*)(p + (size_t)n * 256);
    w.O = (__nv_bfloat16*)(p + (size_t)n * 768);
    return w;
}

dg4i_attn_more attn_more(const dg4_graph* g) {
    dg4i_attn_more m;
    m.nbr_ptr = g->nbr_ptr; m.nbr_idx = g->nbr_idx;
    return m;
}

dg4i_attn_args attn_args(const dg4_graph* g, const dg4_desc* d, const void* Q, int64_t ldq, const void* K,
                         int64_t ldk, const void* V, int64_t ldv, void* O, int64_t ldo) {
    dg4i_attn_args a;
    a.Q = Q; a.ldq = ldq; a.K = K; a.ldk = ldk; a.V = V; a.ldv = ldv; a.O = O; a.ldo = ldo;
    a.nbr_pad = g->nbr_pad; a.node_list = nullptr; a.first = 0; a.count = g->n;
    a.heads = d->heads; a.max_nbr = g->max_class; a.dtype = d->dtype; a.scale = d->scale;
    return a;
}

}  // namespace

void dg4_set_error(const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
}

extern "C" const char* dg4_last_error(void) { return g_err; }

void dg4i_count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

extern "C" int64_t dg4_launch_count(void) { return (int64_t)g_launches.load(std::memory_order_relaxed); }

extern "C" const char* dg4_status_string(dg4_status s) {
    switch (s) {
        case DG4_OK: return "ok";
        case DG4_ERR_INVALID_ARG: return "invalid argument";
        case DG4_ERR_NOT_SORTED: return "CSR is not sorted by destination";
        case DG4_ERR_BAD_DEGREE: return "node with more than two fan-ins";
        case DG4_ERR_BAD_LEVEL: return "levels do not increase along an edge";
        case DG4_ERR_UNSUPPORTED: return "unsupported configuration";
        case DG4_ERR_ALLOC: return "allocation failed";
        case DG4_ERR_CUDA: return "CUDA error";
        case DG4_ERR_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

extern "C" dg4_status dg4_qkv_project(const dg4_graph* g, const dg4_desc* desc, const void* X, int64_t ldx,
                                       const void* W_qkv, void* Q, int64_t ldq, void* K, int64_t ldk, void* V,
                                       int64_t ldv, void* stream) {
    CHECK(dg4i_check_device(g));
    CHECK(check_desc(desc, true));
    CHECK(check_tensor("X", X, ldx, 2, 128));
    CHECK(check_tensor("W_qkv", W_qkv, 128, 2, 128));
    CHECK(check_tensor("Q", Q, ldq, 2, 128));
    CHECK(check_tensor("K", K, ldk, 2, 128));
    CHECK(check_tensor("V", V, ldv, 2, 128));
    dg4i_proj_args a;
    a.A = (const __nv_bfloat16*)X; a.lda = ldx; a.W = (const __nv_bfloat16*)W_qkv; a.n_out = 384;
    a.out[0] = (__nv_bfloat16*)Q; a.ldo[0] = ldq;
    a.out[1] = (__nv_bfloat16*)K; a.ldo[1] = ldk;
    a.out[2] = (__nv_bfloat16*)V; a.ldo[2] = ldv;
    a.R = nullptr; a.ldr = 0; a.row_list = nullptr; a.first = 0; a.rows = g->n; a.status = g->dev_status;
    return dg4i_proj_launch(a, (cudaStream_t)stream);
}

extern "C" dg4_status dg4_sparse_attn_fwd(const dg4_graph* g, const dg4_desc* desc, const void* Q, int64_t ldq,
                                           const void* K, int64_t ldk, const void* V, int64_t ldv, void* O,
                                           int64_t ldo, void* stream) {
    CHECK(dg4i_check_device(g));
    CHECK(check_desc(desc, false));
    const int es = desc->dtype == DG4_BF16 ? 2 : 4;
    CHECK(check_tensor("Q", Q, ldq, es, 128));
    CHECK(check_tensor("K", K, ldk, es, 128));
    CHECK(check_tensor("V", V, ldv, es, 128));
    CHECK(check_tensor("O", O, ldo, es, 128));
    if (O == K || O == V) DG4_FAIL(DG4_ERR_INVALID_ARG, "O must not alias K or V");
    const dg4i_attn_more more = attn_more(g);
    return dg4i_attn_launch(attn_args(g, desc, Q, ldq, K, ldk, V, ldv, O, ldo), &more, (cudaStream_t)stream);
}

extern "C" dg4_status dg4_sparse_attn_additive_fwd(const dg4_graph* g, const dg4_desc* desc, const float* S_dst,
                                                    const float* S_src, float negative_slope, const void* V,
                                                    int64_t ldv, void* O, int64_t ldo, void* stream) {
    CHECK(dg4i_check_device(g));
    CHECK(check_desc(desc, false));
    if (!S_dst || !S_src) DG4_FAIL(DG4_ERR_INVALID_ARG, "null score array");
    if ((((uintptr_t)S_dst) | ((uintptr_t)S_src)) & 3u) DG4_FAIL(DG4_ERR_INVALID_ARG, "score arrays must be 4-byte aligned");
    if (!(negative_slope == negative_slope)) DG4_FAIL(DG4_ERR_INVALID_ARG, "negative_slope is not a number");
    const int es = desc->dtype == DG4_BF16 ? 2 : 4;
    CHECK(check_tensor("V", V, ldv, es, 128));
    CHECK(check_tensor("O", O, ldo, es, 128));
    if (O == V) DG4_FAIL(DG4_ERR_INVALID_ARG, "O must not alias V");
    dg4i_attn_args a = attn_args(g, desc, nullptr, 0, nullptr, 0, V, ldv, O, ldo);
    dg4i_attn_more more = attn_more(g);
    more.s_dst = S_dst; more.s_src = S_src; more.slope = negative_slope;
    return dg4i_attn_additive_launch(a, more, (cudaStream_t)stream);
}

extern "C" dg4_status dg4_out_project(const dg4_graph* g, const dg4_desc* desc, const void* O, int64_t ldo,
                                       const void* W_o, const void* H_res, int64_t ldh, void* H_out, int64_t ldho,
                                       void* stream) {
    CHECK(dg4i_check_device(g));
    CHECK(check_desc(desc, true));
    CHECK(check_tensor("O", O, ldo, 2, 128));
    CHECK(check_tensor("W_o", W_o, 128, 2, 128));
    CHECK(check_tensor("H_out", H_out, ldho, 2, 128));
    const bool res = (desc->flags & DG4_FLAG_RESIDUAL) && H_res;
    if (res) CHECK(check_tensor("H_res", H_res, ldh, 2, 128));
    if (H_out == O) DG4_FAIL(DG4_ERR_INVALID_ARG, "H_out must not alias O");
    dg4i_proj_args a;
    a.A = (const __nv_bfloat16*)O; a.lda = ldo; a.W = (const __nv_bfloat16*)W_o; a.n_out = 128;
    a.out[0] = (__nv_bfloat16*)H_out; a.ldo[0] = ldho; a.out[1] = a.out[2] = nullptr; a.ldo[1] = a.ldo[2] = 0;
    a.R = res ? (const __nv_bfloat16*)H_res : nullptr; a.ldr = ldh; a.row_list = nullptr; a.first = 0; a.rows = g->n;
    a.status = g->dev_status;
    return dg4i_proj_launch(a, (cudaStream_t)stream);
}

extern "C" size_t dg4_layer_workspace_bytes(const dg4_graph* g, const dg4_desc* desc) {
    (void)desc;
    return g ? workspace_bytes(g) : 0;
}

namespace {
dg4_status check_layer_args(const dg4_graph* g, const dg4_desc* desc, const void* H, int64_t ldh, const void* W_qkv,
                            const void* W_o, void* ws, size_t ws_bytes) {
    CHECK(dg4i_check_device(g));
    CHECK(check_desc(desc, true));
    CHECK(check_tensor("H", H, ldh, 2, 128));
    CHECK(check_tensor("W_qkv", W_qkv, 128, 2, 128));
    CHECK(check_tensor("W_o", W_o, 128, 2, 128));
    if (!ws) DG4_FAIL(DG4_ERR_INVALID_ARG, "workspace is null");
    if ((((uintptr_t)ws) & 255u) != 0) DG4_FAIL(DG4_ERR_INVALID_ARG, "workspace is not 256-byte aligned");
    if (ws_bytes < workspace_bytes(g))
        DG4_FAIL(DG4_ERR_INVALID_ARG, "workspace of %zu bytes is below the %zu bytes needed", ws_bytes, workspace_bytes(g));
    return DG4_OK;
}
}  // namespace

extern "C" dg4_status dg4_layer_fwd_parallel(const dg4_graph* g, const dg4_desc* desc, const void* H_in, int64_t ldh,
                                              const void* W_qkv, const void* W_o, void* H_out, int64_t ldho,
                                              void* workspace, size_t workspace_bytes_, void* stream) {
    CHECK(check_layer_args(g, desc, H_in, ldh, W_qkv, W_o, workspace, workspace_bytes_));
    CHECK(check_tensor("H_out", H_out, ldho, 2, 128));
    if (H_out == H_in && ldh != ldho) DG4_FAIL(DG4_ERR_INVALID_ARG, "in-place use needs equal leading dimensions");
    cudaStream_t st = (cudaStream_t)stream;
    Workspace w = carve(workspace, g->n);
    int32_t* status_word = g->dev_status;

    if ((desc->flags & DG4_FLAG_FUSED_LAYER) && dg4i_fused_layer_supported(g, desc)) {
        // K | V of every node first (every node may be gathered by any other), then one kernel for the rest:
        // queries from the X tiles, attention, output projection, residual -- Q and O never leave the chip
        dg4i_proj_args kv;
        kv.A = (const __nv_bfloat16*)H_in; kv.lda = ldh; kv.W = (const __nv_bfloat16*)W_qkv + (size_t)128 * 128; kv.n_out = 256;
        kv.out[0] = w.KV; kv.ldo[0] = 256; kv.out[1] = w.KV + 128; kv.ldo[1] = 256; kv.out[2] = nullptr; kv.ldo[2] = 0;
        kv.R = nullptr; kv.ldr = 0; kv.row_list = nullptr; kv.first = 0; kv.rows = g->n; kv.status = status_word;
        CHECK(dg4i_proj_launch(kv, st));
        return dg4i_fused_layer_launch(g, desc, (const __nv_bfloat16*)H_in, ldh, w.KV, (const __nv_bfloat16*)W_qkv,
                                       (const __nv_bfloat16*)W_o, (__nv_bfloat16*)H_out, ldho, status_word, st);
    }

    dg4i_proj_args p;
    p.A = (const __nv_bfloat16*)H_in; p.lda = ldh; p.W = (const __nv_bfloat16*)W_qkv; p.n_out = 384;
    p.out[0] = w.Q; p.ldo[0] = 128; p.out[1] = w.KV; p.ldo[1] = 256; p.out[2] = w.KV + 128; p.ldo[2] = 256;
    p.R = nullptr; p.ldr = 0; p.row_list = nullptr; p.first = 0; p.rows = g->n; p.status = status_word;
    CHECK(dg4i_proj_launch(p, st));

    const dg4i_attn_more more = attn_more(g);
    CHECK(dg4i_attn_launch(attn_args(g, desc, w.Q, 128, w.KV, 256, w.KV + 128, 256, w.O, 128), &more, st));

    dg4i_proj_args o;
    o.A = w.O; o.lda = 128; o.W = (const __nv_bfloat16*)W_o; o.n_out = 128;
    o.out[0] = (__nv_bfloat16*)H_out; o.ldo[0] = ldho; o.out[1] = o.out[2] = nullptr; o.ldo[1] = o.ldo[2] = 0;
    o.R = (desc->flags & DG4_FLAG_RESIDUAL) ? (const __nv_bfloat16*)H_in : nullptr; o.ldr = ldh;
    o.row_list = nullptr; o.first = 0; o.rows = g->n; o.status = status_word;
    return dg4i_proj_launch(o, st);
}

extern "C" dg4_status dg4_layer_fwd_levelised(const dg4_graph* g, const dg4_desc* desc, void* H, int64_t ldh,
                                               const void* W_qkv, const void* W_o, void* workspace,
                                               size_t workspace_bytes_, int32_t* device_status, void* stream) {
    CHECK(check_layer_args(g, desc, H, ldh, W_qkv, W_o, workspace, workspace_bytes_));
    cudaStream_t st = (cudaStream_t)stream;
    Workspace w = carve(workspace, g->n);
    if (device_status) DG4_CUDA_TRY(cudaMemsetAsync(device_status, 0, sizeof(int32_t), st));
    int32_t* status_word = device_status ? device_status : g->dev_status;

    if (!(desc->flags & DG4_FLAG_LEVEL_LAUNCHES)) {
        // one persistent kernel walks the levels; it projects each tile's own Q | K | V on the fly and fills the
        // K | V table as nodes are updated
        int32_t* sync = (int32_t*)((char*)workspace + tensors_bytes(g->n));
        __nv_bfloat16* kv1[1] = {w.KV};
        const __nv_bfloat16* wq1[1] = {(const __nv_bfloat16*)W_qkv};
        const __nv_bfloat16* wo1[1] = {(const __nv_bfloat16*)W_o};
        return dg4i_levelised_launch(g, desc, 1, kv1, (__nv_bfloat16*)H, ldh, wq1, wo1, sync, status_word, st);
    }

    // Q | K | V of every node from the layer's input
    dg4i_proj_args p;
    p.A = (const __nv_bfloat16*)H; p.lda = ldh; p.W = (const __nv_bfloat16*)W_qkv; p.n_out = 384;
    p.out[0] = w.Q; p.ldo[0] = 128; p.out[1] = w.KV; p.ldo[1] = 256; p.out[2] = w.KV + 128; p.ldo[2] = 256;
    p.R = nullptr; p.ldr = 0; p.row_list = nullptr; p.first = 0; p.rows = g->n; p.status = status_word;
    CHECK(dg4i_proj_launch(p, st));

    // alternative driver: one group of launches per level (attention, output projection, K|V refresh)
    const __nv_bfloat16* W_kv = (const __nv_bfloat16*)W_qkv + (size_t)128 * 128;
    for (int l = 0; l < g->n_levels; ++l) {
        const int first = g->h_level_ptr[l], count = g->h_level_ptr[l + 1] - first;
        if (count <= 0) continue;
        dg4i_attn_args a = attn_args(g, desc, w.Q, 128, w.KV, 256, w.KV + 128, 256, w.O, 128);
        a.node_list = g->level_nodes; a.first = first; a.count = count;
        const dg4i_attn_more more = attn_more(g);
        CHECK(dg4i_attn_launch(a, &more, st));

        dg4i_proj_args o;
        o.A = w.O; o.lda = 128; o.W = (const __nv_bfloat16*)W_o; o.n_out = 128;
        o.out[0] = (__nv_bfloat16*)H; o.ldo[0] = ldh; o.out[1] = o.out[2] = nullptr; o.ldo[1] = o.ldo[2] = 0;
        o.R = (desc->flags & DG4_FLAG_RESIDUAL) ? (const __nv_bfloat16*)H : nullptr; o.ldr = ldh;
        o.row_list = g->level_nodes; o.first = first; o.rows = count; o.status = status_word;
        CHECK(dg4i_proj_launch(o, st));

        if (l + 1 < g->n_levels) {   // refresh K | V of the finished level for the levels above
            dg4i_proj_args k;
            k.A = (const __nv_bfloat16*)H; k.lda = ldh; k.W = W_kv; k.n_out = 256;
            k.out[0] = w.KV; k.ldo[0] = 256; k.out[1] = w.KV + 128; k.ldo[1] = 256; k.out[2] = nullptr; k.ldo[2] = 0;
            k.R = nullptr; k.ldr = 0; k.row_list = g->level_nodes; k.first = first; k.rows = count; k.status = status_word;
            CHECK(dg4i_proj_launch(k, st));
        }
    }
    return DG4_OK;
}

extern "C" size_t dg4_layers_workspace_bytes(const dg4_graph* g, const dg4_desc* desc, int32_t n_layers) {
    (void)desc;
    if (!g || n_layers < 1 || n_layers > DG4I_MAX_LAYERS) return 0;
    return layers_workspace_bytes(g, n_layers);
}

extern "C" dg4_status dg4_layers_fwd_levelised(const dg4_graph* g, const dg4_desc* desc, void* H, int64_t ldh,
                                                int32_t n_layers, const void* const* W_qkv, const void* const* W_o,
                                                void* workspace, size_t workspace_bytes_, int32_t* device_status,
                                                void* stream) {
    CHECK(dg4i_check_device(g));
    if (n_layers < 1 || n_layers > DG4I_MAX_LAYERS)
        DG4_FAIL(DG4_ERR_UNSUPPORTED, "n_layers = %d: between 1 and %d layers per call", n_layers, DG4I_MAX_LAYERS);
    if (!W_qkv || !W_o) DG4_FAIL(DG4_ERR_INVALID_ARG, "null weight list");
    CHECK(check_desc(desc, true));
    CHECK(check_tensor("H", H, ldh, 2, 128));
    for (int k = 0; k < n_layers; ++k) {
        CHECK(check_tensor("W_qkv[k]", W_qkv[k], 128, 2, 128));
        CHECK(check_tensor("W_o[k]", W_o[k], 128, 2, 128));
    }
    if (!workspace) DG4_FAIL(DG4_ERR_INVALID_ARG, "workspace is null");
    if ((((uintptr_t)workspace) & 255u) != 0) DG4_FAIL(DG4_ERR_INVALID_ARG, "workspace is not 256-byte aligned");
    if (workspace_bytes_ < layers_workspace_bytes(g, n_layers))
        DG4_FAIL(DG4_ERR_INVALID_ARG, "workspace of %zu bytes is below the %zu bytes needed", workspace_bytes_,
                 layers_workspace_bytes(g, n_layers));
    cudaStream_t st = (cudaStream_t)stream;

    if (desc->flags & DG4_FLAG_LEVEL_LAUNCHES) {       // comparison driver: layer after layer, a launch group per level
        for (int k = 0; k < n_layers; ++k)
            CHECK(dg4_layer_fwd_levelised(g, desc, H, ldh, W_qkv[k], W_o[k], workspace, workspace_bytes_, device_status, stream));
        return DG4_OK;
    }

    if (device_status) DG4_CUDA_TRY(cudaMemsetAsync(device_status, 0, sizeof(int32_t), st));
    int32_t* status_word = device_status ? device_status : g->dev_status;
    __nv_bfloat16* kv[DG4I_MAX_LAYERS];
    const __nv_bfloat16* wq[DG4I_MAX_LAYERS];
    const __nv_bfloat16* wo[DG4I_MAX_LAYERS];
    const size_t per_layer = layer_tables_bytes(g->n);
    for (int k = 0; k < n_layers; ++k) {
        kv[k] = (__nv_bfloat16*)((char*)workspace + per_layer * (size_t)k);
        wq[k] = (const __nv_bfloat16*)W_qkv[k];
        wo[k] = (const __nv_bfloat16*)W_o[k];
    }
    int32_t* sync = (int32_t*)((char*)workspace + per_layer * (size_t)n_layers);
    // every layer projects its tiles' own Q | K | V on the fly and fills its K | V table as nodes are updated
    return dg4i_levelised_launch(g, desc, n_layers, kv, (__nv_bfloat16*)H, ldh, wq, wo, sync, status_word, st);
}
