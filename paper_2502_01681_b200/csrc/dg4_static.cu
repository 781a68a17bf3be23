// dg4_layer_fwd_parallel_static: the all-nodes-parallel layer for callers that cannot allocate.
//
// The layer needs scratch for its intermediates (Q, K|V and O, 1 KiB per node).  The regular entry point
// takes that scratch from the caller, which means somebody called cudaMalloc (or a framework allocator)
// for it.  Some users of this library cannot: an inference service whose device memory is handed out once
// at start-up and then locked, a plug-in running inside a host application that owns the whole device heap,
// or a latency-critical loop where the implicit device-wide synchronisation of cudaMalloc / cudaFree is
// not acceptable.  For them the scratch lives in a fixed array that is part of the library image itself.
//
// The array is reserved on every GPU on which the library's image is instantiated (at load, or -- with the
// driver's lazy loading -- at the first call on that device) until the process exits, so it is kept modest:
// 32 MiB, i.e. circuits of at most 32 768 nodes.  All calls share it and nothing is cleared
// between calls -- every byte a call reads it has written itself first (Q, K|V and O rows of all its nodes),
// so stale contents are harmless -- but two calls that overlap in time on the GPU (different streams, or
// different host threads) would overwrite each other's intermediates: serialise them.
//
// `g_scratch` below is only a host-side handle in host code: it is not a device address and must never be
// handed to a kernel.  The device address is obtained once per device with cudaGetSymbolAddress while that
// device is current; this happens on the first call for that device (so make that first call outside any
// stream capture).

#include "dg4_internal.h"

#include <mutex>

namespace {

constexpr size_t kScratchBytes = (size_t)32 << 20;
constexpr int64_t kBytesPerNode = 1024;                       // Q 256 + K|V 512 + O 256
constexpr int64_t kMaxNodes = (int64_t)(kScratchBytes / kBytesPerNode);
constexpr int kMaxDevices = 64;

static __device__ __align__(256) unsigned char g_scratch[kScratchBytes];

std::mutex g_mu;
void* g_scratch_addr[kMaxDevices] = {};                       // device address of g_scratch, per device

// Resolves (once per device) the device address of the scratch array on the current device.
dg4_status scratch_for_current_device(int device, void** out) {
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_addr[device]) {
        void* p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_scratch);
        if (e != cudaSuccess || !p) {
            cudaGetLastError();
            DG4_FAIL(DG4_ERR_CUDA, "cudaGetSymbolAddress for the static scratch failed on device %d: %s", device,
                     cudaGetErrorString(e));
        }
        g_scratch_addr[device] = p;
    }
    *out = g_scratch_addr[device];
    return DG4_OK;
}

}  // namespace

extern "C" int64_t dg4_static_max_nodes(void) { return kMaxNodes; }

extern "C" dg4_status dg4_layer_fwd_parallel_static(const dg4_graph* g, const dg4_desc* desc, const void* H_in,
                                                     int64_t ldh, const void* W_qkv, const void* W_o, void* H_out,
                                                     int64_t ldho, void* stream) {
    dg4_status s = dg4i_check_device(g);
    if (s != DG4_OK) return s;
    if ((s = dg4i_check_desc(desc, true)) != DG4_OK) return s;
    if (desc->heads > 16) DG4_FAIL(DG4_ERR_UNSUPPORTED, "heads = %d: must be a power of two up to 16", desc->heads);
    if (g->n > kMaxNodes)
        DG4_FAIL(DG4_ERR_INVALID_ARG,
                 "graph has %d nodes; the static scratch (%zu bytes) holds at most %lld -- use dg4_layer_fwd_parallel "
                 "with a caller-provided workspace", g->n, kScratchBytes, (long long)kMaxNodes);
    if ((s = dg4i_check_tensor("H_in", H_in, ldh, 2, 128)) != DG4_OK) return s;
    if ((s = dg4i_check_tensor("H_out", H_out, ldho, 2, 128)) != DG4_OK) return s;
    if ((s = dg4i_check_tensor("W_qkv", W_qkv, 128, 2, 128)) != DG4_OK) return s;
    if ((s = dg4i_check_tensor("W_o", W_o, 128, 2, 128)) != DG4_OK) return s;
    if (H_out == H_in && ldh != ldho) DG4_FAIL(DG4_ERR_INVALID_ARG, "in-place use needs equal leading dimensions");
    const int cur = g->device;                      // checked above: it is the current device
    if (cur < 0 || cur >= kMaxDevices) DG4_FAIL(DG4_ERR_UNSUPPORTED, "device ordinal %d is out of range", cur);

    void* base = nullptr;
    if ((s = scratch_for_current_device(cur, &base)) != DG4_OK) return s;

    cudaStream_t st = (cudaStream_t)stream;
    const int64_t n = g->n;
    __nv_bfloat16* Q = (__nv_bfloat16*)base;
    __nv_bfloat16* KV = (__nv_bfloat16*)((char*)base + (size_t)n * 256);
    __nv_bfloat16* O = (__nv_bfloat16*)((char*)base + (size_t)n * 768);

    dg4i_proj_args p;
    p.A = (const __nv_bfloat16*)H_in; p.lda = ldh; p.W = (const __nv_bfloat16*)W_qkv; p.n_out = 384;
    p.out[0] = Q; p.ldo[0] = 128; p.out[1] = KV; p.ldo[1] = 256; p.out[2] = KV + 128; p.ldo[2] = 256;
    p.R = nullptr; p.ldr = 0; p.row_list = nullptr; p.first = 0; p.rows = g->n; p.status = g->dev_status;
    if ((s = dg4i_proj_launch(p, st)) != DG4_OK) return s;

    dg4i_attn_args a;
    a.Q = Q; a.ldq = 128; a.K = KV; a.ldk = 256; a.V = KV + 128; a.ldv = 256; a.O = O; a.ldo = 128;
    a.nbr_pad = g->nbr_pad; a.node_list = nullptr; a.first = 0; a.count = g->n;
    a.heads = desc->heads; a.max_nbr = g->max_class; a.dtype = DG4_BF16; a.scale = desc->scale;
    dg4i_attn_more more;
    more.nbr_ptr = g->nbr_ptr; more.nbr_idx = g->nbr_idx;
    if ((s = dg4i_attn_launch(a, &more, st)) != DG4_OK) return s;

    dg4i_proj_args o;
    o.A = O; o.lda = 128; o.W = (const __nv_bfloat16*)W_o; o.n_out = 128;
    o.out[0] = (__nv_bfloat16*)H_out; o.ldo[0] = ldho; o.out[1] = o.out[2] = nullptr; o.ldo[1] = o.ldo[2] = 0;
    o.R = (desc->flags & DG4_FLAG_RESIDUAL) ? (const __nv_bfloat16*)H_in : nullptr; o.ldr = ldh;
    o.row_list = nullptr; o.first = 0; o.rows = g->n; o.status = g->dev_status;
    return dg4i_proj_launch(o, st);
}
