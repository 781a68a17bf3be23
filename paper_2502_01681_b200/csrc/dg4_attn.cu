// Fused sparse attention over the neighbourhood lists (Sec. 3.5): per node and head, dot-product scores
// against at most 7 neighbours, softmax over them, weighted sum of value rows -- in one pass, with the
// scores held in registers (nothing per-edge is written to memory).
//
// Mapping (informed by Sec. 3.7's observation that a warp per node idles 30 of 32 lanes at in-degree <= 2):
// lanes are spread over the FEATURE dimension, not over the edges.  A row of d = 128 elements is split into
// 16-byte pieces, one per lane: 16 lanes per node for bf16 (two nodes per warp), 32 lanes for fp32.  A head
// then spans LPH = lanes / heads adjacent lanes, so a score needs log2(LPH) shuffle steps (one for 8 heads
// in bf16) and the softmax needs no cross-lane traffic at all: every lane of a head holds all of that head's
// scores.  All K and V pieces of a node (up to 14 independent 16-byte loads per lane) are issued before the
// first use, which is what keeps HBM busy.  A node whose neighbourhood is only itself skips Q and K (its
// softmax weight is 1, the case the paper skips as well).

#include "dg4_internal.h"
#include "dg4_attn_core.cuh"

namespace {

using namespace attn;

// BF16: storage type.  LPH: lanes per head.  MAXN: upper bound of the neighbourhood size (3 or 7).
template <bool BF16, int LPH, int MAXN>
__global__ void __launch_bounds__(256) sparse_attn_kernel(dg4i_attn_args a) {
    constexpr int G = BF16 ? 16 : 32;              // lanes per node
    constexpr int EPP = Elem<BF16>::kPerPiece;     // elements per 16-byte piece
    constexpr int ES = BF16 ? 2 : 4;
    const int lane = threadIdx.x & 31;
    const int sub = lane & (G - 1);                // lane within the node's group
    const int grp_base = lane - sub;               // first lane of the group inside the warp
    int slot = (int)(((int64_t)blockIdx.x * blockDim.x + threadIdx.x) / G);
    const bool live = slot < a.count;
    if (!live) slot = a.count - 1;                 // keep whole warps converged for the shuffles
    const int v = a.node_list ? a.node_list[a.first + slot] : a.first + slot;

    const int beg = a.nbr_ptr[v];
    const int cnt = a.nbr_ptr[v + 1] - beg;
    int my_idx = (sub < cnt) ? a.nbr_idx[beg + sub] : v;

    const size_t col = (size_t)sub * EPP * ES;     // byte offset of this lane's piece inside a row
    Piece kq[MAXN], vq[MAXN], qp;
    int u[MAXN];
#pragma unroll
    for (int j = 0; j < MAXN; ++j) u[j] = __shfl_sync(0xffffffffu, my_idx, grp_base + j);
#pragma unroll
    for (int j = 0; j < MAXN; ++j)
        if (j < cnt) vq[j] = ld_piece_nc((const char*)a.V + (size_t)u[j] * a.ldv * ES + col);
    if (cnt > 1) {
        qp = ld_piece_stream((const char*)a.Q + (size_t)v * a.ldq * ES + col);
#pragma unroll
        for (int j = 0; j < MAXN; ++j)
            if (j < cnt) kq[j] = ld_piece_nc((const char*)a.K + (size_t)u[j] * a.ldk * ES + col);
    }
    float acc[EPP];
    const unsigned mask = (G == 32) ? 0xffffffffu : (0xffffu << grp_base);
    attend<BF16, LPH, MAXN>(qp, kq, vq, cnt, a.scale, mask, acc);
    if (live) st_piece_stream((char*)a.O + (size_t)v * a.ldo * ES + col, Elem<BF16>::pack(acc));
}

template <bool BF16, int MAXN>
dg4_status launch_for_heads(const dg4i_attn_args& a, cudaStream_t st) {
    constexpr int G = BF16 ? 16 : 32;
    const int threads = 256;
    const int nodes_per_block = threads / G;
    const unsigned blocks = (unsigned)((a.count + nodes_per_block - 1) / nodes_per_block);
    const int lph = G / a.heads;
    switch (lph) {
        case 1: sparse_attn_kernel<BF16, 1, MAXN><<<blocks, threads, 0, st>>>(a); break;
        case 2: sparse_attn_kernel<BF16, 2, MAXN><<<blocks, threads, 0, st>>>(a); break;
        case 4: sparse_attn_kernel<BF16, 4, MAXN><<<blocks, threads, 0, st>>>(a); break;
        case 8: sparse_attn_kernel<BF16, 8, MAXN><<<blocks, threads, 0, st>>>(a); break;
        case 16: sparse_attn_kernel<BF16, 16, MAXN><<<blocks, threads, 0, st>>>(a); break;
        case 32: sparse_attn_kernel<BF16, 32, MAXN><<<blocks, threads, 0, st>>>(a); break;
        default: DG4_FAIL(DG4_ERR_UNSUPPORTED, "heads = %d is not supported for this dtype", a.heads);
    }
    dg4i_count_launch();
    DG4_CUDA_TRY(cudaGetLastError());
    return DG4_OK;
}

}  // namespace

dg4_status dg4i_attn_launch(const dg4i_attn_args& a, cudaStream_t st) {
    if (a.count <= 0) return DG4_OK;
    const bool bf16 = a.dtype == DG4_BF16;
    const int G = bf16 ? 16 : 32;
    if (a.heads < 1 || a.heads > G || (G % a.heads) != 0)
        DG4_FAIL(DG4_ERR_UNSUPPORTED, "heads = %d: must divide %d", a.heads, G);
    if (a.max_nbr <= 3) return bf16 ? launch_for_heads<true, 3>(a, st) : launch_for_heads<false, 3>(a, st);
    return bf16 ? launch_for_heads<true, 7>(a, st) : launch_for_heads<false, 7>(a, st);
}
