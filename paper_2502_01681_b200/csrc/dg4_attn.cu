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

// resident blocks per SM the compiler must allow for (caps registers per thread)
#ifndef DG4_ATTN_THREADS
#define DG4_ATTN_THREADS 256
#endif
#ifndef DG4_ATTN_MIN_BLOCKS
#define DG4_ATTN_MIN_BLOCKS 3
#endif
// L2 eviction priority of the gathered K | V rows: 1 = ask L2 to keep them (they are gathered again by later nodes)
#ifndef DG4_ATTN_KV_EVICT_LAST
#define DG4_ATTN_KV_EVICT_LAST 0
#endif
// neighbour-table entries are read once: 1 = ask L2 to drop them first
#ifndef DG4_ATTN_PAD_EVICT_FIRST
#define DG4_ATTN_PAD_EVICT_FIRST 0
#endif
// warp-per-node kernel for wider cones: neighbours in flight per half-warp, and resident blocks per SM
#ifndef DG4_WIDE_UN
#define DG4_WIDE_UN 4
#endif
#ifndef DG4_WIDE_MIN_BLOCKS
#define DG4_WIDE_MIN_BLOCKS 3      // measured: 3 blocks of 8 warps beat 4 (8.6 vs 9.5 ms on the 1M-node circuit, 8 hops)
#endif
// 1 = the value rows of table slots beyond |N(v)| are not loaded (the key rows still are, unpredicated)
#ifndef DG4_ATTN_V_PREDICATED
#define DG4_ATTN_V_PREDICATED 0
#endif

namespace {

using namespace attn;

// BF16: storage type.  LPH: lanes per head.  MAXN: upper bound of the neighbourhood size (3 or 7).
// Persistent: a group of G lanes walks the nodes slot, slot + (groups in the grid), ... so that the nodes in
// flight across the GPU at any moment are a contiguous id range (their gathered rows overlap in L2).  The
// fixed-width neighbour entry of the NEXT node is fetched while the current node's rows are in flight, which
// takes the index lookup off the per-node dependency chain (one memory round trip per node instead of three).
template <bool BF16, int LPH, int MAXN>
__global__ void __launch_bounds__(DG4_ATTN_THREADS, DG4_ATTN_MIN_BLOCKS) sparse_attn_kernel(dg4i_attn_args a) {
    constexpr int G = BF16 ? 16 : 32;              // lanes per node
    constexpr int EPP = Elem<BF16>::kPerPiece;     // elements per 16-byte piece
    constexpr int ES = BF16 ? 2 : 4;
    constexpr int W = MAXN + 1;                    // width of a neighbour-table entry
    const int lane = threadIdx.x & 31;
    const int sub = lane & (G - 1);                // lane within the node's group
    const int grp_base = lane - sub;               // first lane of the group inside the warp
    const unsigned mask = (G == 32) ? 0xffffffffu : (0xffffu << grp_base);
    const int stride = (int)(gridDim.x * (blockDim.x / G));
    int slot = (int)((blockIdx.x * blockDim.x + threadIdx.x) / G);
    const size_t col = (size_t)sub * EPP * ES;     // byte offset of this lane's piece inside a row

#if DG4_ATTN_KV_EVICT_LAST
    const uint64_t keep = l2_policy_evict_last();
#define DG4_LD_KV(ptr) ld_piece_nc_hint(ptr, keep)
#else
#define DG4_LD_KV(ptr) ld_piece_nc(ptr)
#endif
#if DG4_ATTN_PAD_EVICT_FIRST
    const uint64_t drop = l2_policy_evict_first();
#define DG4_LD_PAD(ptr) ld_int_nc_hint(ptr, drop)
#else
#define DG4_LD_PAD(ptr) (*(ptr))
#endif
    int v_next = -1, pad_next = 0;
    if (slot < a.count) {
        v_next = a.node_list ? a.node_list[a.first + slot] : a.first + slot;
        if (sub < W) pad_next = DG4_LD_PAD(a.nbr_pad + (size_t)v_next * W + sub);
    }
    for (; slot < a.count; slot += stride) {
        const int v = v_next;
        const int pad = pad_next;
        {   // next node of this group: its table entry arrives while this node's rows are gathered
            const int s2 = slot + stride;
            if (s2 < a.count) {
                v_next = a.node_list ? a.node_list[a.first + s2] : a.first + s2;
                if (sub < W) pad_next = DG4_LD_PAD(a.nbr_pad + (size_t)v_next * W + sub);
            }
        }
        const int cnt = __shfl_sync(mask, pad, grp_base);
        Piece kq[MAXN], vq[MAXN], qp;
        int u[MAXN];
        u[0] = v;
#pragma unroll
        for (int j = 1; j < MAXN; ++j) u[j] = __shfl_sync(mask, pad, grp_base + j);
        // The filler entries of the table repeat v, so every slot names a valid row: all 2 * MAXN + 1 loads are
        // issued without predicates (slots beyond cnt re-read the node's own row, a cache hit), which saves the
        // branches and lets the kernel fit three blocks per SM; the arithmetic below still stops at cnt.
        qp = ld_piece_stream((const char*)a.Q + (size_t)v * a.ldq * ES + col);
#pragma unroll
        for (int j = 0; j < MAXN; ++j) kq[j] = DG4_LD_KV((const char*)a.K + (size_t)u[j] * a.ldk * ES + col);
#pragma unroll
        for (int j = 0; j < MAXN; ++j) {
#if DG4_ATTN_V_PREDICATED
            if (j < cnt)
#endif
            vq[j] = DG4_LD_KV((const char*)a.V + (size_t)u[j] * a.ldv * ES + col);
        }
        float acc[EPP];
        attend<BF16, LPH, MAXN>(qp, kq, vq, cnt, a.scale, mask, acc);
        st_piece_stream((char*)a.O + (size_t)v * a.ldo * ES + col, Elem<BF16>::pack(acc));
    }
#undef DG4_LD_KV
#undef DG4_LD_PAD
}

// Additive (GAT-style) scores: e = LeakyReLU(S_src[u, head] + S_dst[v, head]) from node-level scalars, so a
// neighbour costs one value row and one 4-byte scalar per head instead of a key row; same persistent walk.
template <bool BF16, int LPH, int MAXN>
__global__ void __launch_bounds__(DG4_ATTN_THREADS, DG4_ATTN_MIN_BLOCKS) sparse_attn_additive_kernel(dg4i_attn_args a, dg4i_attn_more x) {
    constexpr int G = BF16 ? 16 : 32;
    constexpr int EPP = Elem<BF16>::kPerPiece;
    constexpr int ES = BF16 ? 2 : 4;
    constexpr int W = MAXN + 1;
    const int lane = threadIdx.x & 31;
    const int sub = lane & (G - 1);
    const int grp_base = lane - sub;
    const unsigned mask = (G == 32) ? 0xffffffffu : (0xffffu << grp_base);
    const int stride = (int)(gridDim.x * (blockDim.x / G));
    int slot = (int)((blockIdx.x * blockDim.x + threadIdx.x) / G);
    const size_t col = (size_t)sub * EPP * ES;
    const int head = sub / LPH;                    // the head this lane's piece belongs to

    int v_next = -1, pad_next = 0;
    if (slot < a.count) {
        v_next = a.node_list ? a.node_list[a.first + slot] : a.first + slot;
        if (sub < W) pad_next = a.nbr_pad[(size_t)v_next * W + sub];
    }
    for (; slot < a.count; slot += stride) {
        const int v = v_next;
        const int pad = pad_next;
        {
            const int s2 = slot + stride;
            if (s2 < a.count) {
                v_next = a.node_list ? a.node_list[a.first + s2] : a.first + s2;
                if (sub < W) pad_next = a.nbr_pad[(size_t)v_next * W + sub];
            }
        }
        const int cnt = __shfl_sync(mask, pad, grp_base);
        Piece vq[MAXN];
        float ss[MAXN];
        int u[MAXN];
        u[0] = v;
#pragma unroll
        for (int j = 1; j < MAXN; ++j) u[j] = __shfl_sync(mask, pad, grp_base + j);
#pragma unroll
        for (int j = 0; j < MAXN; ++j) {
            ss[j] = 0.f;
            if (j < cnt) {
                vq[j] = ld_piece_nc((const char*)a.V + (size_t)u[j] * a.ldv * ES + col);
                if (cnt > 1) ss[j] = __ldg(x.s_src + (size_t)u[j] * a.heads + head);
            }
        }
        const float sd = cnt > 1 ? __ldg(x.s_dst + (size_t)v * a.heads + head) : 0.f;
        float acc[EPP];
        attend_additive<BF16, MAXN>(sd, ss, vq, cnt, x.slope, acc);
        st_piece_stream((char*)a.O + (size_t)v * a.ldo * ES + col, Elem<BF16>::pack(acc));
    }
}

// Wider cones (3 to 8 hops, up to 511 neighbours, Sec. 3.2 with the paper's k = 8): one warp per node, the
// neighbour list in CSR form walked in chunks; for bf16 the two half-warps take alternate neighbours.  Each lane
// keeps an online softmax (running maximum and sum, in log2 units) over the neighbours its half has seen and the
// matching weighted sum of its value piece; the halves are merged at the end.  Four neighbours per half are in
// flight at a time.
// ADDITIVE: scores are LeakyReLU(S_src[u, head] + S_dst[v, head]) from node-level scalars instead of q . k (no
// query or key rows are read).
template <bool BF16, int LPH, bool ADDITIVE>
__global__ void __launch_bounds__(256, DG4_WIDE_MIN_BLOCKS) sparse_attn_wide_kernel(dg4i_attn_args a, dg4i_attn_more x) {
    constexpr int G = BF16 ? 16 : 32;              // lanes per row
    constexpr int HALVES = 32 / G;                 // neighbours a warp handles side by side
    constexpr int EPP = Elem<BF16>::kPerPiece;
    constexpr int ES = BF16 ? 2 : 4;
    constexpr int UN = DG4_WIDE_UN;                // neighbours in flight per half
    const int lane = threadIdx.x & 31;
    const int sub = lane & (G - 1);
    const int half = lane / G;
    const unsigned hmask = (G == 32) ? 0xffffffffu : (0xffffu << (lane - sub));
    const size_t col = (size_t)sub * EPP * ES;
    const int warps = (int)(gridDim.x * (blockDim.x >> 5));
    const float c = a.scale * 1.4426950408889634f;
    for (int slot = (int)((blockIdx.x * blockDim.x + threadIdx.x) >> 5); slot < a.count; slot += warps) {
        const int v = a.node_list ? a.node_list[a.first + slot] : a.first + slot;
        const int beg = x.nbr_ptr[v];
        const int cnt = x.nbr_ptr[v + 1] - beg;
        Piece qp;
        float sd = 0.f;
        if (ADDITIVE) sd = __ldg(x.s_dst + (size_t)v * a.heads + sub / LPH);
        else qp = ld_piece_stream((const char*)a.Q + (size_t)v * a.ldq * ES + col);
        float m = -INFINITY, z = 0.f, acc[EPP];
#pragma unroll
        for (int i = 0; i < EPP; ++i) acc[i] = 0.f;
        for (int base = 0; base < cnt; base += 32) {
            const int my_u = (base + lane < cnt) ? x.nbr_idx[beg + base + lane] : -1;
            const int chunk = cnt - base < 32 ? cnt - base : 32;
            for (int t = 0; t < chunk; t += HALVES * UN) {
                Piece kq[UN], vq[UN];
                int u[UN];
#pragma unroll
                for (int i = 0; i < UN; ++i) {
                    const int j = t + i * HALVES + half;                       // position inside the chunk
                    u[i] = __shfl_sync(0xffffffffu, my_u, j & 31);
                    if (j >= chunk) u[i] = -1;
                }
#pragma unroll
                for (int i = 0; i < UN; ++i) {
                    if (u[i] >= 0) {
                        if (ADDITIVE) kq[i].w[0] = __float_as_uint(__ldg(x.s_src + (size_t)u[i] * a.heads + sub / LPH));
                        else kq[i] = ld_piece_nc((const char*)a.K + (size_t)u[i] * a.ldk * ES + col);
                        vq[i] = ld_piece_nc((const char*)a.V + (size_t)u[i] * a.ldv * ES + col);
                    }
                }
                // scores of the batch first, then ONE rescale of the running sums to the batch's maximum (rescaling
                // per neighbour costs a multiply per accumulator and an exponential each time)
                float s[UN];
#pragma unroll
                for (int i = 0; i < UN; ++i) {
                    if (ADDITIVE) {
                        float e = __uint_as_float(kq[i].w[0]) + sd;
                        e = (e > 0.f ? e : x.slope * e) * 1.4426950408889634f;
                        s[i] = (u[i] >= 0) ? e : -INFINITY;
                    } else {
                        float dot = (u[i] >= 0) ? Elem<BF16>::dot(qp, kq[i]) : 0.f;
#pragma unroll
                        for (int o = LPH / 2; o > 0; o >>= 1) dot += __shfl_xor_sync(hmask, dot, o);
                        s[i] = (u[i] >= 0) ? dot * c : -INFINITY;
                    }
                }
                float m_new = m;
#pragma unroll
                for (int i = 0; i < UN; ++i) m_new = fmaxf(m_new, s[i]);
                if (u[0] >= 0) {                                               // uniform inside a half; a batch's first slot is its lowest position
                    const float keep = fast_exp2(m - m_new);                   // 0 for the first batch (m = -inf)
                    z *= keep;
#pragma unroll
                    for (int e = 0; e < EPP; ++e) acc[e] *= keep;
#pragma unroll
                    for (int i = 0; i < UN; ++i) {
                        if (u[i] >= 0) {
                            const float p = fast_exp2(s[i] - m_new);
                            float vf[EPP];
                            Elem<BF16>::unpack(vq[i], vf);
                            z += p;
#pragma unroll
                            for (int e = 0; e < EPP; ++e) acc[e] = fmaf(p, vf[e], acc[e]);
                        }
                    }
                    m = m_new;
                }
            }
        }
        if (HALVES == 2) {                       // merge the two halves' partial softmaxes
            const float m2 = __shfl_xor_sync(0xffffffffu, m, 16);
            const float z2 = __shfl_xor_sync(0xffffffffu, z, 16);
            const float mm = fmaxf(m, m2);
            const float w1 = fast_exp2(m - mm), w2 = (m2 == -INFINITY) ? 0.f : fast_exp2(m2 - mm);
            z = z * w1 + z2 * w2;
#pragma unroll
            for (int e = 0; e < EPP; ++e) {
                const float a2 = __shfl_xor_sync(0xffffffffu, acc[e], 16);
                acc[e] = acc[e] * w1 + a2 * w2;
            }
        }
        if (half == 0) {
            if (cnt == 1) {                      // a single neighbour (v itself): weight exactly 1
                // acc = 1 * V row, z = 1 already; nothing to normalise
            } else {
                const float inv = fast_rcp(z);
#pragma unroll
                for (int e = 0; e < EPP; ++e) acc[e] *= inv;
            }
            st_piece_stream((char*)a.O + (size_t)v * a.ldo * ES + col, Elem<BF16>::pack(acc));
        }
    }
}

template <bool BF16, int LPH, bool ADDITIVE>
dg4_status launch_wide(const dg4i_attn_args& a, const dg4i_attn_more& x, cudaStream_t st) {
    int dev = 0, sms = 0;
    DG4_CUDA_TRY(cudaGetDevice(&dev));
    DG4_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    const int64_t needed = ((int64_t)a.count + 7) / 8;
    const int64_t resident = (int64_t)sms * DG4_WIDE_MIN_BLOCKS;
    sparse_attn_wide_kernel<BF16, LPH, ADDITIVE><<<(unsigned)(needed < resident ? needed : resident), 256, 0, st>>>(a, x);
    dg4i_count_launch();
    DG4_CUDA_TRY(cudaGetLastError());
    return DG4_OK;
}

template <bool BF16, bool ADDITIVE>
dg4_status launch_wide_heads(const dg4i_attn_args& a, const dg4i_attn_more& x, cudaStream_t st) {
    constexpr int G = BF16 ? 16 : 32;
    switch (G / a.heads) {
        case 1: return launch_wide<BF16, 1, ADDITIVE>(a, x, st);
        case 2: return launch_wide<BF16, 2, ADDITIVE>(a, x, st);
        case 4: return launch_wide<BF16, 4, ADDITIVE>(a, x, st);
        case 8: return launch_wide<BF16, 8, ADDITIVE>(a, x, st);
        case 16: return launch_wide<BF16, 16, ADDITIVE>(a, x, st);
        case 32: if (G == 32) return launch_wide<BF16, (G == 32 ? 32 : 16), ADDITIVE>(a, x, st);
    }
    DG4_FAIL(DG4_ERR_UNSUPPORTED, "heads = %d is not supported for this dtype", a.heads);
}

struct LaunchShape { int sm_count = 0; int blocks_per_sm = 0; };

template <bool BF16, int LPH, int MAXN, bool ADDITIVE>
dg4_status launch_one(const dg4i_attn_args& a, const dg4i_attn_more* x, cudaStream_t st) {
    constexpr int G = BF16 ? 16 : 32;
    const int threads = DG4_ATTN_THREADS;
    static LaunchShape shape[64];
    int dev = 0;
    DG4_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) DG4_FAIL(DG4_ERR_UNSUPPORTED, "device ordinal %d is out of range", dev);
    if (shape[dev].sm_count == 0) {
        int sms = 0, per_sm = 0;
        DG4_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
        if (ADDITIVE) DG4_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, sparse_attn_additive_kernel<BF16, LPH, MAXN>, threads, 0));
        else DG4_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, sparse_attn_kernel<BF16, LPH, MAXN>, threads, 0));
        shape[dev].blocks_per_sm = per_sm > 0 ? per_sm : 1;
        shape[dev].sm_count = sms;
    }
    const int nodes_per_block = threads / G;
    const int64_t needed = ((int64_t)a.count + nodes_per_block - 1) / nodes_per_block;
    const int64_t resident = (int64_t)shape[dev].sm_count * shape[dev].blocks_per_sm;
    const unsigned blocks = (unsigned)(needed < resident ? needed : resident);
    if (ADDITIVE) sparse_attn_additive_kernel<BF16, LPH, MAXN><<<blocks, threads, 0, st>>>(a, *x);
    else sparse_attn_kernel<BF16, LPH, MAXN><<<blocks, threads, 0, st>>>(a);
    dg4i_count_launch();
    DG4_CUDA_TRY(cudaGetLastError());
    return DG4_OK;
}

template <bool BF16, int MAXN, bool ADDITIVE>
dg4_status launch_for_heads(const dg4i_attn_args& a, const dg4i_attn_more* x, cudaStream_t st) {
    constexpr int G = BF16 ? 16 : 32;
    switch (G / a.heads) {
        case 1: return launch_one<BF16, 1, MAXN, ADDITIVE>(a, x, st);
        case 2: return launch_one<BF16, 2, MAXN, ADDITIVE>(a, x, st);
        case 4: return launch_one<BF16, 4, MAXN, ADDITIVE>(a, x, st);
        case 8: return launch_one<BF16, 8, MAXN, ADDITIVE>(a, x, st);
        case 16: return launch_one<BF16, 16, MAXN, ADDITIVE>(a, x, st);
        case 32: if (G == 32) return launch_one<BF16, (G == 32 ? 32 : 16), MAXN, ADDITIVE>(a, x, st);
    }
    DG4_FAIL(DG4_ERR_UNSUPPORTED, "heads = %d is not supported for this dtype", a.heads);
}

}  // namespace

namespace {
template <bool ADDITIVE>
dg4_status attn_dispatch(const dg4i_attn_args& a, const dg4i_attn_more* x, cudaStream_t st) {
    if (a.count <= 0) return DG4_OK;
    const bool bf16 = a.dtype == DG4_BF16;
    const int G = bf16 ? 16 : 32;
    if (a.heads < 1 || a.heads > G || (G % a.heads) != 0)
        DG4_FAIL(DG4_ERR_UNSUPPORTED, "heads = %d: must divide %d", a.heads, G);
    if (a.max_nbr > 7) {
        if (!x || !x->nbr_ptr || !x->nbr_idx) DG4_FAIL(DG4_ERR_INVALID_ARG, "wider cones need the CSR neighbour lists");
        return bf16 ? launch_wide_heads<true, ADDITIVE>(a, *x, st) : launch_wide_heads<false, ADDITIVE>(a, *x, st);
    }
    if (a.max_nbr <= 3) return bf16 ? launch_for_heads<true, 3, ADDITIVE>(a, x, st) : launch_for_heads<false, 3, ADDITIVE>(a, x, st);
    return bf16 ? launch_for_heads<true, 7, ADDITIVE>(a, x, st) : launch_for_heads<false, 7, ADDITIVE>(a, x, st);
}
}  // namespace

dg4_status dg4i_attn_launch(const dg4i_attn_args& a, const dg4i_attn_more* more, cudaStream_t st) {
    return attn_dispatch<false>(a, more, st);
}
dg4_status dg4i_attn_additive_launch(const dg4i_attn_args& a, const dg4i_attn_more& more, cudaStream_t st) {
    return attn_dispatch<true>(a, &more, st);
}
