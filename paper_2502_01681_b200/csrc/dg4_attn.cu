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

namespace {

struct alignas(16) Piece { uint32_t w[4]; };

__device__ __forceinline__ Piece ld_piece(const void* p) {
    Piece r;
    asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.w[0]), "=r"(r.w[1]), "=r"(r.w[2]), "=r"(r.w[3]) : "l"(p));
    return r;
}
// streamed once: streaming (evict-first) policy so that gathered rows keep their place in the caches
__device__ __forceinline__ Piece ld_piece_stream(const void* p) {
    Piece r;
    asm volatile("ld.global.cs.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.w[0]), "=r"(r.w[1]), "=r"(r.w[2]), "=r"(r.w[3]) : "l"(p));
    return r;
}
__device__ __forceinline__ void st_piece_stream(void* p, const Piece& v) {
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};"
                 :: "l"(p), "r"(v.w[0]), "r"(v.w[1]), "r"(v.w[2]), "r"(v.w[3]) : "memory");
}

template <bool BF16> struct Elem;
template <> struct Elem<true> {
    static constexpr int kPerPiece = 8;
    __device__ static __forceinline__ void unpack(const Piece& p, float* f) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            f[2 * i] = __uint_as_float(p.w[i] << 16);
            f[2 * i + 1] = __uint_as_float(p.w[i] & 0xffff0000u);
        }
    }
    __device__ static __forceinline__ Piece pack(const float* f) {
        Piece p;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            __nv_bfloat162 h = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
            p.w[i] = *reinterpret_cast<uint32_t*>(&h);
        }
        return p;
    }
};
template <> struct Elem<false> {
    static constexpr int kPerPiece = 4;
    __device__ static __forceinline__ void unpack(const Piece& p, float* f) {
#pragma unroll
        for (int i = 0; i < 4; ++i) f[i] = __uint_as_float(p.w[i]);
    }
    __device__ static __forceinline__ Piece pack(const float* f) {
        Piece p;
#pragma unroll
        for (int i = 0; i < 4; ++i) p.w[i] = __float_as_uint(f[i]);
        return p;
    }
};

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
        if (j < cnt) vq[j] = ld_piece((const char*)a.V + (size_t)u[j] * a.ldv * ES + col);
    const bool need_scores = cnt > 1;
    if (need_scores) {
        qp = ld_piece_stream((const char*)a.Q + (size_t)v * a.ldq * ES + col);
#pragma unroll
        for (int j = 0; j < MAXN; ++j)
            if (j < cnt) kq[j] = ld_piece((const char*)a.K + (size_t)u[j] * a.ldk * ES + col);
    }

    float acc[EPP];
    if (!need_scores) {
        Elem<BF16>::unpack(vq[0], acc);            // softmax over one element: weight exactly 1
    } else {
        float q[EPP];
        Elem<BF16>::unpack(qp, q);
        const float c = a.scale * 1.4426950408889634f;   // scores kept in log2 units
        float s[MAXN];
        float m = -INFINITY;
#pragma unroll
        for (int j = 0; j < MAXN; ++j) {
            float kf[EPP];
            float dot = 0.f;
            if (j < cnt) {
                Elem<BF16>::unpack(kq[j], kf);
#pragma unroll
                for (int i = 0; i < EPP; ++i) dot = fmaf(q[i], kf[i], dot);
            }
#pragma unroll
            for (int o = LPH / 2; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
            s[j] = (j < cnt) ? dot * c : -INFINITY;
            m = fmaxf(m, s[j]);
        }
        float z = 0.f;
#pragma unroll
        for (int i = 0; i < EPP; ++i) acc[i] = 0.f;
#pragma unroll
        for (int j = 0; j < MAXN; ++j) {
            if (j < cnt) {
                float p = exp2f(s[j] - m);
                z += p;
                float vf[EPP];
                Elem<BF16>::unpack(vq[j], vf);
#pragma unroll
                for (int i = 0; i < EPP; ++i) acc[i] = fmaf(p, vf[i], acc[i]);
            }
        }
        const float inv = 1.0f / z;
#pragma unroll
        for (int i = 0; i < EPP; ++i) acc[i] *= inv;
    }
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
