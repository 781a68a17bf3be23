// Per-node arithmetic of the sparse attention shared by the stand-alone kernel and the levelised kernel:
// a node's row is split into 16-byte pieces, one per lane; a head spans LPH adjacent lanes.
#pragma once

#include <cuda_bf16.h>
#include <stdint.h>

namespace attn {

struct alignas(16) Piece { uint32_t w[4]; };

__device__ __forceinline__ Piece ld_piece_nc(const void* p) {        // read-only for the whole kernel
    Piece r;
    asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.w[0]), "=r"(r.w[1]), "=r"(r.w[2]), "=r"(r.w[3]) : "l"(p));
    return r;
}
// L2 eviction priorities (a 64-bit policy word made once per thread): rows that are gathered again by later nodes
// are asked to stay, data that passes through once is asked to leave first.
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ Piece ld_piece_nc_hint(const void* p, uint64_t pol) {   // read-only, with an L2 policy
    Piece r;
    asm volatile("ld.global.nc.L2::cache_hint.v4.u32 {%0,%1,%2,%3}, [%4], %5;"
                 : "=r"(r.w[0]), "=r"(r.w[1]), "=r"(r.w[2]), "=r"(r.w[3]) : "l"(p), "l"(pol));
    return r;
}
__device__ __forceinline__ int ld_int_nc_hint(const int* p, uint64_t pol) {
    int r;
    asm volatile("ld.global.nc.L2::cache_hint.s32 %0, [%1], %2;" : "=r"(r) : "l"(p), "l"(pol));
    return r;
}
__device__ __forceinline__ Piece ld_piece_cg(const void* p) {        // coherent at L2: data written by other CTAs
    Piece r;
    asm volatile("ld.global.cg.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.w[0]), "=r"(r.w[1]), "=r"(r.w[2]), "=r"(r.w[3]) : "l"(p) : "memory");
    return r;
}
__device__ __forceinline__ Piece ld_piece_stream(const void* p) {    // streamed once: evict-first
    Piece r;
    asm volatile("ld.global.cs.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.w[0]), "=r"(r.w[1]), "=r"(r.w[2]), "=r"(r.w[3]) : "l"(p));
    return r;
}
__device__ __forceinline__ void st_piece_stream(void* p, const Piece& v) {
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};"
                 :: "l"(p), "r"(v.w[0]), "r"(v.w[1]), "r"(v.w[2]), "r"(v.w[3]) : "memory");
}

__device__ __forceinline__ float fast_exp2(float x) {      // 2^x, relative error about 2^-22
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float fast_rcp(float x) {       // 1/x, relative error about 2^-23
    float y;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
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
    // sum over the piece of q[i] * k[i], products and sums in fp32 (a bf16 x bf16 product is exact in fp32).
    // The mixed-precision FMA takes the bf16 halves of the packed words directly: no unpacking instructions.
    __device__ static __forceinline__ float dot(const Piece& q, const Piece& k) {
        float acc = 0.f;
#pragma unroll
        for (int i = 0; i < 4; ++i)
            asm("{\n\t.reg .b16 ql, qh, kl, kh;\n\tmov.b32 {ql, qh}, %1;\n\tmov.b32 {kl, kh}, %2;\n\t"
                "fma.rn.f32.bf16 %0, ql, kl, %0;\n\tfma.rn.f32.bf16 %0, qh, kh, %0;\n\t}"
                : "+f"(acc) : "r"(q.w[i]), "r"(k.w[i]));
        return acc;
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
    __device__ static __forceinline__ float dot(const Piece& q, const Piece& k) {
        float acc = 0.f;
#pragma unroll
        for (int i = 0; i < 4; ++i) acc = fmaf(__uint_as_float(q.w[i]), __uint_as_float(k.w[i]), acc);
        return acc;
    }
};

// Softmax over the scores s[0..cnt) (log2 units, maximum m) and the weighted sum of this lane's value pieces.
template <bool BF16, int MAXN>
__device__ __forceinline__ void softmax_weighted_sum(const float* s, float m, int cnt, const Piece* vq, float* acc) {
    constexpr int EPP = Elem<BF16>::kPerPiece;
    float z = 0.f;
#pragma unroll
    for (int i = 0; i < EPP; ++i) acc[i] = 0.f;
#pragma unroll
    for (int j = 0; j < MAXN; ++j) {
        if (j < cnt) {
            float p = fast_exp2(s[j] - m);
            z += p;
            float vf[EPP];
            Elem<BF16>::unpack(vq[j], vf);
#pragma unroll
            for (int i = 0; i < EPP; ++i) acc[i] = fmaf(p, vf[i], acc[i]);
        }
    }
    const float inv = fast_rcp(z);
#pragma unroll
    for (int i = 0; i < EPP; ++i) acc[i] *= inv;
}

// Scores, softmax and weighted sum for one lane's piece of one node.  qp, kq[j], vq[j]: this lane's pieces
// of the query row and of neighbour j's key / value rows (j < cnt; cnt >= 1).  `mask` names the lanes of this
// node's group: they share cnt, so they take the same path and meet in the score-reduction shuffles; other
// groups of the warp may be on a different path.
template <bool BF16, int LPH, int MAXN>
__device__ __forceinline__ void attend(const Piece& qp, const Piece* kq, const Piece* vq, int cnt, float scale,
                                       unsigned mask, float* acc /*[kPerPiece]*/) {
    if (cnt <= 1) {                                   // softmax over one element: weight exactly 1
        Elem<BF16>::unpack(vq[0], acc);
        return;
    }
    const float c = scale * 1.4426950408889634f;      // scores kept in log2 units
    float s[MAXN];
    float m = -INFINITY;
#pragma unroll
    for (int j = 0; j < MAXN; ++j) {
        float dot = 0.f;
        if (j < cnt) dot = Elem<BF16>::dot(qp, kq[j]);
#pragma unroll
        for (int o = LPH / 2; o > 0; o >>= 1) dot += __shfl_xor_sync(mask, dot, o);
        s[j] = (j < cnt) ? dot * c : -INFINITY;
        m = fmaxf(m, s[j]);
    }
    constexpr int EPP = Elem<BF16>::kPerPiece;
    float z = 0.f;
#pragma unroll
    for (int i = 0; i < EPP; ++i) acc[i] = 0.f;
#pragma unroll
    for (int j = 0; j < MAXN; ++j) {
        if (j < cnt) {
            float p = fast_exp2(s[j] - m);
            z += p;
            float vf[EPP];
            Elem<BF16>::unpack(vq[j], vf);
#pragma unroll
            for (int i = 0; i < EPP; ++i) acc[i] = fmaf(p, vf[i], acc[i]);
        }
    }
    const float inv = fast_rcp(z);
#pragma unroll
    for (int i = 0; i < EPP; ++i) acc[i] *= inv;
}

// Additive-score variant: this lane's head has the node-level scalars s_dst (of the destination) and s_src[j]
// (of neighbour j); score = LeakyReLU(s_src[j] + s_dst).  No cross-lane traffic at all.
template <bool BF16, int MAXN>
__device__ __forceinline__ void attend_additive(float s_dst, const float* s_src, const Piece* vq, int cnt, float slope,
                                                float* acc /*[kPerPiece]*/) {
    if (cnt <= 1) {
        Elem<BF16>::unpack(vq[0], acc);
        return;
    }
    float s[MAXN];
    float m = -INFINITY;
#pragma unroll
    for (int j = 0; j < MAXN; ++j) {
        float x = s_src[j] + s_dst;
        x = (x > 0.f ? x : slope * x) * 1.4426950408889634f;
        s[j] = (j < cnt) ? x : -INFINITY;
        m = fmaxf(m, s[j]);
    }
    softmax_weighted_sum<BF16, MAXN>(s, m, cnt, vq, acc);
}

}  // namespace attn
