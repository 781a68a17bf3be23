// Levelised layers as ONE persistent kernel (Sec. 1 / Sec. 3.4: gates are encoded level by level in
// topological order, each gate once, reading the rows already updated for lower levels).
//
// Work of one tile (16 nodes of one level, for one layer k):
//   1. gather the K | V rows of every neighbour from layer k's K|V table (16 lanes per node, 16 bytes per
//      lane), compute scores, softmax and the weighted value sum in registers, and write the 16 x 128
//      attention tile into shared memory in the tensor core's K-major, 128-byte-swizzled operand layout;
//   2. output projection TRANSPOSED on the tensor cores: D[feature, node] = W_o * O^T (tcgen05.mma, M = 128
//      features, N = 16 nodes, K = 128), so a small tile costs a fraction of a 128-row tile and all warps take
//      part in the epilogue (128 TMEM lanes x 16 columns);
//   3. add the residual, round to bf16, write the new rows to H and -- in operand layout again -- to shared
//      memory;
//   4. from the new rows, again transposed: refresh the tile's K | V rows of layer k (so that higher levels
//      gather updated rows) and, if there is a layer k+1, project that layer's Q | K | V rows of these nodes
//      (a node's own query, key and value always come from its row as the previous layer left it).
//
// Several layers run as a wavefront: layer k+1 may process level l as soon as layer k has finished level l
// (its inputs are that level's new rows) and layer k+1 itself has finished the levels below l.  CTAs are dealt
// to layers round-robin; each keeps its layer's W_o, W_k, W_v and the next layer's W_q, W_k, W_v resident in
// TENSOR memory (six blocks of 128 lanes x 64 columns beside the accumulators) and issues its MMAs with the A
// operand read from there, so the weights are never re-read from shared memory and shared memory holds only the
// node-side tiles.  With n layers the dependent chain is n_levels + n - 1 tile steps long
// instead of n * n_levels, while computing exactly what n successive level-by-level sweeps compute.
//
// Levels are separated by counters in global memory instead of kernel launches: every (layer, level) has an
// arrival counter that only the CTAs owning a tile of it bump (release); before a level in which it has work a
// CTA waits (acquire) until the counter of its layer's previous non-empty level and the counter of the previous
// layer's same level are full.  Completion is transitive, because every CTA that arrived had itself waited the
// same way.  Launched cooperatively (all CTAs co-resident).  Every wait is bounded; on expiry the kernel records
// DG4_ERR_TIMEOUT, raises an abort word that every other wait polls, and all CTAs leave their loops, free
// tensor memory and return.

#include "dg4_internal.h"
#include "dg4_attn_core.cuh"
#include "dg4_sm100.cuh"

#include <mutex>

namespace {

using namespace sm100;
using namespace attn;

constexpr int kTile = 16;                    // nodes per tile
constexpr int kThreads = kTile * 16;         // 16 lanes per node
constexpr int kBHalf = kTile * 128;          // K-half of a kTile-row operand tile
constexpr int kTmemCols = 512;               // six accumulators of kTile columns, then six weight blocks of 64 columns
constexpr int kWCol0 = 6 * kTile;            // first column of the weight blocks W_o | W_k | W_v | next W_q | W_k | W_v
constexpr int kWCols = 64;                   // a 128 x 128 bf16 block: 128 lanes x 64 columns of two elements
constexpr int kStageRow = 1280;              // staging per node: K|V of this layer 512, Q of the next 256, its K|V 512

constexpr int kOffO = 0;                          // attention tile (operand layout)
constexpr int kOffHp = kOffO + 2 * kBHalf;        // new rows (operand layout)
constexpr int kOffHres = kOffHp + 2 * kBHalf;     // residual rows, plain [kTile][256 B]
constexpr int kOffStage = kOffHres + kTile * 256; // output staging, plain [kTile][kStageRow]
constexpr int kOffMisc = kOffStage + kTile * kStageRow;
constexpr int kSmemBytes = kOffMisc + 256 + 1024;
static_assert(kSmemBytes <= 232448, "shared memory budget of one CTA");
static_assert(kWCol0 + 6 * kWCols <= kTmemCols, "tensor memory budget of one CTA");
// Every CTA allocates all of its SM's tensor memory, so two CTAs must never share an SM (the second one's
// allocation would wait for the first, which waits for the second's levels): the launch asks for more than half
// of an SM's shared memory, which rules that out.
constexpr int kLaunchSmemBytes = kSmemBytes > 120 * 1024 ? kSmemBytes : 120 * 1024;

struct Misc {
    uint64_t mma1, mma2, drain;
    uint32_t tmem_base;
    int32_t go, go2;
    int32_t failed;                        // a wait for this CTA's own MMAs ran out: leave at the next level
    int32_t node[kTile];
};

struct LevParams {
    __nv_bfloat16* Q[DG4I_MAX_LAYERS];     // [n, 128] per layer
    __nv_bfloat16* KV[DG4I_MAX_LAYERS];    // [n, 256] per layer
    const __nv_bfloat16* Wo[DG4I_MAX_LAYERS];    // [128, 128] per layer, out x in
    const __nv_bfloat16* Wqkv[DG4I_MAX_LAYERS];  // [384, 128] per layer
    __nv_bfloat16* H;                      // [n, ldh], updated in place by every layer in turn
    int64_t ldh;
    const int32_t* nbr_pad;                // [n, pad_width]
    const int32_t* level_ptr;
    const int32_t* level_nodes;
    int32_t n_levels;
    int32_t n_layers;
    int32_t residual;
    float scale;
    int32_t* arrive;                       // [n_layers, n_levels], zero on entry
    int32_t* abort_word;                   // zero on entry
    int32_t* status;
    uint32_t poll_limit;                   // polls after which a wait gives up
};

__device__ __forceinline__ void st_shared_v4(uint32_t addr, const uint32_t* r) {
    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]) : "memory");
}
__device__ __forceinline__ void ld_shared_v4(uint32_t addr, uint32_t* r) {
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}
__device__ __forceinline__ void st_shared_b16(uint32_t addr, uint16_t v) {
    asm volatile("st.shared.b16 [%0], %1;" ::"r"(addr), "h"(v) : "memory");
}
__device__ __forceinline__ uint16_t ld_shared_b16(uint32_t addr) {
    uint16_t v;
    asm volatile("ld.shared.b16 %0, [%1];" : "=h"(v) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void st_global_v4(void* p, const uint32_t* r) {
    asm volatile("st.global.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]) : "memory");
}
__device__ __forceinline__ int ld_acquire(const int32_t* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void red_release_add(int32_t* p, int v) {
    asm volatile("red.release.gpu.global.add.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ uint16_t bf16_bits(float x) {
    __nv_bfloat16 h = __float2bfloat16_rn(x);
    return *reinterpret_cast<uint16_t*>(&h);
}
// byte offset of element k (0..127) of row `row` in a kTile-row operand tile (two K-halves, 128-byte swizzle)
__device__ __forceinline__ uint32_t operand_offset(int row, int k) {
    return (uint32_t)((k >> 6) * kBHalf) + sw128_offset(row, (k & 63) >> 3) + (uint32_t)((k & 7) * 2);
}

__device__ __forceinline__ void give_up(const LevParams& p) {
    atomicExch(p.abort_word, 1);
    if (p.status) atomicCAS(p.status, 0, (int)DG4_ERR_TIMEOUT);
}

// Polls (acquire) until *counter >= target; false on abort or after `limit` polls (about a second by default).
__device__ __forceinline__ bool wait_counter(const int32_t* counter, int target, const int32_t* abort_word, uint32_t limit) {
    uint32_t polls = 0;
    while (ld_acquire(counter) < target) {
        ++polls;
        if (polls > limit || ((polls & 63u) == 0 && ld_acquire(abort_word) != 0)) return false;
        if (polls > 64) __nanosleep(32);
    }
    return true;
}

template <int LPH, int MAXN>
__global__ void __launch_bounds__(kThreads, 1)
levelised_kernel(LevParams p) {
    extern __shared__ uint8_t smem_raw[];
    constexpr int W = MAXN + 1;                          // width of a neighbour-table entry
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
    Misc* misc = reinterpret_cast<Misc*>(base_ptr + kOffMisc);
    const uint32_t sO = base + kOffO, sHp = base + kOffHp, sHres = base + kOffHres, sSt = base + kOffStage;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int slot = tid >> 4, sub = tid & 15;          // node slot of the tile and lane within the node
    const int grp_base = lane - sub;
    const unsigned gmask = 0xffffu << grp_base;
    const uint32_t bar1 = smem_u32(&misc->mma1), bar2 = smem_u32(&misc->mma2);

    // this CTA's layer, its rank among the CTAs of that layer, and how many CTAs each layer has
    const int layer = (int)blockIdx.x % p.n_layers;
    const int bid = (int)blockIdx.x / p.n_layers;
    auto ctas_of = [&](int k) { return ((int)gridDim.x - k + p.n_layers - 1) / p.n_layers; };
    const int nctas = ctas_of(layer);
    const bool has_next = layer + 1 < p.n_layers;
    const int n_acc = has_next ? 5 : 2;                  // accumulators of the second MMA group

    if (tid == 0) {
        mbar_init(bar1, 1);
        mbar_init(bar2, 1);
        mbar_init(smem_u32(&misc->drain), 1);
        misc->go = 1;
        misc->go2 = 1;
        misc->failed = 0;
        mbar_fence_init();
    }
    if (warp == 0) tmem_alloc(smem_u32(&misc->tmem_base), kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = misc->tmem_base;
    static_assert(kThreads / 32 / 4 * 8 == kTile, "epilogue: every warp reads 8 node columns of its lane quadrant");
    const int q4 = warp & 3, cg = warp >> 2;             // TMEM lane quadrant of the warp; which half of the columns it takes
    const int feat = q4 * 32 + lane;                     // output feature (TMEM lane) this thread holds
    // The weights stay in tensor memory for the whole kernel: row `feat` of every block in lane `feat`, two
    // consecutive bf16 of the row per 32-bit column (the bytes as they lie in global memory).  Each thread copies
    // half a row (128 bytes) of every block of its layer.
    {
        const int n_blocks = has_next ? 6 : 3;
        for (int blk = 0; blk < n_blocks; ++blk) {
            const __nv_bfloat16* wb = blk == 0 ? p.Wo[layer]
                                     : blk < 3 ? p.Wqkv[layer] + (size_t)blk * 128 * 128
                                               : p.Wqkv[layer + 1] + (size_t)(blk - 3) * 128 * 128;
            const uint4* src = reinterpret_cast<const uint4*>(wb + (size_t)feat * 128 + cg * 64);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const uint4 lo = src[2 * c], hi = src[2 * c + 1];
                const uint32_t r[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
                tmem_st_32x8(tmem + ((uint32_t)(q4 * 32) << 16) + (uint32_t)(kWCol0 + blk * kWCols + cg * 32 + c * 8), r);
            }
        }
        tmem_st_wait();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();

    const uint32_t idesc = idesc_bf16_f32(128, kTile);
    // matrix descriptors of the node-side operands; stepping along K only adds to the address field
    const uint64_t dO = smem_desc_sw128(sO), dHp = smem_desc_sw128(sHp);
    uint32_t ph1 = 0, ph2 = 0;
    int last_nonempty = -1, last_participants = 0;
    bool alive = true;
    const uint32_t counter_limit = p.poll_limit > 4u ? p.poll_limit >> 2 : 1u;   // a counter poll is a trip to L2

    const char* kv_tab = (const char*)p.KV[layer];
    const char* q_tab = (const char*)p.Q[layer];
    int32_t* my_arrive = p.arrive + (size_t)layer * p.n_levels;
    const int32_t* prev_arrive = layer > 0 ? p.arrive + (size_t)(layer - 1) * p.n_levels : nullptr;
    const int prev_ctas = layer > 0 ? ctas_of(layer - 1) : 0;

    // The index chain of a tile (node id -> neighbour-table entry) is two dependent loads that do not depend on
    // any other CTA's results.  It is software-pipelined across levels so that none of it sits on the
    // level-to-level critical path: while level l is processed, the node id of this CTA's first tile of level
    // l+2 and the table entry for level l+1 are in flight.
    // The level offsets run four levels ahead in registers: every acquire of a counter drops the L1 contents,
    // so a plain load at the top of a level would cost a trip to L2 on the level-to-level chain.
    auto lp_at = [&](int lv) { return p.level_ptr[lv < p.n_levels ? lv : p.n_levels]; };
    auto stage_node = [&](int lv_first, int lv_end) -> int {   // node of (first tile of this CTA, this slot) of a level
        const int r = bid * kTile + slot;
        return (r < lv_end - lv_first) ? p.level_nodes[lv_first + r] : -1;
    };
    int lp0 = lp_at(0), lp1 = lp_at(1), lp2 = lp_at(2), lp3 = lp_at(3);
    auto pad_of = [&](int v) -> int { return (v >= 0 && sub < W) ? p.nbr_pad[(size_t)v * W + sub] : 0; };
    int v0 = stage_node(lp0, lp1);                     // level l  : node id and this lane's table word
    int pad0 = pad_of(v0);
    int vC = stage_node(lp1, lp2);                     // level l+1: node id

    for (int l = 0; l < p.n_levels && alive; ++l) {
        const int first = lp0;
        const int n_l = lp1 - lp0;
        // issue the next load of every pipelined chain; the results are first used one level later
        const int lp4 = lp_at(l + 4);
        const int vB = stage_node(lp2, lp3);
        const int padC = pad_of(vC);
        const int tiles = (n_l + kTile - 1) / kTile;
        if (n_l > 0 && bid < tiles) {
            bool waited = false;
            int v_nx = -1, pad_nx = 0;           // index chain of this CTA's next tile in a wide level
            for (int tile = bid; tile < tiles; tile += nctas) {
                int v, pad;
                if (tile == bid) {
                    v = v0; pad = pad0;
                } else {                         // further tiles of a wide level: fetched during the tile before
                    v = v_nx; pad = pad_nx;
                }
                {
                    const int r = (tile + nctas) * kTile + slot;
                    v_nx = (tile + nctas < tiles && r < n_l) ? p.level_nodes[first + r] : -1;
                }
                const bool valid = v >= 0;

                if (!waited) {
                    // ---- this layer's previous level and the previous layer's same level must be complete
                    // (two pollers in different warps, so that both counters are watched at the same time)
                    if (tid == 0) {
                        bool go = true;
                        if (misc->failed) go = false;
                        if (go && last_nonempty >= 0) go = wait_counter(my_arrive + last_nonempty, last_participants, p.abort_word, counter_limit);
                        if (!go && ld_acquire(p.abort_word) == 0) give_up(p);
                        if (go && (l & 255) == 0 && ld_acquire(p.abort_word) != 0) go = false;
                        misc->go = go ? 1 : 0;
                    } else if (tid == 32) {
                        bool go = true;
                        if (prev_arrive) go = wait_counter(prev_arrive + l, tiles < prev_ctas ? tiles : prev_ctas, p.abort_word, counter_limit);
                        if (!go && ld_acquire(p.abort_word) == 0) give_up(p);
                        misc->go2 = go ? 1 : 0;
                    }
                    __syncthreads();
                    waited = true;
                    if (!misc->go || !misc->go2) { alive = false; break; }
                }

                // ---- gather and attend
                Piece kq[MAXN], vq[MAXN], qp, hres;
                int u[MAXN];
                const int cnt = valid ? __shfl_sync(gmask, pad, grp_base) : 1;
                u[0] = v;
#pragma unroll
                for (int j = 1; j < MAXN; ++j) u[j] = __shfl_sync(gmask, pad, grp_base + j);
                float acc[8];
                if (valid) {
#pragma unroll
                    for (int j = 0; j < MAXN; ++j)
                        if (j < cnt) vq[j] = ld_piece_cg(kv_tab + (size_t)u[j] * 512 + 256 + sub * 16);
                    if (cnt > 1) {
                        qp = ld_piece_cg(q_tab + (size_t)v * 256 + sub * 16);
#pragma unroll
                        for (int j = 0; j < MAXN; ++j)
                            if (j < cnt) kq[j] = ld_piece_cg(kv_tab + (size_t)u[j] * 512 + sub * 16);
                    }
                    if (p.residual) hres = ld_piece_cg((const char*)p.H + (size_t)v * p.ldh * 2 + sub * 16);
                } else {
                    vq[0].w[0] = vq[0].w[1] = vq[0].w[2] = vq[0].w[3] = 0u;
                }
                if (!valid || !p.residual) hres.w[0] = hres.w[1] = hres.w[2] = hres.w[3] = 0u;
                attend<true, LPH, MAXN>(qp, kq, vq, cnt, p.scale, gmask, acc);
                pad_nx = pad_of(v_nx);           // its node id has arrived by now; the entry is used by the next tile
                {
                    Piece o = Elem<true>::pack(acc);
                    st_shared_v4(sO + (uint32_t)((sub >> 3) * kBHalf) + sw128_offset(slot, sub & 7), o.w);
                    st_shared_v4(sHres + (uint32_t)(slot * 256 + sub * 16), hres.w);
                    if (sub == 0) misc->node[slot] = v;
                }
                fence_proxy_async_smem();
                __syncthreads();

                // ---- output projection, transposed: D[feature, node] = W_o * O^T
                if (tid == 0) {
                    tc_fence_after();
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        const uint32_t b_off = (uint32_t)((ks >> 2) * kBHalf + (ks & 3) * 32);
                        mma_bf16_ta(tmem, tmem + (uint32_t)(kWCol0 + ks * 8), dO + (b_off >> 4), idesc, ks > 0 ? 1u : 0u);
                    }
                    mma_commit(bar1);
                }
                if (!mbar_wait(bar1, ph1, p.poll_limit) && tid == 0) { give_up(p); misc->failed = 1; }
                ph1 ^= 1u;
                tc_fence_after();
                {
                    uint32_t d[8];
                    tmem_ld_32x8(tmem + ((uint32_t)(q4 * 32) << 16) + (uint32_t)(cg * 8), d);
                    tmem_ld_wait();
#pragma unroll
                    for (int nn = 0; nn < 8; ++nn) {
                        const int node = cg * 8 + nn;
                        const uint16_t rb = ld_shared_b16(sHres + (uint32_t)(node * 256 + feat * 2));
                        const float val = __uint_as_float(d[nn]) + __uint_as_float((uint32_t)rb << 16);
                        st_shared_b16(sHp + operand_offset(node, feat), bf16_bits(val));
                    }
                }
                tc_fence_before();
                fence_proxy_async_smem();
                __syncthreads();

                // ---- from the new rows, transposed: this layer's K | V refresh and the next layer's Q | K | V
                if (tid == 0) {
                    tc_fence_after();
                    // K-step outermost: consecutive instructions accumulate into different accumulators, so none
                    // has to wait for the one before it
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        const uint32_t b_off = (uint32_t)((ks >> 2) * kBHalf + (ks & 3) * 32);
#pragma unroll
                        for (int blk = 0; blk < 5; ++blk) {
                            if (blk < n_acc) {
                                mma_bf16_ta(tmem + (uint32_t)(kTile * (1 + blk)),
                                            tmem + (uint32_t)(kWCol0 + (1 + blk) * kWCols + ks * 8), dHp + (b_off >> 4), idesc,
                                            ks > 0 ? 1u : 0u);
                            }
                        }
                    }
                    mma_commit(bar2);
                }
                // meanwhile: the new rows go to H (16 lanes cover one 256-byte row)
                const int node_v = misc->node[slot];
                {
                    uint32_t w4[4];
                    ld_shared_v4(sHp + (uint32_t)((sub >> 3) * kBHalf) + sw128_offset(slot, sub & 7), w4);
                    if (node_v >= 0) st_global_v4((char*)p.H + (size_t)node_v * p.ldh * 2 + sub * 16, w4);
                }
                if (!mbar_wait(bar2, ph2, p.poll_limit) && tid == 0) { give_up(p); misc->failed = 1; }
                ph2 ^= 1u;
                tc_fence_after();
                // accumulator blk (0: K, 1: V, 2: next Q, 3: next K, 4: next V) -> byte offset inside a staging row
                {
                    uint32_t d[5][8];
#pragma unroll
                    for (int blk = 0; blk < 5; ++blk)
                        if (blk < n_acc)
                            tmem_ld_32x8(tmem + ((uint32_t)(q4 * 32) << 16) + (uint32_t)(kTile * (1 + blk) + cg * 8), d[blk]);
                    tmem_ld_wait();
#pragma unroll
                    for (int blk = 0; blk < 5; ++blk) {
                        if (blk < n_acc) {
                            const uint32_t off = (uint32_t)(blk * 256 + feat * 2);
#pragma unroll
                            for (int nn = 0; nn < 8; ++nn)
                                st_shared_b16(sSt + (uint32_t)((cg * 8 + nn) * kStageRow) + off, bf16_bits(__uint_as_float(d[blk][nn])));
                        }
                    }
                }
                tc_fence_before();
                __syncthreads();
                if (node_v >= 0) {
                    const uint32_t row = sSt + (uint32_t)(slot * kStageRow);
                    uint32_t w4[4];
#pragma unroll
                    for (int h = 0; h < 2; ++h) {        // this layer's K | V row
                        ld_shared_v4(row + (uint32_t)((sub + 16 * h) * 16), w4);
                        st_global_v4((char*)p.KV[layer] + (size_t)node_v * 512 + (sub + 16 * h) * 16, w4);
                    }
                    if (has_next) {                      // the next layer's Q row and (not yet updated) K | V row
                        ld_shared_v4(row + (uint32_t)(512 + sub * 16), w4);
                        st_global_v4((char*)p.Q[layer + 1] + (size_t)node_v * 256 + sub * 16, w4);
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            ld_shared_v4(row + (uint32_t)(768 + (sub + 16 * h) * 16), w4);
                            st_global_v4((char*)p.KV[layer + 1] + (size_t)node_v * 512 + (sub + 16 * h) * 16, w4);
                        }
                    }
                }
                __syncthreads();    // the tile's shared buffers may be overwritten from here on
            }
            if (!alive) break;
            // ---- this CTA's part of (layer, level l) is in global memory: arrive on its counter (release)
            // (by a thread that does not poll: the release waits for the CTA's outstanding stores, and the pollers
            // should already be watching the next level's counters meanwhile)
            if (tid == 64) red_release_add(my_arrive + l, 1);
        }
        if (n_l > 0) {
            last_nonempty = l;
            last_participants = tiles < nctas ? tiles : nctas;
        }
        // rotate the pipeline by one level
        v0 = vC; pad0 = padC;
        vC = vB;
        lp0 = lp1; lp1 = lp2; lp2 = lp3; lp3 = lp4;
    }

    // Tensor memory is freed below: every MMA this CTA issued must have completed.  Normally each was waited for
    // right after it was issued; after a wait that ran out, one may still be in flight.
    if (tid == 0) {
        mma_commit(smem_u32(&misc->drain));
        mbar_wait(smem_u32(&misc->drain), 0);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc(tmem, kTmemCols);
    }
}

// ---------------------------------------------------------------------------------------------------
std::mutex g_mu;
int g_sm_count[64] = {};
int g_coop[64] = {};
bool g_dev_known[64] = {};

template <int LPH, int MAXN>
dg4_status launch(const LevParams& p, int grid, cudaStream_t st) {
    auto kern = levelised_kernel<LPH, MAXN>;
    DG4_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kLaunchSmemBytes));
    int per_sm = 0;
    DG4_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kThreads, kLaunchSmemBytes));
    if (per_sm != 1) DG4_FAIL(DG4_ERR_CUDA, "the levelised kernel needs exactly one CTA per SM on this device (got %d)", per_sm);
    void* args[] = {(void*)&p};
    DG4_CUDA_TRY(cudaLaunchCooperativeKernel((const void*)kern, dim3(grid), dim3(kThreads), args, kLaunchSmemBytes, st));
    dg4i_count_launch();
    return DG4_OK;
}

template <int MAXN>
dg4_status launch_heads(int heads, const LevParams& p, int grid, cudaStream_t st) {
    switch (16 / heads) {
        case 1: return launch<1, MAXN>(p, grid, st);
        case 2: return launch<2, MAXN>(p, grid, st);
        case 4: return launch<4, MAXN>(p, grid, st);
        case 8: return launch<8, MAXN>(p, grid, st);
        case 16: return launch<16, MAXN>(p, grid, st);
    }
    DG4_FAIL(DG4_ERR_UNSUPPORTED, "heads = %d is not supported", heads);
}

}  // namespace

size_t dg4i_levelised_sync_bytes(const dg4_graph* g, int n_layers) {
    return ((size_t)g->n_levels * (size_t)n_layers + 64) * sizeof(int32_t);
}

dg4_status dg4i_levelised_launch(const dg4_graph* g, const dg4_desc* desc, int n_layers, __nv_bfloat16* const* Q,
                                 __nv_bfloat16* const* KV, __nv_bfloat16* H, int64_t ldh,
                                 const __nv_bfloat16* const* W_qkv, const __nv_bfloat16* const* W_o, int32_t* sync,
                                 int32_t* status, cudaStream_t st) {
    if (n_layers < 1 || n_layers > DG4I_MAX_LAYERS)
        DG4_FAIL(DG4_ERR_UNSUPPORTED, "n_layers = %d: between 1 and %d layers per call", n_layers, DG4I_MAX_LAYERS);
    int dev = 0;
    DG4_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) DG4_FAIL(DG4_ERR_UNSUPPORTED, "device ordinal %d is out of range", dev);
    {
        std::lock_guard<std::mutex> lock(g_mu);
        if (!g_dev_known[dev]) {
            DG4_CUDA_TRY(cudaDeviceGetAttribute(&g_sm_count[dev], cudaDevAttrMultiProcessorCount, dev));
            DG4_CUDA_TRY(cudaDeviceGetAttribute(&g_coop[dev], cudaDevAttrCooperativeLaunch, dev));
            g_dev_known[dev] = true;
        }
    }
    if (!g_coop[dev]) DG4_FAIL(DG4_ERR_UNSUPPORTED, "device %d cannot launch cooperative kernels", dev);
    if (g_sm_count[dev] < n_layers) DG4_FAIL(DG4_ERR_UNSUPPORTED, "fewer SMs than layers");
    LevParams p;
    for (int k = 0; k < DG4I_MAX_LAYERS; ++k) {
        const int kk = k < n_layers ? k : 0;           // unused slots repeat layer 0 (never read)
        p.Wo[k] = W_o[kk];
        p.Wqkv[k] = W_qkv[kk];
        p.Q[k] = Q[kk];
        p.KV[k] = KV[kk];
    }
    DG4_CUDA_TRY(cudaMemsetAsync(sync, 0, dg4i_levelised_sync_bytes(g, n_layers), st));
    p.H = H; p.ldh = ldh;
    p.nbr_pad = g->nbr_pad; p.level_ptr = g->level_ptr; p.level_nodes = g->level_nodes;
    p.n_levels = g->n_levels; p.n_layers = n_layers;
    p.residual = (desc->flags & DG4_FLAG_RESIDUAL) ? 1 : 0; p.scale = desc->scale;
    p.abort_word = sync; p.arrive = sync + 16; p.status = status; p.poll_limit = dg4i_poll_limit();
    const int grid = g_sm_count[dev];
    if (g->max_class <= 3) return launch_heads<3>(desc->heads, p, grid, st);
    return launch_heads<7>(desc->heads, p, grid, st);
}
