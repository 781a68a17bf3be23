// Levelised layer as ONE persistent kernel (Sec. 1 / Sec. 3.4: gates are encoded level by level in
// topological order, each gate once, reading the rows already updated for lower levels).
//
// Q | K | V of every node have been projected from the layer's input beforehand (a node's own query, key and
// value always come from its row as it was when the layer started).  This kernel then walks the levels.
// For a tile of 16 nodes of the current level a CTA
//   1. gathers the K | V rows of every neighbour (16 lanes per node, 16 bytes per lane), computes scores,
//      softmax and the weighted value sum in registers, and writes the 16 x 128 attention tile into shared
//      memory in the tensor core's K-major, 128-byte-swizzled operand layout;
//   2. runs the output projection TRANSPOSED on the tensor cores: D1[feature, node] = W_o * O^T
//      (tcgen05.mma, M = 128 features, N = 16 nodes, K = 128), so a small tile costs a fraction of a
//      128-row tile and all warps take part in the epilogue (128 TMEM lanes x 16 columns);
//   3. adds the residual, rounds to bf16, writes the new rows to H and -- in operand layout again -- to shared
//      memory, and
//   4. refreshes the tile's K | V rows the same way: D2 = W_k * H'^T and W_v * H'^T, rounded and stored.
// W_o, W_k and W_v stay resident in shared memory for the whole kernel (one TMA load each).
//
// Levels are separated by counters in global memory instead of kernel launches: each level has an arrival
// counter that only the CTAs owning a tile of that level bump (release); before a level in which it has work a
// CTA waits (acquire) until the previous non-empty level's counter is full.  Completion is transitive, because
// every CTA that arrived on that level had itself waited for the level before it.  Launched cooperatively (all CTAs
// co-resident).  Every wait is bounded; on expiry the kernel records DG4_ERR_TIMEOUT, raises an abort word that
// every other wait polls, and all CTAs leave their loops, free tensor memory and return.

#include "dg4_internal.h"
#include "dg4_attn_core.cuh"
#include "dg4_sm100.cuh"

#include <mutex>

namespace {

using namespace sm100;
using namespace attn;

constexpr int kTile = 16;                    // nodes per tile
constexpr int kThreads = kTile * 16;         // 16 lanes per node
constexpr int kWBlock = 2 * 128 * 128;       // one 128 x 128 bf16 weight block: two K-halves of 16 KiB
constexpr int kBHalf = kTile * 128;          // K-half of a kTile-row operand tile
constexpr int kTmemCols = 64;

constexpr int kOffW = 0;                          // W_o | W_k | W_v : 96 KiB
constexpr int kOffO = 3 * kWBlock;                // attention tile (operand layout)
constexpr int kOffHp = kOffO + 2 * kBHalf;        // new rows (operand layout)
constexpr int kOffHres = kOffHp + 2 * kBHalf;     // residual rows, plain [kTile][256 B]
constexpr int kOffKV = kOffHres + kTile * 256;    // K|V staging, plain [kTile][512 B]
constexpr int kOffMisc = kOffKV + kTile * 512;
constexpr int kSmemBytes = kOffMisc + 512 + 1024;

struct Misc {
    uint64_t w_full, mma1, mma2;
    uint32_t tmem_base;
    int32_t go;
    int32_t node[kTile];
};

struct LevParams {
    const __nv_bfloat16* Q;          // [n, 128]
    __nv_bfloat16* KV;               // [n, 256]
    __nv_bfloat16* H;                // [n, ldh]
    int64_t ldh;
    const int32_t* nbr_ptr;
    const int32_t* nbr_idx;
    const int32_t* level_ptr;
    const int32_t* level_nodes;
    int32_t n_levels;
    int32_t residual;
    float scale;
    int32_t* arrive;                 // [n_levels], zero on entry
    int32_t* abort_word;             // zero on entry
    int32_t* status;
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
__device__ __forceinline__ void tmem_ld_32x8(uint32_t taddr, uint32_t* r) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr) : "memory");
}
__device__ __forceinline__ uint16_t bf16_bits(float x) {
    __nv_bfloat16 h = __float2bfloat16_rn(x);
    return *reinterpret_cast<uint16_t*>(&h);
}
// byte offset of element k (0..127) of row `row` in a kTile-row operand tile (two K-halves, 128-byte swizzle)
__device__ __forceinline__ uint32_t operand_offset(int row, int k) {
    return (uint32_t)((k >> 6) * kBHalf) + sw128_offset(row, (k & 63) >> 3) + (uint32_t)((k & 7) * 2);
}

template <int LPH, int MAXN>
__global__ void __launch_bounds__(kThreads, 1)
levelised_kernel(const __grid_constant__ CUtensorMap map_wo, const __grid_constant__ CUtensorMap map_wqkv, LevParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
    Misc* misc = reinterpret_cast<Misc*>(base_ptr + kOffMisc);
    const uint32_t sW = base + kOffW, sO = base + kOffO, sHp = base + kOffHp, sHres = base + kOffHres, sKV = base + kOffKV;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int slot = tid >> 4, sub = tid & 15;          // node slot of the tile and lane within the node
    const int grp_base = lane - sub;
    const uint32_t bar_w = smem_u32(&misc->w_full), bar1 = smem_u32(&misc->mma1), bar2 = smem_u32(&misc->mma2);

    if (tid == 0) {
        mbar_init(bar_w, 1);
        mbar_init(bar1, 1);
        mbar_init(bar2, 1);
        misc->go = 1;
        mbar_fence_init();
        tma_prefetch_desc(&map_wo);
        tma_prefetch_desc(&map_wqkv);
        mbar_expect_tx(bar_w, 3u * kWBlock);
        for (int h = 0; h < 2; ++h) {
            tma_load_2d(sW + h * (kWBlock / 2), &map_wo, h * 64, 0, bar_w);
            tma_load_2d(sW + kWBlock + h * (kWBlock / 2), &map_wqkv, h * 64, 128, bar_w);
            tma_load_2d(sW + 2 * kWBlock + h * (kWBlock / 2), &map_wqkv, h * 64, 256, bar_w);
        }
    }
    if (warp == 0) tmem_alloc(smem_u32(&misc->tmem_base), kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = misc->tmem_base;
    bool weights_ok = mbar_wait(bar_w, 0);
    if (!weights_ok && tid == 0) {
        atomicExch(p.abort_word, 1);
        if (p.status) atomicCAS(p.status, 0, (int)DG4_ERR_TIMEOUT);
    }

    const uint32_t idesc = idesc_bf16_f32(128, kTile);
    static_assert(kThreads / 32 / 4 * 8 == kTile, "epilogue: every warp reads 8 node columns of its lane quadrant");
    const int q4 = warp & 3, cg = warp >> 2;             // epilogue: TMEM lane quadrant and group of 8 node columns
    const int feat = q4 * 32 + lane;                     // output feature this thread holds in the epilogues
    uint32_t ph1 = 0, ph2 = 0;
    int last_nonempty = -1, last_participants = 0;
    bool alive = true;
    const int bid = blockIdx.x, nctas = gridDim.x;

    // The index chain of a tile (node id -> list bounds -> neighbour ids) is three dependent loads that do not
    // depend on any other CTA's results.  It is software-pipelined across levels so that none of it sits on the
    // level-to-level critical path: while level l is processed, the node id of this CTA's first tile of level
    // l+3, the list bounds for level l+2 and the neighbour ids for level l+1 are in flight.
    auto level_first = [&](int lv) { return lv < p.n_levels ? p.level_ptr[lv] : 0; };
    auto level_size = [&](int lv) { return lv < p.n_levels ? p.level_ptr[lv + 1] - p.level_ptr[lv] : 0; };
    auto stage_node = [&](int lv) -> int {            // node of (first tile of this CTA, this slot) at level lv
        const int n_lv = level_size(lv);
        const int r = bid * kTile + slot;
        return (r < n_lv) ? p.level_nodes[level_first(lv) + r] : -1;
    };
    // pipeline state at the top of iteration l:
    int v0 = -1, cnt0 = 1, idx0 = -1;                  // level l  : node id, list length, this lane's neighbour id
    int vC = -1, cntC = 1, begC = 0;                   // level l+1: node id and list bounds
    int vB = -1;                                       // level l+2: node id
    {   // prologue: levels 0, 1, 2
        v0 = stage_node(0);
        vC = stage_node(1);
        vB = stage_node(2);
        int beg0 = 0;
        if (v0 >= 0) { beg0 = p.nbr_ptr[v0]; cnt0 = p.nbr_ptr[v0 + 1] - beg0; }
        if (vC >= 0) { begC = p.nbr_ptr[vC]; cntC = p.nbr_ptr[vC + 1] - begC; }
        idx0 = (v0 >= 0 && sub < cnt0) ? p.nbr_idx[beg0 + sub] : v0;
    }

    for (int l = 0; l < p.n_levels && alive; ++l) {
        const int first = p.level_ptr[l];
        const int n_l = p.level_ptr[l + 1] - first;
        // issue the next load of every pipelined chain; the results are first used one level later
        const int vA = stage_node(l + 3);                                               // level l+3: node id
        int begB = 0, cntB = 1;                                                          // level l+2: list bounds
        if (vB >= 0) { begB = p.nbr_ptr[vB]; cntB = p.nbr_ptr[vB + 1] - begB; }
        const int idxC = (vC >= 0 && sub < cntC) ? p.nbr_idx[begC + sub] : vC;          // level l+1: neighbour id
        const int tiles = (n_l + kTile - 1) / kTile;
        if (n_l > 0 && bid < tiles) {
            bool waited = false;
            for (int tile = bid; tile < tiles; tile += nctas) {
                int v, cnt, my_idx;
                bool valid;
                if (tile == bid) {
                    v = v0; cnt = cnt0; my_idx = idx0; valid = v0 >= 0;
                } else {                         // further tiles of a wide level: plain dependent loads
                    const int r = tile * kTile + slot;
                    valid = r < n_l;
                    v = valid ? p.level_nodes[first + r] : -1;
                    int beg = 0;
                    cnt = 1;
                    if (valid) { beg = p.nbr_ptr[v]; cnt = p.nbr_ptr[v + 1] - beg; }
                    my_idx = (valid && sub < cnt) ? p.nbr_idx[beg + sub] : v;
                }

                if (!waited) {
                    // ---- every tile of the previous non-empty level must have arrived (and nobody has given up)
                    if (tid == 0) {
                        int go = 1;
                        if (last_nonempty >= 0) {
                            uint32_t polls = 0;
                            while (ld_acquire(p.arrive + last_nonempty) < last_participants) {
                                ++polls;
                                if (polls > (1u << 22) || ((polls & 63u) == 0 && ld_acquire(p.abort_word) != 0)) { go = 0; break; }
                                if (polls > 64) __nanosleep(32);
                            }
                            if (!go && ld_acquire(p.abort_word) == 0) {
                                atomicExch(p.abort_word, 1);
                                if (p.status) atomicCAS(p.status, 0, (int)DG4_ERR_TIMEOUT);
                            }
                        }
                        if (go && (l & 255) == 0 && ld_acquire(p.abort_word) != 0) go = 0;
                        misc->go = go;
                    }
                    __syncthreads();
                    waited = true;
                    if (!misc->go) { alive = false; break; }
                }

                // ---- gather and attend
                Piece kq[MAXN], vq[MAXN], qp, hres;
                int u[MAXN];
#pragma unroll
                for (int j = 0; j < MAXN; ++j) u[j] = __shfl_sync(0xffffffffu, my_idx, grp_base + j);
                float acc[8];
                if (valid) {
                    const char* kv = (const char*)p.KV;
#pragma unroll
                    for (int j = 0; j < MAXN; ++j)
                        if (j < cnt) vq[j] = ld_piece_cg(kv + (size_t)u[j] * 512 + 256 + sub * 16);
                    if (cnt > 1) {
                        qp = ld_piece_nc((const char*)p.Q + (size_t)v * 256 + sub * 16);
#pragma unroll
                        for (int j = 0; j < MAXN; ++j)
                            if (j < cnt) kq[j] = ld_piece_cg(kv + (size_t)u[j] * 512 + sub * 16);
                    }
                    if (p.residual) hres = ld_piece_cg((const char*)p.H + (size_t)v * p.ldh * 2 + sub * 16);
                } else {
                    vq[0].w[0] = vq[0].w[1] = vq[0].w[2] = vq[0].w[3] = 0u;
                }
                if (!valid || !p.residual) hres.w[0] = hres.w[1] = hres.w[2] = hres.w[3] = 0u;
                attend<true, LPH, MAXN>(qp, kq, vq, cnt, p.scale, 0xffffu << grp_base, acc);
                {
                    Piece o = Elem<true>::pack(acc);
                    st_shared_v4(sO + (uint32_t)((sub >> 3) * kBHalf) + sw128_offset(slot, sub & 7), o.w);
                    st_shared_v4(sHres + (uint32_t)(slot * 256 + sub * 16), hres.w);
                    if (sub == 0) misc->node[slot] = v;
                }
                fence_proxy_async_smem();
                __syncthreads();

                // ---- output projection, transposed: D1[feature, node] = W_o * O^T
                if (tid == 0) {
                    tc_fence_after();
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        const uint32_t a_off = (uint32_t)((ks >> 2) * (kWBlock / 2) + (ks & 3) * 32);
                        const uint32_t b_off = (uint32_t)((ks >> 2) * kBHalf + (ks & 3) * 32);
                        mma_bf16(tmem, smem_desc_sw128(sW + a_off), smem_desc_sw128(sO + b_off), idesc, ks > 0 ? 1u : 0u);
                    }
                    mma_commit(bar1);
                }
                if (!mbar_wait(bar1, ph1) && tid == 0) {
                    atomicExch(p.abort_word, 1);
                    if (p.status) atomicCAS(p.status, 0, (int)DG4_ERR_TIMEOUT);
                }
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

                // ---- K | V refresh, transposed: D2 = W_k * H'^T and W_v * H'^T
                if (tid == 0) {
                    tc_fence_after();
#pragma unroll
                    for (int blk = 0; blk < 2; ++blk) {
#pragma unroll
                        for (int ks = 0; ks < 8; ++ks) {
                            const uint32_t a_off = (uint32_t)((1 + blk) * kWBlock + (ks >> 2) * (kWBlock / 2) + (ks & 3) * 32);
                            const uint32_t b_off = (uint32_t)((ks >> 2) * kBHalf + (ks & 3) * 32);
                            mma_bf16(tmem + (uint32_t)(kTile + kTile * blk), smem_desc_sw128(sW + a_off),
                                     smem_desc_sw128(sHp + b_off), idesc, ks > 0 ? 1u : 0u);
                        }
                    }
                    mma_commit(bar2);
                }
                // meanwhile: the new rows go to H (16 lanes cover one 256-byte row)
                {
                    const int node_v = misc->node[slot];
                    uint32_t w4[4];
                    ld_shared_v4(sHp + (uint32_t)((sub >> 3) * kBHalf) + sw128_offset(slot, sub & 7), w4);
                    if (node_v >= 0) st_global_v4((char*)p.H + (size_t)node_v * p.ldh * 2 + sub * 16, w4);
                }
                if (!mbar_wait(bar2, ph2) && tid == 0) {
                    atomicExch(p.abort_word, 1);
                    if (p.status) atomicCAS(p.status, 0, (int)DG4_ERR_TIMEOUT);
                }
                ph2 ^= 1u;
                tc_fence_after();
                {
                    uint32_t dk[8], dv[8];
                    tmem_ld_32x8(tmem + ((uint32_t)(q4 * 32) << 16) + (uint32_t)(kTile + cg * 8), dk);
                    tmem_ld_32x8(tmem + ((uint32_t)(q4 * 32) << 16) + (uint32_t)(2 * kTile + cg * 8), dv);
                    tmem_ld_wait();
#pragma unroll
                    for (int nn = 0; nn < 8; ++nn) {
                        const int node = cg * 8 + nn;
                        st_shared_b16(sKV + (uint32_t)(node * 512 + feat * 2), bf16_bits(__uint_as_float(dk[nn])));
                        st_shared_b16(sKV + (uint32_t)(node * 512 + 256 + feat * 2), bf16_bits(__uint_as_float(dv[nn])));
                    }
                }
                tc_fence_before();
                __syncthreads();
                {
                    const int node_v = misc->node[slot];
                    if (node_v >= 0) {
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            uint32_t w4[4];
                            ld_shared_v4(sKV + (uint32_t)(slot * 512 + (sub + 16 * h) * 16), w4);
                            st_global_v4((char*)p.KV + (size_t)node_v * 512 + (sub + 16 * h) * 16, w4);
                        }
                    }
                }
                __syncthreads();    // the tile's shared buffers may be overwritten from here on
            }
            if (!alive) break;
            // ---- this CTA's part of level l is in global memory: arrive on the level's counter (release)
            if (tid == 0) red_release_add(p.arrive + l, 1);
        }
        if (n_l > 0) {
            last_nonempty = l;
            last_participants = tiles < nctas ? tiles : nctas;
        }
        // rotate the pipeline by one level
        v0 = vC; cnt0 = cntC; idx0 = idxC;
        vC = vB; cntC = cntB; begC = begB;
        vB = vA;
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc(tmem, kTmemCols);
    }
}

// ---------------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

std::mutex g_mu;
EncodeTiledFn g_encode = nullptr;
int g_sm_count[64] = {};
int g_coop[64] = {};
bool g_dev_known[64] = {};

dg4_status make_weight_map(CUtensorMap* m, const void* base, int64_t rows) {
    {
        std::lock_guard<std::mutex> lock(g_mu);
        if (!g_encode) {
            void* fn = nullptr;
            cudaDriverEntryPointQueryResult q;
            cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q);
            if (e != cudaSuccess || q != cudaDriverEntryPointSuccess || !fn) {
                cudaGetLastError();
                DG4_FAIL(DG4_ERR_CUDA, "cuTensorMapEncodeTiled is not available from this driver");
            }
            g_encode = (EncodeTiledFn)fn;
        }
    }
    cuuint64_t dims[2] = {128, (cuuint64_t)rows};
    cuuint64_t strides[1] = {256};
    cuuint32_t box[2] = {64, 128};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = g_encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) DG4_FAIL(DG4_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);
    return DG4_OK;
}

template <int LPH, int MAXN>
dg4_status launch(const CUtensorMap& map_wo, const CUtensorMap& map_wqkv, const LevParams& p, int grid, cudaStream_t st) {
    auto kern = levelised_kernel<LPH, MAXN>;
    DG4_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
    int per_sm = 0;
    DG4_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kThreads, kSmemBytes));
    if (per_sm < 1) DG4_FAIL(DG4_ERR_CUDA, "the levelised kernel does not fit on this device");
    void* args[] = {(void*)&map_wo, (void*)&map_wqkv, (void*)&p};
    DG4_CUDA_TRY(cudaLaunchCooperativeKernel((const void*)kern, dim3(grid), dim3(kThreads), args, kSmemBytes, st));
    dg4i_count_launch();
    return DG4_OK;
}

template <int MAXN>
dg4_status launch_heads(int heads, const CUtensorMap& a, const CUtensorMap& b, const LevParams& p, int grid, cudaStream_t st) {
    switch (16 / heads) {
        case 1: return launch<1, MAXN>(a, b, p, grid, st);
        case 2: return launch<2, MAXN>(a, b, p, grid, st);
        case 4: return launch<4, MAXN>(a, b, p, grid, st);
        case 8: return launch<8, MAXN>(a, b, p, grid, st);
        case 16: return launch<16, MAXN>(a, b, p, grid, st);
    }
    DG4_FAIL(DG4_ERR_UNSUPPORTED, "heads = %d is not supported", heads);
}

}  // namespace

size_t dg4i_levelised_sync_bytes(const dg4_graph* g) { return ((size_t)g->n_levels + 64) * sizeof(int32_t); }

// Q, KV: projected from the layer's input for all nodes.  sync: dg4i_levelised_sync_bytes() bytes, 16-byte aligned.
dg4_status dg4i_levelised_launch(const dg4_graph* g, const dg4_desc* desc, const __nv_bfloat16* Q, __nv_bfloat16* KV,
                                 __nv_bfloat16* H, int64_t ldh, const __nv_bfloat16* W_qkv, const __nv_bfloat16* W_o,
                                 int32_t* sync, int32_t* status, cudaStream_t st) {
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
    CUtensorMap map_wo, map_wqkv;
    dg4_status s;
    if ((s = make_weight_map(&map_wo, W_o, 128)) != DG4_OK) return s;
    if ((s = make_weight_map(&map_wqkv, W_qkv, 384)) != DG4_OK) return s;
    DG4_CUDA_TRY(cudaMemsetAsync(sync, 0, dg4i_levelised_sync_bytes(g), st));
    LevParams p;
    p.Q = Q; p.KV = KV; p.H = H; p.ldh = ldh;
    p.nbr_ptr = g->nbr_ptr; p.nbr_idx = g->nbr_idx; p.level_ptr = g->level_ptr; p.level_nodes = g->level_nodes;
    p.n_levels = g->n_levels; p.residual = (desc->flags & DG4_FLAG_RESIDUAL) ? 1 : 0; p.scale = desc->scale;
    p.abort_word = sync; p.arrive = sync + 16; p.status = status;
    const int grid = g_sm_count[dev];
    if (g->max_class <= 3) return launch_heads<3>(desc->heads, map_wo, map_wqkv, p, grid, st);
    return launch_heads<7>(desc->heads, map_wo, map_wqkv, p, grid, st);
}
