// The rest of the Transformer block around the sparse attention (Sec. 3.5 replaces only the attention module
// and keeps the block's structure; the block itself is the original post-norm Transformer layer):
//   row-wise layer normalisation, and the position-wise feed-forward sub-layer with residual and the
//   normalisation that follows it:
//       U = max(0, X W1^T + b1),  W1 [512, 128];     Y = LayerNorm(X + U W2^T + b2),  W2 [128, 512].
//
// ffn_kernel: one persistent CTA per SM, a tile = 128 rows.  The hidden activations never leave the SM.
//   * W1 stays in TENSOR memory for the whole kernel (4 blocks of 128 hidden units x 128 inputs = 4 x 64 columns)
//     and is the A operand of the first product, computed TRANSPOSED per block q of 128 hidden units:
//         D1^T[hidden, row] = W1_q (tensor memory) * X^T (the X tile in shared memory, K-major, as B operand);
//   * the epilogue of block q reads the accumulator as m16n8 fragments, adds b1, applies the ReLU, rounds to bf16
//     and writes the values with transposing matrix stores (8 rows x 32 hidden units each) into shared memory as
//     the K-major, 128-byte-swizzled A operand of the second product: A2[row, hidden of block q];
//   * second product, accumulated over the four blocks: D2[row, out] += A2 * W2_q^T with W2 resident in shared
//     memory (4 chunks of 128 outputs x 128 hidden units, 128 KiB, loaded once by TMA);
//   * final epilogue (thread = row, two threads per row): + b2 + the X row (still in shared memory), mean and
//     variance of the row combined from the two half-rows, gamma / beta, bf16, staged in shared memory and
//     written with a TMA store (the last tile is clipped by the tensor map).
//   The X tile of the next tile is prefetched by TMA while the current one is processed.  Inside a tile the eight
//   worker warps never wait for one another: each arrives on an mbarrier when it has read the accumulator or
//   written its part of the operand, and the warp that issues the products waits on those.
// Every CTA loads its own tiles (no load is shared across CTAs).  Every wait is bounded; after a timeout the kernel records DG4_ERR_TIMEOUT and
// the CTA leaves its tile loop.
#include "dg4_internal.h"
#include "dg4_sm100.cuh"

#include <algorithm>
#include <mutex>

namespace {

using namespace sm100;

constexpr int kTileM = 128;                 // rows per tile
constexpr int kWorkers = 256;               // eight warps: epilogues of both products
constexpr int kThreads = kWorkers + 32;     // and a ninth warp whose first lane issues every tcgen05.mma
constexpr int kHalf = 128 * 128;            // bytes of one K-half (64 bf16 columns) of a 128-row operand tile
constexpr int kTileBytes = 2 * kHalf;       // 32 KiB: a 128 x 128 bf16 operand tile
constexpr int kOffW2 = 0;                   // 4 chunks of W2
constexpr int kOffX = 4 * kTileBytes;       // 2 stages of X tiles
constexpr int kOffA2 = kOffX + 2 * kTileBytes;   // hidden activations of one block; later the output staging
constexpr int kOffMisc = kOffA2 + kTileBytes;
constexpr int kSmemBytes = kOffMisc + 1024 + 128;
static_assert(kSmemBytes <= 232448, "shared memory budget of one CTA");
constexpr int kColD1 = 0, kColD2 = 128, kColW1 = 256, kTmemCols = 512;

struct Misc {
    uint64_t bar_w, bar_x[2], bar_g1, bar_g2, bar_d1free, bar_a2full, bar_drain;
    uint32_t tmem_base;
    int32_t posted;            // tiles whose rows have landed, as told to the issuing thread so far (monotone)
    int32_t stop;              // the workers are leaving: no further products
};

struct FfnParams {
    const __nv_bfloat16* W1;
    const float* b1;
    const float* b2;
    const float* gamma;
    const float* beta;
    float eps;
    int32_t n_tiles;
    int32_t* status;
    uint32_t poll_limit;      // polls after which a pipeline wait gives up
    // rows taken from a list (the level-by-level block): X and Y are then addressed directly, not through tensor maps
    const int32_t* row_list;
    int32_t first, rows;
    const __nv_bfloat16* X; int64_t ldx;
    __nv_bfloat16* Y; int64_t ldy;
};

__device__ __forceinline__ void ld_nc_v4(const void* p, uint32_t* r) {
    asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "l"(p));
}
__device__ __forceinline__ void st_global_v4(void* p, const uint32_t* r) {
    asm volatile("st.global.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]) : "memory");
}

__device__ __forceinline__ void st_shared_v4(uint32_t addr, const uint32_t* r) {
    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]) : "memory");
}
__device__ __forceinline__ void ld_shared_v4(uint32_t addr, uint32_t* r) {
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}
__device__ __forceinline__ void st_shared_f2(uint32_t addr, float a, float b) {
    asm volatile("st.shared.v2.f32 [%0], {%1,%2};" ::"r"(addr), "f"(a), "f"(b) : "memory");
}
__device__ __forceinline__ void ld_shared_f2(uint32_t addr, float& a, float& b) {
    asm volatile("ld.shared.v2.f32 {%0,%1}, [%2];" : "=f"(a), "=f"(b) : "r"(addr) : "memory");
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {   // both rounded to nearest even in one conversion
    uint32_t pk;
    asm("cvt.rn.bf16x2.f32 %0, %2, %1;" : "=r"(pk) : "f"(lo), "f"(hi));
    return pk;
}
// max(0, lo) and max(0, hi) rounded to bf16 in one conversion (lo in the low half)
__device__ __forceinline__ uint32_t relu_pack(float lo, float hi) {
    uint32_t pk;
    asm("cvt.rn.relu.bf16x2.f32 %0, %2, %1;" : "=r"(pk) : "f"(lo), "f"(hi));
    return pk;
}
// barrier (and barrier with an OR reduction) among the eight worker warps only
__device__ __forceinline__ void worker_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kWorkers) : "memory"); }
__device__ __forceinline__ bool worker_sync_or(bool flag) {
    uint32_t out;
    asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.u32 p, %1, 0;\n\tbar.red.or.pred q, 1, %2, p;\n\tselp.u32 %0, 1, 0, q;\n\t}"
                 : "=r"(out) : "r"(flag ? 1u : 0u), "n"(kWorkers) : "memory");
    return out != 0;
}
// byte offset of element k (0..127) of row `row` in a 128-row operand tile (two K-halves, 128-byte swizzle)
__device__ __forceinline__ uint32_t operand_offset(int row, int k) {
    return (uint32_t)((k >> 6) * kHalf) + sw128_offset(row, (k & 63) >> 3) + (uint32_t)((k & 7) * 2);
}
// descriptor address increment of K-step ks (16 elements) inside an operand tile
__device__ __forceinline__ uint64_t kstep(int ks) { return (uint64_t)(((ks >> 2) * kHalf + (ks & 3) * 32) >> 4); }

template <bool LISTED>
__global__ void __launch_bounds__(kThreads, 1)
ffn_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w2,
           const __grid_constant__ CUtensorMap map_y, FfnParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
    Misc* misc = reinterpret_cast<Misc*>(base_ptr + kOffMisc);
    const uint32_t sW2 = base + kOffW2, sX = base + kOffX, sA2 = base + kOffA2;
    const uint32_t bar_w = smem_u32(&misc->bar_w), bar_g1 = smem_u32(&misc->bar_g1), bar_g2 = smem_u32(&misc->bar_g2);
    const uint32_t bar_x[2] = {smem_u32(&misc->bar_x[0]), smem_u32(&misc->bar_x[1])};
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int q4 = warp & 3, cg = warp >> 2;             // TMEM lane quadrant of the warp; which half of the columns it takes
    const int ln = q4 * 32 + lane;                       // TMEM lane of this thread: a hidden unit, later a row
    const uint32_t lane_base = (uint32_t)(q4 * 32) << 16;

    const int first_tile = (int)blockIdx.x;
    if (tid == 0) {
        mbar_init(bar_w, 1);
        mbar_init(bar_x[0], 1);
        mbar_init(bar_x[1], 1);
        mbar_init(bar_g1, 1);
        mbar_init(bar_g2, 1);
        mbar_init(smem_u32(&misc->bar_d1free), kWorkers / 32);     // one arrival per worker warp
        mbar_init(smem_u32(&misc->bar_a2full), kWorkers / 32);
        mbar_init(smem_u32(&misc->bar_drain), 1);
        misc->posted = 0;
        misc->stop = 0;
        mbar_fence_init();
        tma_prefetch_desc(&map_x);
        tma_prefetch_desc(&map_w2);
        tma_prefetch_desc(&map_y);
        if (first_tile < p.n_tiles) {
            mbar_expect_tx(bar_w, 4 * kTileBytes);
            for (int q = 0; q < 4; ++q)
                for (int h = 0; h < 2; ++h)
                    tma_load_2d(sW2 + q * kTileBytes + h * kHalf, &map_w2, q * 128 + h * 64, 0, bar_w);
            if (!LISTED) {
                mbar_expect_tx(bar_x[0], kTileBytes);
                for (int h = 0; h < 2; ++h) tma_load_2d(sX + h * kHalf, &map_x, h * 64, first_tile * kTileM, bar_x[0]);
            }
        }
    }
    if (warp == 0) tmem_alloc(smem_u32(&misc->tmem_base), kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = misc->tmem_base;

    // W1 into tensor memory: hidden unit `ln` of block q in lane `ln`, two consecutive inputs per 32-bit column
    // (the bytes as they lie in global memory); each worker thread copies half a row (128 bytes) of every block.
    float b1v[4][4] = {};                                // b1 of the hidden units this thread holds after a fragment load
    if (warp < 8) {
        for (int q = 0; q < 4; ++q) {
            const uint4* src = reinterpret_cast<const uint4*>(p.W1 + (size_t)(q * 128 + ln) * 128 + cg * 64);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const uint4 lo = src[2 * c], hi = src[2 * c + 1];
                const uint32_t r[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
                tmem_st_32x8(tmem + lane_base + (uint32_t)(kColW1 + q * 64 + cg * 32 + c * 8), r);
            }
#pragma unroll
            for (int m = 0; m < 4; ++m) b1v[q][m] = p.b1[q * 128 + q4 * 32 + 8 * m + (lane >> 2)];
        }
        tmem_st_wait();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();

    const uint32_t idesc = idesc_bf16_f32(128, 128);
    const uint64_t dA2 = smem_desc_sw128(sA2);

    if (warp == 8) {
        // ------------------------------------------------------------------ the issuing thread
        // The order of the products is fixed (per tile: G1(0) G1(1) G2(0) G1(2) G2(1) G1(3) G2(2) G2(3)).  A tile's first
        // product waits for the word that its rows have landed (`posted`); every other first product for all eight
        // worker warps to have read the accumulator D1 (bar_d1free), every second product for all of them to have
        // written their part of the activation buffer (bar_a2full): the warps arrive on those barriers and go on, none
        // waits for another.  Issuing a product keeps the issuing thread busy for about as long as the tensor pipe
        // needs to execute it, which is why no worker does it.
        if (lane == 0) {
            int consumed = 0;
            bool leave = false;
            const uint32_t token_limit = p.poll_limit < (1u << 28) ? p.poll_limit << 2 : p.poll_limit;
            const uint32_t bar_d1free = smem_u32(&misc->bar_d1free), bar_a2full = smem_u32(&misc->bar_a2full);
            uint32_t ph_d1 = 0, ph_a2 = 0;
            int it = 0;
            for (int tile = first_tile; tile < p.n_tiles && !leave; tile += (int)gridDim.x, ++it) {
                const uint64_t dX = smem_desc_sw128(sX + (it & 1) * kTileBytes);
                for (int step = 0; step < 8 && !leave; ++step) {
                    const bool first_product = (step == 0) || (step == 1) || (step == 3) || (step == 5);
                    if (step == 0) {
                        uint32_t polls = 0;
                        while (*reinterpret_cast<volatile int32_t*>(&misc->posted) <= consumed) {
                            if (*reinterpret_cast<volatile int32_t*>(&misc->stop) != 0 || ++polls > token_limit) { leave = true; break; }
                            if (polls > 256) __nanosleep(20);
                        }
                        if (leave || *reinterpret_cast<volatile int32_t*>(&misc->stop) != 0) { leave = true; break; }
                        ++consumed;
                        __threadfence_block();
                        if (it > 0) {                    // block 3 of the tile before is out of D1 (long since: its second product was issued)
                            if (!mbar_wait(bar_d1free, ph_d1, token_limit)) { leave = true; break; }
                            ph_d1 ^= 1u;
                        }
                    } else if (first_product) {
                        if (!mbar_wait(bar_d1free, ph_d1, token_limit)) { leave = true; break; }
                        ph_d1 ^= 1u;
                    } else {
                        if (!mbar_wait(bar_a2full, ph_a2, token_limit)) { leave = true; break; }
                        ph_a2 ^= 1u;
                    }
                    tc_fence_after();
                    // steps 0, 1, 3, 5 are first products of blocks 0..3; steps 2, 4, 6, 7 second products of blocks 0..3
                    const int q = first_product ? (step + 1) / 2 : (step == 7 ? 3 : step / 2 - 1);
                    if (first_product) {             // D1^T = W1_q * X^T
#pragma unroll
                        for (int ks = 0; ks < 8; ++ks)
                            mma_bf16_ta(tmem + kColD1, tmem + (uint32_t)(kColW1 + q * 64 + ks * 8), dX + kstep(ks), idesc, ks > 0 ? 1u : 0u);
                        mma_commit(bar_g1);
                    } else {                         // D2 += A2 * W2_q^T
                        const uint64_t dW2 = smem_desc_sw128(sW2 + q * kTileBytes);
#pragma unroll
                        for (int ks = 0; ks < 8; ++ks)
                            mma_bf16(tmem + kColD2, dA2 + kstep(ks), dW2 + kstep(ks), idesc, (q > 0 || ks > 0) ? 1u : 0u);
                        mma_commit(bar_g2);
                    }
                }
            }
            // tensor memory is freed below: every product issued must have completed
            mma_commit(smem_u32(&misc->bar_drain));
            mbar_wait(smem_u32(&misc->bar_drain), 0);
        }
    } else {
        // ------------------------------------------------------------------ the eight worker warps
        const uint32_t bar_d1free = smem_u32(&misc->bar_d1free), bar_a2full = smem_u32(&misc->bar_a2full);
        auto release_product = [&]() {               // one worker thread: the rows of a tile have landed
            __threadfence_block();
            *reinterpret_cast<volatile int32_t*>(&misc->posted) = misc->posted + 1;
        };
        // The accumulator of a first product holds hidden units in lanes and rows in columns; the operand of the
        // second product wants rows with their hidden units contiguous.  A fragment load followed by a transposing
        // matrix store does that 8 rows x 32 hidden units at a time: thread 8m + j passes the address of row
        // cg*64 + 8c + j, hidden units q4*32 + 8m .. +7 (16 bytes; the swizzle depends on j only).
        const uint32_t a2_addr = sA2 + operand_offset(cg * 64 + (lane & 7), q4 * 32 + 8 * (lane >> 3));
        uint32_t ph_g1 = 0, ph_g2 = 0;
        bool failed = false;
        if (first_tile < p.n_tiles) failed |= !mbar_wait(bar_w, 0, p.poll_limit);

        int it = 0;
        bool g1_released = false;        // the first product of the tile about to start was released during the tile before
        for (int tile = first_tile; tile < p.n_tiles; tile += (int)gridDim.x, ++it) {
            const int s = it & 1;
            const uint32_t sXs = sX + s * kTileBytes;
            const bool has_next = tile + (int)gridDim.x < p.n_tiles;
            if (!LISTED) {
                if (tid == 0 && has_next) {                      // prefetch the next tile's rows into the other stage
                    const int next = tile + (int)gridDim.x;
                    mbar_expect_tx(bar_x[s ^ 1], kTileBytes);
                    for (int h = 0; h < 2; ++h)
                        tma_load_2d(sX + (s ^ 1) * kTileBytes + h * kHalf, &map_x, h * 64, next * kTileM, bar_x[s ^ 1]);
                }
                if (!g1_released) {
                    failed |= !mbar_wait(bar_x[s], (uint32_t)(it >> 1) & 1u, p.poll_limit);
                    worker_sync();
                    if (tid == 0) release_product();         // G1(0)
                }
            } else {
                // listed rows: the workers gather the tile's rows into the same swizzled layout, 16 bytes at a time
                for (int i = tid; i < kTileM * 16; i += kWorkers) {
                    const int row = i >> 4, chunk = i & 15;
                    const int r = tile * kTileM + row;
                    uint32_t v[4] = {0u, 0u, 0u, 0u};
                    if (r < p.rows) ld_nc_v4(p.X + (int64_t)p.row_list[p.first + r] * p.ldx + chunk * 8, v);
                    st_shared_v4(sXs + (uint32_t)((chunk >> 3) * kHalf) + sw128_offset(row, chunk & 7), v);
                }
                fence_proxy_async_smem();
                worker_sync();
                if (tid == 0) release_product();             // G1(0)
            }

            // Per block q of hidden units: the accumulator is read into registers, the next block's first product is
            // released at once (it runs while the values are scattered into the operand buffer), then the second
            // product of this block.  The tensor pipe executes in issue order: G1(0) G1(1) G2(0) G1(2) G2(1) ...
            for (int q = 0; q < 4; ++q) {
                failed |= !mbar_wait(bar_g1, ph_g1, p.poll_limit);         // D1^T of block q is complete
                ph_g1 ^= 1u;
                tc_fence_after();
                uint32_t d[64];
                tmem_ld_16x256b_x8(tmem + lane_base + (uint32_t)(kColD1 + cg * 64), d);                  // lanes +0..15
                tmem_ld_16x256b_x8(tmem + lane_base + (16u << 16) + (uint32_t)(kColD1 + cg * 64), d + 32);  // lanes +16..31
                tmem_ld_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_d1free);      // this warp holds its part of D1^T: G1(q + 1) may overwrite it
                if (!LISTED && q == 0) {                     // the previous tile's store has read the staging buffer
                    if (tid == 0) bulk_wait_read0();
                    worker_sync();
                }
                if (q > 0) {                                 // the previous block's second product has read the buffer
                    failed |= !mbar_wait(bar_g2, ph_g2, p.poll_limit);
                    ph_g2 ^= 1u;
                }
                // d[32u + 4c + 2h + e]: hidden unit q4*32 + 8(2u + h) + lane/4, row cg*64 + 8c + 2(lane%4) + e; bias and
                // ReLU folded into the conversion, then eight rows of 32 hidden units per store
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    uint32_t m[4];
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const int i = 32 * (k >> 1) + 4 * c + 2 * (k & 1);
                        m[k] = relu_pack(__uint_as_float(d[i]) + b1v[q][k], __uint_as_float(d[i + 1]) + b1v[q][k]);
                    }
                    stmatrix_x4_trans(a2_addr + (uint32_t)(c * 1024), m);
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_a2full);      // this warp's part of the operand is written: G2(q)
            }
            // The next tile's rows were requested a tile ago and have landed: its first product may run under this
            // tile's final epilogue (its accumulator is free: every worker has read block 3's before the last barrier).
            g1_released = false;
            if (!LISTED && has_next) {
                if (tid == 0) {
                    failed |= !mbar_wait(bar_x[s ^ 1], (uint32_t)((it + 1) >> 1) & 1u, p.poll_limit);
                    release_product();                       // G1(0) of the next tile
                }
                g1_released = true;
            }
            failed |= !mbar_wait(bar_g2, ph_g2, p.poll_limit);   // D2 is complete; the activation buffer is free
            ph_g2 ^= 1u;
            tc_fence_after();

            // ---- final epilogue: thread = row `ln`, columns cg*64 .. cg*64+63
            {
                float y[64];
                {
                    uint32_t d[64];
                    tmem_ld_32x32(tmem + lane_base + (uint32_t)(kColD2 + cg * 64), d);
                    tmem_ld_32x32(tmem + lane_base + (uint32_t)(kColD2 + cg * 64 + 32), d + 32);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 64; ++j) y[j] = __uint_as_float(d[j]);
                }
                tc_fence_before();
                const float4* b2v = reinterpret_cast<const float4*>(p.b2 + cg * 64);
#pragma unroll
                for (int c = 0; c < 8; ++c) {                // + b2 + the row of X (K-half cg of the X tile)
                    uint32_t w[4];
                    ld_shared_v4(sXs + (uint32_t)(cg * kHalf) + sw128_offset(ln, c), w);
                    const float4 ba = __ldg(b2v + 2 * c), bb = __ldg(b2v + 2 * c + 1);
                    y[c * 8 + 0] += __uint_as_float(w[0] << 16) + ba.x;
                    y[c * 8 + 1] += __uint_as_float(w[0] & 0xffff0000u) + ba.y;
                    y[c * 8 + 2] += __uint_as_float(w[1] << 16) + ba.z;
                    y[c * 8 + 3] += __uint_as_float(w[1] & 0xffff0000u) + ba.w;
                    y[c * 8 + 4] += __uint_as_float(w[2] << 16) + bb.x;
                    y[c * 8 + 5] += __uint_as_float(w[2] & 0xffff0000u) + bb.y;
                    y[c * 8 + 6] += __uint_as_float(w[3] << 16) + bb.z;
                    y[c * 8 + 7] += __uint_as_float(w[3] & 0xffff0000u) + bb.w;
                }
                // mean and sum of squared deviations of the half-row, merged with the other half-row's
                float ms[4] = {0.0f, 0.0f, 0.0f, 0.0f};               // four partial sums: four independent chains
#pragma unroll
                for (int j = 0; j < 64; j += 4) { ms[0] += y[j]; ms[1] += y[j + 1]; ms[2] += y[j + 2]; ms[3] += y[j + 3]; }
                const float m = ((ms[0] + ms[1]) + (ms[2] + ms[3])) * (1.0f / 64.0f);
                float vs[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
                for (int j = 0; j < 64; j += 4) {
                    vs[0] = fmaf(y[j] - m, y[j] - m, vs[0]);
                    vs[1] = fmaf(y[j + 1] - m, y[j + 1] - m, vs[1]);
                    vs[2] = fmaf(y[j + 2] - m, y[j + 2] - m, vs[2]);
                    vs[3] = fmaf(y[j + 3] - m, y[j + 3] - m, vs[3]);
                }
                const float m2 = (vs[0] + vs[1]) + (vs[2] + vs[3]);
                st_shared_f2(sA2 + (uint32_t)((ln * 2 + cg) * 8), m, m2);
                worker_sync();
                float mo, m2o;
                ld_shared_f2(sA2 + (uint32_t)((ln * 2 + (cg ^ 1)) * 8), mo, m2o);
                worker_sync();
                const float mean = 0.5f * (m + mo);
                const float var = (m2 + m2o + 32.0f * (m - mo) * (m - mo)) * (1.0f / 128.0f);
                const float rstd = rsqrtf(var + p.eps);
                const float nmr = -mean * rstd;              // (y - mean) rstd as one fused multiply-add per element
                const float4* gv = reinterpret_cast<const float4*>(p.gamma + cg * 64);
                const float4* bv = reinterpret_cast<const float4*>(p.beta + cg * 64);
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    const float4 ga = __ldg(gv + 2 * c), gb = __ldg(gv + 2 * c + 1);
                    const float4 ba = __ldg(bv + 2 * c), bb = __ldg(bv + 2 * c + 1);
                    uint32_t w[4];
                    w[0] = pack_bf16(fmaf(fmaf(y[c * 8 + 0], rstd, nmr), ga.x, ba.x), fmaf(fmaf(y[c * 8 + 1], rstd, nmr), ga.y, ba.y));
                    w[1] = pack_bf16(fmaf(fmaf(y[c * 8 + 2], rstd, nmr), ga.z, ba.z), fmaf(fmaf(y[c * 8 + 3], rstd, nmr), ga.w, ba.w));
                    w[2] = pack_bf16(fmaf(fmaf(y[c * 8 + 4], rstd, nmr), gb.x, bb.x), fmaf(fmaf(y[c * 8 + 5], rstd, nmr), gb.y, bb.y));
                    w[3] = pack_bf16(fmaf(fmaf(y[c * 8 + 6], rstd, nmr), gb.z, bb.z), fmaf(fmaf(y[c * 8 + 7], rstd, nmr), gb.w, bb.w));
                    st_shared_v4(sA2 + (uint32_t)(cg * kHalf) + sw128_offset(ln, c), w);
                }
            }
            fence_proxy_async_smem();
            const bool stop = worker_sync_or(failed);        // also: the X stage may be refilled from here on
            if (!LISTED) {
                if (tid == 0 && !stop) {
                    tma_store_2d(&map_y, 0, tile * kTileM, sA2);
                    tma_store_2d(&map_y, 64, tile * kTileM, sA2 + kHalf);
                    bulk_commit();
                }
            } else if (!stop) {
                for (int i = tid; i < kTileM * 16; i += kWorkers) {
                    const int row = i >> 4, chunk = i & 15;
                    const int r = tile * kTileM + row;
                    if (r < p.rows) {
                        uint32_t v[4];
                        ld_shared_v4(sA2 + (uint32_t)((chunk >> 3) * kHalf) + sw128_offset(row, chunk & 7), v);
                        st_global_v4(p.Y + (int64_t)p.row_list[p.first + r] * p.ldy + chunk * 8, v);
                    }
                }
                worker_sync();                               // the staging buffer is rewritten by the next tile
            }
            if (stop) {
                // A wait ran out somewhere in this CTA.  Every worker went through the whole tile (nothing above
                // branches on `failed`), so all of them are here.  Before the CTA may leave, what it started must
                // have ended: the weight copy and the copies of this tile's and of the prefetched tile's rows (these
                // waits keep the default limit: a copy that was started does land); the issuing thread waits for the
                // products.
                if (tid == 0) {
                    if (p.status) atomicCAS(p.status, 0, (int)DG4_ERR_TIMEOUT);
                    mbar_wait(bar_w, 0);
                    if (!LISTED) {
                        mbar_wait(bar_x[s], (uint32_t)(it >> 1) & 1u);
                        if (tile + (int)gridDim.x < p.n_tiles) mbar_wait(bar_x[s ^ 1], (uint32_t)((it + 1) >> 1) & 1u);
                    }
                }
                break;
            }
        }
        if (tid == 0) {
            *reinterpret_cast<volatile int32_t*>(&misc->stop) = 1;   // releases the issuing thread from its wait
            bulk_wait_all();
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc(tmem, kTmemCols);
    }
}

// ---- row-wise layer normalisation: half a warp per row, eight columns (16 bytes) per lane -----------
__global__ void __launch_bounds__(256)
layernorm_kernel(const __nv_bfloat16* X, int64_t ldx, const float* __restrict__ gamma,
                 const float* __restrict__ beta, float eps, __nv_bfloat16* Y, int64_t ldy, int n,
                 const int32_t* __restrict__ row_list, int list_first) {   // Y may be X; rows from a list if row_list != NULL
    const int sub = threadIdx.x & 15;
    const int groups = (int)((gridDim.x * blockDim.x) >> 4);
    const float4 ga = __ldg(reinterpret_cast<const float4*>(gamma) + 2 * sub), gb = __ldg(reinterpret_cast<const float4*>(gamma) + 2 * sub + 1);
    const float4 ba = __ldg(reinterpret_cast<const float4*>(beta) + 2 * sub), bb = __ldg(reinterpret_cast<const float4*>(beta) + 2 * sub + 1);
    const int first = (int)((blockIdx.x * blockDim.x + threadIdx.x) >> 4);
    // whole warps stay in the loop together (the shuffles name all 32 lanes): rows are dealt two per warp, and
    // every half-warp keeps four rows in flight
    const int hw = (threadIdx.x >> 4) & 1;
    for (int base_row = first - hw; base_row < n; base_row += 4 * groups) {
        uint4 w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int row = base_row + hw + i * groups;
            w[i] = make_uint4(0u, 0u, 0u, 0u);
            if (row < n) w[i] = *reinterpret_cast<const uint4*>(X + (size_t)(row_list ? row_list[list_first + row] : row) * ldx + sub * 8);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int row = base_row + hw + i * groups;
            float x[8] = {__uint_as_float(w[i].x << 16), __uint_as_float(w[i].x & 0xffff0000u), __uint_as_float(w[i].y << 16),
                          __uint_as_float(w[i].y & 0xffff0000u), __uint_as_float(w[i].z << 16), __uint_as_float(w[i].z & 0xffff0000u),
                          __uint_as_float(w[i].w << 16), __uint_as_float(w[i].w & 0xffff0000u)};
            float sum = 0.0f;
#pragma unroll
            for (int j = 0; j < 8; ++j) sum += x[j];
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
            const float mean = sum * (1.0f / 128.0f);
            float sq = 0.0f;
#pragma unroll
            for (int j = 0; j < 8; ++j) { x[j] -= mean; sq += x[j] * x[j]; }
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
            const float rstd = rsqrtf(sq * (1.0f / 128.0f) + eps);
            uint4 out;
            out.x = pack_bf16(x[0] * rstd * ga.x + ba.x, x[1] * rstd * ga.y + ba.y);
            out.y = pack_bf16(x[2] * rstd * ga.z + ba.z, x[3] * rstd * ga.w + ba.w);
            out.z = pack_bf16(x[4] * rstd * gb.x + bb.x, x[5] * rstd * gb.y + bb.y);
            out.w = pack_bf16(x[6] * rstd * gb.z + bb.z, x[7] * rstd * gb.w + bb.w);
            if (row < n) *reinterpret_cast<uint4*>(Y + (size_t)(row_list ? row_list[list_first + row] : row) * ldy + sub * 8) = out;
        }
    }
}

// ---------------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
std::mutex g_mu;
EncodeTiledFn g_encode = nullptr;
bool g_attr_set[64] = {};
int g_sm_count[64] = {};

// [rows, cols] bf16 row-major with leading dimension ld; box = 64 columns x 128 rows, 128-byte swizzle
dg4_status make_map(CUtensorMap* m, const void* base, int64_t rows, int64_t cols, int64_t ld) {
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
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)(ld * 2)};
    cuuint32_t box[2] = {64, 128};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = g_encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) DG4_FAIL(DG4_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);
    return DG4_OK;
}

bool aligned16(const void* p) { return (((uintptr_t)p) & 15u) == 0; }

dg4_status check_rows(const char* name, const void* p, int64_t ld) {
    if (!p) DG4_FAIL(DG4_ERR_INVALID_ARG, "%s is null", name);
    if (!aligned16(p)) DG4_FAIL(DG4_ERR_INVALID_ARG, "%s is not 16-byte aligned", name);
    if (ld < 128) DG4_FAIL(DG4_ERR_INVALID_ARG, "leading dimension of %s (%lld) is below 128", name, (long long)ld);
    if ((ld * 2) % 16 != 0)
        DG4_FAIL(DG4_ERR_INVALID_ARG, "leading dimension of %s (%lld elements) is not a multiple of 16 bytes", name, (long long)ld);
    return DG4_OK;
}

dg4_status check_vec(const char* name, const float* p) {
    if (!p) DG4_FAIL(DG4_ERR_INVALID_ARG, "%s is null", name);
    if (!aligned16(p)) DG4_FAIL(DG4_ERR_INVALID_ARG, "%s is not 16-byte aligned", name);
    return DG4_OK;
}

dg4_status check_common(const dg4_graph* g, const dg4_desc* desc, float eps) {
    dg4_status dev_ok = dg4i_check_device(g);
    if (dev_ok != DG4_OK) return dev_ok;
    if (!desc) DG4_FAIL(DG4_ERR_INVALID_ARG, "null descriptor");
    if (desc->d != 128) DG4_FAIL(DG4_ERR_UNSUPPORTED, "d = %d: only d = 128 is supported", desc->d);
    if (desc->dtype != DG4_BF16) DG4_FAIL(DG4_ERR_UNSUPPORTED, "the block's dense parts are bf16 only");
    if (!(eps >= 0.0f) || eps > 3.0e38f) DG4_FAIL(DG4_ERR_INVALID_ARG, "eps must be finite and not negative");
    return DG4_OK;
}

#define CHECK(expr) do { dg4_status _s = (expr); if (_s != DG4_OK) return _s; } while (0)

}  // namespace

namespace {

struct RowSet {                       // which rows a call works on: 0 .. rows-1, or row_list[first .. first+rows-1]
    const int32_t* row_list = nullptr;
    int32_t first = 0;
    int32_t rows = 0;
};

dg4_status layernorm_launch(const void* X, int64_t ldx, const float* gamma, const float* beta, float eps, void* Y,
                            int64_t ldy, const RowSet& rs, cudaStream_t st) {
    if (rs.rows <= 0) return DG4_OK;
    const int blocks = (int)std::min<int64_t>(((int64_t)rs.rows + 15) / 16, 148 * 8);
    layernorm_kernel<<<blocks, 256, 0, st>>>((const __nv_bfloat16*)X, ldx, gamma, beta, eps, (__nv_bfloat16*)Y, ldy,
                                             rs.rows, rs.row_list, rs.first);
    DG4_CUDA_TRY(cudaGetLastError());
    dg4i_count_launch();
    return DG4_OK;
}

dg4_status ffn_launch(const dg4_graph* g, const void* X, int64_t ldx, const void* W1, const float* b1, const void* W2,
                      const float* b2, const float* gamma, const float* beta, float eps, void* Y, int64_t ldy,
                      const RowSet& rs, cudaStream_t st) {
    if (rs.rows <= 0) return DG4_OK;
    int dev = 0;
    DG4_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) DG4_FAIL(DG4_ERR_UNSUPPORTED, "device ordinal %d is out of range", dev);
    {
        std::lock_guard<std::mutex> lock(g_mu);
        if (!g_attr_set[dev]) {
            DG4_CUDA_TRY(cudaFuncSetAttribute(ffn_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
            DG4_CUDA_TRY(cudaFuncSetAttribute(ffn_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
            DG4_CUDA_TRY(cudaDeviceGetAttribute(&g_sm_count[dev], cudaDevAttrMultiProcessorCount, dev));
            g_attr_set[dev] = true;
        }
    }
    CUtensorMap map_x, map_w2, map_y;
    CHECK(make_map(&map_w2, W2, 128, 512, 512));
    map_x = map_y = map_w2;                      // placeholders when the rows come from a list
    if (!rs.row_list) {
        CHECK(make_map(&map_x, X, rs.rows, 128, ldx));
        CHECK(make_map(&map_y, Y, rs.rows, 128, ldy));
    }
    FfnParams p;
    p.W1 = (const __nv_bfloat16*)W1; p.b1 = b1; p.b2 = b2; p.gamma = gamma; p.beta = beta; p.eps = eps;
    p.n_tiles = (rs.rows + kTileM - 1) / kTileM;
    p.status = g->dev_status;
    p.poll_limit = dg4i_poll_limit();
    p.row_list = rs.row_list; p.first = rs.first; p.rows = rs.rows;
    p.X = (const __nv_bfloat16*)X; p.ldx = ldx; p.Y = (__nv_bfloat16*)Y; p.ldy = ldy;
    const int grid = std::min(p.n_tiles, g_sm_count[dev]);
    if (rs.row_list) ffn_kernel<true><<<grid, kThreads, kSmemBytes, st>>>(map_x, map_w2, map_y, p);
    else ffn_kernel<false><<<grid, kThreads, kSmemBytes, st>>>(map_x, map_w2, map_y, p);
    DG4_CUDA_TRY(cudaGetLastError());
    dg4i_count_launch();
    return DG4_OK;
}

dg4_status check_ffn_args(const void* W1, const float* b1, const void* W2, const float* b2, const float* gamma,
                          const float* beta, int32_t d_ff) {
    if (d_ff != 512) DG4_FAIL(DG4_ERR_UNSUPPORTED, "d_ff = %d: only d_ff = 4 d = 512 is supported", d_ff);
    if (!W1 || !W2) DG4_FAIL(DG4_ERR_INVALID_ARG, "null weight matrix");
    if (!aligned16(W1) || !aligned16(W2)) DG4_FAIL(DG4_ERR_INVALID_ARG, "weight matrices must be 16-byte aligned");
    CHECK(check_vec("b1", b1));
    CHECK(check_vec("b2", b2));
    CHECK(check_vec("gamma", gamma));
    CHECK(check_vec("beta", beta));
    return DG4_OK;
}

}  // namespace

extern "C" dg4_status dg4_layernorm_fwd(const dg4_graph* g, const dg4_desc* desc, const void* X, int64_t ldx,
                                         const float* gamma, const float* beta, float eps, void* Y, int64_t ldy,
                                         void* stream) {
    CHECK(check_common(g, desc, eps));
    CHECK(check_rows("X", X, ldx));
    CHECK(check_rows("Y", Y, ldy));
    CHECK(check_vec("gamma", gamma));
    CHECK(check_vec("beta", beta));
    RowSet all;
    all.rows = g->n;
    return layernorm_launch(X, ldx, gamma, beta, eps, Y, ldy, all, (cudaStream_t)stream);
}

extern "C" dg4_status dg4_ffn_fwd(const dg4_graph* g, const dg4_desc* desc, const void* X, int64_t ldx, const void* W1,
                                   const float* b1, const void* W2, const float* b2, const float* gamma,
                                   const float* beta, float eps, int32_t d_ff, void* Y, int64_t ldy, void* stream) {
    CHECK(check_common(g, desc, eps));
    CHECK(check_ffn_args(W1, b1, W2, b2, gamma, beta, d_ff));
    CHECK(check_rows("X", X, ldx));
    CHECK(check_rows("Y", Y, ldy));
    RowSet all;
    all.rows = g->n;
    return ffn_launch(g, X, ldx, W1, b1, W2, b2, gamma, beta, eps, Y, ldy, all, (cudaStream_t)stream);
}

/* The whole block in level-by-level order (the order of Sec. 1 / Sec. 3.4 applied to the block of Sec. 3.5): one group
 * of launches per level -- attention for the level's nodes, output projection with residual, LayerNorm, feed-forward
 * sub-layer with its LayerNorm (rows taken from the level's node list, updated in place), then the K | V rows of the
 * level are refreshed from the new rows so that higher levels gather block outputs. */
extern "C" dg4_status dg4_block_fwd_levelised(const dg4_graph* g, const dg4_desc* desc, void* H, int64_t ldh,
                                               const void* W_qkv, const void* W_o, const float* ln1_gamma,
                                               const float* ln1_beta, const void* W1, const float* b1, const void* W2,
                                               const float* b2, const float* ln2_gamma, const float* ln2_beta, float eps,
                                               int32_t d_ff, void* workspace, size_t workspace_bytes, void* stream) {
    CHECK(check_common(g, desc, eps));
    CHECK(dg4i_check_desc(desc, true));
    CHECK(check_rows("H", H, ldh));
    if (!W_qkv || !W_o || !aligned16(W_qkv) || !aligned16(W_o)) DG4_FAIL(DG4_ERR_INVALID_ARG, "W_qkv / W_o null or misaligned");
    CHECK(check_vec("ln1_gamma", ln1_gamma));
    CHECK(check_vec("ln1_beta", ln1_beta));
    CHECK(check_ffn_args(W1, b1, W2, b2, ln2_gamma, ln2_beta, d_ff));
    if (!workspace) DG4_FAIL(DG4_ERR_INVALID_ARG, "workspace is null");
    if ((((uintptr_t)workspace) & 255u) != 0) DG4_FAIL(DG4_ERR_INVALID_ARG, "workspace is not 256-byte aligned");
    if (workspace_bytes < dg4_layer_workspace_bytes(g, desc))
        DG4_FAIL(DG4_ERR_INVALID_ARG, "workspace of %zu bytes is below the %zu bytes needed", workspace_bytes,
                 dg4_layer_workspace_bytes(g, desc));
    cudaStream_t st = (cudaStream_t)stream;
    __nv_bfloat16* Hb = (__nv_bfloat16*)H;
    __nv_bfloat16* Q = (__nv_bfloat16*)workspace;
    __nv_bfloat16* KV = Q + (size_t)g->n * 128;
    __nv_bfloat16* O = Q + (size_t)g->n * 384;
    if (!(desc->flags & DG4_FLAG_LEVEL_LAUNCHES) && (size_t)g->n * 256 >= dg4i_levelised_sync_bytes(g, 2)) {
        // one persistent kernel: attention-stage and feed-forward-stage CTAs hand the levels to one another (the
        // counters live where the launch-group driver keeps its Q table, which this path does not need)
        dg4i_block_tail tail;
        tail.ln1_gamma = ln1_gamma; tail.ln1_beta = ln1_beta; tail.W1 = (const __nv_bfloat16*)W1; tail.b1 = b1;
        tail.W2 = (const __nv_bfloat16*)W2; tail.b2 = b2; tail.ln2_gamma = ln2_gamma; tail.ln2_beta = ln2_beta; tail.eps = eps;
        __nv_bfloat16* kv1[1] = {KV};
        const __nv_bfloat16* wq1[1] = {(const __nv_bfloat16*)W_qkv};
        const __nv_bfloat16* wo1[1] = {(const __nv_bfloat16*)W_o};
        return dg4i_levelised_launch(g, desc, 1, kv1, Hb, ldh, wq1, wo1, (int32_t*)workspace, g->dev_status, st, &tail);
    }
    // Q | K | V of every node from the block's input: a node's own query, key and value never change
    CHECK(dg4_qkv_project(g, desc, H, ldh, W_qkv, Q, 128, KV, 256, KV + 128, 256, stream));
    const __nv_bfloat16* W_kv = (const __nv_bfloat16*)W_qkv + (size_t)128 * 128;
    for (int l = 0; l < g->n_levels; ++l) {
        RowSet lev;
        lev.row_list = g->level_nodes; lev.first = g->h_level_ptr[l]; lev.rows = g->h_level_ptr[l + 1] - lev.first;
        if (lev.rows <= 0) continue;
        dg4i_attn_args a;
        a.Q = Q; a.ldq = 128; a.K = KV; a.ldk = 256; a.V = KV + 128; a.ldv = 256; a.O = O; a.ldo = 128;
        a.nbr_pad = g->nbr_pad; a.node_list = g->level_nodes; a.first = lev.first; a.count = lev.rows;
        a.heads = desc->heads; a.max_nbr = g->max_class; a.dtype = desc->dtype; a.scale = desc->scale;
        dg4i_attn_more more;
        more.nbr_ptr = g->nbr_ptr; more.nbr_idx = g->nbr_idx;
        CHECK(dg4i_attn_launch(a, &more, st));
        dg4i_proj_args o;
        o.A = O; o.lda = 128; o.W = (const __nv_bfloat16*)W_o; o.n_out = 128;
        o.out[0] = Hb; o.ldo[0] = ldh; o.out[1] = o.out[2] = nullptr; o.ldo[1] = o.ldo[2] = 0;
        o.R = Hb; o.ldr = ldh; o.row_list = g->level_nodes; o.first = lev.first; o.rows = lev.rows; o.status = g->dev_status;
        CHECK(dg4i_proj_launch(o, st));
        CHECK(layernorm_launch(H, ldh, ln1_gamma, ln1_beta, eps, H, ldh, lev, st));
        CHECK(ffn_launch(g, H, ldh, W1, b1, W2, b2, ln2_gamma, ln2_beta, eps, H, ldh, lev, st));
        if (l + 1 < g->n_levels) {
            dg4i_proj_args k;
            k.A = Hb; k.lda = ldh; k.W = W_kv; k.n_out = 256;
            k.out[0] = KV; k.ldo[0] = 256; k.out[1] = KV + 128; k.ldo[1] = 256; k.out[2] = nullptr; k.ldo[2] = 0;
            k.R = nullptr; k.ldr = 0; k.row_list = g->level_nodes; k.first = lev.first; k.rows = lev.rows; k.status = g->dev_status;
            CHECK(dg4i_proj_launch(k, st));
        }
    }
    return DG4_OK;
}

extern "C" size_t dg4_blocks_workspace_bytes(const dg4_graph* g, const dg4_desc* desc, int32_t n_blocks) {
    (void)desc;
    if (!g || n_blocks < 1 || n_blocks > DG4I_MAX_LAYERS) return 0;
    const size_t tables = (((size_t)g->n * 512 + 255) / 256) * 256 * (size_t)n_blocks;
    return tables + ((dg4i_levelised_sync_bytes(g, 2 * n_blocks) + 255) / 256) * 256;
}

/* Several blocks in level-by-level order as ONE wavefront: the attention stage and the feed-forward stage of every
 * block are pipeline stages of one persistent kernel; block k+1 takes a level as soon as block k has finished it. */
extern "C" dg4_status dg4_blocks_fwd_levelised(const dg4_graph* g, const dg4_desc* desc, void* H, int64_t ldh,
                                                int32_t n_blocks, const void* const* W_qkv, const void* const* W_o,
                                                const float* const* ln1_gamma, const float* const* ln1_beta,
                                                const void* const* W1, const float* const* b1, const void* const* W2,
                                                const float* const* b2, const float* const* ln2_gamma,
                                                const float* const* ln2_beta, float eps, int32_t d_ff, void* workspace,
                                                size_t workspace_bytes, void* stream) {
    CHECK(check_common(g, desc, eps));
    CHECK(dg4i_check_desc(desc, true));
    CHECK(check_rows("H", H, ldh));
    if (n_blocks < 1 || n_blocks > DG4I_MAX_LAYERS)
        DG4_FAIL(DG4_ERR_UNSUPPORTED, "n_blocks = %d: between 1 and %d blocks per call", n_blocks, DG4I_MAX_LAYERS);
    if (!W_qkv || !W_o || !ln1_gamma || !ln1_beta || !W1 || !b1 || !W2 || !b2 || !ln2_gamma || !ln2_beta)
        DG4_FAIL(DG4_ERR_INVALID_ARG, "null parameter array");
    dg4i_block_tail tails[DG4I_MAX_LAYERS];
    const __nv_bfloat16* wq[DG4I_MAX_LAYERS];
    const __nv_bfloat16* wo[DG4I_MAX_LAYERS];
    __nv_bfloat16* kv[DG4I_MAX_LAYERS];
    if (!workspace) DG4_FAIL(DG4_ERR_INVALID_ARG, "workspace is null");
    if ((((uintptr_t)workspace) & 255u) != 0) DG4_FAIL(DG4_ERR_INVALID_ARG, "workspace is not 256-byte aligned");
    if (workspace_bytes < dg4_blocks_workspace_bytes(g, desc, n_blocks))
        DG4_FAIL(DG4_ERR_INVALID_ARG, "workspace of %zu bytes is below the %zu bytes needed", workspace_bytes,
                 dg4_blocks_workspace_bytes(g, desc, n_blocks));
    const size_t table = (((size_t)g->n * 512 + 255) / 256) * 256;
    for (int k = 0; k < n_blocks; ++k) {
        if (!W_qkv[k] || !W_o[k] || !aligned16(W_qkv[k]) || !aligned16(W_o[k]))
            DG4_FAIL(DG4_ERR_INVALID_ARG, "W_qkv / W_o of block %d null or misaligned", k);
        CHECK(check_vec("ln1_gamma", ln1_gamma[k]));
        CHECK(check_vec("ln1_beta", ln1_beta[k]));
        CHECK(check_ffn_args(W1[k], b1[k], W2[k], b2[k], ln2_gamma[k], ln2_beta[k], d_ff));
        tails[k].ln1_gamma = ln1_gamma[k]; tails[k].ln1_beta = ln1_beta[k];
        tails[k].W1 = (const __nv_bfloat16*)W1[k]; tails[k].b1 = b1[k];
        tails[k].W2 = (const __nv_bfloat16*)W2[k]; tails[k].b2 = b2[k];
        tails[k].ln2_gamma = ln2_gamma[k]; tails[k].ln2_beta = ln2_beta[k]; tails[k].eps = eps;
        wq[k] = (const __nv_bfloat16*)W_qkv[k]; wo[k] = (const __nv_bfloat16*)W_o[k];
        kv[k] = (__nv_bfloat16*)((char*)workspace + table * (size_t)k);
    }
    int32_t* sync = (int32_t*)((char*)workspace + table * (size_t)n_blocks);
    return dg4i_levelised_launch(g, desc, n_blocks, kv, (__nv_bfloat16*)H, ldh, wq, wo, sync, g->dev_status,
                                 (cudaStream_t)stream, tails);
}

extern "C" dg4_status dg4_block_fwd_parallel(const dg4_graph* g, const dg4_desc* desc, const void* H_in, int64_t ldh,
                                              const void* W_qkv, const void* W_o, const float* ln1_gamma,
                                              const float* ln1_beta, const void* W1, const float* b1, const void* W2,
                                              const float* b2, const float* ln2_gamma, const float* ln2_beta, float eps,
                                              int32_t d_ff, void* H_out, int64_t ldho, void* workspace,
                                              size_t workspace_bytes, void* stream) {
    CHECK(check_common(g, desc, eps));
    if (!workspace) DG4_FAIL(DG4_ERR_INVALID_ARG, "workspace is null");
    if ((((uintptr_t)workspace) & 255u) != 0) DG4_FAIL(DG4_ERR_INVALID_ARG, "workspace is not 256-byte aligned");
    if (workspace_bytes < dg4_layer_workspace_bytes(g, desc))
        DG4_FAIL(DG4_ERR_INVALID_ARG, "workspace of %zu bytes is below the %zu bytes needed", workspace_bytes,
                 dg4_layer_workspace_bytes(g, desc));
    if (d_ff != 512) DG4_FAIL(DG4_ERR_UNSUPPORTED, "d_ff = %d: only d_ff = 4 d = 512 is supported", d_ff);
    // workspace rows: Q [n,128] | K|V [n,256] | O [n,128]; the Q table is free once the attention has run and
    // then holds the attention sub-layer's output
    __nv_bfloat16* Q = (__nv_bfloat16*)workspace;
    __nv_bfloat16* KV = Q + (size_t)g->n * 128;
    __nv_bfloat16* O = Q + (size_t)g->n * 384;
    __nv_bfloat16* H1 = Q;
    dg4_desc with_res = *desc;
    with_res.flags |= DG4_FLAG_RESIDUAL;     // the block always has its residual connections
    CHECK(dg4_qkv_project(g, desc, H_in, ldh, W_qkv, Q, 128, KV, 256, KV + 128, 256, stream));
    CHECK(dg4_sparse_attn_fwd(g, desc, Q, 128, KV, 256, KV + 128, 256, O, 128, stream));
    CHECK(dg4_out_project(g, &with_res, O, 128, W_o, H_in, ldh, H1, 128, stream));
    CHECK(dg4_layernorm_fwd(g, desc, H1, 128, ln1_gamma, ln1_beta, eps, H1, 128, stream));
    return dg4_ffn_fwd(g, desc, H1, 128, W1, b1, W2, b2, ln2_gamma, ln2_beta, eps, d_ff, H_out, ldho, stream);
}
