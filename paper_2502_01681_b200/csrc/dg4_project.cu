// Dense projections of the layer on the 5th-generation tensor cores: Y = A * W^T with K = 128, bf16 operands,
// fp32 accumulation in tensor memory, one rounding to bf16 per stored element.  Used for
// [Q|K|V] = X * W_qkv^T, H' = O * W_o^T (+ residual) and, in the per-level driver, for refreshing the K|V rows
// of a finished level.
//
// One persistent CTA per SM, ten warps:
//   warp 0  producer: brings the weight matrix into shared memory once (TMA), then streams 128-row tiles of A
//           (and of the residual, if any) through a 2-stage ring -- by TMA when the rows are contiguous, by
//           16-byte gathers written in the same 128-byte-swizzled layout when the rows come from a list;
//   warp 1  owns the tensor memory allocation and issues tcgen05.mma (one lane): for every tile and every
//           128-column block of the output, 8 MMAs of 128x128x16 into one of four 128-column accumulator slots;
//   warps 2-9  epilogue: each warp owns 32 rows x 64 columns of a block: tcgen05.ld, residual add, rounding to
//           bf16, and a 128-byte-swizzled staging tile in shared memory.  Contiguous rows leave by TMA store
//           (two 64-column boxes per block, double-buffered staging, ragged last tile clipped by the tensor
//           map); listed rows leave by 16-byte stores, four rows per warp instruction.
// The stages are coupled only by mbarriers, so loads, MMAs and stores of neighbouring tiles overlap.  The work is
// bound by HBM traffic (96 flop per byte for QKV, below the machine's ridge), which is why nothing here tries to
// raise tensor-pipe occupancy beyond what hides the memory time.
//
// Every mbarrier wait is bounded; on expiry the kernel records DG4_ERR_TIMEOUT in the status word and raises an
// abort flag in shared memory.  Leaving is arranged so that no warp can be left waiting for another one: a wait's
// result is made uniform across the warp before anything branches on it; the eight epilogue warps, which meet at
// a named barrier once per item when they store by TMA, take the decision to leave together (one thread samples
// the flag before that barrier, all read the sample after it); the producer then waits for the tensor copies it
// has started, the MMA thread for the MMAs it has issued, the storing thread for its stores, and only then is
// tensor memory freed.

#include "dg4_internal.h"
#include "dg4_sm100.cuh"

#include <mutex>

namespace {

using namespace sm100;

constexpr int kEpiWarps = 8;
constexpr int kThreads = 32 * (2 + kEpiWarps);
constexpr int kTileM = 128;
constexpr int kHalfBytes = 128 * 128;             // a 128-row x 64-column bf16 box: 128 rows x 128 bytes
constexpr int kTileBytes = 2 * kHalfBytes;        // 32 KiB
constexpr int kStages = 2;
constexpr int kSlots = 4;                         // accumulator slots of 128 columns
constexpr int kTmemCols = 512;

// shared memory map (offsets from a 1024-byte aligned base)
constexpr int kOffW = 0;                                  // 3 blocks x 32 KiB; with one block, the other two hold
constexpr int kOffR = kTileBytes;                         //   the residual ring (2 x 32 KiB)
constexpr int kOffA = 3 * kTileBytes;                     // 2 stages x 32 KiB
constexpr int kOffStage = kOffA + kStages * kTileBytes;   // 2 x 32 KiB output staging
constexpr int kOffBar = kOffStage + 2 * kTileBytes;
constexpr int kSmemBytes = kOffBar + 256 + 1024;          // barriers + slack for manual alignment

struct Bars {
    uint64_t w_full;
    uint64_t a_full[kStages];
    uint64_t a_empty[kStages];
    uint64_t r_empty[kStages];
    uint64_t acc_full[kSlots];
    uint64_t acc_empty[kSlots];
    uint64_t drain;            // error path only: completion of the MMAs still in flight
    uint32_t tmem_base;
    uint32_t abort_flag;
    uint32_t epi_stop[2];      // the epilogue warps' common decision to leave, per item parity
};

struct ProjParams {
    dg4i_proj_args a;
    int32_t n_blocks;         // n_out / 128
    int32_t n_tiles;
    int32_t* status;          // device status word (nullable)
    uint32_t poll_limit;      // polls after which a pipeline wait gives up
};

__device__ __forceinline__ void ld_nc_v4(const void* p, uint32_t* r) {
    asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "l"(p));
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, const uint32_t* r) {
    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]) : "memory");
}
__device__ __forceinline__ void ld_shared_v4(uint32_t addr, uint32_t* r) {
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}
__device__ __forceinline__ void st_global_v4(void* p, const uint32_t* r) {
    asm volatile("st.global.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]) : "memory");
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ void epi_barrier() { asm volatile("bar.sync 1, %0;" ::"n"(kEpiWarps * 32) : "memory"); }

__device__ __forceinline__ void raise_timeout(Bars* bars, int32_t* status) {
    atomicExch(&bars->abort_flag, 1u);
    if (status) atomicCAS(status, 0, (int)DG4_ERR_TIMEOUT);
}

struct OutMaps { CUtensorMap m[3]; };

template <bool LISTED>
__global__ void __launch_bounds__(kThreads, 1)
proj_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_w,
               const __grid_constant__ CUtensorMap map_r, const __grid_constant__ OutMaps map_o, ProjParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
    Bars* bars = reinterpret_cast<Bars*>(base_ptr + kOffBar);
    const uint32_t sW = base + kOffW, sR = base + kOffR, sA = base + kOffA, sStage = base + kOffStage;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nb = p.n_blocks;
    const bool has_res = p.a.R != nullptr;             // only with a single output block (checked by the host)
    volatile uint32_t* abort_flag = &bars->abort_flag;

    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bars->w_full), 1);
        for (int s = 0; s < kStages; ++s) {
            mbar_init(smem_u32(&bars->a_full[s]), 1);
            mbar_init(smem_u32(&bars->a_empty[s]), 1);
            mbar_init(smem_u32(&bars->r_empty[s]), kEpiWarps);
        }
        for (int s = 0; s < kSlots; ++s) { mbar_init(smem_u32(&bars->acc_full[s]), 1); mbar_init(smem_u32(&bars->acc_empty[s]), kEpiWarps); }
        mbar_init(smem_u32(&bars->drain), 1);
        bars->abort_flag = 0;
        bars->epi_stop[0] = bars->epi_stop[1] = 0;
        mbar_fence_init();
        tma_prefetch_desc(&map_w);
        if (!LISTED) {
            tma_prefetch_desc(&map_a);
            if (has_res) tma_prefetch_desc(&map_r);
            for (int j = 0; j < nb; ++j) tma_prefetch_desc(&map_o.m[j]);
        }
    }
    if (warp == 1) tmem_alloc(smem_u32(&bars->tmem_base), kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = bars->tmem_base;

    const int my_tiles = (p.n_tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;

    if (warp == 0) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            mbar_expect_tx(smem_u32(&bars->w_full), (uint32_t)(nb * kTileBytes));
            for (int j = 0; j < nb; ++j)
                for (int h = 0; h < 2; ++h)
                    tma_load_2d(sW + (j * 2 + h) * kHalfBytes, &map_w, h * 64, j * 128, smem_u32(&bars->w_full));
        }
        int armed = 0;
        for (int i = 0; i < my_tiles; ++i) {
            if (__any_sync(0xffffffffu, *abort_flag != 0)) break;
            const int tile = blockIdx.x + i * gridDim.x;
            const int s = i % kStages;
            const uint32_t ph = (uint32_t)(i / kStages) & 1u;
            if (!mbar_wait_warp(smem_u32(&bars->a_empty[s]), ph ^ 1u, p.poll_limit)) { raise_timeout(bars, p.status); break; }
            const uint32_t dst = sA + s * kTileBytes;
            if (!LISTED) {
                if (has_res && !mbar_wait_warp(smem_u32(&bars->r_empty[s]), ph ^ 1u, p.poll_limit)) { raise_timeout(bars, p.status); break; }
                if (lane == 0) {
                    const uint32_t bar = smem_u32(&bars->a_full[s]);
                    mbar_expect_tx(bar, (uint32_t)(has_res ? 2 * kTileBytes : kTileBytes));
                    tma_load_2d(dst, &map_a, 0, tile * kTileM, bar);
                    tma_load_2d(dst + kHalfBytes, &map_a, 64, tile * kTileM, bar);
                    if (has_res) {
                        tma_load_2d(sR + s * kTileBytes, &map_r, 0, tile * kTileM, bar);
                        tma_load_2d(sR + s * kTileBytes + kHalfBytes, &map_r, 64, tile * kTileM, bar);
                    }
                }
                armed = i + 1;
            } else {
                // two rows per warp instruction: lanes 0-15 one row, lanes 16-31 the next; 16 bytes per lane
                const int chunk = lane & 15, half = chunk >> 3, c8 = chunk & 7;
#pragma unroll 4
                for (int it = 0; it < 64; ++it) {
                    const int row = it * 2 + (lane >> 4);
                    const int r = tile * kTileM + row;
                    uint32_t v[4] = {0u, 0u, 0u, 0u};
                    if (r < p.a.rows) {
                        const int64_t rid = p.a.row_list[p.a.first + r];
                        ld_nc_v4(p.a.A + rid * p.a.lda + chunk * 8, v);
                    }
                    st_shared_v4(dst + half * kHalfBytes + sw128_offset(row, c8), v);
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bars->a_full[s]));
            }
        }
        // do not leave with tensor copies still landing in shared memory: normally the MMAs have consumed them all
        // long before; after an abort they may not have (these waits keep the default limit: a copy that was
        // started does land)
        if (lane == 0) {
            mbar_wait(smem_u32(&bars->w_full), 0);
            if (!LISTED)
                for (int i = (armed > kStages ? armed - kStages : 0); i < armed; ++i)
                    mbar_wait(smem_u32(&bars->a_full[i % kStages]), (uint32_t)(i / kStages) & 1u);
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc = idesc_bf16_f32(128, 128);
            bool ok = mbar_wait(smem_u32(&bars->w_full), 0, p.poll_limit);
            if (!ok) raise_timeout(bars, p.status);
            int item = 0;
            for (int i = 0; i < my_tiles && ok && !*abort_flag; ++i) {
                const int s = i % kStages;
                if (!mbar_wait(smem_u32(&bars->a_full[s]), (uint32_t)(i / kStages) & 1u, p.poll_limit)) { raise_timeout(bars, p.status); break; }
                tc_fence_after();
                const uint32_t a_base = sA + s * kTileBytes;
                for (int j = 0; j < nb; ++j, ++item) {
                    const int slot = item % kSlots;
                    if (!mbar_wait(smem_u32(&bars->acc_empty[slot]), ((uint32_t)(item / kSlots) & 1u) ^ 1u, p.poll_limit)) {
                        raise_timeout(bars, p.status); ok = false; break;
                    }
                    tc_fence_after();
                    const uint32_t d = tmem + (uint32_t)(slot * 128);
                    const uint32_t b_base = sW + j * kTileBytes;
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        const uint32_t off = (uint32_t)((ks >> 2) * kHalfBytes + (ks & 3) * 32);
                        mma_bf16(d, smem_desc_sw128(a_base + off), smem_desc_sw128(b_base + off), idesc, ks > 0 ? 1u : 0u);
                    }
                    mma_commit(smem_u32(&bars->acc_full[slot]));
                }
                mma_commit(smem_u32(&bars->a_empty[s]));   // the stage is free once these MMAs have read it
            }
            // tensor memory is freed below, so every MMA issued above must have completed (normally the epilogue
            // has waited for each of them; after an abort it may have left first)
            mma_commit(smem_u32(&bars->drain));
            mbar_wait(smem_u32(&bars->drain), 0);
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..9)
        const int ew = warp - 2;
        const int quad = warp & 3;                       // TMEM lane quadrant this warp may read
        const int half = ew >> 2;                        // which 64-column box of a block this warp produces
        const int my_row = quad * 32 + lane;             // row of the tile held by this thread
        const bool issuer = (ew == 0 && lane == 0);      // the one thread that issues (and waits for) TMA stores
        int item = 0;
        bool ok = true;          // no wait of this warp has run out (the same for all its lanes)
        bool stop = false;
        for (int i = 0; i < my_tiles && !stop; ++i) {
            // listed rows: the warps of the epilogue never wait for one another, so each may leave on its own
            if (LISTED && __any_sync(0xffffffffu, *abort_flag != 0)) break;
            const int tile = blockIdx.x + i * gridDim.x;
            const int s = i % kStages;
            const int r_own = tile * kTileM + my_row;
            int64_t rid_own = -1;
            if (r_own < p.a.rows) rid_own = LISTED ? (int64_t)p.a.row_list[p.a.first + r_own] : (int64_t)p.a.first + r_own;
            for (int j = 0; j < nb; ++j, ++item) {
                const int slot = item % kSlots;
                const uint32_t stage = sStage + (uint32_t)((item & 1) * kTileBytes + half * kHalfBytes);
                if (ok && !mbar_wait_warp(smem_u32(&bars->acc_full[slot]), (uint32_t)(item / kSlots) & 1u, p.poll_limit)) {
                    raise_timeout(bars, p.status);
                    ok = false;
                }
                if (LISTED && !ok) { stop = true; break; }
                const bool add_res = (j == 0) && has_res;
                if (ok) {
                    tc_fence_after();
                    const uint32_t t_addr = tmem + ((uint32_t)(quad * 32) << 16) + (uint32_t)(slot * 128 + half * 64);
#pragma unroll 1
                    for (int q = 0; q < 2; ++q) {
                        uint32_t acc[32];
                        tmem_ld_32x32(t_addr + (uint32_t)(q * 32), acc);
                        uint32_t res[16];
                        if (add_res) {
                            if (!LISTED) {                   // residual tile sits in shared memory in box layout
#pragma unroll
                                for (int c = 0; c < 4; ++c)
                                    ld_shared_v4(sR + (uint32_t)(s * kTileBytes + half * kHalfBytes) + sw128_offset(my_row, q * 4 + c), res + 4 * c);
                            } else if (rid_own >= 0) {
#pragma unroll
                                for (int c = 0; c < 4; ++c) ld_nc_v4(p.a.R + rid_own * p.a.ldr + half * 64 + q * 32 + c * 8, res + 4 * c);
                            } else {
#pragma unroll
                                for (int c = 0; c < 16; ++c) res[c] = 0u;
                            }
                        }
                        tmem_ld_wait();
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            uint32_t out[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                float lo = __uint_as_float(acc[c * 8 + 2 * e]), hi = __uint_as_float(acc[c * 8 + 2 * e + 1]);
                                if (add_res) {
                                    lo += __uint_as_float(res[4 * c + e] << 16);
                                    hi += __uint_as_float(res[4 * c + e] & 0xffff0000u);
                                }
                                out[e] = pack_bf16(lo, hi);
                            }
                            st_shared_v4(stage + sw128_offset(my_row, q * 4 + c), out);
                        }
                    }
                    // all tensor-memory (and residual) reads of this item are done: hand the buffers back
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) {
                        mbar_arrive(smem_u32(&bars->acc_empty[slot]));
                        if (add_res && !LISTED) mbar_arrive(smem_u32(&bars->r_empty[s]));
                    }
                }
                if (!LISTED) {
                    // staging -> global by TMA.  The issuer first makes sure the previous item's store has finished
                    // reading ITS staging buffer (the one the next item will overwrite) and samples the abort flag;
                    // then everybody meets, and everybody acts on that one sample: the eight warps go on to the
                    // next item together or leave together.  (A warp whose own wait ran out keeps coming to this
                    // barrier, without touching tensor memory, until the common decision says leave: at the
                    // latest at the next item, because its flag was raised before it arrived here.)
                    fence_proxy_async_smem();
                    if (issuer) {
                        bulk_wait_read0();
                        bars->epi_stop[item & 1] = *abort_flag;
                    }
                    epi_barrier();
                    stop = reinterpret_cast<volatile uint32_t*>(bars->epi_stop)[item & 1] != 0;
                    if (stop) break;
                    if (issuer) {
                        const uint32_t src = sStage + (uint32_t)((item & 1) * kTileBytes);
                        tma_store_2d(&map_o.m[j], 0, tile * kTileM, src);
                        tma_store_2d(&map_o.m[j], 64, tile * kTileM, src + kHalfBytes);
                        bulk_commit();
                    }
                } else {
                    // 8 lanes cover the 128 bytes this warp produced of a row: four rows per instruction
                    __nv_bfloat16* outp = p.a.out[j];
                    const int64_t ldo = p.a.ldo[j];
                    const int c8 = lane & 7;
#pragma unroll 4
                    for (int it = 0; it < 8; ++it) {
                        const int lr = it * 4 + (lane >> 3);
                        const int64_t rid = __shfl_sync(0xffffffffu, (long long)rid_own, lr);
                        uint32_t v[4];
                        ld_shared_v4(stage + sw128_offset(quad * 32 + lr, c8), v);
                        if (rid >= 0) st_global_v4(outp + rid * ldo + half * 64 + c8 * 8, v);
                    }
                    __syncwarp();
                    // the staging rows of this warp are rewritten two items later by this warp only
                }
            }
        }
        if (!LISTED && issuer) bulk_wait_all();
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem, kTmemCols);
    }
}

// ---------------------------------------------------------------------------------------------------
// host side: tensor maps and launch
// ---------------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

std::mutex g_mu;
EncodeTiledFn g_encode = nullptr;
bool g_attr_set[64] = {};
int g_sm_count[64] = {};

dg4_status get_encoder(EncodeTiledFn* fn) {
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_encode) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q);
        if (e != cudaSuccess || q != cudaDriverEntryPointSuccess || !p) {
            cudaGetLastError();
            DG4_FAIL(DG4_ERR_CUDA, "cuTensorMapEncodeTiled is not available from this driver");
        }
        g_encode = (EncodeTiledFn)p;
    }
    *fn = g_encode;
    return DG4_OK;
}

// [rows, 128] bf16 row-major with leading dimension ld; box = 64 columns x box_rows rows, 128-byte swizzle.
dg4_status make_map(CUtensorMap* m, const void* base, int64_t rows, int64_t ld, int box_rows = 128) {
    EncodeTiledFn enc;
    dg4_status s = get_encoder(&enc);
    if (s != DG4_OK) return s;
    cuuint64_t dims[2] = {128, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)(ld * 2)};
    cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) DG4_FAIL(DG4_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);
    return DG4_OK;
}

}  // namespace

dg4_status dg4i_make_row_map(CUtensorMap_st* map, const void* base, int64_t rows, int64_t ld, int box_rows) {
    return make_map(map, base, rows, ld, box_rows);
}

dg4_status dg4i_proj_launch(const dg4i_proj_args& a, cudaStream_t st) {
    if (a.rows <= 0) return DG4_OK;
    if (a.n_out != 128 && a.n_out != 256 && a.n_out != 384)
        DG4_FAIL(DG4_ERR_UNSUPPORTED, "projection width %d is not supported", a.n_out);
    if (a.R && a.n_out != 128) DG4_FAIL(DG4_ERR_UNSUPPORTED, "a residual needs a 128-column projection");
    int dev = 0;
    DG4_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) DG4_FAIL(DG4_ERR_UNSUPPORTED, "device ordinal %d is out of range", dev);
    {
        std::lock_guard<std::mutex> lock(g_mu);
        if (!g_attr_set[dev]) {
            DG4_CUDA_TRY(cudaFuncSetAttribute(proj_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
            DG4_CUDA_TRY(cudaFuncSetAttribute(proj_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
            DG4_CUDA_TRY(cudaDeviceGetAttribute(&g_sm_count[dev], cudaDevAttrMultiProcessorCount, dev));
            g_attr_set[dev] = true;
        }
    }
    ProjParams p;
    p.a = a;
    p.n_blocks = a.n_out / 128;
    p.n_tiles = (a.rows + kTileM - 1) / kTileM;
    p.status = a.status;
    p.poll_limit = dg4i_poll_limit();
    CUtensorMap map_a, map_w, map_r;
    OutMaps map_o;
    dg4_status s = make_map(&map_w, a.W, a.n_out, 128);
    if (s != DG4_OK) return s;
    map_a = map_r = map_w;                       // placeholders for the maps a mode does not use
    for (int j = 0; j < 3; ++j) map_o.m[j] = map_w;
    const int grid = p.n_tiles < g_sm_count[dev] ? p.n_tiles : g_sm_count[dev];
    if (!a.row_list) {
        // contiguous rows: every map starts at the first row, so tile coordinates start at 0
        if ((s = make_map(&map_a, a.A + (int64_t)a.first * a.lda, a.rows, a.lda)) != DG4_OK) return s;
        if (a.R && (s = make_map(&map_r, a.R + (int64_t)a.first * a.ldr, a.rows, a.ldr)) != DG4_OK) return s;
        for (int j = 0; j < p.n_blocks; ++j)
            if ((s = make_map(&map_o.m[j], a.out[j] + (int64_t)a.first * a.ldo[j], a.rows, a.ldo[j])) != DG4_OK) return s;
        proj_tc_kernel<false><<<grid, kThreads, kSmemBytes, st>>>(map_a, map_w, map_r, map_o, p);
    } else {
        proj_tc_kernel<true><<<grid, kThreads, kSmemBytes, st>>>(map_a, map_w, map_r, map_o, p);
    }
    dg4i_count_launch();
    DG4_CUDA_TRY(cudaGetLastError());
    return DG4_OK;
}
