// The all-nodes-parallel layer behind its K | V projection as ONE kernel (Sec. 3.5: Q = X W_q^T, sparse attention
// over the neighbourhood, H' = O W_o^T + X): per 128-node tile the query rows are projected on the tensor cores
// from the X tile, the attention is gathered and computed exactly as in the stand-alone attention kernel, and
// its output tile goes straight into the output projection.  Neither Q nor O ever exists in global memory: of
// the layer's traffic that removes the Q write + read and the O write + read (1 KiB of 3.4 KiB per node).
// K | V of ALL nodes must exist before any node attends, so that projection stays a kernel of its own in front.
// Results are bit for bit those of the three-kernel path (same products, same roundings, same order of sums).
//
// OPT-IN (DG4_FLAG_FUSED_LAYER): measured on the 10M-node circuit the layer takes 5.9 ms this way against 5.95 ms
// as three kernels -- the traffic saved is paid back twice.  (1) A gathered row waits in L1 between request and
// arrival, so the gather needs most of the SM's 256 KiB as L1 to keep enough requests in flight: the stand-alone
// attention kernel slows from 3.1 to 3.6 and 5.9 ms when 168 and 216 KiB are taken away as shared memory, and
// this kernel's tiles and weights take 224 KiB.  (2) The gather is also bound by issue slots (65 % busy on its
// own), and the epilogues share them.  A variant with the weights in tensor memory, transposed products and
// 64-node tiles (112 KiB of shared memory) cured (1) but not (2): its epilogues scatter two-byte elements and
// execute half as many instructions again as the gather itself (6.1 ms).
//
// One persistent CTA per SM; tile s of a CTA is tile blockIdx.x + s * gridDim.x of the node range, so the
// tiles in flight across the GPU cover a contiguous id range and the gathered rows overlap in L2.  Warps:
//   warp 0      producer: W_q and W_o once, then the X tiles through a 2-stage ring (TMA, 128-byte swizzle);
//   warp 1      issues tcgen05.mma (one lane): Q(s) = X(s) W_q^T, a tile ahead of the gather; H(s) = O(s) W_o^T
//               once the gather of tile s is complete;
//   warps 4-7   epilogues (thread = node row): Q(s) out of tensor memory, rounded to bf16, into buffer s % 3 in
//               the tensor core's operand layout, while the tile's input rows move from the X stage into
//               tensor memory (64 columns of packed bf16) for the residual; later H(s) out of tensor memory,
//               + those rows, rounded, into the same buffer, which then leaves by TMA store;
//   warps 8-27  gather and attend, 16 lanes per node, two nodes per warp at a time: a lane reads its 16-byte
//               piece of the node's Q row from buffer s % 3, gathers the neighbours' K and V pieces, and writes
//               its piece of O back INTO THE SAME PLACE, which is where the output projection's A operand is read.
//               Node pairs are dealt round-robin across tile boundaries, so no warp idles at the end of a tile.
// Three buffers rotate: while the gather warps work on tile s, buffer (s+1) % 3 receives Q(s+1) and buffer
// (s-1) % 3 carries O(s-1) -> H(s-1) -> store.  The roles are coupled by mbarriers only; the roles that wait long
// wait suspended (try_wait with a time hint) so that they leave the issue slots to the gather warps.  Twenty
// gather warps keep nearly as many loads in flight as the stand-alone kernel's 24 (measured there: 3.15 vs
// 3.09 ms at 20 vs 24 warps per SM, 3.52 ms at 16); the register file allows them because the producer and
// issuer warps give registers back (setmaxnreg).
//
// Every wait is bounded; on expiry the kernel records DG4_ERR_TIMEOUT, raises an abort flag that every loop
// reads, each role waits for the asynchronous work it started itself, and tensor memory is freed last.

#include "dg4_internal.h"
#include "dg4_attn_core.cuh"
#include "dg4_sm100.cuh"

#include <cuda.h>
#include <mutex>

namespace {

using namespace sm100;
using namespace attn;

constexpr int kGatherWarps = 20;
constexpr int kFirstEpiWarp = 4, kFirstGatherWarp = 8;
constexpr int kThreads = 32 * (kFirstGatherWarp + kGatherWarps);     // 896
constexpr int kTileM = 128;
constexpr int kPairs = kTileM / 2;                // node pairs (one warp's unit of work) per tile
constexpr int kHalfBytes = 128 * 128;             // a 128-row x 64-column bf16 box
constexpr int kTileBytes = 2 * kHalfBytes;        // 32 KiB
constexpr int kXStages = 2, kBufs = 3;
constexpr int kTmemCols = 512;
constexpr int kColQ = 0, kColH = 128, kColStash = 256;   // accQ | accH (128 columns each) | 3 x 64 columns of input rows
constexpr int kRegsIdle = 56, kRegsEpi = 88;      // 128*56 + 128*88 + 640*72 = 64512 = 896 threads * 72 at launch

constexpr int kOffWq = 0;
constexpr int kOffWo = kTileBytes;
constexpr int kOffX = 2 * kTileBytes;
constexpr int kOffQO = kOffX + kXStages * kTileBytes;
constexpr int kOffBar = kOffQO + kBufs * kTileBytes;
constexpr int kSmemBytes = kOffBar + 256 + 1024;  // barriers + slack for manual alignment
static_assert(kSmemBytes <= 232448, "shared memory budget of one CTA");

struct Bars {
    uint64_t w_full;
    uint64_t x_full[kXStages], x_empty[kXStages];
    uint64_t accq_full, accq_empty;
    uint64_t acch_full, acch_empty;
    uint64_t q_full[kBufs];        // Q(s) is in buffer s % 3
    uint64_t o_full[kBufs];        // all 64 node pairs of tile s have written their O pieces
    uint64_t drain;
    uint32_t tmem_base;
    uint32_t abort_flag;
    uint32_t epi_stop[2];
};
static_assert(sizeof(Bars) <= 256, "barrier block");

struct FusedParams {
    const __nv_bfloat16* X;        // [n, ldx] layer input (queries are projected from it; residual)
    int64_t ldx;
    const __nv_bfloat16* KV;       // [n, 256] K | V of every node
    const int32_t* nbr_pad;        // [n, MAXN + 1]
    int32_t n;
    int32_t n_tiles;
    int32_t residual;
    float scale;
    int32_t* status;
    uint32_t poll_limit;
};

__device__ __forceinline__ void st_shared_v4(uint32_t addr, const uint32_t* r) {
    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]) : "memory");
}
__device__ __forceinline__ void ld_shared_v4(uint32_t addr, uint32_t* r) {
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ void epi_barrier() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
template <int N> __device__ __forceinline__ void regs_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N> __device__ __forceinline__ void regs_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }

__device__ __forceinline__ void raise_timeout(Bars* bars, int32_t* status) {
    atomicExch(&bars->abort_flag, 1u);
    if (status) atomicCAS(status, 0, (int)DG4_ERR_TIMEOUT);
}

// byte offset of the 16-byte piece `piece` (0..15) of row `row` in a 128-row operand tile (two 64-column boxes)
__device__ __forceinline__ uint32_t tile_piece(int row, int piece) {
    return (uint32_t)((piece >> 3) * kHalfBytes) + sw128_offset(row, piece & 7);
}

template <int LPH, int MAXN>
__global__ void __launch_bounds__(kThreads, 1)
fused_layer_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_wq,
                   const __grid_constant__ CUtensorMap map_wo, const __grid_constant__ CUtensorMap map_out, FusedParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
    Bars* bars = reinterpret_cast<Bars*>(base_ptr + kOffBar);
    const uint32_t sWq = base + kOffWq, sWo = base + kOffWo, sX = base + kOffX, sQO = base + kOffQO;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile uint32_t* abort_flag = &bars->abort_flag;

    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bars->w_full), 1);
        // an X stage is free once the Q product has read it (1 arrival) and the epilogue warps have copied the
        // rows for the residual (4)
        for (int s = 0; s < kXStages; ++s) { mbar_init(smem_u32(&bars->x_full[s]), 1); mbar_init(smem_u32(&bars->x_empty[s]), 5); }
        mbar_init(smem_u32(&bars->accq_full), 1); mbar_init(smem_u32(&bars->accq_empty), 4);
        mbar_init(smem_u32(&bars->acch_full), 1); mbar_init(smem_u32(&bars->acch_empty), 4);
        for (int s = 0; s < kBufs; ++s) { mbar_init(smem_u32(&bars->q_full[s]), 4); mbar_init(smem_u32(&bars->o_full[s]), kPairs); }
        mbar_init(smem_u32(&bars->drain), 1);
        bars->abort_flag = 0;
        bars->epi_stop[0] = bars->epi_stop[1] = 0;
        mbar_fence_init();
        tma_prefetch_desc(&map_x);
        tma_prefetch_desc(&map_wq);
        tma_prefetch_desc(&map_wo);
        tma_prefetch_desc(&map_out);
    }
    if (warp == 1) tmem_alloc(smem_u32(&bars->tmem_base), kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = bars->tmem_base;
    const int my_tiles = (p.n_tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;

    if (warp < kFirstEpiWarp) {
        regs_dec<kRegsIdle>();
        if (warp == 0) {
            // ---------------------------------------------------------------- producer
            int armed = 0;
            if (lane == 0) {
                mbar_expect_tx(smem_u32(&bars->w_full), (uint32_t)(2 * kTileBytes));
                for (int h = 0; h < 2; ++h) {
                    tma_load_2d(sWq + h * kHalfBytes, &map_wq, h * 64, 0, smem_u32(&bars->w_full));
                    tma_load_2d(sWo + h * kHalfBytes, &map_wo, h * 64, 0, smem_u32(&bars->w_full));
                }
                for (int s = 0; s < my_tiles; ++s) {
                    if (*abort_flag) break;
                    const int st = s % kXStages;
                    if (!mbar_wait_relaxed(smem_u32(&bars->x_empty[st]), (((uint32_t)(s / kXStages)) & 1u) ^ 1u, p.poll_limit)) {
                        raise_timeout(bars, p.status);
                        break;
                    }
                    const int tile = blockIdx.x + s * gridDim.x;
                    const uint32_t bar = smem_u32(&bars->x_full[st]);
                    mbar_expect_tx(bar, (uint32_t)kTileBytes);
                    tma_load_2d(sX + st * kTileBytes, &map_x, 0, tile * kTileM, bar);
                    tma_load_2d(sX + st * kTileBytes + kHalfBytes, &map_x, 64, tile * kTileM, bar);
                    armed = s + 1;
                }
                // do not leave with tensor copies still landing in shared memory (a copy that was started does land)
                mbar_wait(smem_u32(&bars->w_full), 0);
                for (int s = (armed > kXStages ? armed - kXStages : 0); s < armed; ++s)
                    mbar_wait(smem_u32(&bars->x_full[s % kXStages]), ((uint32_t)(s / kXStages)) & 1u);
            }
        } else if (warp == 1) {
            // ---------------------------------------------------------------- MMA issuer
            // step s: Q(s+1) first -- it depends on nothing the gather warps do, so the query rows of a tile are
            // ready a whole tile ahead -- then H(s-1), which waits for the gather of tile s-1
            if (lane == 0) {
                const uint32_t idesc = idesc_bf16_f32(128, 128);
                bool ok = mbar_wait(smem_u32(&bars->w_full), 0, p.poll_limit);
                if (!ok) raise_timeout(bars, p.status);
                for (int s = -1; s <= my_tiles && ok && !*abort_flag; ++s) {
                    const int a = s + 1;
                    if (a < my_tiles) {                          // Q(a) = X(a) W_q^T
                        const int st = a % kXStages;
                        ok = mbar_wait_relaxed(smem_u32(&bars->x_full[st]), ((uint32_t)(a / kXStages)) & 1u, p.poll_limit) &&
                             mbar_wait_relaxed(smem_u32(&bars->accq_empty), ((uint32_t)a & 1u) ^ 1u, p.poll_limit);
                        if (!ok) { raise_timeout(bars, p.status); break; }
                        tc_fence_after();
                        const uint32_t a_base = sX + st * kTileBytes;
#pragma unroll
                        for (int ks = 0; ks < 8; ++ks) {
                            const uint32_t off = (uint32_t)((ks >> 2) * kHalfBytes + (ks & 3) * 32);
                            mma_bf16(tmem + kColQ, smem_desc_sw128(a_base + off), smem_desc_sw128(sWq + off), idesc, ks > 0 ? 1u : 0u);
                        }
                        mma_commit(smem_u32(&bars->accq_full));
                        mma_commit(smem_u32(&bars->x_empty[st]));
                    }
                    if (s >= 1) {                                // H(t) = O(t) W_o^T
                        const int t = s - 1, buf = t % kBufs;
                        ok = mbar_wait_relaxed(smem_u32(&bars->o_full[buf]), ((uint32_t)(t / kBufs)) & 1u, p.poll_limit) &&
                             mbar_wait_relaxed(smem_u32(&bars->acch_empty), ((uint32_t)t & 1u) ^ 1u, p.poll_limit);
                        if (!ok) { raise_timeout(bars, p.status); break; }
                        tc_fence_after();
                        const uint32_t a_base = sQO + buf * kTileBytes;
#pragma unroll
                        for (int ks = 0; ks < 8; ++ks) {
                            const uint32_t off = (uint32_t)((ks >> 2) * kHalfBytes + (ks & 3) * 32);
                            mma_bf16(tmem + kColH, smem_desc_sw128(a_base + off), smem_desc_sw128(sWo + off), idesc, ks > 0 ? 1u : 0u);
                        }
                        mma_commit(smem_u32(&bars->acch_full));
                    }
                }
                // tensor memory is freed below: every MMA issued above must have completed
                mma_commit(smem_u32(&bars->drain));
                mbar_wait(smem_u32(&bars->drain), 0);
            }
        }
    } else if (warp < kFirstGatherWarp) {
        // -------------------------------------------------------------------- epilogues (warps 4..7)
        regs_inc<kRegsEpi>();
        const int quad = warp & 3;
        const int my_row = quad * 32 + lane;
        const bool issuer = (warp == kFirstEpiWarp && lane == 0);
        const uint32_t t_lane = (uint32_t)(quad * 32) << 16;
        bool ok = true, stop = false;
        int step = 0;
        for (int s = -1; s <= my_tiles && !stop; ++s) {
            // ---- Q(a), a = s+1: tensor memory -> bf16 -> buffer a % 3 (free once the store of tile a-3 has read
            // it); the tile's input rows, which the residual needs two steps later, move from the X stage into
            // tensor memory meanwhile (the stage is handed back to the producer right away)
            const int a = s + 1;
            if (a < my_tiles) {
                if (issuer) {
                    bulk_wait_read0();
                    bars->epi_stop[step & 1] = *abort_flag;
                }
                epi_barrier();
                stop = reinterpret_cast<volatile uint32_t*>(bars->epi_stop)[step & 1] != 0;
                ++step;
                if (stop) break;
                const int buf = a % kBufs, st = a % kXStages;
                // (the X stage has landed long before the product that read it completes; waiting on its barrier as
                // well makes the copied bytes visible to this thread's own loads)
                if (ok && !(mbar_wait_relaxed_warp(smem_u32(&bars->accq_full), (uint32_t)a & 1u, p.poll_limit) &&
                            mbar_wait_relaxed_warp(smem_u32(&bars->x_full[st]), ((uint32_t)(a / kXStages)) & 1u, p.poll_limit))) {
                    raise_timeout(bars, p.status);
                    ok = false;
                }
                if (ok) {
                    tc_fence_after();
                    if (p.residual) {
                        const uint32_t src = sX + st * kTileBytes;
                        const uint32_t t_stash = tmem + t_lane + (uint32_t)(kColStash + (a % kBufs) * 64);
#pragma unroll
                        for (int c = 0; c < 8; ++c) {
                            uint32_t xr[8];
                            ld_shared_v4(src + tile_piece(my_row, 2 * c), xr);
                            ld_shared_v4(src + tile_piece(my_row, 2 * c + 1), xr + 4);
                            tmem_st_32x8(t_stash + (uint32_t)(c * 8), xr);
                        }
                    }
                    const uint32_t dst = sQO + buf * kTileBytes;
#pragma unroll 1
                    for (int q = 0; q < 4; ++q) {
                        uint32_t acc[32];
                        tmem_ld_32x32(tmem + t_lane + (uint32_t)(kColQ + q * 32), acc);
                        tmem_ld_wait();
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            uint32_t out[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e)
                                out[e] = pack_bf16(__uint_as_float(acc[c * 8 + 2 * e]), __uint_as_float(acc[c * 8 + 2 * e + 1]));
                            st_shared_v4(dst + tile_piece(my_row, q * 4 + c), out);
                        }
                    }
                    tmem_st_wait();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) {
                        mbar_arrive(smem_u32(&bars->accq_empty));
                        mbar_arrive(smem_u32(&bars->x_empty[st]));
                        mbar_arrive(smem_u32(&bars->q_full[buf]));
                    }
                }
            }
            // ---- H(t), t = s-1: tensor memory + residual -> bf16 -> buffer t % 3 -> TMA store
            if (s >= 1) {
                const int t = s - 1, buf = t % kBufs;
                const int tile = blockIdx.x + t * gridDim.x;
                if (ok && !mbar_wait_relaxed_warp(smem_u32(&bars->acch_full), (uint32_t)t & 1u, p.poll_limit)) {
                    raise_timeout(bars, p.status);
                    ok = false;
                }
                if (ok) {
                    tc_fence_after();
                    const uint32_t dst = sQO + buf * kTileBytes;
                    const uint32_t t_stash = tmem + t_lane + (uint32_t)(kColStash + (t % kBufs) * 64);
#pragma unroll 1
                    for (int q = 0; q < 4; ++q) {
                        uint32_t acc[32];
                        uint32_t res[16];
                        tmem_ld_32x32(tmem + t_lane + (uint32_t)(kColH + q * 32), acc);
                        if (p.residual) {
                            tmem_ld_32x8(t_stash + (uint32_t)(q * 16), res);
                            tmem_ld_32x8(t_stash + (uint32_t)(q * 16 + 8), res + 8);
                        } else {
#pragma unroll
                            for (int c = 0; c < 16; ++c) res[c] = 0u;
                        }
                        tmem_ld_wait();
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            uint32_t out[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const float lo = __uint_as_float(acc[c * 8 + 2 * e]) + __uint_as_float(res[4 * c + e] << 16);
                                const float hi = __uint_as_float(acc[c * 8 + 2 * e + 1]) + __uint_as_float(res[4 * c + e] & 0xffff0000u);
                                out[e] = pack_bf16(lo, hi);
                            }
                            st_shared_v4(dst + tile_piece(my_row, q * 4 + c), out);
                        }
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&bars->acch_empty));
                }
                fence_proxy_async_smem();
                if (issuer) bars->epi_stop[step & 1] = *abort_flag;
                epi_barrier();
                stop = reinterpret_cast<volatile uint32_t*>(bars->epi_stop)[step & 1] != 0;
                ++step;
                if (stop) break;
                if (issuer) {
                    const uint32_t src = sQO + buf * kTileBytes;
                    tma_store_2d(&map_out, 0, tile * kTileM, src);
                    tma_store_2d(&map_out, 64, tile * kTileM, src + kHalfBytes);
                    bulk_commit();
                }
            }
        }
        if (issuer) bulk_wait_all();
    } else {
        // -------------------------------------------------------------------- gather and attend (warps 8..27)
        constexpr int W = MAXN + 1;
        const int g = warp - kFirstGatherWarp;
        const int sub = lane & 15;
        const int grp_base = lane - sub;
        const unsigned mask = 0xffffu << grp_base;
        const int total = my_tiles * kPairs;
        const size_t col = (size_t)sub * 16;
        int s_ready = -1;
        auto node_of = [&](int P) -> int {
            const int tile = blockIdx.x + (P >> 6) * gridDim.x;
            return tile * kTileM + 2 * (P & (kPairs - 1)) + (lane >> 4);
        };
        int v_next = 0, pad_next = 0;
        if (g < total) {
            const int v = node_of(g);
            v_next = v < p.n ? v : 0;                     // rows past the end stand in as node 0; their output is clipped
            if (sub < W) pad_next = p.nbr_pad[(size_t)v_next * W + sub];
        }
        for (int P = g; P < total; P += kGatherWarps) {
            if (__any_sync(0xffffffffu, *abort_flag != 0)) break;
            const int s = P >> 6;
            const int row = 2 * (P & (kPairs - 1)) + (lane >> 4);
            const int v = v_next, pad = pad_next;
            if (P + kGatherWarps < total) {               // the next node's table entry arrives under this node's gather
                const int v2 = node_of(P + kGatherWarps);
                v_next = v2 < p.n ? v2 : 0;
                if (sub < W) pad_next = p.nbr_pad[(size_t)v_next * W + sub];
            }
            const int cnt = __shfl_sync(mask, pad, grp_base);
            Piece kq[MAXN], vq[MAXN], qp;
            int u[MAXN];
            u[0] = v;
#pragma unroll
            for (int j = 1; j < MAXN; ++j) u[j] = __shfl_sync(mask, pad, grp_base + j);
            // filler entries of the table repeat v: all loads go out without predicates (predicating them off was
            // measured slower here as in the stand-alone kernel)
#pragma unroll
            for (int j = 0; j < MAXN; ++j) kq[j] = ld_piece_nc((const char*)p.KV + (size_t)u[j] * 512 + col);
#pragma unroll
            for (int j = 0; j < MAXN; ++j) vq[j] = ld_piece_nc((const char*)p.KV + (size_t)u[j] * 512 + 256 + col);
            if (s != s_ready) {                           // the tile's query rows must have been projected
                if (!mbar_wait_warp(smem_u32(&bars->q_full[s % kBufs]), ((uint32_t)(s / kBufs)) & 1u, p.poll_limit)) {
                    raise_timeout(bars, p.status);
                    break;
                }
                s_ready = s;
            }
            const uint32_t place = sQO + (uint32_t)((s % kBufs) * kTileBytes) + tile_piece(row, sub);
            ld_shared_v4(place, qp.w);
            float acc[8];
            attend<true, LPH, MAXN>(qp, kq, vq, cnt, p.scale, mask, acc);
            const Piece o = Elem<true>::pack(acc);
            st_shared_v4(place, o.w);
            fence_proxy_async_smem();                     // the output projection reads the tile through the async proxy
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&bars->o_full[s % kBufs]));
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem, kTmemCols);
    }
}

// ---------------------------------------------------------------------------------------------------
std::mutex g_mu;
int g_sm_count[64] = {};
bool g_dev_known[64] = {};

template <int LPH, int MAXN>
dg4_status launch(const CUtensorMap& mx, const CUtensorMap& mwq, const CUtensorMap& mwo, const CUtensorMap& mout,
                  const FusedParams& p, int grid, cudaStream_t st) {
    auto kern = fused_layer_kernel<LPH, MAXN>;
    DG4_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
    kern<<<grid, kThreads, kSmemBytes, st>>>(mx, mwq, mwo, mout, p);
    dg4i_count_launch();
    DG4_CUDA_TRY(cudaGetLastError());
    return DG4_OK;
}

template <int MAXN>
dg4_status launch_heads(int heads, const CUtensorMap& mx, const CUtensorMap& mwq, const CUtensorMap& mwo,
                        const CUtensorMap& mout, const FusedParams& p, int grid, cudaStream_t st) {
    switch (16 / heads) {
        case 1: return launch<1, MAXN>(mx, mwq, mwo, mout, p, grid, st);
        case 2: return launch<2, MAXN>(mx, mwq, mwo, mout, p, grid, st);
        case 4: return launch<4, MAXN>(mx, mwq, mwo, mout, p, grid, st);
        case 8: return launch<8, MAXN>(mx, mwq, mwo, mout, p, grid, st);
        case 16: return launch<16, MAXN>(mx, mwq, mwo, mout, p, grid, st);
    }
    DG4_FAIL(DG4_ERR_UNSUPPORTED, "heads = %d is not supported", heads);
}

}  // namespace

bool dg4i_fused_layer_supported(const dg4_graph* g, const dg4_desc* desc) {
    const int h = desc->heads;
    return !g->wide && g->nbr_pad != nullptr && g->max_class <= 7 && desc->dtype == DG4_BF16 && h >= 1 && h <= 16 &&
           (h & (h - 1)) == 0;
}

dg4_status dg4i_fused_layer_launch(const dg4_graph* g, const dg4_desc* desc, const __nv_bfloat16* X, int64_t ldx,
                                   const __nv_bfloat16* KV, const __nv_bfloat16* W_q, const __nv_bfloat16* W_o,
                                   __nv_bfloat16* H_out, int64_t ldho, int32_t* status, cudaStream_t st) {
    if (g->n <= 0) return DG4_OK;
    int dev = 0;
    DG4_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) DG4_FAIL(DG4_ERR_UNSUPPORTED, "device ordinal %d is out of range", dev);
    {
        std::lock_guard<std::mutex> lock(g_mu);
        if (!g_dev_known[dev]) {
            DG4_CUDA_TRY(cudaDeviceGetAttribute(&g_sm_count[dev], cudaDevAttrMultiProcessorCount, dev));
            g_dev_known[dev] = true;
        }
    }
    CUtensorMap mx, mwq, mwo, mout;
    dg4_status s;
    if ((s = dg4i_make_row_map(&mx, X, g->n, ldx, kTileM)) != DG4_OK) return s;
    if ((s = dg4i_make_row_map(&mwq, W_q, 128, 128, 128)) != DG4_OK) return s;
    if ((s = dg4i_make_row_map(&mwo, W_o, 128, 128, 128)) != DG4_OK) return s;
    if ((s = dg4i_make_row_map(&mout, H_out, g->n, ldho, kTileM)) != DG4_OK) return s;
    FusedParams p;
    p.X = X; p.ldx = ldx; p.KV = KV; p.nbr_pad = g->nbr_pad; p.n = g->n;
    p.n_tiles = (g->n + kTileM - 1) / kTileM;
    p.residual = (desc->flags & DG4_FLAG_RESIDUAL) ? 1 : 0;
    p.scale = desc->scale; p.status = status; p.poll_limit = dg4i_poll_limit();
    const int grid = p.n_tiles < g_sm_count[dev] ? p.n_tiles : g_sm_count[dev];
    if (g->max_class <= 3) return launch_heads<3>(desc->heads, mx, mwq, mwo, mout, p, grid, st);
    return launch_heads<7>(desc->heads, mx, mwq, mwo, mout, p, grid, st);
}
