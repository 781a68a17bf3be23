// Levelised layers as ONE persistent kernel (Sec. 1 / Sec. 3.4: gates are encoded level by level in
// topological order, each gate once, reading the rows already updated for lower levels).
//
// Work of one tile (16 nodes of one level, for one layer k), in two parts:
//   PROLOGUE (depends only on the layer below): the tile's input rows -- H as layer k-1 left it, or the caller's
//      rows for the first layer -- are brought into shared memory in the tensor core's K-major, 128-byte-swizzled
//      operand layout, and Q | K | V of the tile's own nodes are computed from them TRANSPOSED on the tensor
//      cores: D[feature, node] = W * X^T (tcgen05.mma, M = 128 features, N = 16 nodes, K = 128).  A node's own
//      query, key and value always come from its row as the previous layer left it, and nobody else ever reads
//      them (other nodes gather its K | V only after its update), so they stay on chip: no Q table, no up-front
//      projection of all nodes.
//   MAIN (depends on the level below in the same layer):
//   1. gather the K | V rows of every OTHER neighbour from layer k's K|V table (16 lanes per node, 16 bytes per
//      lane), compute scores, softmax and the weighted value sum in registers, and write the 16 x 128
//      attention tile into shared memory in operand layout;
//   2. output projection by warp-level MMAs (mma.sync m16n8k16, W_o in shared memory): warp w computes output
//      features 16w .. 16w+15 of all 16 nodes, and the result is in registers when the last instruction retires.
//      This product sits on the level-to-level chain, and an asynchronous tcgen05 group costs an order / issue /
//      commit / barrier / tcgen05.ld round trip that for its 8 instructions is longer than the product itself;
//   3. add the residual (the input rows still in shared memory), round to bf16, write the new rows to H and --
//      in operand layout again -- to shared memory;
//   4. from the new rows, transposed (tcgen05.mma, 16 instructions: here the asynchronous path is the cheaper
//      one): the tile's K | V rows of layer k, stored to the table so that higher levels gather updated rows.
//      While that product runs, the lanes ask L2 (prefetch, nothing waits for it) for what the coming levels'
//      first loads will want: node ids, neighbour-table entries, input rows, the next level's neighbours' K | V.
// The prologue of a CTA's NEXT tile is folded into the main part of the current one: the next tile's rows are
// requested once the layer below is known to have finished them, they are written to the second input buffer
// before the barrier that precedes step 4, and their Q | K | V product is issued right behind step 4's MMAs, so
// it runs while the CTA stores its rows, arrives and waits for the level to complete.  The level-to-level chain
// is then wait -> gather -> W_o -> K|V refresh -> arrive; the projections of the next tile hide in the hand-off.
// A CTA that has no tile in a level but has one in the next does that prologue while it is idle.
// The tcgen05 MMAs are issued by a thread of a ninth warp that does nothing else: issuing an M128 x N16 x K16 instruction
// occupies the issuing thread for about as long as the tensor pipe needs to execute it, so a worker thread that
// issued the next tile's 24 instructions would hold up its own warp's epilogue (and with it the level) for their
// whole duration.  The workers hand the issuing thread one order at a time (a word in shared memory and an
// mbarrier arrival) and wait only for the completion barrier of the product they need next.  Both sides wait
// suspended (try_wait with a time hint) rather than polling: a polling warp takes issue slots from the warp that
// shares its scheduler -- from the issuing thread while the workers wait for its product, from the workers'
// attention while the issuing thread waits for an order (measured: 2 % of the whole sweep).
//
// Cones wider than two hops (MAXN = 0) come as lists instead of the fixed-width table: step 1 then walks a node's
// list in batches of four entries with an online softmax, two batches in flight.  A tile's time is then the serial
// walk of its longest list, so narrow levels are spread over all of the layer's CTAs and the slots a tile has
// left over take replicas of its nodes, each walking a share of the list; the shares are merged in shared memory.
//
// The whole Transformer block level by level (block mode, Sec. 3.5 with the order of Sec. 1 / Sec. 3.4): the CTAs are
// dealt alternately to an attention stage -- the tile described above without step 4 -- and a feed-forward stage,
// which keeps W1 in tensor memory and W2 in shared memory and turns the attention stage's rows of a level into
// the block's output rows (LayerNorm, two transposed products with bias / ReLU between them, residual, LayerNorm)
// and refreshes the level's K | V rows from THOSE.  Both stages take the same tiles, so the kernel is launched as
// clusters of two -- an attention-stage CTA and the feed-forward-stage CTA of
// the same tiles -- and a tile's rows go from one to the other on chip: the feed-forward CTA reads them out of its
// partner's shared memory as soon as the partner's arrival on a barrier in ITS shared memory says they are there
// (no trip through global memory, no wait for the rest of the level).  The way back is a level's worth: the
// attention stage of the next level waits for the feed-forward stage's counter of this one, as the layers of a
// wavefront wait for theirs.
//
// Several layers run as a wavefront: layer k+1 may process level l as soon as layer k has finished level l
// (its inputs are that level's new rows) and layer k+1 itself has finished the levels below l.  CTAs are dealt
// to layers round-robin; each keeps its layer's W_k, W_v and W_q resident in TENSOR memory (blocks of 128 lanes
// x 64 columns beside the accumulators) and issues its tcgen05 MMAs with the A operand read from there, so
// those weights are never re-read from shared memory, which holds the node-side tiles and W_o.  With n
// layers the dependent chain is n_levels + n - 1 tile steps long instead of n * n_levels, while computing exactly
// what n successive level-by-level sweeps compute.
//
// Levels are separated by counters in global memory instead of kernel launches: every (layer, level) has an
// arrival counter that only the CTAs owning a tile of it bump (release); before a level in which it has work a
// CTA waits (acquire) until the counter of its layer's previous non-empty level and the counter of the previous
// layer's same level are full.  Completion is transitive, because every CTA that arrived had itself waited the
// same way.  Launched cooperatively (all CTAs co-resident).  Every wait is bounded; on expiry the kernel records
// DG4_ERR_TIMEOUT, raises an abort word that every other wait polls, and all CTAs leave their loops, wait for the
// MMAs they have issued, free tensor memory and return.

#include "dg4_internal.h"
#include "dg4_attn_core.cuh"
#include "dg4_sm100.cuh"

#include <stdlib.h>
#include <mutex>

namespace {

using namespace sm100;
using namespace attn;

constexpr int kTile = 16;                    // node slots per tile
constexpr int kMergeRow = 12;                // floats a lane parks for the merge of a split list: m, z, 8 sums (+ padding)
constexpr int kWorkers = kTile * 16;         // 16 lanes per node: eight warps that gather, attend and run the epilogues
constexpr int kThreads = kWorkers + 32;      // and a ninth warp whose first lane issues every tcgen05.mma
constexpr int kBHalf = kTile * 128;          // K-half of a kTile-row operand tile
constexpr int kTileOp = 2 * kBHalf;          // a kTile x 128 bf16 tile in operand layout (4 KiB)
constexpr int kTmemCols = 512;
constexpr int kAccK2 = 1, kAccV2 = 2, kAccQ = 3, kAccK = 4, kAccV = 5;   // accumulators of kTile columns (slot 0 unused)
constexpr int kWCol0 = 64;                   // weight blocks at kWCol0 + blk * 64: W_k at 128, W_v at 192, W_q at 256
// a CTA that runs the feed-forward stage of the block instead keeps W1 where W_q would be (four blocks from column
// 256) and has its own accumulators beside K2 | V2: the four hidden blocks and the second product
constexpr int kColW1 = 256, kColD1 = 3 * kTile, kColD2 = 7 * kTile;
constexpr int kWCols = 64;                   // a 128 x 128 bf16 block: 128 lanes x 64 columns of two elements
constexpr int kBlkK = 1, kBlkV = 2, kBlkQ = 3;            // weight blocks in tensor memory (slot 0 unused)
constexpr int kStageRow = 768 + 16;          // staging per node: Q 256 | K 256 | V 256 (+ padding against bank conflicts)

constexpr int kOffO = 0;                               // attention tile (operand layout)
constexpr int kOffHp = kOffO + kTileOp;                // new rows (operand layout)
constexpr int kOffX = kOffHp + kTileOp;                // input rows of the current and of the next tile (operand layout)
constexpr int kOffHres = kOffX + 2 * kTileOp;          // the same rows, plain [kTile][256 B], twice
constexpr int kOffStage = kOffHres + 2 * kTile * 256;  // staging, plain [kTile][kStageRow]
constexpr int kOffMerge = kOffStage + kTile * kStageRow;        // wide cones: partial softmaxes of a node's replicas
constexpr int kOffAct = ((kOffMerge + kWorkers * kMergeRow * 4 + 1023) / 1024) * 1024;   // feed-forward stage: hidden activations, 4 tiles
constexpr int kOffS32 = kOffAct + 4 * kTileOp;                  // feed-forward stage: second product in fp32, [kTile][128]
constexpr int kOffMisc = kOffS32 + kTile * 128 * 4;
constexpr int kWHalf = 128 * 128;                      // K-half of a 128-row weight block: 128 rows x 128 bytes
constexpr int kWBlock = 2 * kWHalf;                    // a 128 x 128 bf16 block in shared memory (32 KiB)
constexpr int kOffWs = ((kOffMisc + 256 + 1023) / 1024) * 1024;   // W_o for the warp-level output projection; W2 (4 blocks) in a feed-forward CTA
constexpr int kSmemBytes = kOffWs + kWBlock + 1024;              // layers: W_o
constexpr int kSmemBytesBlock = kOffWs + 4 * kWBlock + 1024;     // blocks: room for W2 in the feed-forward-stage CTAs
static_assert(kSmemBytesBlock <= 232448, "shared memory budget of one CTA");
static_assert(kWCol0 + 4 * kWCols <= kTmemCols && kColW1 + 4 * kWCols <= kTmemCols && 6 * kTile <= kWCol0 + kWCols &&
              kColD2 + kTile <= kWCol0 + kWCols, "tensor memory budget of one CTA");
static_assert((kOffX % 1024) == 0 && (kOffHp % 1024) == 0 && (kTileOp % 1024) == 0, "operand tiles are 1024-byte aligned");
// Every CTA allocates all of its SM's tensor memory, so two CTAs must never share an SM (the second one's
// allocation would wait for the first, which waits for the second's levels): the launch asks for more than half
// of an SM's shared memory, which rules that out.
// (Blocks ask for more: only then is the rest of the SM's 256 KiB, which the gathers use as L1, given up.)
constexpr int kLaunchSmemBytes = kSmemBytes > 120 * 1024 ? kSmemBytes : 120 * 1024;
static_assert(kSmemBytesBlock > 120 * 1024, "one CTA per SM in block mode too");

enum : int32_t { kCmdExit = 0, kCmdQkv = 1, kCmdKv = 2, kCmdKvThenQkv = 3, kCmdFfn1 = 4, kCmdFfn2 = 5 };

struct Misc {
    uint64_t mma0, mma1, mma2, drain;
    uint64_t pair_rows;                    // feed-forward CTA of a pair: the attention CTA's rows of the next tile are in ITS shared memory
    uint64_t pair_taken;                   // attention CTA of a pair: the feed-forward CTA has read them
    uint64_t cmd_bar;                      // the workers' next order for the issuing thread is in `cmd`
    int32_t cmd, cmd_buf;
    uint32_t tmem_base;
    int32_t go, go2;
    int32_t failed;                        // a wait for this CTA's own MMAs ran out: leave at the next level
    int32_t pre_ok;                        // the layer below has finished the rows of this CTA's next tile (checked mid-tile)
    int32_t pre_early;                     // the same, already known at the top of the tile
    int32_t node[kTile];
};

struct LevParams {
    __nv_bfloat16* KV[DG4I_MAX_LAYERS];    // [n, 256] per layer: K | V of the nodes the layer has updated so far
    const __nv_bfloat16* Wo[DG4I_MAX_LAYERS];    // [128, 128] per layer, out x in
    const __nv_bfloat16* Wqkv[DG4I_MAX_LAYERS];  // [384, 128] per layer
    __nv_bfloat16* H;                      // [n, ldh], updated in place by every layer in turn
    int64_t ldh;
    const int32_t* nbr_pad;                // [n, pad_width] (cones of at most two hops)
    const int32_t* nbr_ptr;                // [n + 1], [n_nbr]: the cones as lists (wider cones)
    const int32_t* nbr_idx;
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
    // The whole Transformer block level by level (block != 0, n_layers == 2): the CTAs of "layer" 0 run the
    // attention sub-layer of a level, those of "layer" 1 its LayerNorm, feed-forward sub-layer, LayerNorm and the
    // K | V refresh from the block's output rows; the two hand each level to one another through the counters.
    // Several blocks: n_layers == 2 x blocks, "layer" 2k is block k's attention stage, 2k+1 its feed-forward stage,
    // and the stages of all blocks form one wavefront.
    int32_t block;
    int32_t paired;                        // launched as clusters of two: CTA 2j (attention stage) and 2j+1 (feed-forward stage)
                                           // take the same tiles, and the rows go from one to the other on chip
    float eps;
    const float* ln1_gamma[DG4I_MAX_LAYERS]; const float* ln1_beta[DG4I_MAX_LAYERS];
    const __nv_bfloat16* W1[DG4I_MAX_LAYERS];              // [512, 128]
    const float* b1[DG4I_MAX_LAYERS];                      // [512]
    const __nv_bfloat16* W2[DG4I_MAX_LAYERS];              // [128, 512]
    const float* b2[DG4I_MAX_LAYERS];                      // [128]
    const float* ln2_gamma[DG4I_MAX_LAYERS]; const float* ln2_beta[DG4I_MAX_LAYERS];
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
// NB accumulators (lanes = 128 output features, 16 columns = the tile's nodes, kTile columns apart) into the staging
// rows as bf16: the warp reads its 32 lanes x 8 nodes as m16n8 fragments and writes, per accumulator, one transposing
// matrix store -- 8 nodes x 32 features, 16 bytes (8 features) per node and matrix.  `taddr`: the first accumulator
// at this warp's lanes and columns; `st_addr`: thread 8m + j passes staging row j of the warp's 8 nodes at
// features 8m of the warp's 32.
__device__ __forceinline__ uint32_t pack_bf16x2_of_bits(uint32_t lo, uint32_t hi) {   // fp32 bit patterns in, as tcgen05.ld delivers them
    uint32_t pk;
    asm("cvt.rn.bf16x2.f32 %0, %2, %1;" : "=r"(pk) : "f"(__uint_as_float(lo)), "f"(__uint_as_float(hi)));
    return pk;
}
template <int NB>
__device__ __forceinline__ void accumulators_to_stage(uint32_t taddr, uint32_t st_addr) {
    uint32_t r[NB][8];
#pragma unroll
    for (int blk = 0; blk < NB; ++blk) {
        tmem_ld_16x256b_x1(taddr + (uint32_t)(blk * kTile), r[blk]);
        tmem_ld_16x256b_x1(taddr + (16u << 16) + (uint32_t)(blk * kTile), r[blk] + 4);
    }
    tmem_ld_wait();
#pragma unroll
    for (int blk = 0; blk < NB; ++blk) {
        const uint32_t m[4] = {pack_bf16x2_of_bits(r[blk][0], r[blk][1]), pack_bf16x2_of_bits(r[blk][2], r[blk][3]),
                               pack_bf16x2_of_bits(r[blk][4], r[blk][5]), pack_bf16x2_of_bits(r[blk][6], r[blk][7])};
        stmatrix_x4_trans(st_addr + (uint32_t)(blk * 256), m);
    }
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
// byte offset of the 16-byte piece `sub` (0..15) of row `row` in the same layout
__device__ __forceinline__ uint32_t operand_piece(int row, int sub) {
    return (uint32_t)((sub >> 3) * kBHalf) + sw128_offset(row, sub & 7);
}

__device__ __forceinline__ void give_up(const LevParams& p) {
    atomicExch(p.abort_word, 1);
    if (p.status) atomicCAS(p.status, 0, (int)DG4_ERR_TIMEOUT);
}

// byte offset of the 16-byte piece `chunk` (0..15) of row `row` in a 128-row weight block (same swizzle)
__device__ __forceinline__ uint32_t weight_piece(int row, int chunk) {
    return (uint32_t)((chunk >> 3) * kWHalf) + sw128_offset(row, chunk & 7);
}
// warp-level tensor-core product (synchronous: the result is in registers when the instruction retires), used for
// the two 16-node products that sit on the level-to-level chain
__device__ __forceinline__ void prefetch_l2(const void* ptr) {
    asm volatile("prefetch.global.L2 [%0];" ::"l"(ptr));
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t* r) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}
__device__ __forceinline__ void mma_m16n8k16(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void st_shared_b32(uint32_t addr, uint32_t v) {
    asm volatile("st.shared.b32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ uint32_t ld_shared_b32(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&h);
}

// ---- the two CTAs of a cluster (a block's attention stage and its feed-forward stage, paired tile by tile) ----
__device__ __forceinline__ uint32_t in_cta(uint32_t smem_addr, uint32_t rank) {      // the same address in the cluster's CTA `rank`
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_in_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ bool mbar_wait_from_cluster(uint32_t bar, uint32_t parity, uint32_t limit) {   // bounded, suspended
    const uint32_t tries = (limit >> 4) + 1u;
    for (uint32_t i = 0; i < tries; ++i) {
        uint32_t ok;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(ok) : "r"(bar), "r"(parity), "r"(kRelaxedWaitNs) : "memory");
        if (ok) return true;
    }
    return false;
}
__device__ __forceinline__ void ld_cluster_v4(uint32_t cluster_addr, uint32_t* r) {
    asm volatile("ld.shared::cluster.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// barrier among the eight worker warps only (the issuing warp never joins it)
__device__ __forceinline__ void worker_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kWorkers) : "memory"); }

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

// BLOCK: the whole Transformer block (attention-stage and feed-forward-stage CTAs) instead of attention layers.
template <int LPH, int MAXN, bool BLOCK>
__global__ void __launch_bounds__(kThreads, 1)
levelised_kernel(LevParams p) {
    extern __shared__ uint8_t smem_raw[];
    constexpr bool WIDE = (MAXN == 0);                   // cones wider than two hops: CSR lists instead of the table
    constexpr int NK = WIDE ? 1 : MAXN;
    constexpr int W = WIDE ? 2 : MAXN + 1;               // words of a node's index entry: table row, or its list bounds
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
    Misc* misc = reinterpret_cast<Misc*>(base_ptr + kOffMisc);
    const uint32_t sO = base + kOffO, sHp = base + kOffHp, sX = base + kOffX, sHres = base + kOffHres, sSt = base + kOffStage;
    const uint32_t sW = base + kOffWs;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int slot = tid >> 4, sub = tid & 15;          // node slot of the tile and lane within the node
    const int grp_base = lane - sub;
    const unsigned gmask = 0xffffu << grp_base;
    const uint32_t bar0 = smem_u32(&misc->mma0), bar2 = smem_u32(&misc->mma2);

    // this CTA's layer, its rank among the CTAs of that layer, and how many CTAs each layer has
    const int layer = (int)blockIdx.x % p.n_layers;
    const int bid = (int)blockIdx.x / p.n_layers;
    auto ctas_of = [&](int k) { return ((int)gridDim.x - k + p.n_layers - 1) / p.n_layers; };
    const int nctas = ctas_of(layer);

    if (tid == 0) {
        mbar_init(bar0, 1);
        mbar_init(bar2, 1);
        mbar_init(smem_u32(&misc->mma1), 1);
        mbar_init(smem_u32(&misc->pair_rows), 1);
        mbar_init(smem_u32(&misc->pair_taken), 1);
        mbar_init(smem_u32(&misc->drain), 1);
        mbar_init(smem_u32(&misc->cmd_bar), 1);
        misc->cmd = kCmdExit;
        misc->cmd_buf = 0;
        misc->go = 1;
        misc->go2 = 1;
        misc->failed = 0;
        misc->pre_ok = 0;
        misc->pre_early = 0;
        mbar_fence_init();
    }
    if (warp == 0) tmem_alloc(smem_u32(&misc->tmem_base), kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = misc->tmem_base;
    static_assert(kWorkers / 32 / 4 * 8 == kTile, "epilogue: every warp reads 8 node columns of its lane quadrant");
    const int q4 = warp & 3, cg = warp >> 2;             // TMEM lane quadrant of the warp; which half of the columns it takes
    const int feat = q4 * 32 + lane;                     // output feature (TMEM lane) this thread holds
    // where this thread points a transposing matrix store of its warp's 8 nodes x 32 features (see accumulators_to_stage)
    const uint32_t stage_frag = sSt + (uint32_t)((cg * 8 + (lane & 7)) * kStageRow + (q4 * 32 + 8 * (lane >> 3)) * 2);
    const uint32_t lane_base = (uint32_t)(q4 * 32) << 16;
    // The weights stay in tensor memory for the whole kernel: row `feat` of every block in lane `feat`, two
    // consecutive bf16 of the row per 32-bit column (the bytes as they lie in global memory).  Each thread copies
    // half a row (128 bytes) of every block of its layer.
    const bool paired = BLOCK && p.paired != 0;
    if (paired) cluster_sync_all();        // the partner's barriers are initialised before anything arrives on them
    const bool ffn_stage = BLOCK && (layer & 1) != 0;
    const int wl = BLOCK ? layer >> 1 : layer;         // whose weights and K | V table this CTA works with
    if (warp < 8 && ffn_stage) {
        // W_k, W_v as everywhere; W1's four blocks of 128 hidden units in tensor memory; W2 in shared memory as
        // four 128 x 128 blocks (block c = hidden units 128c .. 128c+127) in the swizzled K-major layout
        for (int blk = 1; blk <= 6; ++blk) {
            const __nv_bfloat16* wb = blk <= 2 ? p.Wqkv[wl] + (size_t)blk * 128 * 128 : p.W1[wl] + (size_t)(blk - 3) * 128 * 128;
            const uint32_t col0 = blk <= 2 ? (uint32_t)(kWCol0 + blk * kWCols) : (uint32_t)(kColW1 + (blk - 3) * kWCols);
            const uint4* src = reinterpret_cast<const uint4*>(wb + (size_t)feat * 128 + cg * 64);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const uint4 lo = src[2 * c], hi = src[2 * c + 1];
                const uint32_t r[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
                tmem_st_32x8(tmem + lane_base + col0 + (uint32_t)(cg * 32 + c * 8), r);
            }
        }
        tmem_st_wait();
        for (int i = tid; i < 4 * 128 * 16; i += kWorkers) {
            const int c = i >> 11, row = (i >> 4) & 127, chunk = i & 15;
            const uint4 v = *reinterpret_cast<const uint4*>(p.W2[wl] + (size_t)row * 512 + c * 128 + chunk * 8);
            const uint32_t r[4] = {v.x, v.y, v.z, v.w};
            st_shared_v4(sW + (uint32_t)(c * kWBlock) + weight_piece(row, chunk), r);
        }
        fence_proxy_async_smem();
    } else if (warp < 8) {
        for (int blk = kBlkK; blk <= kBlkQ; ++blk) {
            const __nv_bfloat16* wb = blk == kBlkQ ? p.Wqkv[wl]
                                                    : p.Wqkv[wl] + (size_t)blk * 128 * 128;     // kBlkK = 1, kBlkV = 2
            const uint4* src = reinterpret_cast<const uint4*>(wb + (size_t)feat * 128 + cg * 64);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const uint4 lo = src[2 * c], hi = src[2 * c + 1];
                const uint32_t r[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
                tmem_st_32x8(tmem + lane_base + (uint32_t)(kWCol0 + blk * kWCols + cg * 32 + c * 8), r);
            }
        }
        tmem_st_wait();
        // W_o once more in shared memory (same 128-byte swizzle): the B operand of the warp-level output projection
        for (int i = tid; i < 128 * 16; i += kWorkers) {
            const int row = i >> 4, chunk = i & 15;
            const uint4 v = *reinterpret_cast<const uint4*>(p.Wo[wl] + (size_t)row * 128 + chunk * 8);
            const uint32_t r[4] = {v.x, v.y, v.z, v.w};
            st_shared_v4(sW + weight_piece(row, chunk), r);
        }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();

    const uint32_t idesc = idesc_bf16_f32(128, kTile);
    // matrix descriptors of the node-side operands; stepping along K only adds to the address field
    const uint64_t dHp = smem_desc_sw128(sHp);
    const uint64_t dX[2] = {smem_desc_sw128(sX), smem_desc_sw128(sX + kTileOp)};
    // issues Q | K | V = W * X^T for the rows in input buffer b (one thread)
    auto issue_qkv = [&](int b) {
        tc_fence_after();
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            const uint32_t b_off = (uint32_t)((ks >> 2) * kBHalf + (ks & 3) * 32);
            mma_bf16_ta(tmem + (uint32_t)(kTile * kAccQ), tmem + (uint32_t)(kWCol0 + kBlkQ * kWCols + ks * 8), dX[b] + (b_off >> 4), idesc, ks > 0 ? 1u : 0u);
            mma_bf16_ta(tmem + (uint32_t)(kTile * kAccK), tmem + (uint32_t)(kWCol0 + kBlkK * kWCols + ks * 8), dX[b] + (b_off >> 4), idesc, ks > 0 ? 1u : 0u);
            mma_bf16_ta(tmem + (uint32_t)(kTile * kAccV), tmem + (uint32_t)(kWCol0 + kBlkV * kWCols + ks * 8), dX[b] + (b_off >> 4), idesc, ks > 0 ? 1u : 0u);
        }
        mma_commit(bar0);
    };
    if (warp == 8) {
        // ---------------------------------------------------------------- the issuing thread
        if (lane == 0) {
            const uint32_t cmd_bar = smem_u32(&misc->cmd_bar);
            uint32_t phc = 0;
            int strikes = 0;
            for (;;) {
                if (!mbar_wait_relaxed(cmd_bar, phc, p.poll_limit)) {
                    // no order for a long time: normal while the CTA idles through levels in which it has no tile,
                    // unless the run was aborted meanwhile; a bound on the total keeps even that wait finite
                    if (ld_acquire(p.abort_word) != 0) break;
                    if (++strikes >= 64) { give_up(p); break; }
                    continue;
                }
                phc ^= 1u;
                strikes = 0;
                const int cmd = *reinterpret_cast<volatile int32_t*>(&misc->cmd);
                const int b = *reinterpret_cast<volatile int32_t*>(&misc->cmd_buf);
                if (cmd == kCmdExit) break;
                if (cmd == kCmdQkv) {
                    issue_qkv(b);
                } else if (cmd == kCmdFfn1) {
                    // hidden^T = W1 * Y1^T, four blocks of 128 hidden units (rows in input buffer 0)
                    tc_fence_after();
#pragma unroll
                    for (int blk = 0; blk < 4; ++blk)
#pragma unroll
                        for (int ks = 0; ks < 8; ++ks) {
                            const uint32_t b_off = (uint32_t)((ks >> 2) * kBHalf + (ks & 3) * 32);
                            mma_bf16_ta(tmem + (uint32_t)(kColD1 + blk * kTile), tmem + (uint32_t)(kColW1 + blk * kWCols + ks * 8), dX[0] + (b_off >> 4), idesc, ks > 0 ? 1u : 0u);
                        }
                    mma_commit(bar0);
                } else if (cmd == kCmdFfn2) {
                    // out^T = W2 * act^T: W2's block c from shared memory as the A operand, the activation tile c as B
                    tc_fence_after();
#pragma unroll
                    for (int c = 0; c < 4; ++c)
#pragma unroll
                        for (int ks = 0; ks < 8; ++ks) {
                            const uint32_t a_off = (uint32_t)(c * kWBlock + (ks >> 2) * kWHalf + (ks & 3) * 32);
                            const uint32_t b_off = (uint32_t)(c * kTileOp + (ks >> 2) * kBHalf + (ks & 3) * 32);
                            mma_bf16(tmem + (uint32_t)kColD2, smem_desc_sw128(sW + a_off), smem_desc_sw128(base + kOffAct + b_off), idesc, (c > 0 || ks > 0) ? 1u : 0u);
                        }
                    mma_commit(smem_u32(&misc->mma1));
                } else {
                    // from the new rows, transposed: this layer's K | V refresh; right behind it, if ordered, the next
                    // tile's Q | K | V (it runs while this tile's rows are stored and the level completes)
                    tc_fence_after();
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        const uint32_t b_off = (uint32_t)((ks >> 2) * kBHalf + (ks & 3) * 32);
                        mma_bf16_ta(tmem + (uint32_t)(kTile * kAccK2), tmem + (uint32_t)(kWCol0 + kBlkK * kWCols + ks * 8), dHp + (b_off >> 4), idesc, ks > 0 ? 1u : 0u);
                        mma_bf16_ta(tmem + (uint32_t)(kTile * kAccV2), tmem + (uint32_t)(kWCol0 + kBlkV * kWCols + ks * 8), dHp + (b_off >> 4), idesc, ks > 0 ? 1u : 0u);
                    }
                    mma_commit(bar2);
                    if (cmd == kCmdKvThenQkv) issue_qkv(b);
                }
            }
            // Tensor memory is freed below: every MMA issued must have completed.  Normally each was waited for by
            // the workers; after a wait that ran out, one may still be in flight.
            mma_commit(smem_u32(&misc->drain));
            mbar_wait(smem_u32(&misc->drain), 0);
        }
    } else {
        // ---------------------------------------------------------------- the eight worker warps
        // hands the issuing thread its next order (one worker thread, after the barrier that made the operands
        // of that order visible)
        auto post = [&](int cmd, int b) {
            misc->cmd = cmd;
            misc->cmd_buf = b;
            mbar_arrive(smem_u32(&misc->cmd_bar));
        };
        uint32_t ph0 = 0, ph2 = 0;
        // lane's place in the warp-level products: g = row of the 8 x 8 sub-matrix it holds, t = column pair
        const int mg = lane >> 2, mt = lane & 3;
        const int a_row = lane & 15, a_chunk = lane >> 4;                       // A fragments: the 16-node tile
        const int b_row = (lane & 7) + ((lane >> 4) << 3), b_chunk = (lane >> 3) & 1;   // B fragments: 16 weight rows
        int last_nonempty = -1, last_participants = 0, last_participants_ffn = 0;
        bool alive = true;
        const uint32_t counter_limit = p.poll_limit > 4u ? p.poll_limit >> 2 : 1u;   // a counter poll is a trip to L2

        const char* kv_tab = (const char*)p.KV[wl];
        int32_t* my_arrive = p.arrive + (size_t)layer * p.n_levels;
        const int32_t* prev_arrive = layer > 0 ? p.arrive + (size_t)(layer - 1) * p.n_levels : nullptr;
        const int prev_ctas = layer > 0 ? ctas_of(layer - 1) : 0;
        // Nodes per tile of a level.  With the fixed-width table: 16, on as few CTAs as that takes (spreading a
        // narrow level over all CTAs was measured 2 % slower: more arrivals per level, nothing saved).  With cone
        // lists, where a tile's time is the serial walk of its longest list, a level narrower than ctas x 16
        // nodes is spread over all the layer's CTAs, and the slots a tile has left over take REPLICAS of its
        // nodes: replica q of `parts` walks every parts-th batch of the list, and the partial softmaxes are
        // merged through shared memory.
        auto per_tile = [&](int n_level, int ctas) {
            if (!WIDE) return kTile;
            const int t = (n_level + ctas - 1) / ctas;
            return t < 1 ? 1 : (t > kTile ? kTile : t);
        };
        auto tiles_of = [&](int n_level, int ctas) { const int t = per_tile(n_level, ctas); return (n_level + t - 1) / t; };
        // arrivals on the layer below's counter for a level of n_level nodes (one per CTA that owns a tile of it)
        auto prev_target = [&](int n_level) { const int t = tiles_of(n_level, prev_ctas); return t < prev_ctas ? t : prev_ctas; };

        // this lane's piece of node v's input row (zero for an empty slot) into input buffer b, both layouts
        auto stage_input = [&](int b, const Piece& x) {
            st_shared_v4(sX + (uint32_t)(b * kTileOp) + operand_piece(slot, sub), x.w);
            st_shared_v4(sHres + (uint32_t)(b * kTile * 256 + slot * 256 + sub * 16), x.w);
        };
        auto load_input = [&](int v) {
            Piece x;
            if (v >= 0) x = ld_piece_cg((const char*)p.H + (size_t)v * p.ldh * 2 + sub * 16);
            else x.w[0] = x.w[1] = x.w[2] = x.w[3] = 0u;
            return x;
        };

        // The index chain of a tile (node id -> neighbour-table entry) is two dependent loads that do not depend on
        // any other CTA's results.  It is software-pipelined across levels so that none of it sits on the
        // level-to-level critical path: while level l is processed, the node id of this CTA's first tile of level
        // l+2 and the table entry for level l+1 are in flight.
        // The level offsets run four levels ahead in registers: every acquire of a counter drops the L1 contents,
        // so a plain load at the top of a level would cost a trip to L2 on the level-to-level chain.
        auto lp_at = [&](int lv) { return p.level_ptr[lv < p.n_levels ? lv : p.n_levels]; };
        auto stage_node = [&](int lv_first, int lv_end) -> int {   // node of (first tile of this CTA, this slot) of a level
            const int t = per_tile(lv_end - lv_first, nctas);
            const int r = bid * t + slot % t;
            return (slot / t < kTile / t && r < lv_end - lv_first) ? p.level_nodes[lv_first + r] : -1;
        };
        int lp0 = lp_at(0), lp1 = lp_at(1), lp2 = lp_at(2), lp3 = lp_at(3);
        auto pad_of = [&](int v) -> int {
            if (v < 0 || sub >= W) return 0;
            return WIDE ? p.nbr_ptr[v + sub] : p.nbr_pad[(size_t)v * W + sub];
        };
        int v0 = stage_node(lp0, lp1);                     // level l  : node id and this lane's table word
        int pad0 = pad_of(v0);
        int vC = stage_node(lp1, lp2);                     // level l+1: node id

        if (ffn_stage) {
            // ------------------------------------------------------------ a block's feed-forward stage
            // Per tile of 16 nodes of a level whose attention stage has arrived: rows a (attention sub-layer output)
            // -> LayerNorm -> y1 (bf16) -> hidden^T = W1 y1^T (four blocks) -> + b1, ReLU, bf16 -> out^T = W2 act^T
            // -> + b2 + y1 -> LayerNorm -> block output rows (bf16) to H -> K | V refresh from them -> arrive.
            // Lanes own 8 features of a node in the row-wise parts and one feature (hidden unit) of 8 nodes in the
            // epilogues that read tensor memory; the two views meet in shared memory.
            const uint32_t bar1 = smem_u32(&misc->mma1);
            const uint32_t sAct = base + kOffAct, sS32 = base + kOffS32;
            uint32_t ph1 = 0, ph_rows = 0;
            float g1[8], be1[8], g2[8], be2[8], bo[8], bh[4];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                g1[i] = __ldg(p.ln1_gamma[wl] + sub * 8 + i); be1[i] = __ldg(p.ln1_beta[wl] + sub * 8 + i);
                g2[i] = __ldg(p.ln2_gamma[wl] + sub * 8 + i); be2[i] = __ldg(p.ln2_beta[wl] + sub * 8 + i);
                bo[i] = __ldg(p.b2[wl] + sub * 8 + i);
            }
#pragma unroll
            for (int blk = 0; blk < 4; ++blk) bh[blk] = __ldg(p.b1[wl] + blk * 128 + feat);
            auto layer_norm = [&](float* x, const float* g, const float* b) {     // over the node's 128 features (16 lanes)
                float sum = 0.f;
#pragma unroll
                for (int i = 0; i < 8; ++i) sum += x[i];
#pragma unroll
                for (int o = 8; o > 0; o >>= 1) sum += __shfl_xor_sync(gmask, sum, o);
                const float mean = sum * (1.0f / 128.0f);
                float sq = 0.f;
#pragma unroll
                for (int i = 0; i < 8; ++i) { x[i] -= mean; sq += x[i] * x[i]; }
#pragma unroll
                for (int o = 8; o > 0; o >>= 1) sq += __shfl_xor_sync(gmask, sq, o);
                const float rstd = rsqrtf(sq * (1.0f / 128.0f) + p.eps);
#pragma unroll
                for (int i = 0; i < 8; ++i) x[i] = x[i] * rstd * g[i] + b[i];
            };
            for (int l = 0; l < p.n_levels && alive; ++l) {
                const int first = p.level_ptr[l];
                const int n_l = p.level_ptr[l + 1] - first;
                // the same tiles as the attention stage (with cone lists: T_l nodes in the first T_l slots; the other
                // slots, which held replicas there, are empty here)
                const int T_l = per_tile(n_l, nctas);
                const int tiles = n_l > 0 ? (n_l + T_l - 1) / T_l : 0;
                if (n_l <= 0 || bid >= tiles) continue;
                bool waited = false;
                for (int tile = bid; tile < tiles; tile += nctas) {
                    const int r = tile * T_l + slot;
                    const int v = (slot < T_l && r < n_l) ? p.level_nodes[first + r] : -1;
                    if (!paired && !waited) {          // the attention stage has stored this level's rows
                        if (tid == 0) {
                            bool go = misc->failed == 0;
                            if (go) go = wait_counter(prev_arrive + l, prev_target(n_l), p.abort_word, counter_limit);
                            if (!go && ld_acquire(p.abort_word) == 0) give_up(p);
                            misc->go = go ? 1 : 0;
                        }
                        worker_sync();
                        waited = true;
                        if (!misc->go) { alive = false; break; }
                    }
                    // ---- first LayerNorm, rows into the operand tile
                    float x[8];
                    if (paired) {
                        // the partner CTA has just finished the same tile: its rows are read out of its shared memory
                        if (tid == 0) {
                            bool go = misc->failed == 0 && mbar_wait_from_cluster(smem_u32(&misc->pair_rows), ph_rows, p.poll_limit);
                            if (!go && ld_acquire(p.abort_word) == 0) give_up(p);
                            misc->go = go ? 1 : 0;
                        }
                        worker_sync();
                        if (!misc->go) { alive = false; break; }
                        mbar_wait_from_cluster(smem_u32(&misc->pair_rows), ph_rows, p.poll_limit);   // complete: acquires for this thread
                        ph_rows ^= 1u;
                        Piece a;
                        ld_cluster_v4(in_cta(sHp + operand_piece(slot, sub), 0), a.w);
                        Elem<true>::unpack(a, x);
                    } else {
                        const Piece a = load_input(v);
                        Elem<true>::unpack(a, x);
                    }
                    layer_norm(x, g1, be1);
                    const Piece y1 = Elem<true>::pack(x);
                    st_shared_v4(sX + operand_piece(slot, sub), y1.w);
                    if (sub == 0) misc->node[slot] = v;
                    fence_proxy_async_smem();
                    worker_sync();
                    if (tid == 0) {
                        post(kCmdFfn1, 0);
                        if (paired) mbar_arrive_in_cluster(in_cta(smem_u32(&misc->pair_taken), 0));   // every lane has its rows
                    }
                    // ---- hidden units: + b1, ReLU, bf16, into the four activation tiles (operand layout)
                    if (!mbar_wait_relaxed(bar0, ph0, p.poll_limit) && tid == 0) { give_up(p); misc->failed = 1; }
                    ph0 ^= 1u;
                    tc_fence_after();
#pragma unroll
                    for (int blk = 0; blk < 4; ++blk) {
                        uint32_t d[8];
                        tmem_ld_32x8(tmem + lane_base + (uint32_t)(kColD1 + blk * kTile + cg * 8), d);
                        tmem_ld_wait();
#pragma unroll
                        for (int nn = 0; nn < 8; ++nn) {
                            const float hval = fmaxf(__uint_as_float(d[nn]) + bh[blk], 0.f);
                            st_shared_b16(sAct + (uint32_t)(blk * kTileOp) + operand_offset(cg * 8 + nn, feat), bf16_bits(hval));
                        }
                    }
                    tc_fence_before();
                    fence_proxy_async_smem();
                    worker_sync();
                    if (tid == 0) post(kCmdFfn2, 0);
                    // ---- second product out of tensor memory into [node][feature] fp32
                    if (!mbar_wait_relaxed(bar1, ph1, p.poll_limit) && tid == 0) { give_up(p); misc->failed = 1; }
                    ph1 ^= 1u;
                    tc_fence_after();
                    {
                        uint32_t d[8];
                        tmem_ld_32x8(tmem + lane_base + (uint32_t)(kColD2 + cg * 8), d);
                        tmem_ld_wait();
#pragma unroll
                        for (int nn = 0; nn < 8; ++nn) st_shared_b32(sS32 + (uint32_t)(((cg * 8 + nn) * 128 + feat) * 4), d[nn]);
                    }
                    tc_fence_before();
                    worker_sync();
                    // ---- + b2 + y1, second LayerNorm, the block's output rows
                    {
                        uint32_t w8[8];
                        ld_shared_v4(sS32 + (uint32_t)((slot * 128 + sub * 8) * 4), w8);
                        ld_shared_v4(sS32 + (uint32_t)((slot * 128 + sub * 8 + 4) * 4), w8 + 4);
                        float y[8];
                        Elem<true>::unpack(y1, y);
#pragma unroll
                        for (int i = 0; i < 8; ++i) x[i] = __uint_as_float(w8[i]) + bo[i] + y[i];
                    }
                    layer_norm(x, g2, be2);
                    const Piece out = Elem<true>::pack(x);
                    if (v >= 0) st_global_v4((char*)p.H + (size_t)v * p.ldh * 2 + sub * 16, out.w);
                    st_shared_v4(sHp + operand_piece(slot, sub), out.w);
                    fence_proxy_async_smem();
                    worker_sync();
                    // ---- K | V of the new rows into the table
                    if (tid == 0) post(kCmdKv, 0);
                    if (!mbar_wait_relaxed(bar2, ph2, p.poll_limit) && tid == 0) { give_up(p); misc->failed = 1; }
                    ph2 ^= 1u;
                    tc_fence_after();
                    accumulators_to_stage<2>(tmem + lane_base + (uint32_t)(kTile * kAccK2 + cg * 8), stage_frag);
                    tc_fence_before();
                    worker_sync();
                    if (v >= 0) {
                        const uint32_t row = sSt + (uint32_t)(slot * kStageRow);
                        uint32_t w4[4];
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            ld_shared_v4(row + (uint32_t)((sub + 16 * h) * 16), w4);
                            st_global_v4((char*)p.KV[wl] + (size_t)v * 512 + (sub + 16 * h) * 16, w4);
                        }
                    }
                    worker_sync();
                }
                if (!alive) break;
                if (tid == 64) red_release_add(my_arrive + l, 1);
            }
            if (tid == 0) post(kCmdExit, 0);
        } else {
        bool pro_ready = false;      // the Q | K | V product of this CTA's next tile has been issued (rows in buffer `buf`)
        int buf = 0;
        bool rows_out = false;       // paired: a tile's rows are in sHp for the partner
        uint32_t ph_taken = 0;

        for (int l = 0; l < p.n_levels && alive; ++l) {
            const int first = lp0;
            const int n_l = lp1 - lp0;
            // the next load of every pipelined chain (results first used one level later) is issued together with
            // the tile's gather loads, whose latency the tile waits out anyway: issued here at the top, the first
            // wait on anything else would also wait for them
            int lp4 = 0, vB = -1, padC = 0;
            auto issue_chains = [&]() {
                lp4 = lp_at(l + 4);
                vB = stage_node(lp2, lp3);
                padC = pad_of(vC);
            };
            const int T_l = per_tile(n_l, nctas);                         // nodes per tile in this level
            const int tiles = (n_l + T_l - 1) / T_l;
            const int tiles_next = tiles_of(lp2 - lp1, nctas);            // tiles of level l + 1
            if (!(n_l > 0 && bid < tiles)) issue_chains();
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
                    const bool more_here = tile + nctas < tiles;
                    {
                        const int r = (tile + nctas) * T_l + slot % T_l;
                        v_nx = (more_here && slot / T_l < kTile / T_l && r < n_l) ? p.level_nodes[first + r] : -1;
                    }
                    const bool valid = v >= 0;
                    // which tile comes next for this CTA, and may its rows be requested already?  Asked twice: at the
                    // top of the tile (then the rows travel under the gather) and, if the layer below was not ready
                    // yet, once more in the middle of it
                    const bool next_level_tile = !more_here && l + 1 < p.n_levels && bid < tiles_next;
                    const bool want_pre = more_here || next_level_tile;
                    auto next_rows_ready = [&]() -> int {
                        if (!want_pre) return 0;
                        if (next_level_tile && prev_arrive) return ld_acquire(prev_arrive + l + 1) >= prev_target(lp2 - lp1) ? 1 : 0;
                        return 1;
                    };
                    if (waited && tid == 32) misc->pre_early = next_rows_ready();   // visible after the barrier below

                    // ---- this tile's own Q | K | V: read from tensor memory if the product was issued during the
                    // tile before, else brought up from scratch below (after the counters)
                    auto epilogue_qkv = [&]() {
                        if (!mbar_wait_relaxed(bar0, ph0, p.poll_limit) && tid == 0) { give_up(p); misc->failed = 1; }
                        ph0 ^= 1u;
                        tc_fence_after();
                        accumulators_to_stage<3>(tmem + lane_base + (uint32_t)(kTile * kAccQ + cg * 8), stage_frag);
                        tc_fence_before();
                    };
                    if (pro_ready) epilogue_qkv();

                    if (!waited) {
                        // ---- this layer's previous level must be complete, and (unless the prologue already saw it)
                        // the previous layer's same level: two pollers in different warps, so that both counters are
                        // watched at the same time
                        if (tid == 0) {
                            bool go = true;
                            if (misc->failed) go = false;
                            // (as a block's attention stage: the level below is complete when the feed-forward stage has
                            // refreshed its K | V rows)
                            if (go && last_nonempty >= 0)
                                go = BLOCK ? wait_counter(p.arrive + (size_t)(layer + 1) * p.n_levels + last_nonempty, last_participants_ffn, p.abort_word, counter_limit)
                                             : wait_counter(my_arrive + last_nonempty, last_participants, p.abort_word, counter_limit);
                            if (!go && ld_acquire(p.abort_word) == 0) give_up(p);
                            if (go && (l & 255) == 0 && ld_acquire(p.abort_word) != 0) go = false;
                            misc->go = go ? 1 : 0;
                        } else if (tid == 32) {
                            bool go = true;
                            if (prev_arrive && !pro_ready) go = wait_counter(prev_arrive + l, prev_target(n_l), p.abort_word, counter_limit);
                            if (!go && ld_acquire(p.abort_word) == 0) give_up(p);
                            misc->go2 = go ? 1 : 0;
                            misc->pre_early = go ? next_rows_ready() : 0;
                        }
                        worker_sync();
                        waited = true;
                        if (!misc->go || !misc->go2) { alive = false; break; }
                    } else if (pro_ready) {
                        worker_sync();             // the staged Q | K | V are visible to every lane
                    }
                    if (!pro_ready) {
                        // from scratch (a CTA's first tile, or the layer below was not ready in time): rows -> shared
                        // memory -> product -> staging
                        stage_input(buf, load_input(v));
                        fence_proxy_async_smem();
                        worker_sync();
                        if (tid == 0) post(kCmdQkv, buf);
                        epilogue_qkv();
                        worker_sync();
                    }
                    const uint32_t sHres_cur = sHres + (uint32_t)(buf * kTile * 256);

                    // ---- gather and attend
                    float acc[8];
                    Piece xpre;
                    const int v_pre = more_here ? v_nx : vC;
                    const bool pre_early = want_pre && misc->pre_early != 0;
                    if constexpr (!WIDE) {
                        Piece kq[NK], vq[NK], qp;
                        int u[NK];
                        const int cnt = valid ? __shfl_sync(gmask, pad, grp_base) : 1;
                        u[0] = v;
#pragma unroll
                        for (int j = 1; j < MAXN; ++j) u[j] = __shfl_sync(gmask, pad, grp_base + j);
                        if (valid) {
#pragma unroll
                            for (int j = 1; j < MAXN; ++j)
                                if (j < cnt) vq[j] = ld_piece_cg(kv_tab + (size_t)u[j] * 512 + 256 + sub * 16);
#pragma unroll
                            for (int j = 1; j < MAXN; ++j)
                                if (j < cnt) kq[j] = ld_piece_cg(kv_tab + (size_t)u[j] * 512 + sub * 16);
                        }
                        if (tile == bid) issue_chains();
                        if (pre_early) xpre = load_input(v_pre);                      // the next tile's input rows
                        else if (tid == 32) misc->pre_ok = next_rows_ready();         // second look; read after the next barrier
                        {   // the node's own query, key and value: from the staging rows
                            const uint32_t row = sSt + (uint32_t)(slot * kStageRow + sub * 16);
                            ld_shared_v4(row, qp.w);
                            ld_shared_v4(row + 256, kq[0].w);
                            ld_shared_v4(row + 512, vq[0].w);
                        }
                        attend<true, LPH, NK>(qp, kq, vq, cnt, p.scale, gmask, acc);
                    } else {
                        // cones wider than two hops: the node's list (CSR, the node itself included) is walked 16
                        // entries at a time -- one entry per lane of the node's group -- with four neighbours' rows
                        // in flight and an online softmax (running maximum and sum in log2 units, one rescale per
                        // batch of four).  The node's own entry takes the key and value projected on chip.
                        const int beg = valid ? __shfl_sync(gmask, pad, grp_base) : 0;
                        const int cnt = valid ? __shfl_sync(gmask, pad, grp_base + 1) - beg : 0;
                        if (tile == bid) issue_chains();
                        if (pre_early) xpre = load_input(v_pre);
                        else if (tid == 32) misc->pre_ok = next_rows_ready();
                        Piece qp, k_own, v_own;
                        {
                            const uint32_t row = sSt + (uint32_t)(slot * kStageRow + sub * 16);
                            ld_shared_v4(row, qp.w);
                            ld_shared_v4(row + 256, k_own.w);
                            ld_shared_v4(row + 512, v_own.w);
                        }
                        constexpr int UN = 4;
                        const float c = p.scale * 1.4426950408889634f;
                        const int parts = kTile / T_l, part = slot / T_l;      // replicas of a node, and which one this is
                        float m = -INFINITY, z = 0.f;
#pragma unroll
                        for (int e = 0; e < 8; ++e) acc[e] = 0.f;
                        // Batches of UN entries; this replica takes batches part, part + parts, ...  A 16-lane load
                        // brings the entries of four of its batches (one group), one group ahead of their use; the
                        // rows of batch k+1 are requested before batch k is consumed.
                        const int n_batches = (cnt + UN - 1) / UN;
                        const int nb = part < n_batches ? (n_batches - part + parts - 1) / parts : 0;   // this replica's
                        auto idx_group = [&](int j) -> int {
                            const int pos = (part + (4 * j + (sub >> 2)) * parts) * UN + (sub & 3);
                            return pos < cnt ? p.nbr_idx[beg + pos] : -1;
                        };
                        int g0 = nb > 0 ? idx_group(0) : -1, g1 = nb > 4 ? idx_group(1) : -1;
                        auto issue = [&](int k, int* u, Piece* kq, Piece* vq) {
                            const int j = k >> 2;
                            if ((k & 3) == 0 && k > 0 && 4 * (j + 1) < nb) {       // entering group j: fetch group j+1
                                if (j & 1) g0 = idx_group(j + 1); else g1 = idx_group(j + 1);
                            }
                            const int src = (j & 1) ? g1 : g0;
#pragma unroll
                            for (int i = 0; i < UN; ++i) u[i] = __shfl_sync(gmask, src, grp_base + (k & 3) * 4 + i);
#pragma unroll
                            for (int i = 0; i < UN; ++i) {
                                if (u[i] >= 0 && u[i] != v) {
                                    kq[i] = ld_piece_cg(kv_tab + (size_t)u[i] * 512 + sub * 16);
                                    vq[i] = ld_piece_cg(kv_tab + (size_t)u[i] * 512 + 256 + sub * 16);
                                }
                            }
                        };
                        auto consume = [&](const int* u, Piece* kq, Piece* vq) {
                            float sc[UN];
#pragma unroll
                            for (int i = 0; i < UN; ++i) {
                                if (u[i] == v) { kq[i] = k_own; vq[i] = v_own; }
                                float dot = (u[i] >= 0) ? Elem<true>::dot(qp, kq[i]) : 0.f;
#pragma unroll
                                for (int o = LPH / 2; o > 0; o >>= 1) dot += __shfl_xor_sync(gmask, dot, o);
                                sc[i] = (u[i] >= 0) ? dot * c : -INFINITY;
                            }
                            float m_new = m;
#pragma unroll
                            for (int i = 0; i < UN; ++i) m_new = fmaxf(m_new, sc[i]);
                            const float keep = fast_exp2(m - m_new);            // 0 for the first batch (m = -inf)
                            z *= keep;
#pragma unroll
                            for (int e = 0; e < 8; ++e) acc[e] *= keep;
#pragma unroll
                            for (int i = 0; i < UN; ++i) {
                                if (u[i] >= 0) {
                                    const float pw = fast_exp2(sc[i] - m_new);
                                    float vf[8];
                                    Elem<true>::unpack(vq[i], vf);
                                    z += pw;
#pragma unroll
                                    for (int e = 0; e < 8; ++e) acc[e] = fmaf(pw, vf[e], acc[e]);
                                }
                            }
                            m = m_new;
                        };
                        {
                            Piece kA[UN], vA[UN], kB[UN], vB[UN];
                            int uA[UN], uB[UN];
                            if (nb > 0) issue(0, uA, kA, vA);
                            for (int k = 0; k < nb; k += 2) {
                                if (k + 1 < nb) issue(k + 1, uB, kB, vB);
                                consume(uA, kA, vA);
                                if (k + 2 < nb) issue(k + 2, uA, kA, vA);
                                if (k + 1 < nb) consume(uB, kB, vB);
                            }
                        }
                        // merge the replicas' partial softmaxes into replica 0 (a replica that saw nothing has m = -inf)
                        float* mine = reinterpret_cast<float*>(base_ptr + kOffMerge) + (size_t)tid * kMergeRow;
                        mine[0] = m; mine[1] = z;
#pragma unroll
                        for (int e = 0; e < 8; ++e) mine[2 + e] = acc[e];
                        worker_sync();
                        if (part == 0) {
                            for (int q = 1; q < parts; ++q) {
                                const float* other = mine + (size_t)q * T_l * 16 * kMergeRow;
                                const float m2 = other[0], z2 = other[1];
                                if (m2 == -INFINITY) continue;
                                const float mm = fmaxf(m, m2);
                                const float w1 = fast_exp2(m - mm), w2 = fast_exp2(m2 - mm);
                                z = z * w1 + z2 * w2;
#pragma unroll
                                for (int e = 0; e < 8; ++e) acc[e] = acc[e] * w1 + other[2 + e] * w2;
                                m = mm;
                            }
                        } else {
#pragma unroll
                            for (int e = 0; e < 8; ++e) acc[e] = 0.f;           // a replica's row of the O tile is never used
                            z = 1.f;
                        }
                        if (cnt == 1 && part == 0) {
                            Elem<true>::unpack(v_own, acc);                     // softmax over one element: weight exactly 1
                        } else if (cnt > 1 && part == 0) {
                            const float inv = fast_rcp(z);
#pragma unroll
                            for (int e = 0; e < 8; ++e) acc[e] *= inv;
                        }
                    }
                    pad_nx = pad_of(v_nx);           // its node id has arrived by now; the entry is used by the next tile
                    {
                        Piece o = Elem<true>::pack(acc);
                        st_shared_v4(sO + operand_piece(slot, sub), o.w);
                        if (sub == 0) misc->node[slot] = (WIDE && slot / T_l != 0) ? -1 : v;   // replicas store nothing
                    }
                    worker_sync();

                    // ---- output projection for the 16 nodes by warp-level MMAs (m16n8k16): warp w computes output
                    // features 16w .. 16w+15 for all nodes; the result is in registers when the last one retires
                    // (the asynchronous tcgen05 path costs an order / commit / barrier round trip per product, which
                    // at N = 16 is longer than the product itself)
                    const bool pre_ok = pre_early || (want_pre && misc->pre_ok != 0);
                    if (pre_ok && !pre_early) xpre = load_input(v_pre);
                    if (paired && rows_out) {          // the partner has read the previous tile's rows out of sHp
                        if (!mbar_wait_from_cluster(smem_u32(&misc->pair_taken), ph_taken, p.poll_limit) && tid == 0) { give_up(p); misc->failed = 1; }
                        ph_taken ^= 1u;
                    }
                    {
                        float acc_o[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
                        for (int ks = 0; ks < 8; ++ks) {
                            uint32_t af[4], bf[4];
                            ldmatrix_x4(sO + operand_piece(a_row, 2 * ks + a_chunk), af);
                            ldmatrix_x4(sW + weight_piece(16 * warp + b_row, 2 * ks + b_chunk), bf);
                            mma_m16n8k16(acc_o[0], af, bf[0], bf[1]);
                            mma_m16n8k16(acc_o[1], af, bf[2], bf[3]);
                        }
                        // residual, rounding, new rows into shared memory in operand layout (two features per store)
#pragma unroll
                        for (int nt = 0; nt < 2; ++nt) {
                            const int f = 16 * warp + 8 * nt + 2 * mt;
#pragma unroll
                            for (int hrow = 0; hrow < 2; ++hrow) {
                                const int node = mg + 8 * hrow;
                                const uint32_t rb = p.residual ? ld_shared_b32(sHres_cur + (uint32_t)(node * 256 + f * 2)) : 0u;
                                const float lo = acc_o[nt][2 * hrow] + __uint_as_float(rb << 16);
                                const float hi = acc_o[nt][2 * hrow + 1] + __uint_as_float(rb & 0xffff0000u);
                                st_shared_b32(sHp + operand_offset(node, f), pack_bf16x2(lo, hi));
                            }
                        }
                    }
                    if (pre_ok) stage_input(buf ^ 1, xpre);
                    fence_proxy_async_smem();
                    worker_sync();

                    // ---- from the new rows, transposed on the tcgen05 path (issued by the ninth warp): this layer's
                    // K | V refresh; right behind it the next tile's Q | K | V, which runs while this tile's rows are
                    // stored and the level completes.  (Measured: for the 8-instruction W_o product the warp-level
                    // path wins, its fixed cost being nil; for these 16 instructions the asynchronous path does:
                    // a warp-level m16n8k16 occupies its sub-partition for about 32 clocks.)
                    // (as a block's attention stage there is no refresh here: the feed-forward stage does it, from the
                    // block's output rows)
                    if (tid == 0) {
                        if (!BLOCK) post(pre_ok ? kCmdKvThenQkv : kCmdKv, buf ^ 1);
                        else if (pre_ok) post(kCmdQkv, buf ^ 1);
                        // (paired: the rows stay on chip -- the partner reads them out of this CTA's shared memory)
                        if (paired) mbar_arrive_in_cluster(in_cta(smem_u32(&misc->pair_rows), 1));
                    }
                    rows_out = true;
                    const int node_v = misc->node[slot];
                    if (!paired) {
                        uint32_t w4[4];
                        ld_shared_v4(sHp + operand_piece(slot, sub), w4);
                        if (node_v >= 0) st_global_v4((char*)p.H + (size_t)node_v * p.ldh * 2 + sub * 16, w4);
                    }
                    if (!more_here) {
                        // While the product runs: ask L2 for the lines the coming levels' first loads will want (a
                        // prefetch has no destination register, so nothing ever waits for it).  Without this the
                        // index-chain loads and the neighbours' K | V rows of a large circuit come from DRAM, and
                        // that latency is on the level-to-level chain.
                        const int t3 = per_tile(lp4 - lp3, nctas);
                        const int r3 = bid * t3 + slot;
                        if (sub == 0 && slot < t3 && r3 < lp4 - lp3) prefetch_l2(p.level_nodes + lp3 + r3);   // node ids, level l+3
                        if (vB >= 0) {                                                            // level l+2's node
                            if (sub == 0) prefetch_l2(WIDE ? (const void*)(p.nbr_ptr + vB) : (const void*)(p.nbr_pad + (size_t)vB * W));
                            if ((sub & 1) == 0) prefetch_l2((const char*)p.H + (size_t)vB * p.ldh * 2 + sub * 16);
                        }
                        if (!WIDE && vC >= 0) {                                                   // level l+1's node
                            const int cnt_c = __shfl_sync(gmask, padC, grp_base);
#pragma unroll
                            for (int j = 1; j < MAXN; ++j) {
                                const int uj = __shfl_sync(gmask, padC, grp_base + j);
                                if (j < cnt_c) prefetch_l2(kv_tab + (size_t)uj * 512 + sub * 32);
                            }
                        }
                    }
                    if (!BLOCK) {
                    if (!mbar_wait_relaxed(bar2, ph2, p.poll_limit) && tid == 0) { give_up(p); misc->failed = 1; }
                    ph2 ^= 1u;
                    tc_fence_after();
                    accumulators_to_stage<2>(tmem + lane_base + (uint32_t)(kTile * kAccK2 + cg * 8), stage_frag);
                    tc_fence_before();
                    worker_sync();
                    if (node_v >= 0) {
                        const uint32_t row = sSt + (uint32_t)(slot * kStageRow);
                        uint32_t w4[4];
#pragma unroll
                        for (int h = 0; h < 2; ++h) {        // this layer's K | V row
                            ld_shared_v4(row + (uint32_t)((sub + 16 * h) * 16), w4);
                            st_global_v4((char*)p.KV[wl] + (size_t)node_v * 512 + (sub + 16 * h) * 16, w4);
                        }
                    }
                    }
                    worker_sync();    // the tile's shared buffers may be overwritten from here on
                    pro_ready = pre_ok;
                    if (pre_ok) buf ^= 1;
                }
                if (!alive) break;
                // ---- this CTA's part of (layer, level l) is in global memory: arrive on its counter (release)
                // (by a thread that does not poll: the release waits for the CTA's outstanding stores, and the pollers
                // should already be watching the next level's counters meanwhile)
                // (the attention CTA of a pair has handed its rows over on chip; nobody reads its counter)
                if (tid == 64 && !paired) red_release_add(my_arrive + l, 1);
            } else if (!pro_ready && l + 1 < p.n_levels && bid < tiles_next) {
                // ---- no tile in this level but one in the next: bring that tile up while there is nothing else to do
                if (tid == 32) {
                    bool go = true;
                    if (prev_arrive) go = wait_counter(prev_arrive + l + 1, prev_target(lp2 - lp1), p.abort_word, counter_limit);
                    if (!go && ld_acquire(p.abort_word) == 0) give_up(p);
                    misc->go2 = go ? 1 : 0;
                }
                worker_sync();
                if (!misc->go2) { alive = false; break; }
                stage_input(buf, load_input(vC));
                fence_proxy_async_smem();
                worker_sync();
                if (tid == 0) post(kCmdQkv, buf);
                pro_ready = true;
            }
            if (n_l > 0) {
                last_nonempty = l;
                last_participants = tiles < nctas ? tiles : nctas;
                if (BLOCK) {      // the feed-forward stage takes the same tiles
                    const int t1 = tiles_of(n_l, ctas_of(layer + 1));
                    last_participants_ffn = t1 < ctas_of(layer + 1) ? t1 : ctas_of(layer + 1);
                }
            }
            // rotate the pipeline by one level
            v0 = vC; pad0 = padC;
            vC = vB;
            lp0 = lp1; lp1 = lp2; lp2 = lp3; lp3 = lp4;
        }
        if (tid == 0) post(kCmdExit, 0);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc(tmem, kTmemCols);
    }
    if (paired) cluster_sync_all();        // neither CTA of a pair leaves while the other may still touch its shared memory
}

// ---------------------------------------------------------------------------------------------------
std::mutex g_mu;
int g_sm_count[64] = {};
int g_coop[64] = {};
bool g_dev_known[64] = {};

template <int LPH, int MAXN, bool BLOCK>
dg4_status launch_mode(const LevParams& p, int grid, cudaStream_t st) {
    auto kern = levelised_kernel<LPH, MAXN, BLOCK>;
    const int smem = p.block ? kSmemBytesBlock : kLaunchSmemBytes;
    DG4_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytesBlock));
    int per_sm = 0;
    DG4_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kThreads, smem));
    if (per_sm != 1) DG4_FAIL(DG4_ERR_CUDA, "the levelised kernel needs exactly one CTA per SM on this device (got %d)", per_sm);
    if (BLOCK && p.paired) {
        // clusters of two: CTA 2j runs an attention stage, CTA 2j+1 the feed-forward stage of the same tiles
        LevParams q = p;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(grid & ~1));
        cfg.blockDim = dim3(kThreads);
        cfg.dynamicSmemBytes = (size_t)smem;
        cfg.stream = st;
        cudaLaunchAttribute attrs[2];
        attrs[0].id = cudaLaunchAttributeCooperative;
        attrs[0].val.cooperative = 1;
        attrs[1].id = cudaLaunchAttributeClusterDimension;
        attrs[1].val.clusterDim.x = 2; attrs[1].val.clusterDim.y = 1; attrs[1].val.clusterDim.z = 1;
        cfg.attrs = attrs;
        cfg.numAttrs = 2;
        int clusters = 0;
        cudaError_t e = cudaOccupancyMaxActiveClusters(&clusters, kern, &cfg);
        if (e == cudaSuccess && clusters * 2 >= (grid & ~1)) {
            DG4_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, q));
            dg4i_count_launch();
            return DG4_OK;
        }
        cudaGetLastError();
        q.paired = 0;                      // not all pairs can be resident together: plain cooperative launch
        void* args2[] = {(void*)&q};
        DG4_CUDA_TRY(cudaLaunchCooperativeKernel((const void*)kern, dim3(grid), dim3(kThreads), args2, smem, st));
        dg4i_count_launch();
        return DG4_OK;
    }
    void* args[] = {(void*)&p};
    DG4_CUDA_TRY(cudaLaunchCooperativeKernel((const void*)kern, dim3(grid), dim3(kThreads), args, smem, st));
    dg4i_count_launch();
    return DG4_OK;
}

template <int LPH, int MAXN>
dg4_status launch(const LevParams& p, int grid, cudaStream_t st) {
    return p.block ? launch_mode<LPH, MAXN, true>(p, grid, st) : launch_mode<LPH, MAXN, false>(p, grid, st);
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

dg4_status dg4i_levelised_launch(const dg4_graph* g, const dg4_desc* desc, int n_layers,
                                 __nv_bfloat16* const* KV, __nv_bfloat16* H, int64_t ldh,
                                 const __nv_bfloat16* const* W_qkv, const __nv_bfloat16* const* W_o, int32_t* sync,
                                 int32_t* status, cudaStream_t st, const dg4i_block_tail* block) {
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
        p.KV[k] = KV[kk];
    }
    DG4_CUDA_TRY(cudaMemsetAsync(sync, 0, dg4i_levelised_sync_bytes(g, block ? 2 * n_layers : n_layers), st));
    p.H = H; p.ldh = ldh;
    p.nbr_pad = g->nbr_pad; p.nbr_ptr = g->nbr_ptr; p.nbr_idx = g->nbr_idx;
    p.level_ptr = g->level_ptr; p.level_nodes = g->level_nodes;
    p.n_levels = g->n_levels; p.n_layers = n_layers;
    p.residual = (desc->flags & DG4_FLAG_RESIDUAL) ? 1 : 0; p.scale = desc->scale;
    p.abort_word = sync; p.arrive = sync + 16; p.status = status; p.poll_limit = dg4i_poll_limit();
    p.block = 0; p.paired = 0; p.eps = 0.f;
    for (int k = 0; k < DG4I_MAX_LAYERS; ++k) {
        p.ln1_gamma[k] = p.ln1_beta[k] = p.b1[k] = p.b2[k] = p.ln2_gamma[k] = p.ln2_beta[k] = nullptr;
        p.W1[k] = p.W2[k] = nullptr;
    }
    if (block) {
        // two kinds of CTA per block, dealt round-robin: attention stage ("layer" 2k) and feed-forward stage (2k+1)
        if (g_sm_count[dev] < 2 * n_layers) DG4_FAIL(DG4_ERR_UNSUPPORTED, "fewer SMs than stages");
        p.block = 1; p.n_layers = 2 * n_layers; p.eps = block[0].eps; p.residual = 1;
        // both stages take the same tiles, so CTA 2j and CTA 2j+1 can be paired
        p.paired = ((g_sm_count[dev] & ~1) >= 2 * 2 * n_layers) ? 1 : 0;
        // (a profiler that cannot replay a cooperative launch in clusters gets the plain cooperative launch, whose
        // stages hand over through the level counters: on request, or when a tool has injected itself into the process)
        if (getenv("DG4_NO_CLUSTER_PAIRS") || getenv("NV_COMPUTE_PROFILER_PERFWORKS_DIR") || getenv("CUDA_INJECTION64_PATH"))
            p.paired = 0;
        for (int k = 0; k < n_layers; ++k) {
            p.ln1_gamma[k] = block[k].ln1_gamma; p.ln1_beta[k] = block[k].ln1_beta; p.W1[k] = block[k].W1; p.b1[k] = block[k].b1;
            p.W2[k] = block[k].W2; p.b2[k] = block[k].b2; p.ln2_gamma[k] = block[k].ln2_gamma; p.ln2_beta[k] = block[k].ln2_beta;
        }
    }
    const int grid = g_sm_count[dev];
    if (g->wide) return launch_heads<0>(desc->heads, p, grid, st);
    if (g->max_class <= 3) return launch_heads<3>(desc->heads, p, grid, st);
    return launch_heads<7>(desc->heads, p, grid, st);
}
