// Graph prep: host validation + upload, then device kernels that build the neighbourhood CSR
// (cone_k(v), Sec. 3.2 / virtual edges of Sec. 3.5), the level buckets (levels as in Eq. 1) and the
// degree-class orderings.  All integer work; results are defined uniquely (see include/dg4.h), so they
// can be compared bit for bit.
//
// Device algorithms: per-node cone expansion in registers (at most 7 members), a reduce-then-scan
// exclusive prefix sum, atomics-based histograms, and a stable least-significant-digit radix pass
// (1024-element tiles, warp match + per-warp digit counters for the stable in-tile rank).

#include "dg4_internal.h"

#include <mutex>
#include <new>
#include <thread>
#include <vector>
#include <stdlib.h>
#include <string.h>

namespace {

constexpr int kTile = 1024;          // elements per block in the radix pass
constexpr int kScanThreads = 256;
constexpr int kScanItems = 8;
constexpr int kScanTile = kScanThreads * kScanItems;

// ------------------------------------------------------------------------------------------------
// cone_k(v) for k in {1, 2}: members other than v, ascending, duplicates collapsed.  Returns the count.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ int insert_sorted(int* a, int cnt, int x) {
    int pos = 0;
    while (pos < cnt && a[pos] < x) ++pos;
    if (pos < cnt && a[pos] == x) return cnt;
    for (int i = cnt; i > pos; --i) a[i] = a[i - 1];
    a[pos] = x;
    return cnt + 1;
}

__device__ __forceinline__ int cone_members(int v, const int32_t* __restrict__ row_ptr,
                                            const int32_t* __restrict__ col_idx, int hops, int* m /*[6]*/) {
    int cnt = 0;
    int b = row_ptr[v], e = row_ptr[v + 1];
    for (int i = b; i < e; ++i) {
        int u = col_idx[i];
        cnt = insert_sorted(m, cnt, u);
        if (hops >= 2) {
            int b2 = row_ptr[u], e2 = row_ptr[u + 1];
            for (int k = b2; k < e2; ++k) cnt = insert_sorted(m, cnt, col_idx[k]);
        }
    }
    return cnt;
}

__global__ void cone_count_kernel(int n, const int32_t* __restrict__ row_ptr, const int32_t* __restrict__ col_idx,
                                  int hops, int32_t* __restrict__ cnt_out /*[n+1]*/) {
    int v = blockIdx.x * blockDim.x + threadIdx.x;
    if (v == 0) cnt_out[n] = 0;
    if (v >= n) return;
    int m[6];
    cnt_out[v] = 1 + cone_members(v, row_ptr, col_idx, hops, m);
}

__global__ void cone_fill_kernel(int n, const int32_t* __restrict__ row_ptr, const int32_t* __restrict__ col_idx,
                                 int hops, const int32_t* __restrict__ nbr_ptr, int32_t* __restrict__ nbr_idx,
                                 int pad_width, int32_t* __restrict__ nbr_pad) {
    int v = blockIdx.x * blockDim.x + threadIdx.x;
    if (v >= n) return;
    int m[6];
    int c = cone_members(v, row_ptr, col_idx, hops, m);
    int o = nbr_ptr[v];
    nbr_idx[o] = v;
    for (int i = 0; i < c; ++i) nbr_idx[o + 1 + i] = m[i];
    // fixed-width copy for the attention kernels: [ |N(v)|, the members other than v ascending, v as filler ]
    int32_t* row = nbr_pad + (size_t)v * pad_width;
    row[0] = c + 1;
    for (int i = 1; i < pad_width; ++i) row[i] = (i - 1 < c) ? m[i - 1] : v;
}

// ------------------------------------------------------------------------------------------------
// exclusive prefix sum (int32), reduce-then-scan
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ int warp_inclusive_scan(int x) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int y = __shfl_up_sync(0xffffffffu, x, o);
        if ((threadIdx.x & 31) >= o) x += y;
    }
    return x;
}

// exclusive scan of one value per thread over the block; *total receives the block sum
template <int THREADS>
__device__ __forceinline__ int block_exclusive_scan(int x, int* total) {
    __shared__ int warp_tot[THREADS / 32];
    __shared__ int s_total;
    int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    int inc = warp_inclusive_scan(x);
    if (lane == 31) warp_tot[w] = inc;
    __syncthreads();
    if (w == 0) {
        int t = (lane < THREADS / 32) ? warp_tot[lane] : 0;
        int ti = warp_inclusive_scan(t);
        if (lane < THREADS / 32) warp_tot[lane] = ti - t;
        if (lane == 31) s_total = ti;
    }
    __syncthreads();
    int r = inc - x + warp_tot[w];
    *total = s_total;
    __syncthreads();
    return r;
}

__global__ void __launch_bounds__(kScanThreads) scan_reduce_kernel(const int32_t* __restrict__ in, int64_t n,
                                                                    int32_t* __restrict__ block_sums) {
    int64_t base = (int64_t)blockIdx.x * kScanTile + (int64_t)threadIdx.x * kScanItems;
    int s = 0;
#pragma unroll
    for (int i = 0; i < kScanItems; ++i)
        if (base + i < n) s += in[base + i];
    int total;
    block_exclusive_scan<kScanThreads>(s, &total);
    if (threadIdx.x == 0) block_sums[blockIdx.x] = total;
}

__global__ void __launch_bounds__(1024) scan_sums_kernel(int32_t* __restrict__ block_sums, int nb) {
    int carry = 0;
    for (int base = 0; base < nb; base += 1024) {
        int i = base + threadIdx.x;
        int x = (i < nb) ? block_sums[i] : 0;
        int total;
        int ex = block_exclusive_scan<1024>(x, &total);
        if (i < nb) block_sums[i] = carry + ex;
        carry += total;
    }
}

__global__ void __launch_bounds__(kScanThreads) scan_apply_kernel(const int32_t* in, int32_t* out, int64_t n,
                                                                   const int32_t* __restrict__ block_sums) {
    int64_t base = (int64_t)blockIdx.x * kScanTile + (int64_t)threadIdx.x * kScanItems;
    int x[kScanItems];
    int s = 0;
#pragma unroll
    for (int i = 0; i < kScanItems; ++i) {
        x[i] = (base + i < n) ? in[base + i] : 0;
        s += x[i];
    }
    int total;
    int ex = block_exclusive_scan<kScanThreads>(s, &total) + block_sums[blockIdx.x];
#pragma unroll
    for (int i = 0; i < kScanItems; ++i) {
        if (base + i < n) out[base + i] = ex;
        ex += x[i];
    }
}

dg4_status exclusive_scan(const int32_t* in, int32_t* out, int64_t n, int32_t* block_sums, cudaStream_t st) {
    if (n <= 0) return DG4_OK;
    int nb = (int)((n + kScanTile - 1) / kScanTile);
    scan_reduce_kernel<<<nb, kScanThreads, 0, st>>>(in, n, block_sums);
    dg4i_count_launch();
    scan_sums_kernel<<<1, 1024, 0, st>>>(block_sums, nb);
    dg4i_count_launch();
    scan_apply_kernel<<<nb, kScanThreads, 0, st>>>(in, out, n, block_sums);
    dg4i_count_launch();
    DG4_CUDA_TRY(cudaGetLastError());
    return DG4_OK;
}

// ------------------------------------------------------------------------------------------------
// histograms:  level_ptr counts, and (segment, class) counts
// ------------------------------------------------------------------------------------------------
__global__ void level_hist_kernel(int n, const int32_t* __restrict__ level, int32_t* __restrict__ hist) {
    int v = blockIdx.x * blockDim.x + threadIdx.x;
    int key = (v < n) ? level[v] : -1;
    // lanes of a warp that hold the same level add once, through their lowest lane
    unsigned peers = __match_any_sync(0xffffffffu, key);
    if (key >= 0 && (peers & ((1u << (threadIdx.x & 31)) - 1u)) == 0) atomicAdd(&hist[key], __popc(peers));
}

// segment of v: v / chunk (by_level == 0) or level[v].  A block of 256 consecutive ids lies inside one chunk
// (chunks are multiples of 1024), so in chunk mode the block first counts in shared memory and then issues at
// most max_class global atomics; in level mode the counters are spread over the levels and contention is low.
__global__ void __launch_bounds__(256) class_hist_kernel(int n, const int32_t* __restrict__ nbr_ptr,
                                                         const int32_t* __restrict__ level, int by_level, int chunk,
                                                         int max_class, int32_t* __restrict__ hist) {
    __shared__ int local[8];
    int v = blockIdx.x * blockDim.x + threadIdx.x;
    if (by_level) {
        if (v >= n) return;
        int cls = nbr_ptr[v + 1] - nbr_ptr[v];
        atomicAdd(&hist[(int64_t)level[v] * (max_class + 1) + (cls - 1)], 1);
        return;
    }
    if (threadIdx.x < 8) local[threadIdx.x] = 0;
    __syncthreads();
    if (v < n) atomicAdd(&local[nbr_ptr[v + 1] - nbr_ptr[v] - 1], 1);
    __syncthreads();
    if (threadIdx.x < max_class && local[threadIdx.x] > 0) {
        int seg = chunk > 0 ? (int)(((int64_t)blockIdx.x * blockDim.x) / chunk) : 0;
        atomicAdd(&hist[(int64_t)seg * (max_class + 1) + threadIdx.x], local[threadIdx.x]);
    }
}

// ------------------------------------------------------------------------------------------------
// one stable radix pass over a sequence of node ids
//   key of an element = (level[id] >> shift) & (RADIX-1)          (by_class == 0)
//                     = |N(id)| = nbr_ptr[id+1] - nbr_ptr[id]      (by_class == 1; RADIX = 8)
//   The sequence is cut into segments of bpc tiles; counters are laid out (segment, digit, tile) so one
//   exclusive scan of the whole counter array yields every element's destination.
//   SCATTER == false: count digits per tile.  SCATTER == true: place elements.
// ------------------------------------------------------------------------------------------------
template <int RADIX, bool SCATTER>
__global__ void __launch_bounds__(kTile) radix_pass_kernel(int n, const int32_t* __restrict__ src /*nullable*/,
                                                           const int32_t* __restrict__ level, int shift,
                                                           const int32_t* __restrict__ nbr_ptr, int by_class,
                                                           int bpc, int32_t* __restrict__ counters,
                                                           int32_t* __restrict__ dst) {
    __shared__ int wcount[kTile / 32][RADIX];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    for (int i = threadIdx.x; i < (kTile / 32) * RADIX; i += kTile) (&wcount[0][0])[i] = 0;
    __syncthreads();

    int i = blockIdx.x * kTile + threadIdx.x;
    bool valid = i < n;
    int id = 0, digit = RADIX;     // RADIX = "no element"
    if (valid) {
        id = src ? src[i] : i;
        digit = by_class ? (nbr_ptr[id + 1] - nbr_ptr[id]) : ((level[id] >> shift) & (RADIX - 1));
    }
    unsigned peers = __match_any_sync(0xffffffffu, digit);
    int rank_in_warp = __popc(peers & ((1u << lane) - 1u));
    if (valid && rank_in_warp == 0) wcount[w][digit] = __popc(peers);
    __syncthreads();

    int seg = blockIdx.x / bpc, tile_in_seg = blockIdx.x - seg * bpc;
    int64_t slot_base = (int64_t)seg * RADIX * bpc + tile_in_seg;
    if (!SCATTER) {
        for (int dgt = threadIdx.x; dgt < RADIX; dgt += kTile) {
            int tot = 0;
#pragma unroll 8
            for (int ww = 0; ww < kTile / 32; ++ww) tot += wcount[ww][dgt];
            counters[slot_base + (int64_t)dgt * bpc] = tot;
        }
    } else if (valid) {
        int before = 0;
        for (int ww = 0; ww < w; ++ww) before += wcount[ww][digit];
        dst[counters[slot_base + (int64_t)digit * bpc] + before + rank_in_warp] = id;
    }
}

template <int RADIX>
dg4_status radix_pass(dg4_graph* g, const int32_t* src, int shift, int by_class, int bpc, int n_seg,
                      int32_t* dst, cudaStream_t st) {
    int nb = (g->n + kTile - 1) / kTile;
    int64_t len = (int64_t)n_seg * RADIX * bpc;
    DG4_CUDA_TRY(cudaMemsetAsync(g->hist, 0, len * sizeof(int32_t), st));
    radix_pass_kernel<RADIX, false><<<nb, kTile, 0, st>>>(g->n, src, g->level, shift, g->nbr_ptr, by_class, bpc,
                                                          g->hist, nullptr);
    dg4i_count_launch();
    dg4_status s = exclusive_scan(g->hist, g->hist, len, g->block_sums, st);
    if (s != DG4_OK) return s;
    radix_pass_kernel<RADIX, true><<<nb, kTile, 0, st>>>(g->n, src, g->level, shift, g->nbr_ptr, by_class, bpc,
                                                         g->hist, dst);
    dg4i_count_launch();
    DG4_CUDA_TRY(cudaGetLastError());
    return DG4_OK;
}

int bits_for(int n_levels) {
    int b = 1;
    while ((1ll << b) < n_levels) ++b;
    return b;
}

// sort `first` (nullable = identity) by level, stable, into dst
dg4_status sort_by_level(dg4_graph* g, const int32_t* first, int32_t* dst, cudaStream_t st) {
    int nb = (g->n + kTile - 1) / kTile;
    int passes = (bits_for(g->n_levels) + 7) / 8;
    const int32_t* src = first;
    for (int p = 0; p < passes; ++p) {
        // ping-pong between the two scratch sequences; never write the buffer being read
        int32_t* out = (p == passes - 1) ? dst : ((src == g->seq_a) ? g->seq_b : g->seq_a);
        dg4_status s = radix_pass<256>(g, src, 8 * p, 0, nb, 1, out, st);
        if (s != DG4_OK) return s;
        src = out;
    }
    return DG4_OK;
}

}  // namespace

dg4_status dg4i_exclusive_scan(const int32_t* in, int32_t* out, int64_t n, int32_t* block_sums, cudaStream_t st) {
    return exclusive_scan(in, out, n, block_sums, st);
}

// ------------------------------------------------------------------------------------------------
// device pass (a2..a4).  first_time: stops after the neighbourhood sizes are known so that the caller can
// size nbr_idx; it is then called again with first_time == false.
// ------------------------------------------------------------------------------------------------
dg4_status dg4i_graph_device_pass(dg4_graph* g, cudaStream_t st, bool sizes_only) {
    const int n = g->n;
    const int tb = 256, nbk = (n + tb - 1) / tb;
    dg4_status s;

    if (!g->wide) {
        // neighbourhood sizes -> nbr_ptr
        cone_count_kernel<<<nbk, tb, 0, st>>>(n, g->row_ptr, g->col_idx, g->hops, g->nbr_ptr);
        dg4i_count_launch();
        if ((s = exclusive_scan(g->nbr_ptr, g->nbr_ptr, (int64_t)n + 1, g->block_sums, st)) != DG4_OK) return s;
        if (sizes_only) return DG4_OK;
        cone_fill_kernel<<<nbk, tb, 0, st>>>(n, g->row_ptr, g->col_idx, g->hops, g->nbr_ptr, g->nbr_idx, g->pad_width, g->nbr_pad);
        dg4i_count_launch();
    }

    // level buckets
    DG4_CUDA_TRY(cudaMemsetAsync(g->level_ptr, 0, ((size_t)g->n_levels + 1) * sizeof(int32_t), st));
    level_hist_kernel<<<nbk, tb, 0, st>>>(n, g->level, g->level_ptr);
    dg4i_count_launch();
    if ((s = exclusive_scan(g->level_ptr, g->level_ptr, (int64_t)g->n_levels + 1, g->block_sums, st)) != DG4_OK) return s;
    if ((s = sort_by_level(g, nullptr, g->level_nodes, st)) != DG4_OK) return s;

    if (g->wide) {            // wider cones: lists come from dg4i_build_wide_cones; no class orderings
        DG4_CUDA_TRY(cudaGetLastError());
        return DG4_OK;
    }

    // degree-class order inside id chunks
    const int mc1 = g->max_class + 1;
    int nb = (n + kTile - 1) / kTile;
    int bpc = g->perm_chunk > 0 ? g->perm_chunk / kTile : nb;
    DG4_CUDA_TRY(cudaMemsetAsync(g->class_ptr, 0, ((size_t)g->n_chunks * mc1 + 1) * sizeof(int32_t), st));
    class_hist_kernel<<<nbk, tb, 0, st>>>(n, g->nbr_ptr, g->level, 0, g->perm_chunk, g->max_class, g->class_ptr);
    dg4i_count_launch();
    if ((s = exclusive_scan(g->class_ptr, g->class_ptr, (int64_t)g->n_chunks * mc1 + 1, g->block_sums, st)) != DG4_OK) return s;
    if ((s = radix_pass<8>(g, nullptr, 0, 1, bpc, g->n_chunks, g->perm, st)) != DG4_OK) return s;

    // degree-class order inside level buckets: stable by class, then stable by level
    DG4_CUDA_TRY(cudaMemsetAsync(g->level_class_ptr, 0, ((size_t)g->n_levels * mc1 + 1) * sizeof(int32_t), st));
    class_hist_kernel<<<nbk, tb, 0, st>>>(n, g->nbr_ptr, g->level, 1, 0, g->max_class, g->level_class_ptr);
    dg4i_count_launch();
    if ((s = exclusive_scan(g->level_class_ptr, g->level_class_ptr, (int64_t)g->n_levels * mc1 + 1, g->block_sums, st)) != DG4_OK) return s;
    if ((s = radix_pass<8>(g, nullptr, 0, 1, nb, 1, g->seq_a, st)) != DG4_OK) return s;
    if ((s = sort_by_level(g, g->seq_a, g->level_perm, st)) != DG4_OK) return s;

    DG4_CUDA_TRY(cudaGetLastError());
    return DG4_OK;
}

// ------------------------------------------------------------------------------------------------
// public entry points
// ------------------------------------------------------------------------------------------------
namespace {

struct DeviceGuard {
    int prev = -1;
    bool ok = false;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) prev = -1;
        ok = cudaSetDevice(dev) == cudaSuccess;
    }
    ~DeviceGuard() {
        if (prev >= 0) cudaSetDevice(prev);
    }
};

// Frees the handle.  With `ordered` set, pooled device memory is released in the order of `st` (work enqueued
// there before may still use it) and nothing waits; otherwise every buffer is released with cudaFree, which
// waits for the device.
void free_graph(dg4_graph* g, bool ordered = false, cudaStream_t st = nullptr) {
    if (!g) return;
    int32_t* bufs[] = {g->nbr_pad, g->row_ptr, g->col_idx, g->level, g->nbr_ptr, g->nbr_idx, g->level_ptr, g->level_nodes,
                       g->perm, g->class_ptr, g->level_perm, g->level_class_ptr, g->seq_a, g->seq_b, g->hist,
                       g->block_sums, g->dev_status};
    for (int32_t* b : bufs) {
        if (!b) continue;
        if (ordered && g->pooled) cudaFreeAsync(b, st);
        else cudaFree(b);
    }
    free(g->h_level_ptr);
    delete g;
}

// The library's own memory pool of a device (handles of cones up to two hops allocate from it in stream order).
// Freed memory stays in the pool, so that creating a handle while kernels run does not have to ask the driver for
// new memory (which would wait for them).
std::mutex g_pool_mu;
cudaMemPool_t g_pool[64] = {};
dg4_status device_pool(int dev, cudaMemPool_t* out) {
    if (dev < 0 || dev >= 64) DG4_FAIL(DG4_ERR_UNSUPPORTED, "device ordinal %d is out of range", dev);
    std::lock_guard<std::mutex> lock(g_pool_mu);
    if (!g_pool[dev]) {
        cudaMemPoolProps props = {};
        props.allocType = cudaMemAllocationTypePinned;
        props.handleTypes = cudaMemHandleTypeNone;
        props.location.type = cudaMemLocationTypeDevice;
        props.location.id = dev;
        cudaMemPool_t pool = nullptr;
        DG4_CUDA_TRY(cudaMemPoolCreate(&pool, &props));
        uint64_t keep = UINT64_MAX;
        DG4_CUDA_TRY(cudaMemPoolSetAttribute(pool, cudaMemPoolAttrReleaseThreshold, &keep));
        g_pool[dev] = pool;
    }
    *out = g_pool[dev];
    return DG4_OK;
}

// Small device-to-host read-backs of graph creation.  A kernel writes the words into pinned host memory that the
// device has mapped, and the host copies them out after the stream has drained: a copy-engine transfer of the same
// few bytes would queue behind whatever large device-to-host copy the caller has in flight on another stream and
// hold graph creation up for its whole length.  One staging buffer per process, grown on demand, taken in turn.
__global__ void publish_words_kernel(const int32_t* __restrict__ src, int32_t* dst, int64_t count) {
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < count; i += (int64_t)gridDim.x * blockDim.x)
        dst[i] = src[i];
}
std::mutex g_stage_mu;
int32_t* g_stage = nullptr;
int64_t g_stage_words = 0;
dg4_status read_words(int32_t* host_dst, const int32_t* dev_src, int64_t count, cudaStream_t st, const char* what) {
    if (count <= 0) return DG4_OK;
    std::lock_guard<std::mutex> lock(g_stage_mu);
    if (g_stage_words < count) {
        if (g_stage) cudaFreeHost(g_stage);
        g_stage = nullptr;
        g_stage_words = 0;
        const int64_t words = 2 * count > 4096 ? 2 * count : 4096;
        void* mem = nullptr;
        cudaError_t e = cudaHostAlloc(&mem, (size_t)words * 4, cudaHostAllocPortable | cudaHostAllocMapped);
        if (e != cudaSuccess) { cudaGetLastError(); DG4_FAIL(DG4_ERR_ALLOC, "pinned staging buffer of %lld bytes: %s", (long long)words * 4, cudaGetErrorString(e)); }
        g_stage = (int32_t*)mem;
        g_stage_words = words;
    }
    int32_t* dev_view = nullptr;
    cudaError_t e = cudaHostGetDevicePointer((void**)&dev_view, g_stage, 0);
    if (e != cudaSuccess) { cudaGetLastError(); DG4_FAIL(DG4_ERR_CUDA, "%s failed: %s", what, cudaGetErrorString(e)); }
    const int blocks = (int)((count + 255) / 256 < 64 ? (count + 255) / 256 : 64);
    publish_words_kernel<<<blocks, 256, 0, st>>>(dev_src, dev_view, count);
    dg4i_count_launch();
    if ((e = cudaGetLastError()) != cudaSuccess || (e = cudaStreamSynchronize(st)) != cudaSuccess)
        DG4_FAIL(DG4_ERR_CUDA, "%s failed: %s", what, cudaGetErrorString(e));
    memcpy(host_dst, g_stage, (size_t)count * 4);
    return DG4_OK;
}

template <typename T>
dg4_status dalloc(T** p, int64_t count, cudaMemPool_t pool, cudaStream_t st) {
    if (count < 1) count = 1;
    const size_t bytes = (size_t)count * sizeof(T);
    cudaError_t e = pool ? cudaMallocFromPoolAsync((void**)p, bytes, pool, st) : cudaMalloc((void**)p, bytes);
    if (e != cudaSuccess) {
        *p = nullptr;
        cudaGetLastError();
        dg4_set_error("device allocation of %lld bytes failed: %s", (long long)bytes, cudaGetErrorString(e));
        return DG4_ERR_ALLOC;
    }
    return DG4_OK;
}

}  // namespace

extern "C" dg4_status dg4_graph_create(int32_t n_nodes, const int32_t* row_ptr, const int32_t* col_idx,
                                        const int32_t* level, int32_t hops, int32_t perm_chunk, int32_t device,
                                        dg4_graph** out) {
    if (!row_ptr || !level || !out) DG4_FAIL(DG4_ERR_INVALID_ARG, "null pointer argument");
    if (n_nodes < 1) DG4_FAIL(DG4_ERR_INVALID_ARG, "n_nodes must be >= 1 (got %d)", n_nodes);
    if (hops < 1 || hops > 8) DG4_FAIL(DG4_ERR_UNSUPPORTED, "hops must be between 1 and 8 (got %d)", hops);
    if (perm_chunk < 0 || (perm_chunk % kTile) != 0)
        DG4_FAIL(DG4_ERR_INVALID_ARG, "perm_chunk must be 0 or a positive multiple of %d (got %d)", kTile, perm_chunk);

    // ---- a1: validation on the host (node ranges checked by a few threads; the error of the lowest node wins)
    if (row_ptr[0] != 0) DG4_FAIL(DG4_ERR_NOT_SORTED, "row_ptr[0] must be 0");
    const int64_t n_edges = row_ptr[n_nodes];
    if (n_edges < 0) DG4_FAIL(DG4_ERR_NOT_SORTED, "row_ptr[n_nodes] is negative");
    if (n_edges > 0 && !col_idx) DG4_FAIL(DG4_ERR_INVALID_ARG, "col_idx is null but the graph has edges");
    struct Finding { dg4_status code = DG4_OK; int32_t node = 0; char msg[160] = ""; int32_t max_level = 0; };
    auto check_range = [&](int32_t v0, int32_t v1, Finding* f) {
        auto fail = [&](dg4_status c, int32_t v, const char* fmt, int a0, int a1, int a2, int a3) {
            f->code = c; f->node = v;
            snprintf(f->msg, sizeof(f->msg), fmt, a0, a1, a2, a3);
        };
        for (int32_t v = v0; v < v1; ++v) {
            const int32_t b = row_ptr[v], e = row_ptr[v + 1];
            if (e < b || b < 0 || e > n_edges) return fail(DG4_ERR_NOT_SORTED, v, "row_ptr is not non-decreasing within [0, %d] at node %d", (int)n_edges, v, 0, 0);
            if (e - b > 2) return fail(DG4_ERR_BAD_DEGREE, v, "node %d has %d fan-ins (an AIG node has at most 2)", v, e - b, 0, 0);
            if (level[v] < 0) return fail(DG4_ERR_BAD_LEVEL, v, "node %d has negative level %d", v, level[v], 0, 0);
            for (int32_t i = b; i < e; ++i) {
                const int32_t u = col_idx[i];
                if (u < 0 || u >= n_nodes) return fail(DG4_ERR_BAD_LEVEL, v, "edge %d: source id %d out of range", i, u, 0, 0);
                if (level[u] >= level[v])
                    return fail(DG4_ERR_BAD_LEVEL, v, "edge %d -> %d: level %d is not below level %d", u, v, level[u], level[v]);
            }
            if (level[v] > f->max_level) f->max_level = level[v];
        }
    };
    int n_thr = (int)std::thread::hardware_concurrency();
    if (n_thr > 16) n_thr = 16;
    if (n_thr < 1 || n_nodes < (1 << 18)) n_thr = 1;
    std::vector<Finding> found((size_t)n_thr);
    if (n_thr == 1) {
        check_range(0, n_nodes, &found[0]);
    } else {
        std::vector<std::thread> pool;
        const int64_t per = ((int64_t)n_nodes + n_thr - 1) / n_thr;
        for (int t = 0; t < n_thr; ++t) {
            const int64_t v0 = per * t, v1 = (v0 + per < n_nodes) ? v0 + per : n_nodes;
            if (v0 >= v1) continue;
            pool.emplace_back(check_range, (int32_t)v0, (int32_t)v1, &found[(size_t)t]);
        }
        for (auto& th : pool) th.join();
    }
    int32_t max_level = 0;
    for (const Finding& f : found) {              // ranges are in node order: the first finding is the lowest node
        if (f.code != DG4_OK) DG4_FAIL(f.code, "%s", f.msg);
        if (f.max_level > max_level) max_level = f.max_level;
    }
    if (max_level >= n_nodes) DG4_FAIL(DG4_ERR_BAD_LEVEL, "max level %d is not below the node count", max_level);

    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || device < 0 || device >= ndev) {
        cudaGetLastError();
        DG4_FAIL(DG4_ERR_CUDA, "CUDA device %d is not available (%d devices visible)", device, ndev);
    }
    DeviceGuard guard(device);
    if (!guard.ok) DG4_FAIL(DG4_ERR_CUDA, "cudaSetDevice(%d) failed", device);

    dg4_graph* g = new (std::nothrow) dg4_graph();
    if (!g) DG4_FAIL(DG4_ERR_ALLOC, "host allocation failed");
    g->device = device;
    g->n = n_nodes;
    g->e = n_edges;
    g->hops = hops;
    g->max_class = (1 << (hops + 1)) - 1;
    g->wide = hops > 2;
    g->pad_width = g->wide ? 0 : g->max_class + 1;   // 4 or 8 int32: 16 or 32 bytes per node
    g->n_levels = max_level + 1;
    g->perm_chunk = (perm_chunk >= n_nodes) ? 0 : perm_chunk;
    g->n_chunks = g->perm_chunk > 0 ? (n_nodes + g->perm_chunk - 1) / g->perm_chunk : 1;

    const int64_t n = n_nodes;
    const int64_t nb = (n + kTile - 1) / kTile;
    const int64_t bpc = g->perm_chunk > 0 ? g->perm_chunk / kTile : nb;
    const int64_t mc1 = g->wide ? 1 : g->max_class + 1;   // no class arrays for wider cones
    int64_t hist_len = 256 * nb;
    if (hist_len < g->n_chunks * 8 * bpc) hist_len = g->n_chunks * 8 * bpc;
    g->hist_len = hist_len;
    int64_t longest = hist_len;
    if (longest < n + 1) longest = n + 1;
    if (longest < (int64_t)g->n_levels * mc1 + 1) longest = (int64_t)g->n_levels * mc1 + 1;
    if (longest < (int64_t)g->n_chunks * mc1 + 1) longest = (int64_t)g->n_chunks * mc1 + 1;
    g->block_sums_len = (longest + kScanTile - 1) / kScanTile + 1;

    dg4_status s = DG4_OK;
    auto fail = [&](dg4_status code) { free_graph(g); return code; };
    // Uploads and the prep kernels run on a stream of their own that does not wait for (or hold up) the work the
    // caller has in flight on other streams; it is drained before the handle is returned.  Device memory comes
    // from the library's pool in the order of that stream (plain cudaMalloc for cones of more than two hops).
    struct PrepStream {
        cudaStream_t st = nullptr;
        ~PrepStream() { if (st) cudaStreamDestroy(st); }
    } prep;
    if (cudaStreamCreateWithFlags(&prep.st, cudaStreamNonBlocking) != cudaSuccess) { dg4_set_error("cudaStreamCreate failed"); return fail(DG4_ERR_CUDA); }
    const cudaStream_t st = prep.st;
    cudaMemPool_t pool = nullptr;
    if (!g->wide) {
        if ((s = device_pool(device, &pool)) != DG4_OK) return fail(s);
        g->pooled = true;
    }
#define TRY_ALLOC(ptr, cnt) if ((s = dalloc(&(ptr), (cnt), pool, st)) != DG4_OK) return fail(s)
    TRY_ALLOC(g->row_ptr, n + 1);
    TRY_ALLOC(g->col_idx, n_edges);
    TRY_ALLOC(g->level, n);
    TRY_ALLOC(g->nbr_ptr, n + 1);
    TRY_ALLOC(g->level_ptr, (int64_t)g->n_levels + 1);
    TRY_ALLOC(g->level_nodes, n);
    TRY_ALLOC(g->perm, n);
    TRY_ALLOC(g->class_ptr, (int64_t)g->n_chunks * mc1 + 1);
    TRY_ALLOC(g->level_perm, n);
    TRY_ALLOC(g->level_class_ptr, (int64_t)g->n_levels * mc1 + 1);
    TRY_ALLOC(g->seq_a, n);
    TRY_ALLOC(g->seq_b, n);
    TRY_ALLOC(g->hist, g->hist_len);
    TRY_ALLOC(g->block_sums, g->block_sums_len);
    TRY_ALLOC(g->dev_status, 1);
    if (cudaMemsetAsync(g->dev_status, 0, sizeof(int32_t), st) != cudaSuccess) { dg4_set_error("cudaMemset failed"); return fail(DG4_ERR_CUDA); }

    auto cuda_fail = [&](cudaError_t e, const char* what) {
        dg4_set_error("%s failed: %s", what, cudaGetErrorString(e));
        free_graph(g);
        return DG4_ERR_CUDA;
    };
    cudaError_t ce;
    if ((ce = cudaMemcpyAsync(g->row_ptr, row_ptr, (size_t)(n + 1) * 4, cudaMemcpyHostToDevice, st)) != cudaSuccess) return cuda_fail(ce, "upload of row_ptr");
    if (n_edges > 0 && (ce = cudaMemcpyAsync(g->col_idx, col_idx, (size_t)n_edges * 4, cudaMemcpyHostToDevice, st)) != cudaSuccess) return cuda_fail(ce, "upload of col_idx");
    if ((ce = cudaMemcpyAsync(g->level, level, (size_t)n * 4, cudaMemcpyHostToDevice, st)) != cudaSuccess) return cuda_fail(ce, "upload of level");

    // sizes first, so that nbr_idx can be allocated exactly
    if (g->wide) {
        if ((ce = cudaStreamSynchronize(st)) != cudaSuccess) return cuda_fail(ce, "upload");
        if ((s = dg4i_build_wide_cones(g)) != DG4_OK) return fail(s);
    } else {
        if ((s = dg4i_graph_device_pass(g, st, true)) != DG4_OK) return fail(s);
        int32_t total = 0;
        if ((s = read_words(&total, g->nbr_ptr + n, 1, st, "read of neighbourhood total")) != DG4_OK) return fail(s);
        g->n_nbr = total;
        TRY_ALLOC(g->nbr_idx, g->n_nbr);
        TRY_ALLOC(g->nbr_pad, n * g->pad_width);
    }
#undef TRY_ALLOC
    if ((s = dg4i_graph_device_pass(g, g->wide ? (cudaStream_t)0 : st, false)) != DG4_OK) return fail(s);

    g->h_level_ptr = (int32_t*)malloc(((size_t)g->n_levels + 1) * sizeof(int32_t));
    if (!g->h_level_ptr) { dg4_set_error("host allocation failed"); return fail(DG4_ERR_ALLOC); }
    if (g->wide && (ce = cudaDeviceSynchronize()) != cudaSuccess) return cuda_fail(ce, "graph prep");
    if ((s = read_words(g->h_level_ptr, g->level_ptr, (int64_t)g->n_levels + 1, st, "read of level_ptr")) != DG4_OK) return fail(s);
    *out = g;
    return DG4_OK;
}

extern "C" dg4_status dg4_graph_rebuild(dg4_graph* g, void* stream) {
    dg4_status dev_ok = dg4i_check_device(g);
    if (dev_ok != DG4_OK) return dev_ok;
    if (g->wide) DG4_FAIL(DG4_ERR_UNSUPPORTED, "rebuild is available for cones of at most two hops");
    return dg4i_graph_device_pass(g, (cudaStream_t)stream, false);
}

extern "C" dg4_status dg4_graph_destroy(dg4_graph* g) {
    if (!g) return DG4_OK;
    DeviceGuard guard(g->device);
    free_graph(g);
    return DG4_OK;
}

extern "C" dg4_status dg4_graph_destroy_async(dg4_graph* g, void* stream) {
    if (!g) return DG4_OK;
    DeviceGuard guard(g->device);
    free_graph(g, true, (cudaStream_t)stream);
    return DG4_OK;
}

extern "C" dg4_status dg4_memory_trim(int32_t device) {
    if (device < 0 || device >= 64) DG4_FAIL(DG4_ERR_INVALID_ARG, "device ordinal %d is out of range", device);
    cudaMemPool_t pool = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_pool_mu);
        pool = g_pool[device];
    }
    if (!pool) return DG4_OK;                 // nothing was ever allocated on this device
    DeviceGuard guard(device);
    DG4_CUDA_TRY(cudaDeviceSynchronize());
    DG4_CUDA_TRY(cudaMemPoolTrimTo(pool, 0));
    return DG4_OK;
}

extern "C" dg4_status dg4_graph_info(const dg4_graph* g, dg4_graph_info_t* out) {
    if (!g || !out) DG4_FAIL(DG4_ERR_INVALID_ARG, "null pointer argument");
    out->n_nodes = g->n;
    out->n_edges = g->e;
    out->n_nbr = g->n_nbr;
    out->n_levels = g->n_levels;
    out->max_class = g->max_class;
    out->hops = g->hops;
    out->perm_chunk = g->perm_chunk;
    out->n_chunks = g->n_chunks;
    out->device = g->device;
    return DG4_OK;
}

namespace {
const int32_t* array_of(const dg4_graph* g, dg4_array_id which, int64_t* len) {
    const int64_t mc1 = g->max_class + 1;
    switch (which) {
        case DG4_ARR_NBR_PTR: *len = (int64_t)g->n + 1; return g->nbr_ptr;
        case DG4_ARR_NBR_IDX: *len = g->n_nbr; return g->nbr_idx;
        case DG4_ARR_NBR_PAD: *len = g->wide ? 0 : (int64_t)g->n * g->pad_width; return g->wide ? nullptr : g->nbr_pad;
        case DG4_ARR_LEVEL_PTR: *len = (int64_t)g->n_levels + 1; return g->level_ptr;
        case DG4_ARR_LEVEL_NODES: *len = g->n; return g->level_nodes;
        case DG4_ARR_PERM: *len = g->wide ? 0 : g->n; return g->wide ? nullptr : g->perm;
        case DG4_ARR_CLASS_PTR: *len = g->wide ? 0 : g->n_chunks * mc1; return g->wide ? nullptr : g->class_ptr;
        case DG4_ARR_LEVEL_PERM: *len = g->wide ? 0 : g->n; return g->wide ? nullptr : g->level_perm;
        case DG4_ARR_LEVEL_CLASS_PTR: *len = g->wide ? 0 : g->n_levels * mc1; return g->wide ? nullptr : g->level_class_ptr;
    }
    *len = 0;
    return nullptr;
}
}  // namespace

extern "C" const int32_t* dg4_graph_device_array(const dg4_graph* g, dg4_array_id which) {
    if (!g) return nullptr;
    int64_t len;
    return array_of(g, which, &len);
}

extern "C" dg4_status dg4_graph_export(const dg4_graph* g, dg4_array_id which, int32_t* host_dst, int64_t capacity,
                                        int64_t* n_written) {
    if (!g) DG4_FAIL(DG4_ERR_INVALID_ARG, "null graph");
    int64_t len = 0;
    const int32_t* src = array_of(g, which, &len);
    if (!src) DG4_FAIL(which >= 0 && which <= DG4_ARR_NBR_PAD ? DG4_ERR_UNSUPPORTED : DG4_ERR_INVALID_ARG,
                       "array %d does not exist for this graph", (int)which);
    if (n_written) *n_written = len;
    if (!host_dst) return DG4_OK;
    if (capacity < len) DG4_FAIL(DG4_ERR_INVALID_ARG, "capacity %lld is below the array length %lld", (long long)capacity, (long long)len);
    DeviceGuard guard(g->device);
    DG4_CUDA_TRY(cudaDeviceSynchronize());
    DG4_CUDA_TRY(cudaMemcpy(host_dst, src, (size_t)len * 4, cudaMemcpyDeviceToHost));
    return DG4_OK;
}

extern "C" dg4_status dg4_graph_poll_status(const dg4_graph* g, int32_t* out) {
    if (!g || !out) DG4_FAIL(DG4_ERR_INVALID_ARG, "null pointer argument");
    DeviceGuard guard(g->device);
    DG4_CUDA_TRY(cudaDeviceSynchronize());
    DG4_CUDA_TRY(cudaMemcpy(out, g->dev_status, sizeof(int32_t), cudaMemcpyDeviceToHost));
    return DG4_OK;
}
