// Algorithm 1 (graph partition): which nodes' cones the partition collects.  Roots are the nodes on levels
// k, k + delta, ... plus the nodes without fan-out, grouped by level and ordered by id inside a level; the cone
// of a root is its neighbourhood list in the graph handle (created with hops = k).  Integer work: a fan-out
// mark per node, a flag per position of the (level, id) ordering, an exclusive scan and a stable compaction.

#include "dg4_internal.h"

namespace {

__global__ void mark_fanout_kernel(int64_t e, const int32_t* __restrict__ col_idx, int32_t* __restrict__ has_out) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < e) has_out[col_idx[i]] = 1;            // every writer stores the same value
}

__global__ void root_flag_kernel(int n, const int32_t* __restrict__ level_nodes, const int32_t* __restrict__ level,
                                 const int32_t* __restrict__ has_out, int k, int delta, int32_t* __restrict__ flag) {
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i == 0) flag[n] = 0;
    if (i >= n) return;
    const int v = level_nodes[i];
    const int lv = level[v];
    const bool on_stride = lv >= k && ((lv - k) % delta) == 0;
    flag[i] = (on_stride || !has_out[v]) ? 1 : 0;
}

__global__ void root_compact_kernel(int n, const int32_t* __restrict__ level_nodes, const int32_t* __restrict__ pos,
                                    int32_t* __restrict__ roots) {
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n && pos[i + 1] != pos[i]) roots[pos[i]] = level_nodes[i];
}

__global__ void group_ptr_kernel(int n_levels, const int32_t* __restrict__ level_ptr, const int32_t* __restrict__ pos,
                                 int32_t* __restrict__ group_ptr) {
    int l = blockIdx.x * blockDim.x + threadIdx.x;
    if (l <= n_levels) group_ptr[l] = pos[level_ptr[l]];
}

}  // namespace

extern "C" dg4_status dg4_graph_partition(const dg4_graph* g, int32_t delta, int32_t* roots, int32_t* group_ptr,
                                           int64_t* n_roots) {
    if (!g || !roots || !group_ptr || !n_roots) DG4_FAIL(DG4_ERR_INVALID_ARG, "null pointer argument");
    if (delta < 1) DG4_FAIL(DG4_ERR_INVALID_ARG, "delta must be at least 1 (got %d)", delta);
    int cur = -1;
    DG4_CUDA_TRY(cudaGetDevice(&cur));
    if (cur != g->device) DG4_FAIL(DG4_ERR_INVALID_ARG, "the graph lives on device %d but device %d is current", g->device, cur);
    const int n = g->n;
    int32_t *has_out = nullptr, *pos = nullptr;
    auto cleanup = [&]() { cudaFree(has_out); cudaFree(pos); };
    if (cudaMalloc(&has_out, (size_t)n * 4) != cudaSuccess || cudaMalloc(&pos, ((size_t)n + 1) * 4) != cudaSuccess) {
        cudaGetLastError();
        cleanup();
        DG4_FAIL(DG4_ERR_ALLOC, "device allocation of the partition scratch failed");
    }
    const int tb = 256;
    dg4_status s = DG4_OK;
    cudaError_t ce = cudaMemset(has_out, 0, (size_t)n * 4);
    if (ce == cudaSuccess && g->e > 0) {
        mark_fanout_kernel<<<(unsigned)((g->e + tb - 1) / tb), tb>>>(g->e, g->col_idx, has_out);
        dg4i_count_launch();
    }
    root_flag_kernel<<<(n + tb) / tb, tb>>>(n, g->level_nodes, g->level, has_out, g->hops, delta, pos);
    dg4i_count_launch();
    if (ce == cudaSuccess) s = dg4i_exclusive_scan(pos, pos, (int64_t)n + 1, g->block_sums, 0);
    if (ce == cudaSuccess && s == DG4_OK) {
        root_compact_kernel<<<(n + tb - 1) / tb, tb>>>(n, g->level_nodes, pos, roots);
        group_ptr_kernel<<<(g->n_levels + tb) / tb, tb>>>(g->n_levels, g->level_ptr, pos, group_ptr);
        dg4i_count_launch(2);
        int32_t total = 0;
        ce = cudaMemcpy(&total, pos + n, 4, cudaMemcpyDeviceToHost);
        if (ce == cudaSuccess) ce = cudaDeviceSynchronize();
        *n_roots = total;
    }
    cleanup();
    if (s != DG4_OK) return s;
    if (ce != cudaSuccess) DG4_FAIL(DG4_ERR_CUDA, "graph partition failed: %s", cudaGetErrorString(ce));
    return DG4_OK;
}
