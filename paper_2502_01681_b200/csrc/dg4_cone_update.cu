// The updating strategy of Sec. 3.4 on top of Algorithm 1's partition, with the table of historical embeddings
// resident on the device (the paper keeps it on the host and moves rows with Push / Pull; a B200 holds the table
// of a 10M-gate circuit many times over).  Cones are encoded level group by level group (l = k, k + delta, ...),
// inside a group in mini-batches of `batch` consecutive cones.  Per mini-batch:
//   1. collect the sub-graph: the union S of the mini-batch's cones (the handle's lists for hops = k); one warp
//      per cone stamps its members and appends those seen for the first time;
//   2. build the sub-graph's attention lists in local numbering: a gate that an earlier mini-batch has updated is
//      frozen (it attends to itself only: its in-edges are removed); any other gate attends to itself and to
//      the members of its own cone that are present in S, in ascending id (so that the order of summation does
//      not depend on the order in which the gates were collected);
//   3. gather the gates' rows from the table (a gate never updated before still has its input row there);
//   4. run the layers on the sub-graph: QKV projection, fused attention over the local lists, output projection
//      with residual -- the library's own kernels on the mini-batch's buffers;
//   5. store the rows of the gates that were not frozen back into the table and mark every gate of S as updated.
// The memory needed does not grow with the circuit beyond three int32 per gate: the buffers are sized by the
// mini-batch (at most batch * (2^(k+1) - 1) gates).
// The host drives the loop and reads one number per mini-batch (the size of S) back from the device, so this
// call waits on its stream between mini-batches.

#include "dg4_internal.h"

#include <algorithm>
#include <vector>

namespace {

constexpr int kWarpsPerBlock = 8;

__global__ void __launch_bounds__(kWarpsPerBlock * 32)
collect_members_kernel(const int32_t* __restrict__ roots, int first, int count, const int32_t* __restrict__ cone_ptr,
                       const int32_t* __restrict__ cone_idx, int stamp_id, int32_t* stamp, int32_t* pos,
                       int32_t* members, int32_t* n_members) {
    const int w = (int)((blockIdx.x * blockDim.x + threadIdx.x) >> 5), lane = threadIdx.x & 31;
    if (w >= count) return;
    const int r = roots[first + w];
    for (int e = cone_ptr[r] + lane; e < cone_ptr[r + 1]; e += 32) {
        const int u = cone_idx[e];
        if (atomicExch(&stamp[u], stamp_id) != stamp_id) {      // first sighting of u in this mini-batch
            const int p = atomicAdd(n_members, 1);
            members[p] = u;
            pos[u] = p;
        }
    }
}

// sizes of the local lists (lptr[i] = size of gate i's list; lptr[m] = 0, ready for the exclusive scan)
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
list_size_kernel(int m, const int32_t* __restrict__ members, const int32_t* __restrict__ updated,
                 const int32_t* __restrict__ cone_ptr, const int32_t* __restrict__ cone_idx,
                 const int32_t* __restrict__ stamp, int stamp_id, int32_t* __restrict__ lptr) {
    const int i = (int)((blockIdx.x * blockDim.x + threadIdx.x) >> 5), lane = threadIdx.x & 31;
    if (i > m) return;
    if (i == m) { if (lane == 0) lptr[m] = 0; return; }
    const int v = members[i];
    int cnt = 0;
    if (!updated[v])
        for (int e = cone_ptr[v] + 1 + lane; e < cone_ptr[v + 1]; e += 32) cnt += (stamp[cone_idx[e]] == stamp_id);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
    if (lane == 0) lptr[i] = 1 + cnt;
}

// the lists themselves: the gate first, then its present cone members in ascending id, as local positions
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
list_fill_kernel(int m, const int32_t* __restrict__ members, const int32_t* __restrict__ updated,
                 const int32_t* __restrict__ cone_ptr, const int32_t* __restrict__ cone_idx,
                 const int32_t* __restrict__ stamp, int stamp_id, const int32_t* __restrict__ pos,
                 const int32_t* __restrict__ lptr, int32_t* __restrict__ lidx) {
    const int i = (int)((blockIdx.x * blockDim.x + threadIdx.x) >> 5), lane = threadIdx.x & 31;
    if (i >= m) return;
    const int v = members[i];
    int out = lptr[i];
    if (lane == 0) lidx[out] = i;
    out += 1;
    if (updated[v]) return;
    const int beg = cone_ptr[v] + 1, end = cone_ptr[v + 1];
    for (int base = beg; base < end; base += 32) {               // whole warp stays in the loop (ballots)
        const int e = base + lane;
        const int u = e < end ? cone_idx[e] : -1;
        const bool present = u >= 0 && stamp[u] == stamp_id;
        const unsigned mask = __ballot_sync(0xffffffffu, present);
        if (present) lidx[out + __popc(mask & ((1u << lane) - 1u))] = pos[u];
        out += __popc(mask);
    }
}

// rows of the table -> the mini-batch's buffer (16 lanes per row, 16 bytes per lane)
__global__ void __launch_bounds__(256)
gather_rows_kernel(int m, const int32_t* __restrict__ members, const __nv_bfloat16* __restrict__ table, int64_t ldh,
                   __nv_bfloat16* __restrict__ rows) {
    const int i = (int)((blockIdx.x * blockDim.x + threadIdx.x) >> 4), sub = threadIdx.x & 15;
    if (i >= m) return;
    const uint4 w = *reinterpret_cast<const uint4*>(table + (size_t)members[i] * ldh + sub * 8);
    *reinterpret_cast<uint4*>(rows + (size_t)i * 128 + sub * 8) = w;
}

// the buffer's rows of the gates that were not frozen -> the table; every gate of the sub-graph is marked
__global__ void __launch_bounds__(256)
store_rows_kernel(int m, const int32_t* __restrict__ members, int32_t* updated, int32_t* stored,
                  const __nv_bfloat16* __restrict__ rows, __nv_bfloat16* table, int64_t ldh) {
    const int i = (int)((blockIdx.x * blockDim.x + threadIdx.x) >> 4), sub = threadIdx.x & 15;
    if (i >= m) return;
    const int v = members[i];
    const bool frozen = updated[v] != 0;                          // read by all 16 lanes before lane 0 writes it
    __syncwarp();
    if (!frozen) {
        const uint4 w = *reinterpret_cast<const uint4*>(rows + (size_t)i * 128 + sub * 8);
        *reinterpret_cast<uint4*>(table + (size_t)v * ldh + sub * 8) = w;
    }
    if (sub == 0) {
        if (!frozen && stored) stored[v] += 1;
        updated[v] = 1;
    }
}

size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

struct Layout {
    int64_t m_max, cap;
    size_t roots, group_ptr, stamp, pos, updated, members, lptr, lidx, sums, count, rows, q, kv, o, total;
};

Layout layout_of(const dg4_graph* g, int batch) {
    Layout L;
    const int64_t maxc = std::min<int64_t>(g->max_class, g->n);
    L.m_max = std::min<int64_t>((int64_t)batch * maxc, g->n);
    L.cap = L.m_max * maxc;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t at = off; off = align256(off + bytes); return at; };
    L.roots = take((size_t)g->n * 4);
    L.group_ptr = take(((size_t)g->n_levels + 1) * 4);
    L.stamp = take((size_t)g->n * 4);
    L.pos = take((size_t)g->n * 4);
    L.updated = take((size_t)g->n * 4);
    L.members = take((size_t)L.m_max * 4);
    L.lptr = take(((size_t)L.m_max + 1) * 4);
    L.lidx = take((size_t)L.cap * 4);
    L.sums = take(((size_t)L.m_max / 256 + 64) * 4);
    L.count = take(256);
    L.rows = take((size_t)L.m_max * 256);
    L.q = take((size_t)L.m_max * 256);
    L.kv = take((size_t)L.m_max * 512);
    L.o = take((size_t)L.m_max * 256);
    L.total = off;
    return L;
}

dg4_status check_common(const dg4_graph* g, const dg4_desc* desc, int32_t delta, int32_t batch) {
    dg4_status s = dg4i_check_device(g);
    if (s != DG4_OK) return s;
    if ((s = dg4i_check_desc(desc, true)) != DG4_OK) return s;
    if (desc->heads > 16) DG4_FAIL(DG4_ERR_UNSUPPORTED, "heads = %d: must be a power of two up to 16", desc->heads);
    if (delta < 1) DG4_FAIL(DG4_ERR_INVALID_ARG, "delta must be at least 1 (got %d)", delta);
    if (batch < 1 || batch > 65536) DG4_FAIL(DG4_ERR_INVALID_ARG, "batch must be between 1 and 65536 cones (got %d)", batch);
    return DG4_OK;
}

}  // namespace

extern "C" size_t dg4_cone_update_workspace_bytes(const dg4_graph* g, const dg4_desc* desc, int32_t batch) {
    (void)desc;
    if (!g || batch < 1 || batch > 65536) return 0;
    return layout_of(g, batch).total;
}

extern "C" dg4_status dg4_cone_update_fwd(const dg4_graph* g, const dg4_desc* desc, void* H, int64_t ldh,
                                           int32_t n_layers, const void* const* W_qkv, const void* const* W_o,
                                           int32_t delta, int32_t batch, void* workspace, size_t workspace_bytes,
                                           int32_t* stored, int64_t* n_batches, void* stream) {
    dg4_status s = check_common(g, desc, delta, batch);
    if (s != DG4_OK) return s;
    if (n_layers < 1 || n_layers > 64) DG4_FAIL(DG4_ERR_UNSUPPORTED, "n_layers = %d: between 1 and 64 layers per call", n_layers);
    if (!W_qkv || !W_o) DG4_FAIL(DG4_ERR_INVALID_ARG, "null weight list");
    if ((s = dg4i_check_tensor("H", H, ldh, 2, 128)) != DG4_OK) return s;
    for (int j = 0; j < n_layers; ++j) {
        if ((s = dg4i_check_tensor("W_qkv[j]", W_qkv[j], 128, 2, 128)) != DG4_OK) return s;
        if ((s = dg4i_check_tensor("W_o[j]", W_o[j], 128, 2, 128)) != DG4_OK) return s;
    }
    if (!workspace) DG4_FAIL(DG4_ERR_INVALID_ARG, "workspace is null");
    if ((((uintptr_t)workspace) & 255u) != 0) DG4_FAIL(DG4_ERR_INVALID_ARG, "workspace is not 256-byte aligned");
    const Layout L = layout_of(g, batch);
    if (workspace_bytes < L.total)
        DG4_FAIL(DG4_ERR_INVALID_ARG, "workspace of %zu bytes is below the %zu bytes needed", workspace_bytes, L.total);
    cudaStream_t st = (cudaStream_t)stream;
    char* ws = (char*)workspace;
    int32_t* roots = (int32_t*)(ws + L.roots);
    int32_t* group_ptr = (int32_t*)(ws + L.group_ptr);
    int32_t* stamp = (int32_t*)(ws + L.stamp);
    int32_t* pos = (int32_t*)(ws + L.pos);
    int32_t* updated = (int32_t*)(ws + L.updated);
    int32_t* members = (int32_t*)(ws + L.members);
    int32_t* lptr = (int32_t*)(ws + L.lptr);
    int32_t* lidx = (int32_t*)(ws + L.lidx);
    int32_t* sums = (int32_t*)(ws + L.sums);
    int32_t* count = (int32_t*)(ws + L.count);
    __nv_bfloat16* rows = (__nv_bfloat16*)(ws + L.rows);
    __nv_bfloat16* q = (__nv_bfloat16*)(ws + L.q);
    __nv_bfloat16* kv = (__nv_bfloat16*)(ws + L.kv);
    __nv_bfloat16* o = (__nv_bfloat16*)(ws + L.o);

    // Algorithm 1: the roots, grouped by level (a graph-prep call: it synchronises the device)
    DG4_CUDA_TRY(cudaStreamSynchronize(st));
    int64_t n_roots = 0;
    if ((s = dg4_graph_partition(g, delta, roots, group_ptr, &n_roots)) != DG4_OK) return s;
    std::vector<int32_t> gp((size_t)g->n_levels + 1);
    DG4_CUDA_TRY(cudaMemcpy(gp.data(), group_ptr, gp.size() * 4, cudaMemcpyDeviceToHost));
    DG4_CUDA_TRY(cudaMemsetAsync(stamp, 0, (size_t)g->n * 4, st));
    DG4_CUDA_TRY(cudaMemsetAsync(updated, 0, (size_t)g->n * 4, st));
    if (stored) DG4_CUDA_TRY(cudaMemsetAsync(stored, 0, (size_t)g->n * 4, st));

    dg4_desc with_res = *desc;                 // the residual flag is honoured as given
    int64_t batches = 0;
    const int tpb = kWarpsPerBlock * 32;
    for (int l = 0; l < g->n_levels; ++l) {
        for (int b0 = gp[l]; b0 < gp[l + 1]; b0 += batch) {
            const int cones = std::min(batch, gp[l + 1] - b0);
            const int stamp_id = (int)(batches + 1);
            DG4_CUDA_TRY(cudaMemsetAsync(count, 0, 4, st));
            collect_members_kernel<<<(cones + kWarpsPerBlock - 1) / kWarpsPerBlock, tpb, 0, st>>>(
                roots, b0, cones, g->nbr_ptr, g->nbr_idx, stamp_id, stamp, pos, members, count);
            dg4i_count_launch();
            int32_t m = 0;
            DG4_CUDA_TRY(cudaMemcpyAsync(&m, count, 4, cudaMemcpyDeviceToHost, st));
            DG4_CUDA_TRY(cudaStreamSynchronize(st));
            if (m < 1 || m > L.m_max) DG4_FAIL(DG4_ERR_CUDA, "mini-batch %lld collected %d gates (capacity %lld)", (long long)batches, m, (long long)L.m_max);
            list_size_kernel<<<(m + 1 + kWarpsPerBlock - 1) / kWarpsPerBlock, tpb, 0, st>>>(m, members, updated, g->nbr_ptr, g->nbr_idx, stamp, stamp_id, lptr);
            dg4i_count_launch();
            if ((s = dg4i_exclusive_scan(lptr, lptr, (int64_t)m + 1, sums, st)) != DG4_OK) return s;
            list_fill_kernel<<<(m + kWarpsPerBlock - 1) / kWarpsPerBlock, tpb, 0, st>>>(m, members, updated, g->nbr_ptr, g->nbr_idx, stamp, stamp_id, pos, lptr, lidx);
            gather_rows_kernel<<<(m + 15) / 16, 256, 0, st>>>(m, members, (const __nv_bfloat16*)H, ldh, rows);
            dg4i_count_launch(2);
            for (int j = 0; j < n_layers; ++j) {
                dg4i_proj_args p;
                p.A = rows; p.lda = 128; p.W = (const __nv_bfloat16*)W_qkv[j]; p.n_out = 384;
                p.out[0] = q; p.ldo[0] = 128; p.out[1] = kv; p.ldo[1] = 256; p.out[2] = kv + 128; p.ldo[2] = 256;
                p.R = nullptr; p.ldr = 0; p.row_list = nullptr; p.first = 0; p.rows = m; p.status = g->dev_status;
                if ((s = dg4i_proj_launch(p, st)) != DG4_OK) return s;
                dg4i_attn_args a;
                a.Q = q; a.ldq = 128; a.K = kv; a.ldk = 256; a.V = kv + 128; a.ldv = 256; a.O = o; a.ldo = 128;
                a.nbr_pad = nullptr; a.node_list = nullptr; a.first = 0; a.count = m;
                a.heads = desc->heads; a.max_nbr = 8;          // CSR lists of any length: the warp-per-gate kernel
                a.dtype = DG4_BF16; a.scale = desc->scale;
                dg4i_attn_more more;
                more.nbr_ptr = lptr; more.nbr_idx = lidx;
                if ((s = dg4i_attn_launch(a, &more, st)) != DG4_OK) return s;
                dg4i_proj_args op;
                op.A = o; op.lda = 128; op.W = (const __nv_bfloat16*)W_o[j]; op.n_out = 128;
                op.out[0] = rows; op.ldo[0] = 128; op.out[1] = op.out[2] = nullptr; op.ldo[1] = op.ldo[2] = 0;
                op.R = (with_res.flags & DG4_FLAG_RESIDUAL) ? rows : nullptr; op.ldr = 128;
                op.row_list = nullptr; op.first = 0; op.rows = m; op.status = g->dev_status;
                if ((s = dg4i_proj_launch(op, st)) != DG4_OK) return s;
            }
            store_rows_kernel<<<(m + 15) / 16, 256, 0, st>>>(m, members, updated, stored, rows, (__nv_bfloat16*)H, ldh);
            dg4i_count_launch();
            ++batches;
        }
    }
    DG4_CUDA_TRY(cudaGetLastError());
    if (n_batches) *n_batches = batches;
    return DG4_OK;
}
