// Neighbourhood lists for wider cones, cone_k(v) with k = 3 .. 8 (Sec. 3.2; the paper's own setting is k = 8,
// at most 2^(k+1) - 1 = 511 members).  Built by k doubling passes over sorted duplicate-free lists:
//     L_1(v) = fan-ins of v,      L_j(v) = fan-ins(v)  U  L_{j-1}(a)  U  L_{j-1}(b)      (a, b the fan-ins of v)
// Each pass is a count kernel, an exclusive scan and a fill kernel (a three-way merge per node); the last pass
// writes the final CSR directly: v first, then L_k(v) ascending.

#include "dg4_internal.h"

namespace {

struct Lists { const int32_t* ptr; const int32_t* idx; };   // ptr == nullptr: every list is empty

// Merges fan-ins(v), L(a), L(b) in ascending order without duplicates.  WRITE: stores to out; returns the count.
template <bool WRITE>
__device__ __forceinline__ int merge_node(int v, const int32_t* __restrict__ row_ptr, const int32_t* __restrict__ col_idx,
                                          Lists prev, int32_t* out) {
    int c[2], nc = 0;
    const int b0 = row_ptr[v], e0 = row_ptr[v + 1];
    for (int i = b0; i < e0; ++i) {
        int u = col_idx[i];
        if (nc == 0 || c[0] != u) c[nc++] = u;
    }
    if (nc == 2 && c[0] > c[1]) { int t = c[0]; c[0] = c[1]; c[1] = t; }
    int pa = 0, ea = 0, pb = 0, eb = 0;
    if (prev.ptr) {
        if (nc > 0) { pa = prev.ptr[c[0]]; ea = prev.ptr[c[0] + 1]; }
        if (nc > 1) { pb = prev.ptr[c[1]]; eb = prev.ptr[c[1] + 1]; }
    }
    int pc = 0, n_out = 0, last = -1;
    const int kBig = 0x7fffffff;
    while (true) {
        const int xa = pa < ea ? prev.idx[pa] : kBig;
        const int xb = pb < eb ? prev.idx[pb] : kBig;
        const int xc = pc < nc ? c[pc] : kBig;
        int x = xa < xb ? xa : xb;
        x = x < xc ? x : xc;
        if (x == kBig) break;
        if (xa == x) ++pa;
        if (xb == x) ++pb;
        if (xc == x) ++pc;
        if (x != last) {
            if (WRITE) out[n_out] = x;
            ++n_out;
            last = x;
        }
    }
    return n_out;
}

__global__ void wide_count_kernel(int n, const int32_t* __restrict__ row_ptr, const int32_t* __restrict__ col_idx,
                                  Lists prev, int extra, int32_t* __restrict__ cnt /*[n+1]*/,
                                  unsigned long long* __restrict__ total) {
    int v = blockIdx.x * blockDim.x + threadIdx.x;
    if (v == 0) cnt[n] = 0;
    if (v >= n) return;
    int c = merge_node<false>(v, row_ptr, col_idx, prev, nullptr) + extra;
    cnt[v] = c;
    atomicAdd(total, (unsigned long long)c);
}

__global__ void wide_fill_kernel(int n, const int32_t* __restrict__ row_ptr, const int32_t* __restrict__ col_idx,
                                 Lists prev, int with_self, const int32_t* __restrict__ out_ptr,
                                 int32_t* __restrict__ out_idx) {
    int v = blockIdx.x * blockDim.x + threadIdx.x;
    if (v >= n) return;
    int32_t* dst = out_idx + out_ptr[v];
    if (with_self) *dst++ = v;
    merge_node<true>(v, row_ptr, col_idx, prev, dst);
}

}  // namespace

// Fills g->nbr_ptr and allocates + fills g->nbr_idx (sets g->n_nbr).  Synchronises; for dg4_graph_create only.
dg4_status dg4i_build_wide_cones(dg4_graph* g) {
    const int n = g->n;
    const int tb = 128, nbk = (n + tb - 1) / tb;
    unsigned long long* d_total = nullptr;
    int32_t *ptr_a = nullptr, *idx_a = nullptr, *ptr_b = nullptr, *idx_b = nullptr;
    dg4_status result = DG4_OK;
    auto cleanup = [&]() {
        cudaFree(d_total); cudaFree(ptr_a); cudaFree(idx_a); cudaFree(ptr_b); cudaFree(idx_b);
    };
#define WIDE_TRY(expr)                                                                            \
    do {                                                                                          \
        cudaError_t _e = (expr);                                                                  \
        if (_e != cudaSuccess) {                                                                  \
            dg4_set_error("%s failed: %s", #expr, cudaGetErrorString(_e));                        \
            cleanup();                                                                            \
            return _e == cudaErrorMemoryAllocation ? DG4_ERR_ALLOC : DG4_ERR_CUDA;                \
        }                                                                                         \
    } while (0)
    WIDE_TRY(cudaMalloc(&d_total, sizeof(unsigned long long)));
    WIDE_TRY(cudaMalloc(&ptr_a, ((size_t)n + 1) * 4));
    WIDE_TRY(cudaMalloc(&ptr_b, ((size_t)n + 1) * 4));
    Lists prev{nullptr, nullptr};
    for (int j = 1; j <= g->hops; ++j) {
        const bool last = j == g->hops;
        int32_t* out_ptr = last ? g->nbr_ptr : ((j & 1) ? ptr_a : ptr_b);
        WIDE_TRY(cudaMemset(d_total, 0, sizeof(unsigned long long)));
        wide_count_kernel<<<nbk, tb>>>(n, g->row_ptr, g->col_idx, prev, last ? 1 : 0, out_ptr, d_total);
        dg4i_count_launch();
        unsigned long long total = 0;
        WIDE_TRY(cudaMemcpy(&total, d_total, sizeof(total), cudaMemcpyDeviceToHost));
        if (total > 0x7fffffffull) {
            cleanup();
            DG4_FAIL(DG4_ERR_UNSUPPORTED, "the %d-hop neighbourhood lists hold %llu entries; the limit is 2^31 - 1", j, total);
        }
        if ((result = dg4i_exclusive_scan(out_ptr, out_ptr, (int64_t)n + 1, g->block_sums, 0)) != DG4_OK) { cleanup(); return result; }
        int32_t* out_idx = nullptr;
        WIDE_TRY(cudaMalloc(&out_idx, (size_t)(total > 0 ? total : 1) * 4));
        wide_fill_kernel<<<nbk, tb>>>(n, g->row_ptr, g->col_idx, prev, last ? 1 : 0, out_ptr, out_idx);
        dg4i_count_launch();
        WIDE_TRY(cudaDeviceSynchronize());
        if (last) {
            g->nbr_idx = out_idx;
            g->n_nbr = (int64_t)total;
        } else {
            int32_t*& slot = (j & 1) ? idx_a : idx_b;
            cudaFree(slot);                       // the list of two passes ago
            slot = out_idx;
            prev = Lists{out_ptr, out_idx};
        }
    }
#undef WIDE_TRY
    cleanup();
    return DG4_OK;
}
