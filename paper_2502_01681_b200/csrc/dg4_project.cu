// Dense projections of the layer: Y = A * W^T with K = 128, bf16 operands, fp32 accumulation, one rounding
// to bf16 per stored element.  Used for [Q|K|V] = X * W_qkv^T, H' = O * W_o^T (+ residual) and, in levelised
// mode, for refreshing the K|V rows of a finished level.
//
// First, plain CUDA-core version: 16 rows per block staged in shared memory, one output column per thread
// and 128-column block.  Correct for any row list; the tensor-core kernel replaces it.

#include "dg4_internal.h"

namespace {

constexpr int kRows = 16;

__global__ void __launch_bounds__(128) proj_simple_kernel(dg4i_proj_args a) {
    __shared__ float xs[kRows][128];
    __shared__ int rid[kRows];
    const int r0 = blockIdx.x * kRows;
    if (threadIdx.x < kRows) {
        int r = r0 + threadIdx.x;
        rid[threadIdx.x] = (r < a.rows) ? (a.row_list ? a.row_list[a.first + r] : a.first + r) : -1;
    }
    __syncthreads();
    for (int i = threadIdx.x; i < kRows * 128; i += 128) {
        int r = i >> 7, c = i & 127;
        xs[r][c] = rid[r] >= 0 ? __bfloat162float(a.A[(size_t)rid[r] * a.lda + c]) : 0.f;
    }
    __syncthreads();
    for (int c = threadIdx.x; c < a.n_out; c += 128) {
        float acc[kRows];
#pragma unroll
        for (int r = 0; r < kRows; ++r) acc[r] = 0.f;
        const __nv_bfloat16* w = a.W + (size_t)c * 128;
        for (int k = 0; k < 128; ++k) {
            float wk = __bfloat162float(w[k]);
#pragma unroll
            for (int r = 0; r < kRows; ++r) acc[r] = fmaf(xs[r][k], wk, acc[r]);
        }
        const int blk = c >> 7, cc = c & 127;
#pragma unroll
        for (int r = 0; r < kRows; ++r) {
            if (rid[r] < 0) continue;
            float y = acc[r];
            if (blk == 0 && a.R) y += __bfloat162float(a.R[(size_t)rid[r] * a.ldr + cc]);
            a.out[blk][(size_t)rid[r] * a.ldo[blk] + cc] = __float2bfloat16_rn(y);
        }
    }
}

}  // namespace

dg4_status dg4i_proj_launch(const dg4i_proj_args& a, cudaStream_t st) {
    if (a.rows <= 0) return DG4_OK;
    if (a.n_out != 128 && a.n_out != 256 && a.n_out != 384)
        DG4_FAIL(DG4_ERR_UNSUPPORTED, "projection width %d is not supported", a.n_out);
    unsigned blocks = (unsigned)((a.rows + kRows - 1) / kRows);
    proj_simple_kernel<<<blocks, 128, 0, st>>>(a);
    dg4i_count_launch();
    DG4_CUDA_TRY(cudaGetLastError());
    return DG4_OK;
}
