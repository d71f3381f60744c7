// The paper's own kernel model (Section 4.1.1, Listing 1) on sm_100a, kept as the baseline the
// other kernels of this library are measured against and as the subject of the layout study of
// Section 4.1.1: one thread group per block, one thread per output coordinate working along its row
// of the block, the block's slice of the input fetched by the whole group through the column index
// array, partial sums in several registers, the result stored through the row index array.
// Geometry as in Section 5: a size x size matrix with n_blocks identical square blocks, one per
// block-row.  fp32, one input vector, no bias, no activation.
//
// Three physical layouts of M_block (rightmost axis fastest):
//   BRC  block, row, column   (row-major within a block: a thread reads consecutive addresses)
//   BCR  block, column, row   (column-major within a block: a warp reads consecutive addresses)
//   CBR  column, block, row   (column c of all blocks next to each other)
#include <cuda_runtime.h>

#include <new>
#include <vector>

#include "pp.h"

struct pp_listing1 {
    int size = 0, n_blocks = 0, edge = 0, layout = 0;
    float* d_values = nullptr;
    int32_t* d_row_perm = nullptr;
    int32_t* d_col_perm = nullptr;
};

namespace {

template <int LAYOUT>
__device__ __forceinline__ size_t element(int blk, int row, int c, int E, int nb) {
    if (LAYOUT == PP_LAYOUT_BRC) return ((size_t)blk * E + row) * E + c;
    if (LAYOUT == PP_LAYOUT_BCR) return ((size_t)blk * E + c) * E + row;
    return ((size_t)c * nb + blk) * E + row;
}

template <int LAYOUT>
__global__ void listing1_kernel(const float* __restrict__ m_block, const int32_t* __restrict__ p_col,
                                const int32_t* __restrict__ p_row, const float* __restrict__ a_in,
                                float* __restrict__ a_out, int E, int nb) {
    extern __shared__ float a_local[];           // [E] input slice, then reused for the group store
    const int blk = blockIdx.x, row = threadIdx.x;
    a_local[row] = a_in[p_col[blk * E + row]];   // group fetch through the column index array
    __syncthreads();
    float acc[4] = {0.0f, 0.0f, 0.0f, 0.0f};      // several partial accumulators, reduced at the end
    int c = 0;
    for (; c + 4 <= E; c += 4) {
#pragma unroll
        for (int q = 0; q < 4; ++q) acc[q] = fmaf(m_block[element<LAYOUT>(blk, row, c + q, E, nb)], a_local[c + q], acc[q]);
    }
    for (; c < E; ++c) acc[0] = fmaf(m_block[element<LAYOUT>(blk, row, c, E, nb)], a_local[c], acc[0]);
    const float sum = (acc[0] + acc[1]) + (acc[2] + acc[3]);
    __syncthreads();
    a_local[row] = sum;
    __syncthreads();
    a_out[p_row[blk * E + row]] = a_local[row];   // group store through the row index array
}

bool is_perm(const int32_t* p, int n) {
    std::vector<unsigned char> seen((size_t)n, 0);
    for (int k = 0; k < n; ++k) {
        if (p[k] < 0 || p[k] >= n || seen[(size_t)p[k]]) return false;
        seen[(size_t)p[k]] = 1;
    }
    return true;
}

}  // namespace

extern "C" {

pp_status_t pp_listing1_pack(int size, int n_blocks, pp_layout_t layout, const float* block_values, float* out) {
    if (size <= 0 || n_blocks <= 0 || size % n_blocks != 0 || !block_values || !out) return PP_ERR_INVALID_ARG;
    if (layout != PP_LAYOUT_BRC && layout != PP_LAYOUT_BCR && layout != PP_LAYOUT_CBR) return PP_ERR_INVALID_ARG;
    const int E = size / n_blocks;
    for (int b = 0; b < n_blocks; ++b)
        for (int r = 0; r < E; ++r)
            for (int c = 0; c < E; ++c) {
                const float v = block_values[((size_t)b * E + r) * E + c];
                size_t dst;
                if (layout == PP_LAYOUT_BRC) dst = ((size_t)b * E + r) * E + c;
                else if (layout == PP_LAYOUT_BCR) dst = ((size_t)b * E + c) * E + r;
                else dst = ((size_t)c * n_blocks + b) * E + r;
                out[dst] = v;
            }
    return PP_OK;
}

pp_status_t pp_listing1_create(pp_listing1_t** out, int size, int n_blocks, pp_layout_t layout,
                               const int32_t* row_perm, const int32_t* col_perm, const float* block_values) {
    if (!out) return PP_ERR_INVALID_ARG;
    *out = nullptr;
    if (size <= 0 || n_blocks <= 0 || size % n_blocks != 0 || !row_perm || !col_perm || !block_values)
        return PP_ERR_INVALID_ARG;
    if (layout != PP_LAYOUT_BRC && layout != PP_LAYOUT_BCR && layout != PP_LAYOUT_CBR) return PP_ERR_INVALID_ARG;
    const int E = size / n_blocks;
    if (E > 1024) return PP_ERR_UNSUPPORTED;        // one thread per block row
    if (!is_perm(row_perm, size) || !is_perm(col_perm, size)) return PP_ERR_BAD_PERM;
    pp_listing1* h = new (std::nothrow) pp_listing1();
    if (!h) return PP_ERR_ALLOC;
    h->size = size; h->n_blocks = n_blocks; h->edge = E; h->layout = (int)layout;
    const size_t n = (size_t)n_blocks * E * E;
    std::vector<float> packed;
    try { packed.resize(n); } catch (const std::bad_alloc&) { delete h; return PP_ERR_ALLOC; }
    pp_listing1_pack(size, n_blocks, layout, block_values, packed.data());
    bool ok = cudaMalloc(&h->d_values, n * sizeof(float)) == cudaSuccess &&
              cudaMalloc(&h->d_row_perm, (size_t)size * 4) == cudaSuccess &&
              cudaMalloc(&h->d_col_perm, (size_t)size * 4) == cudaSuccess;
    ok = ok && cudaMemcpy(h->d_values, packed.data(), n * sizeof(float), cudaMemcpyHostToDevice) == cudaSuccess &&
         cudaMemcpy(h->d_row_perm, row_perm, (size_t)size * 4, cudaMemcpyHostToDevice) == cudaSuccess &&
         cudaMemcpy(h->d_col_perm, col_perm, (size_t)size * 4, cudaMemcpyHostToDevice) == cudaSuccess;
    if (!ok) {
        const cudaError_t e = cudaGetLastError();
        pp_listing1_destroy(h);
        return e == cudaErrorMemoryAllocation ? PP_ERR_ALLOC : PP_ERR_CUDA;
    }
    *out = h;
    return PP_OK;
}

pp_status_t pp_listing1_destroy(pp_listing1_t* h) {
    if (!h) return PP_OK;
    cudaFree(h->d_values);
    cudaFree(h->d_row_perm);
    cudaFree(h->d_col_perm);
    delete h;
    return PP_OK;
}

pp_status_t pp_listing1_forward(pp_listing1_t* h, const float* x, float* y, void* cuda_stream) {
    if (!h || !x || !y || x == y) return PP_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const size_t smem = (size_t)h->edge * sizeof(float);
    if (h->layout == PP_LAYOUT_BRC)
        listing1_kernel<PP_LAYOUT_BRC><<<h->n_blocks, h->edge, smem, s>>>(h->d_values, h->d_col_perm, h->d_row_perm, x, y, h->edge, h->n_blocks);
    else if (h->layout == PP_LAYOUT_BCR)
        listing1_kernel<PP_LAYOUT_BCR><<<h->n_blocks, h->edge, smem, s>>>(h->d_values, h->d_col_perm, h->d_row_perm, x, y, h->edge, h->n_blocks);
    else
        listing1_kernel<PP_LAYOUT_CBR><<<h->n_blocks, h->edge, smem, s>>>(h->d_values, h->d_col_perm, h->d_row_perm, x, y, h->edge, h->n_blocks);
    return cudaGetLastError() == cudaSuccess ? PP_OK : PP_ERR_CUDA;
}

}  // extern "C"
