// Layout study of Section 4.1.1 on sm_100a: plain fp32 kernels over the three physical layouts of M_block the
// paper compares, crossed with two ways of giving the work to threads.  They are the yardstick the library's
// own kernels are measured against and nothing else uses them.
//
// Geometry as in Section 5: a size x size matrix with n_blocks identical square blocks of edge E, block k on
// pivoted rows and columns [k E, (k+1) E).  One input vector, no bias, no activation.
//
// Layouts (rightmost axis fastest):
//   BRC  block, row, column   (row-major within a block)
//   BCR  block, column, row   (column-major within a block)
//   CBR  column, block, row   (column c of all blocks next to each other)
// Mappings:
//   rows per lane   a lane owns one output row and walks its columns; the 32 lanes of a warp are 32 consecutive
//                   rows, so a warp's load touches consecutive addresses when ROWS are contiguous (BCR, CBR);
//   lanes along K   a warp owns four output rows and its lanes stride over the columns; a warp's load touches
//                   consecutive addresses when COLUMNS are contiguous (BRC); one shuffle tree per row at the end.
// Both stage the block's slice of the input through the column index array into shared memory, 1024 columns at
// a time, keep their sums in registers and store straight through the row index array.
#include <cuda_runtime.h>

#include <new>
#include <vector>

#include "pp.h"

struct pp_layout_study {
    int size = 0, n_blocks = 0, edge = 0, layout = 0, mapping = 0;
    float* d_values = nullptr;
    int32_t* d_row_perm = nullptr;
    int32_t* d_col_perm = nullptr;
};

namespace {

constexpr int kChunk = 1024;      // columns of the input slice staged at a time
constexpr int kRowThreads = 128;  // rows-per-lane mapping: rows (threads) per CTA
constexpr int kKWarps = 8;        // lanes-along-K mapping: warps per CTA
constexpr int kKRows = 4;         // ... and rows per warp

template <int LAYOUT>
__device__ __forceinline__ size_t element(int blk, int row, int c, int E, int nb) {
    if (LAYOUT == PP_LAYOUT_BRC) return ((size_t)blk * E + row) * E + c;
    if (LAYOUT == PP_LAYOUT_BCR) return ((size_t)blk * E + c) * E + row;
    return ((size_t)c * nb + blk) * E + row;
}

// columns [c0, c0 + n) of block blk's input slice, gathered through the column index array
__device__ __forceinline__ void stage_slice(float* xs, const float* __restrict__ x, const int32_t* __restrict__ p_col,
                                            int blk, int E, int c0, int n) {
    __syncthreads();                                  // the previous chunk has been consumed
    for (int c = threadIdx.x; c < n; c += blockDim.x) xs[c] = x[p_col[blk * E + c0 + c]];
    __syncthreads();
}

template <int LAYOUT>
__global__ void __launch_bounds__(kRowThreads) rows_per_lane_kernel(const float* __restrict__ w, const int32_t* __restrict__ p_col,
                                                                    const int32_t* __restrict__ p_row, const float* __restrict__ x,
                                                                    float* __restrict__ y, int E, int nb, int ctas_per_block) {
    __shared__ float xs[kChunk];
    const int blk = blockIdx.x / ctas_per_block;
    const int row = (blockIdx.x % ctas_per_block) * kRowThreads + threadIdx.x;
    const bool live = row < E;
    float acc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
    for (int c0 = 0; c0 < E; c0 += kChunk) {
        const int n = min(kChunk, E - c0);
        stage_slice(xs, x, p_col, blk, E, c0, n);
        if (!live) continue;
        int c = 0;
        for (; c + 4 <= n; c += 4) {
#pragma unroll
            for (int q = 0; q < 4; ++q) acc[q] = fmaf(w[element<LAYOUT>(blk, row, c0 + c + q, E, nb)], xs[c + q], acc[q]);
        }
        for (; c < n; ++c) acc[0] = fmaf(w[element<LAYOUT>(blk, row, c0 + c, E, nb)], xs[c], acc[0]);
    }
    if (live) y[p_row[blk * E + row]] = (acc[0] + acc[1]) + (acc[2] + acc[3]);
}

template <int LAYOUT>
__global__ void __launch_bounds__(kKWarps * 32) lanes_along_k_kernel(const float* __restrict__ w, const int32_t* __restrict__ p_col,
                                                                     const int32_t* __restrict__ p_row, const float* __restrict__ x,
                                                                     float* __restrict__ y, int E, int nb, int ctas_per_block) {
    __shared__ float xs[kChunk];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int blk = blockIdx.x / ctas_per_block;
    const int row0 = ((blockIdx.x % ctas_per_block) * kKWarps + warp) * kKRows;
    float acc[kKRows];
#pragma unroll
    for (int r = 0; r < kKRows; ++r) acc[r] = 0.0f;
    for (int c0 = 0; c0 < E; c0 += kChunk) {
        const int n = min(kChunk, E - c0);
        stage_slice(xs, x, p_col, blk, E, c0, n);
        for (int c = lane; c < n; c += 32) {
            const float xv = xs[c];
#pragma unroll
            for (int r = 0; r < kKRows; ++r)
                if (row0 + r < E) acc[r] = fmaf(w[element<LAYOUT>(blk, row0 + r, c0 + c, E, nb)], xv, acc[r]);
        }
    }
#pragma unroll
    for (int r = 0; r < kKRows; ++r) {
        float v = acc[r];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
        if (lane == 0 && row0 + r < E) y[p_row[blk * E + row0 + r]] = v;
    }
}

bool is_perm(const int32_t* p, int n) {
    std::vector<unsigned char> seen((size_t)n, 0);
    for (int k = 0; k < n; ++k) {
        if (p[k] < 0 || p[k] >= n || seen[(size_t)p[k]]) return false;
        seen[(size_t)p[k]] = 1;
    }
    return true;
}

bool known(pp_layout_t layout, pp_mapping_t mapping) {
    return (layout == PP_LAYOUT_BRC || layout == PP_LAYOUT_BCR || layout == PP_LAYOUT_CBR) &&
           (mapping == PP_MAP_ROWS_PER_LANE || mapping == PP_MAP_LANES_ALONG_K);
}

template <int LAYOUT>
cudaError_t launch(const pp_layout_study* h, const float* x, float* y, cudaStream_t s) {
    if (h->mapping == PP_MAP_ROWS_PER_LANE) {
        const int per_block = (h->edge + kRowThreads - 1) / kRowThreads;
        rows_per_lane_kernel<LAYOUT><<<h->n_blocks * per_block, kRowThreads, 0, s>>>(h->d_values, h->d_col_perm, h->d_row_perm, x, y,
                                                                                    h->edge, h->n_blocks, per_block);
    } else {
        const int rows_per_cta = kKWarps * kKRows;
        const int per_block = (h->edge + rows_per_cta - 1) / rows_per_cta;
        lanes_along_k_kernel<LAYOUT><<<h->n_blocks * per_block, kKWarps * 32, 0, s>>>(h->d_values, h->d_col_perm, h->d_row_perm, x, y,
                                                                                     h->edge, h->n_blocks, per_block);
    }
    return cudaGetLastError();
}

}  // namespace

extern "C" {

pp_status_t pp_layout_pack(int size, int n_blocks, pp_layout_t layout, const float* block_values, float* out) {
    if (size <= 0 || n_blocks <= 0 || size % n_blocks != 0 || !block_values || !out) return PP_ERR_INVALID_ARG;
    if (!known(layout, PP_MAP_ROWS_PER_LANE)) return PP_ERR_INVALID_ARG;
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

pp_status_t pp_layout_create(pp_layout_study_t** out, int size, int n_blocks, pp_layout_t layout, pp_mapping_t mapping,
                             const int32_t* row_perm, const int32_t* col_perm, const float* block_values) {
    if (!out) return PP_ERR_INVALID_ARG;
    *out = nullptr;
    if (size <= 0 || n_blocks <= 0 || size % n_blocks != 0 || !row_perm || !col_perm || !block_values)
        return PP_ERR_INVALID_ARG;
    if (!known(layout, mapping)) return PP_ERR_INVALID_ARG;
    const int E = size / n_blocks;
    if (!is_perm(row_perm, size) || !is_perm(col_perm, size)) return PP_ERR_BAD_PERM;
    pp_layout_study* h = new (std::nothrow) pp_layout_study();
    if (!h) return PP_ERR_ALLOC;
    h->size = size; h->n_blocks = n_blocks; h->edge = E; h->layout = (int)layout; h->mapping = (int)mapping;
    const size_t n = (size_t)n_blocks * E * E;
    std::vector<float> packed;
    try { packed.resize(n); } catch (const std::bad_alloc&) { delete h; return PP_ERR_ALLOC; }
    pp_layout_pack(size, n_blocks, layout, block_values, packed.data());
    bool ok = cudaMalloc(&h->d_values, n * sizeof(float)) == cudaSuccess &&
              cudaMalloc(&h->d_row_perm, (size_t)size * 4) == cudaSuccess &&
              cudaMalloc(&h->d_col_perm, (size_t)size * 4) == cudaSuccess;
    ok = ok && cudaMemcpy(h->d_values, packed.data(), n * sizeof(float), cudaMemcpyHostToDevice) == cudaSuccess &&
         cudaMemcpy(h->d_row_perm, row_perm, (size_t)size * 4, cudaMemcpyHostToDevice) == cudaSuccess &&
         cudaMemcpy(h->d_col_perm, col_perm, (size_t)size * 4, cudaMemcpyHostToDevice) == cudaSuccess;
    if (!ok) {
        const cudaError_t e = cudaGetLastError();
        pp_layout_destroy(h);
        return e == cudaErrorMemoryAllocation ? PP_ERR_ALLOC : PP_ERR_CUDA;
    }
    *out = h;
    return PP_OK;
}

pp_status_t pp_layout_destroy(pp_layout_study_t* h) {
    if (!h) return PP_OK;
    cudaFree(h->d_values);
    cudaFree(h->d_row_perm);
    cudaFree(h->d_col_perm);
    delete h;
    return PP_OK;
}

pp_status_t pp_layout_forward(pp_layout_study_t* h, const float* x, float* y, void* cuda_stream) {
    if (!h || !x || !y || x == y) return PP_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t e;
    if (h->layout == PP_LAYOUT_BRC) e = launch<PP_LAYOUT_BRC>(h, x, y, s);
    else if (h->layout == PP_LAYOUT_BCR) e = launch<PP_LAYOUT_BCR>(h, x, y, s);
    else e = launch<PP_LAYOUT_CBR>(h, x, y, s);
    return e == cudaSuccess ? PP_OK : PP_ERR_CUDA;
}

}  // extern "C"
