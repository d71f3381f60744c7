// Launch interface of the streaming block-sparse matrix-vector kernels.
#pragma once
#include <cuda_runtime.h>

#include "pp_internal.h"

namespace pp {

enum OutMode : int {
    OUT_SCATTER_F32 = 0,   // y[b][scatter_idx[i]] = v   (original row order, Listing 1 step 9)
    OUT_PIVOTED_F32 = 1,   // y[b][i] = v                (pivoted order, feeds a folded next layer)
    OUT_PIVOTED_F16 = 2,   // same, rounded to nearest-even binary16
    OUT_SCATTER_F16 = 3    // y[b][scatter_idx[i]] = v rounded to binary16 (chain: the consumer's pivoted column order)
};

struct GemvArgs {
    const void* values;          // fragment-ordered tile values
    const WorkItem* items;
    const int32_t* tile_col;
    const int32_t* gather_idx;   // pivoted column -> index into x, -1 = reads 0; NULL = identity
    const int32_t* scatter_idx;  // pivoted row -> original row, -1 = padding
    const float* bias_piv;
    const void* x;               // [batch][ldx]
    void* y;                     // [batch][ldy]
    float* partials;             // [n_slots][B][kMaxGroupBatch]
    int* counters;               // [Mb], zero between launches
    int ldx, ldy;
    int x_limit;                 // with gather_idx == NULL: columns >= x_limit read 0
    int batch;                   // columns in this launch (<= group limit of the kernel)
    int act;
    int out_mode;
    int xs_stride;               // shared-memory row stride of the staged x, in elements
};

// Enqueue one launch over n_items work items.  batch <= 32 (fp16) or 8 (fp32).
cudaError_t launch_gemv(pp_dtype_t dt, int B, const GemvArgs& a, int n_items, int max_item_tiles,
                        cudaStream_t stream);

// Pre-pass: out[b][j] = x[b][gather_idx[j]] for j < n_pad (0 where the index is -1); out is [batch][n_pad].
cudaError_t launch_pivot_x(pp_dtype_t dt, const void* x, int ldx, int n, const int32_t* gather_idx, int n_pad, void* out,
                           int batch, cudaStream_t stream);

inline int gemv_group_batch(pp_dtype_t dt) { return dt == PP_F16 ? kMaxGroupBatch : 8; }

}  // namespace pp
