// Launch interface of the persistent streaming kernels (batch <= 8).
#pragma once
#include <cuda_runtime.h>

#include "pp_internal.h"

namespace pp {

struct StreamArgs {
    const void* values;          // fragment-ordered tile values (one linear fragment sequence)
    const int32_t* xoff;         // [F] element offset into the staged pivoted x of each fragment's columns
    const int32_t* strip_start;  // [S+1]
    const CtaDesc* cta_desc;     // [grid]
    const StripInfo* strip_info; // [S]
    const int32_t* gather_idx;   // pivoted column -> index into x, -1 = reads 0; NULL = identity
    const int32_t* scatter_idx;  // pivoted row -> original row, -1 = padding
    const float* bias_piv;
    const void* x;               // [batch][ldx]
    void* y;                     // [batch][ldy]
    float* partials;             // [stream_slots][rows_per_strip * kStreamMaxBatch]
    int* counters;               // [S], zero between launches
    int ldx, ldy;
    int x_limit;                 // with gather_idx == NULL: columns >= x_limit read 0
    int n_pad;                   // pivoted columns staged into shared memory
    int xs_stride;               // shared-memory row stride of the staged x, in elements
    int batch;
    int act;
    int out_mode;                // pp::OutMode
};

// Shared memory the kernel needs for this (dtype, n_pad, batch); the caller falls back to the
// chunked kernel when it exceeds kStreamSmemLimit.
size_t stream_smem_bytes(pp_dtype_t dt, int B, int n_pad, int batch);
constexpr size_t kStreamSmemLimit = 200 * 1024;

cudaError_t launch_stream(pp_dtype_t dt, int B, const StreamArgs& a, int grid, cudaStream_t stream);

}  // namespace pp
