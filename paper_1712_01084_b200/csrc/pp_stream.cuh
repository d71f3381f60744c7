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
    const uint16_t* gather16;    // staging mode 4: the same map as 16-bit entries index + 1 (0 = reads 0)
    const int32_t* scatter_idx;  // pivoted row -> original row, -1 = padding
    const float* bias_piv;
    const void* x;               // [batch][ldx]
    void* y;                     // [batch][ldy]
    float* partials;             // [stream_slots][rows_per_strip * kStreamMaxBatch]
    int* counters;               // [S], zero between launches
    int* status;                 // raised to 1 when the bounded wait for the copy of x gave up; may be NULL
    int wait_polls;              // polls before the bounded wait for the copy of x gives up (0: the kernel's default; set by the launcher)
    int x_ready;                 // 1: the caller promises that x was complete before anything still in flight in the stream was
                                 // enqueued, so x is fetched BEFORE the dependency wait, which moves in front of the first write
                                 // to y or scratch (set by the launcher from tuning key 17)
    unsigned long long* trace;   // diagnostic builds (PP_TRACE): [grid][8] time stamps of the kernel's phases; else unused
    int ldx, ldy;
    int x_limit;                 // with gather_idx == NULL: columns >= x_limit read 0
    int n_pad;                   // pivoted columns staged into shared memory
    int x_len;                   // elements of an x row that gather_idx may name
    int max_rows;                // most pivoted rows (strips x rows per strip) any CTA of the plan lists
    int raw_stride;              // staging mode 1: row stride of the shared-memory copy of x (set by the launcher)
    int xs_stride;               // shared-memory row stride of the staged x, in elements
    int batch;
    int act;
    int out_mode;                // pp::OutMode
    int stage_mode;              // 0: gather x from global memory; 1: copy x and gather_idx to shared
                                 // memory, permute there (needs 16-byte aligned rows); 2: x is already
                                 // in pivoted order (gather_idx == NULL), copy it (same alignment rule);
                                 // 3: batch 1 only: copy x and gather_idx as in 1 and read x through the
                                 // index array inside the multiply loop (no permutation pass);
                                 // 4: as 3 with the 16-bit index table (half the shared memory)
};

// Shared memory the kernel needs for this (dtype, n_pad, batch); the caller falls back to the
// chunked kernel when it exceeds kStreamSmemLimit.
size_t stream_smem_bytes(pp_dtype_t dt, int B, int n_pad, int x_len, int max_rows, int batch, int stage_mode);
// Ring depth a launch picks, and the dynamic shared memory of a launch with that depth (max_rows as in the plan).
int stream_pick_depth(pp_dtype_t dt, int B, int n_pad, int x_len, int max_rows, int batch, int stage_mode, int grid,
                      int frags_per_warp);
int stream_frags_per_warp(const CtaDesc* host_table, int grid);   // average over the plan's CTAs
size_t stream_launch_smem(pp_dtype_t dt, int B, int n_pad, int x_len, int max_rows, int batch, int stage_mode, int depth);
extern int g_stream_depth;   // weight-ring slots per warp: 4, 6 or 8; 0 = chosen per launch
extern int g_stream_pdl;     // 1: launch with programmatic stream serialization
constexpr size_t kStreamSmemLimit = 224 * 1024;

// A chain of fp16 layers in one cooperative kernel (batch <= 8).  `layers` holds one complete StreamArgs per layer
// (as stream_finish_args leaves them; cta_desc must point to the plan in device memory); x of the first and y of
// the last layer come with the launch.
constexpr int kChainMaxLayers = 8;
struct ChainLaunch {
    const StreamArgs* layers;    // device, [n_layers]
    const int* grids;            // device, [n_layers]: CTAs of each layer's plan (<= the launch's grid)
    const void* x;               // input of layer 0
    void* y;                     // output of the last layer
    unsigned* counter;           // device, zero between launches: arrivals at the layer boundaries
    int* status;                 // raised to 1 when a bounded wait gave up
    int n_layers;
    int region_bytes;            // bytes of one of the two shared-memory regions the layers alternate between
    int polls;                   // polls of a boundary wait before it gives up (0: default)
    unsigned long long* trace;   // diagnostic builds (PP_TRACE): [n_layers][320][8] phase stamps; else unused
};
void stream_finish_args(pp_dtype_t dt, StreamArgs& a);       // strides and rounding the launcher applies to a layer's arguments
int chain_resident_ctas(size_t smem, int depth);            // CTAs of the chain kernel the device holds at once (0: no cooperative launch)
// smem: 2 * region_bytes; depth: weight copies each warp keeps in flight (4 or 8), the same for every layer
cudaError_t launch_chain_f16(const ChainLaunch& P, int grid, size_t smem, int depth, cudaStream_t stream);
extern int g_stream_wait_polls;
extern int g_stream_x_ready;   // tuning key 17: value of StreamArgs::x_ready for launches through launch_stream

// host_table: the plan's CTA ranges in host memory (grid entries); small plans travel to the
// kernel inside its parameters so that no CTA starts with a dependent global load.
cudaError_t launch_stream(pp_dtype_t dt, int B, const StreamArgs& a, const CtaDesc* host_table, int grid,
                          cudaStream_t stream);

}  // namespace pp
