// Launch interface of the tensor-core tile path (fp16, B = 64, batch chunks of up to 128).
#pragma once
#include <cuda_runtime.h>

#include "pp_internal.h"

namespace pp {

constexpr int kTileBatch = 128;     // batch rows one launch handles (the M side of the MMA)

struct TileArgs {
    const int32_t* row_ptr;      // [Mb+1] first kept tile of each block-row
    const int32_t* col_ptr;      // [Mb+1] start of each block-row's run in tile_col
    const int32_t* tile_col;     // tile-column index of every kept tile
    const int32_t* scatter_idx;  // pivoted row -> original row, -1 = padding
    const float* bias_piv;
    const unsigned char* tiles_sw;   // kept tiles in step order, each an 8 KiB swizzled shared-memory image
    const int32_t* tile_pos;         // sorted-tile index -> position in tiles_sw
    const unsigned char* x_sw;       // [N_pad / 64] blocks of 16 KiB: 128 batch rows x 64 columns, swizzled (scratch)
    float* y;                    // [batch][ldy], first row of this chunk
    int* status;                 // raised to 1 when a bounded wait gave up
    int ldy;
    int batch;                   // rows of this chunk (1..kTileBatch)
    int act;
    int pivoted;                 // 1: y[b][pivoted row] (Section 4.2.2), 0: y[b][scatter_idx[pivoted row]]
    int polls;                   // polls after which a bounded wait gives up (0: the kernels' own limit; set by the launcher)
    // clustered kernel only
    const TileStep* steps;       // steps of all groups
    const int32_t* parts;        // [groups][kTileRows + 1] step boundaries of each cluster's CTAs
    int Mb;
};

// Host: the shared-memory image (128-byte swizzle) of one 64 x 64 row-major fp16 tile, 8 KiB.
void swizzle_tile_64x64(const void* row_major, void* out);

// Enqueue the gather pre-pass (x -> a.x_sw) and one of the tile kernels for one batch chunk:
// use_cluster picks the kernel in which a cluster of kTileRows CTAs shares the X blocks of kTileRows block-rows.
cudaError_t launch_tile(const TileArgs& a, const void* x, int ldx, int n, const int32_t* gather_idx, int n_pad, int Mb,
                        bool use_cluster, cudaStream_t stream);

}  // namespace pp
