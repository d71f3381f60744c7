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
    float* y;                    // [batch][ldy], first row of this chunk
    int* status;                 // raised to 1 when a bounded wait gave up
    int ldy;
    int batch;                   // rows of this chunk (1..kTileBatch)
    int act;
};

struct TilePlan;                 // tensor maps of one layer (host object)

// d_tiles_rm: sorted kept tiles, each 64 x 64 row-major fp16; d_x_piv: [kTileBatch][n_pad] fp16 scratch.
// Returns NULL when the driver's tensor-map encoder is unavailable or refuses the shapes.
TilePlan* tile_plan_create(void* d_tiles_rm, int64_t T, void* d_x_piv, int n_pad);
void tile_plan_destroy(TilePlan* p);

// Enqueue the gather pre-pass and the tile kernel for one batch chunk.
cudaError_t launch_tile(const TilePlan* plan, const TileArgs& a, const void* x, int ldx, int n, const int32_t* gather_idx,
                        int n_pad, void* d_x_piv, int Mb, cudaStream_t stream);

}  // namespace pp
