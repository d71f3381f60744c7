// Launch interface of the tensor-core tile path (fp16, B = 64, batch chunks of up to 128).
#pragma once
#include <cuda_runtime.h>

#include "pp_internal.h"

namespace pp {

constexpr int kTileBatch = 128;     // batch rows one launch handles (the M side of the MMA)

// Persistent tile kernel: the steps of all groups (kTileRows block-rows each) form one sequence that is cut into
// one contiguous range per CTA, balanced by bytes.  A unit is the part of one group that one CTA computes.
struct TileUnit {
    int32_t step_begin, step_end;   // steps of the unit (may be empty: a group without tiles still emits act(bias))
    int32_t group;
    int32_t part;                   // position of this unit among the units of its group
    int32_t n_parts;                // units of the group (1: the unit stores the group's rows itself)
    int32_t first_unit;             // global index of the group's first unit
    int32_t pad[2];
};
static_assert(sizeof(TileUnit) == 32, "read as two 16-byte words");

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
    // clustered and persistent kernels
    const TileStep* steps;       // steps of all groups
    const int32_t* parts;        // [groups][kTileRows + 1] step boundaries of each cluster's CTAs
    int Mb;
    // persistent kernel only (plan built at layer creation for the device's SM count)
    const TileUnit* units;       // units in (group, step) order; a CTA's units are consecutive
    const int32_t* cta_unit;     // [persist_ctas + 1] first unit of every CTA
    float* unit_partials;        // [n_units][8 chunks][kTileBatch rows][32] partial sums of units whose group is split
    int* group_sync;             // [groups][2] arrivals / readers done; zero between launches
    int persist_ctas;            // CTAs of the plan (0: no plan)
    unsigned long long* trace;   // diagnostic builds (PP_TRACE): [persist_ctas][8] time stamps of the persistent kernel's phases
};

// Host: plan of the persistent tile kernel (pp_pack.cpp).
void build_tile_units(const pp_packed* pk, int n_ctas, std::vector<TileUnit>& units, std::vector<int32_t>& cta_unit);

// Host: the shared-memory image (128-byte swizzle) of one 64 x 64 row-major fp16 tile, 8 KiB.
void swizzle_tile_64x64(const void* row_major, void* out);

// Enqueue the gather pre-pass (x -> a.x_sw) and one of the tile kernels for one batch chunk:
// use_cluster picks the kernel in which a cluster of kTileRows CTAs shares the X blocks of kTileRows block-rows.
// kernel: 0 one block-row per CTA, 2 clustered, 3 persistent (needs a.units / a.persist_ctas)
cudaError_t launch_tile(const TileArgs& a, const void* x, int ldx, int n, const int32_t* gather_idx, int n_pad, int Mb,
                        int kernel, cudaStream_t stream);
// Bytes of unit_partials for n_units units.
inline size_t tile_unit_partial_bytes(size_t n_units) { return n_units * 8 * (size_t)kTileBatch * 32 * 4; }

}  // namespace pp
