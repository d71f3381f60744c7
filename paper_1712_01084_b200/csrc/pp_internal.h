// Internal structures shared by the host packer, the API layer and the kernels.
#pragma once
#include <cstdint>
#include <vector>

#include "pp.h"

namespace pp {

// One unit of kernel work: a run of consecutive kept tiles of one block-row.
// The fragment indices are in 512-byte units into the packed value array.
struct WorkItem {
    int32_t frag_base;    // fragment of (row-group 0, first tile of the run, k-fragment 0)
    int32_t rg_stride;    // fragments between consecutive row-groups of this block-row
    int32_t nf;           // fragments per row-group in this run (= ntiles * frags_per_tile_row)
    int32_t col_off;      // index into tile_col[] of the run's first tile
    int32_t ntiles;       // tiles in the run (0 for a block-row without tiles)
    int32_t br;           // block-row
    int32_t part_nparts;  // part | (nparts << 16): position of this run among the block-row's runs
    int32_t slot_base;    // first partial-sum slot of the block-row (valid when nparts > 1)
};
static_assert(sizeof(WorkItem) == 32, "WorkItem is read as two 16-byte words");

constexpr int kMaxGroupBatch = 32;   // batch columns one streaming-kernel launch handles
constexpr int kMaxRunColumns = 2048;  // pivoted columns (tiles x B) one work item may span

// --- persistent streaming kernel (batch <= kStreamMaxBatch) ---------------------------------
// A strip is one row-group of one block-row: its fragments are contiguous in the value array
// and the strips follow each other in (block-row, row-group) order, so the whole layer is one
// linear fragment sequence.  The plan cuts that sequence into one contiguous range per CTA.
struct CtaDesc {
    int32_t p_begin, p_end;   // fragment positions [p_begin, p_end) streamed by this CTA
    int32_t s_first, s_count; // strips this CTA contributes to (consecutive); the first/last may be shared
};
struct StripInfo {
    int32_t first_cta;        // first CTA that lists this strip
    int32_t nparts;           // CTAs that list it (1: no cross-CTA reduction)
    int32_t slot_base;        // first global partial-sum slot (valid when nparts > 1)
    int32_t pad;
};
static_assert(sizeof(CtaDesc) == 16 && sizeof(StripInfo) == 16, "read as 16-byte words");
// --- clustered tensor-core tile kernel (fp16, B = 64) -------------------------------------------
// kTileRows consecutive block-rows form a group that one thread-block cluster of kTileRows CTAs
// computes.  A step is one tile-column some block-row of the group has a tile in; the CTA that owns
// the step fetches that X block once and multiplies it with the (up to kTileRows) tiles of the step.
constexpr int kTileRows = 4;
struct TileStep {
    int32_t col;                 // tile-column
    int32_t tile[kTileRows];     // sorted-tile index per block-row of the group, -1: no tile there
    int32_t ntiles;
    int32_t pos;                 // position of the step's first tile in the step-ordered tile images
    int32_t pad;
};
static_assert(sizeof(TileStep) == 32, "read as two 16-byte words");
extern int g_tile_cluster;   // batched fp16 B = 64 layers: 0 one block-row per CTA, 2 the clustered kernel, 3 the persistent kernel, 1 automatic
extern int g_tile_persist_auto;   // 1: the automatic choice is the persistent kernel whenever the layer has a plan for it
constexpr int kStreamWarps = 16;          // warps per CTA
constexpr int kStreamMaxStrips = 48;      // strips one CTA may list
constexpr int kStreamMaxBatch = 8;
extern int g_use_stream;
extern int g_tile_min_batch;  // fp16 B = 64 layers take the tensor-core tile path from this batch on (0: never)
extern int g_prepass;         // 1: permute multi-column inputs in a pre-pass when the kernel cannot do it in shared memory
extern int g_link_identity;  // 1: chain links whose folded map is the identity store pivoted rows directly (Section 4.2.3)
extern int g_lstm_persist;  // 1: recurrent cells run all steps in one cooperative kernel when the gate weights fit shared memory
extern int g_host_link_kernels;   // 1: pp_forward_host moves page-locked, device-addressable host buffers with kernels instead of copy-engine transfers
extern int g_chain_fused;    // 1: chains of fp16 layers run as one cooperative kernel when they qualify
extern int g_stage_direct;   // batch 1: read x through the index array instead of permuting it first

// "Done once" bookkeeping for settings that belong to a device, not to the process (the opt-in to more than
// 48 KiB of dynamic shared memory, cudaFuncSetAttribute, is one): one flag per device ordinal.  Ordinals beyond
// the table are never marked, so the setting is simply applied again on every launch there.
struct PerDeviceOnce {
    static constexpr int kMaxDevices = 64;
    bool done[kMaxDevices] = {};
    bool is_done(int dev) const { return dev >= 0 && dev < kMaxDevices && done[dev]; }
    void mark(int dev) { if (dev >= 0 && dev < kMaxDevices) done[dev] = true; }
};

// Geometry of the fragment layout for a (dtype, B) pair.
struct FragGeom {
    int rg_rows;   // rows covered by one fragment (row-group height)
    int kf;        // columns covered by one fragment
    int n_rg;      // row-groups per tile      = B / rg_rows
    int fpt;       // fragments per tile per row-group = B / kf
};
inline FragGeom frag_geom(pp_dtype_t dt, int B) {
    FragGeom g;
    if (dt == PP_F16) { g.rg_rows = 16; g.kf = 16; }
    else { g.rg_rows = B < 32 ? B : 32; g.kf = 128 / g.rg_rows; }
    g.n_rg = B / g.rg_rows;
    g.fpt = B / g.kf;
    return g;
}

}  // namespace pp

// Host-side result of packing one layer.
struct pp_packed {
    int M, N, B, Mb, Nb, Mpad, Npad;
    int64_t T;
    pp_dtype_t wdtype;
    std::vector<int32_t> row_perm, col_perm, inv_row_perm;   // copies of the caller's arrays
    std::vector<int32_t> row_ptr, col_ptr, tile_col;         // block-row-compressed index arrays
    std::vector<int32_t> gather_idx, scatter_idx;
    std::vector<uint16_t> gather16;                          // gather_idx + 1 as 16-bit entries (when N_pad < 65536)
    std::vector<float> bias_piv;
    std::vector<unsigned char> values;                       // fragment-ordered tile values
    std::vector<unsigned char> tiles_rm;                     // fp16, B = 64 only: tiles as swizzled 8 KiB images in step order
                                                             // (group, tile-column, block-row) for the tensor-core path
    std::vector<int32_t> tile_pos;                           // sorted-tile index -> position in tiles_rm
    std::vector<pp::TileStep> tile_steps;                    // fp16, B = 64 only: steps of all groups, group after group
    std::vector<int32_t> tile_parts;                         // [groups][kTileRows + 1] step boundaries of the cluster's CTAs
    std::vector<pp::WorkItem> items;
    // plan of the persistent streaming kernel
    std::vector<int32_t> strip_start;   // [S+1] fragment position of each strip
    std::vector<int32_t> xoff;          // [F] per fragment: element offset of its columns in the pivoted x
    std::vector<pp::CtaDesc> cta_desc;
    std::vector<pp::StripInfo> strip_info;
    int stream_slots;
    int max_item_tiles;
    int n_slots;
    bool has_bias;
};
