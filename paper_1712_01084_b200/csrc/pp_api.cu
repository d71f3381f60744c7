// C entry points that own device memory: layers, forward calls, folded chains.
#include <cuda_runtime.h>

#include <algorithm>
#include <new>
#include <vector>

#include "pp_gemv.cuh"
#include "pp_internal.h"
#include "pp_lstm.cuh"
#include "pp_stream.cuh"
#include "pp_tile.cuh"

struct pp_layer {
    pp_packed* pk = nullptr;       // host copy (index arrays are needed again when chains are folded)
    // One read-only device allocation holds every packed array (small tables first, tile values
    // last), so a forward call touches few pages; one more holds the scratch both kernels write.
    unsigned char* d_arena = nullptr;
    size_t arena_bytes = 0;
    unsigned char* d_scratch = nullptr;
    size_t scratch_bytes = 0;
    // views into the arena
    void* d_values = nullptr;
    pp::WorkItem* d_items = nullptr;
    int32_t* d_tile_col = nullptr;
    int32_t* d_gather = nullptr;
    uint16_t* d_gather16 = nullptr;  // 16-bit form of d_gather (NULL when N_pad >= 65536)
    int32_t* d_scatter = nullptr;
    float* d_bias = nullptr;
    int32_t* d_xoff = nullptr;
    int32_t* d_strip_start = nullptr;
    pp::CtaDesc* d_cta_desc = nullptr;
    pp::StripInfo* d_strip_info = nullptr;
    // views into the scratch allocation
    float* d_partials = nullptr;   // chunked kernel: [n_slots][B][kMaxGroupBatch]
    int* d_counters = nullptr;     // chunked kernel: [Mb]
    float* d_spartials = nullptr;  // persistent kernel: [stream_slots][rows per strip][kStreamMaxBatch]
    int* d_scounters = nullptr;    // persistent kernel: [S]
    unsigned char* d_xstage = nullptr;   // [kMaxGroupBatch][N_pad] input in pivoted order (pre-pass output)
    int n_items = 0;
    int max_item_tiles = 0;
    int stream_grid = 0;
    int stream_max_rows = 0;       // most pivoted rows one CTA of the persistent plan lists
    // tensor-core tile path (fp16, B = 64): row_ptr, col_ptr and the row-major tiles in one block,
    // the permuted-input chunk and the status word in another
    unsigned char* d_tile = nullptr;
    size_t tile_bytes = 0;
    int32_t* d_row_ptr = nullptr;
    int32_t* d_col_ptr = nullptr;
    void* d_tiles_rm = nullptr;
    int32_t* d_tile_pos = nullptr;       // sorted-tile index -> position in the step-ordered tile images
    int32_t* d_tile_parts = nullptr;     // clustered tile kernel: step boundaries per group
    pp::TileStep* d_tile_steps = nullptr;
    int n_tile_steps = 0;
    unsigned char* d_tile_scratch = nullptr;
    // persistent tile kernel: units, first unit of every CTA, partial-sum slots, group counters (one allocation)
    unsigned char* d_persist = nullptr;
    pp::TileUnit* d_units = nullptr;
    int32_t* d_cta_unit = nullptr;
    float* d_unit_partials = nullptr;
    int* d_group_sync = nullptr;
    size_t group_sync_bytes = 0;
    int persist_ctas = 0;
    void* d_x_piv = nullptr;
    int* d_status = nullptr;
    bool tile_ok = false;
    // staging buffers of pp_forward_host (grown on demand, never shrunk)
    unsigned char* d_host_x = nullptr;
    float* d_host_y = nullptr;
    int host_batch = 0;
};

struct pp_lstm {
    pp_layer* gates = nullptr;
    int I = 0, H = 0, max_steps = 0;
    int32_t* d_inv_row = nullptr;
    int32_t* d_inv_col = nullptr;
    void* d_z = nullptr;           // [max_steps + 1][N_pad] inputs of every step in pivoted order
    float* d_g = nullptr;          // [M_pad] gate pre-activations in pivoted order; the persistent cell uses the
                                   // allocation as [2][M_pad] 8-byte packets
    unsigned int* d_sync = nullptr;   // persistent cell: [1] status word
    int persist_grid = 0;          // CTAs of the persistent cell (0: layer does not qualify)
    int persist_strips = 0;        // strips per CTA
    size_t persist_smem = 0;
};

struct pp_chain {
    std::vector<pp_layer*> layers;
    std::vector<pp_act_t> acts;
    std::vector<int32_t*> d_q;     // entry l (l >= 1): folded map of the link l-1 -> l, as a STORE map of layer l-1:
                                   // pivoted row of layer l-1 -> pivoted column of layer l (-1: padding row)
    std::vector<void*> d_inter;    // output of layer l in layer l+1's pivoted column order, element type of layer l+1
    std::vector<char> identity;    // entry l (l >= 1): the folded map of the link l-1 -> l is the identity (Section 4.2.3)
    bool out_pivoted = false;      // the last layer leaves its output in pivoted row order (Section 4.2.2)
    int max_batch = 0;
    // one-kernel execution (fp16 layers, batch <= 8): per batch size the layers' kernel arguments in device memory
    pp::StreamArgs* d_fused_args = nullptr;   // [kStreamMaxBatch][n_layers]
    int* d_fused_grids = nullptr;             // [n_layers]
    unsigned* d_fused_sync = nullptr;         // [0] arrival counter, [1] status word
    int fused_grid = 0;                       // CTAs of the launch (0: the chain runs layer by layer)
    size_t fused_region[pp::kStreamMaxBatch + 1] = {}; // bytes of one shared-memory region per batch size (0: that batch runs layer by layer)
    int fused_depth[pp::kStreamMaxBatch + 1] = {};     // weight copies per warp in flight for that batch size (4 or 8)
};

namespace {

// Persistent cell: fp16 gate layers whose strips, dealt out 1, 2, 4, 8 or 16 to a CTA, fit the shared
// memory of at most one CTA per SM -- and a grid that size can be resident at once (cooperative launch).
void lstm_plan_persistent(pp_lstm* R) {
    const pp_packed* pk = R->gates->pk;
    R->persist_grid = 0;
    if (pk->wdtype != PP_F16 || R->H > 4 * 512 || pk->Npad % 8 != 0 || pk->Mpad >= 65536 || pk->Npad >= 65536) return;
    const int S = (int)pk->strip_start.size() - 1;
    int dev = 0, sms = 0, coop = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess || !coop) {
        cudaGetLastError();
        return;
    }
    for (int ns = 1; ns <= 16; ns *= 2) {
        const int grid = (S + ns - 1) / ns;
        if (grid > sms) continue;
        int max_frags = 0;
        for (int c = 0; c < grid; ++c) {
            const int s0 = c * ns, s1 = std::min(S, s0 + ns);
            max_frags = std::max(max_frags, pk->strip_start[(size_t)s1] - pk->strip_start[(size_t)s0]);
        }
        const size_t smem = pp::lstm_persist_smem(max_frags, pk->Npad, pk->Mpad);
        if (smem == 0) return;       // more strips per CTA only need more
        R->persist_grid = grid; R->persist_strips = ns; R->persist_smem = smem;
        return;
    }
}

}  // namespace

namespace {

template <typename T>
bool upload(T** dst, const void* src, size_t bytes) {
    *dst = nullptr;
    if (cudaMalloc(reinterpret_cast<void**>(dst), bytes ? bytes : 16) != cudaSuccess) return false;
    if (bytes && cudaMemcpy(*dst, src, bytes, cudaMemcpyHostToDevice) != cudaSuccess) return false;
    return true;
}

void free_layer(pp_layer* L) {
    if (!L) return;
    cudaFree(L->d_arena);
    cudaFree(L->d_scratch);
    cudaFree(L->d_tile);
    cudaFree(L->d_tile_scratch);
    cudaFree(L->d_persist);
    cudaFree(L->d_host_x);
    cudaFree(L->d_host_y);
    pp_pack_destroy(L->pk);
    delete L;
}

size_t round256(size_t n) { return (n + 255) / 256 * 256; }

// Section sizes of the arena and the scratch allocation, in a fixed order.
struct LayerLayout {
    size_t off[11];       // cta_desc, strip_start, strip_info, scatter, bias, gather, tile_col, items, xoff, values, gather16
    size_t arena_bytes;
    size_t soff[6];       // partials, counters, spartials, scounters, pivoted-x staging, status word
    size_t scratch_bytes;
};

LayerLayout layer_layout(const pp_packed* pk) {
    const pp::FragGeom g = pp::frag_geom(pk->wdtype, pk->B);
    const size_t esz = pk->wdtype == PP_F16 ? 2 : 4;
    const size_t S = pk->strip_info.size();
    const size_t F = (size_t)pk->T * g.n_rg * g.fpt;
    const size_t sz[11] = {pk->cta_desc.size() * sizeof(pp::CtaDesc), (S + 1) * 4, S * sizeof(pp::StripInfo),
                           (size_t)pk->Mpad * 4, (size_t)pk->Mpad * 4, (size_t)pk->Npad * 4, pk->tile_col.size() * 4,
                           pk->items.size() * sizeof(pp::WorkItem), F * 4, (size_t)pk->T * pk->B * pk->B * esz,
                           pk->gather16.size() * 2};
    LayerLayout lo;
    size_t pos = 0;
    for (int i = 0; i < 11; ++i) { lo.off[i] = pos; pos += round256(sz[i]); }
    lo.arena_bytes = pos ? pos : 256;
    const size_t ssz[6] = {(size_t)pk->n_slots * pk->B * pp::kMaxGroupBatch * 4, (size_t)pk->Mb * 4,
                           (size_t)pk->stream_slots * g.rg_rows * pp::kStreamMaxBatch * 4, (S ? S : 1) * 4,
                           (size_t)pp::kMaxGroupBatch * pk->Npad * esz, 4};
    pos = 0;
    for (int i = 0; i < 6; ++i) { lo.soff[i] = pos; pos += round256(ssz[i]); }
    lo.scratch_bytes = pos;
    return lo;
}

// Allocate both device blocks and point the views into them.
bool alloc_layer(pp_layer* L, const LayerLayout& lo) {
    const bool pk_has16 = !L->pk->gather16.empty();
    if (cudaMalloc(reinterpret_cast<void**>(&L->d_arena), lo.arena_bytes) != cudaSuccess) return false;
    if (cudaMalloc(reinterpret_cast<void**>(&L->d_scratch), lo.scratch_bytes) != cudaSuccess) return false;
    if (cudaMemset(L->d_scratch, 0, lo.scratch_bytes) != cudaSuccess) return false;
    // the persistent kernel's exchange slots rest at an all-ones NaN pattern
    if (cudaMemset(L->d_scratch + lo.soff[2], 0xff, lo.soff[3] - lo.soff[2]) != cudaSuccess) return false;
    L->arena_bytes = lo.arena_bytes;
    L->scratch_bytes = lo.scratch_bytes;
    unsigned char* a = L->d_arena;
    L->d_cta_desc = reinterpret_cast<pp::CtaDesc*>(a + lo.off[0]);
    L->d_strip_start = reinterpret_cast<int32_t*>(a + lo.off[1]);
    L->d_strip_info = reinterpret_cast<pp::StripInfo*>(a + lo.off[2]);
    L->d_scatter = reinterpret_cast<int32_t*>(a + lo.off[3]);
    L->d_bias = reinterpret_cast<float*>(a + lo.off[4]);
    L->d_gather = reinterpret_cast<int32_t*>(a + lo.off[5]);
    L->d_tile_col = reinterpret_cast<int32_t*>(a + lo.off[6]);
    L->d_items = reinterpret_cast<pp::WorkItem*>(a + lo.off[7]);
    L->d_xoff = reinterpret_cast<int32_t*>(a + lo.off[8]);
    L->d_values = a + lo.off[9];
    L->d_gather16 = pk_has16 ? reinterpret_cast<uint16_t*>(a + lo.off[10]) : nullptr;
    unsigned char* sc = L->d_scratch;
    L->d_partials = reinterpret_cast<float*>(sc + lo.soff[0]);
    L->d_counters = reinterpret_cast<int*>(sc + lo.soff[1]);
    L->d_spartials = reinterpret_cast<float*>(sc + lo.soff[2]);
    L->d_scounters = reinterpret_cast<int*>(sc + lo.soff[3]);
    L->d_xstage = sc + lo.soff[4];
    L->d_status = reinterpret_cast<int*>(sc + lo.soff[5]);     // zeroed with the scratch block; every kernel of the layer raises this word
    return true;
}

// Plan of the persistent tile kernel for this device (one CTA per SM; see build_tile_units) and its device
// blocks.  false: allocation failed.
bool persist_setup(pp_layer* L) {
    const pp_packed* pk = L->pk;
    if (pp::g_tile_cluster != 3) return true;       // opt-in: the partial-sum slots are 128 KiB per unit (tens of MiB for a large layer)
    int dev = 0, sms = 0, coop = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess) {
        cudaGetLastError();
        return true;                                  // no plan: the other tile kernels remain
    }
    if (!coop || sms < 1) return true;
    const int G = sms;
    const int groups = (pk->Mb + pp::kTileRows - 1) / pp::kTileRows;
    std::vector<pp::TileUnit> units;
    std::vector<int32_t> cta_unit;
    try {
        pp::build_tile_units(pk, G, units, cta_unit);
    } catch (const std::bad_alloc&) {
        return false;
    }
    const size_t ub = round256(units.size() * sizeof(pp::TileUnit)), cb = round256(((size_t)G + 1) * 4);
    const size_t gb = round256((size_t)groups * 2 * 4), pb = round256(pp::tile_unit_partial_bytes(units.size()));
    if (cudaMalloc(reinterpret_cast<void**>(&L->d_persist), ub + cb + gb + pb) != cudaSuccess) return false;
    L->d_units = reinterpret_cast<pp::TileUnit*>(L->d_persist);
    L->d_cta_unit = reinterpret_cast<int32_t*>(L->d_persist + ub);
    L->d_group_sync = reinterpret_cast<int*>(L->d_persist + ub + cb);
    L->d_unit_partials = reinterpret_cast<float*>(L->d_persist + ub + cb + gb);
    L->group_sync_bytes = gb;
    if (cudaMemcpy(L->d_units, units.data(), units.size() * sizeof(pp::TileUnit), cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMemcpy(L->d_cta_unit, cta_unit.data(), cta_unit.size() * 4, cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMemset(L->d_group_sync, 0, gb) != cudaSuccess)
        return false;
    L->persist_ctas = G;
    return true;
}

// Device blocks and tensor maps of the tensor-core tile path.  `host` uploads from the packed layer,
// otherwise the weights block is copied from another layer's.  A layer that is not eligible, or a
// driver without the tensor-map encoder, simply has no tile path (tile_plan stays NULL).
bool tile_setup(pp_layer* L, const pp_layer* from) {
    const pp_packed* pk = L->pk;
    if (pk->wdtype != PP_F16 || pk->B != 64) return true;
    if (!from && pp::g_tile_min_batch == 0) return true;      // the tile path is switched off: no second copy of the weights
    if (from && !from->tile_ok) return true;
    const size_t rp = round256((size_t)(pk->Mb + 1) * 4), tb = (size_t)pk->T * 64 * 64 * 2;
    const int groups = (pk->Mb + pp::kTileRows - 1) / pp::kTileRows;
    const size_t pb = round256((size_t)groups * (pp::kTileRows + 1) * 4);
    L->n_tile_steps = from ? from->n_tile_steps : (int)pk->tile_steps.size();
    const size_t sb = round256((size_t)L->n_tile_steps * sizeof(pp::TileStep));
    const size_t qb = round256((size_t)pk->T * 4);
    L->tile_bytes = 2 * rp + pb + sb + qb + round256(tb);
    if (cudaMalloc(reinterpret_cast<void**>(&L->d_tile), L->tile_bytes) != cudaSuccess) return false;
    const size_t xb = round256((size_t)pp::kTileBatch * pk->Npad * 2);
    if (cudaMalloc(reinterpret_cast<void**>(&L->d_tile_scratch), xb + 256) != cudaSuccess) return false;
    if (cudaMemset(L->d_tile_scratch, 0, xb + 256) != cudaSuccess) return false;
    L->d_row_ptr = reinterpret_cast<int32_t*>(L->d_tile);
    L->d_col_ptr = reinterpret_cast<int32_t*>(L->d_tile + rp);
    L->d_tile_parts = reinterpret_cast<int32_t*>(L->d_tile + 2 * rp);
    L->d_tile_steps = reinterpret_cast<pp::TileStep*>(L->d_tile + 2 * rp + pb);
    L->d_tile_pos = reinterpret_cast<int32_t*>(L->d_tile + 2 * rp + pb + sb);
    L->d_tiles_rm = L->d_tile + 2 * rp + pb + sb + qb;
    L->d_x_piv = L->d_tile_scratch;
    if (from) {
        if (from->tile_bytes != L->tile_bytes ||
            cudaMemcpy(L->d_tile, from->d_tile, L->tile_bytes, cudaMemcpyDeviceToDevice) != cudaSuccess) return false;
    } else {
        if (cudaMemcpy(L->d_row_ptr, pk->row_ptr.data(), (size_t)(pk->Mb + 1) * 4, cudaMemcpyHostToDevice) != cudaSuccess ||
            cudaMemcpy(L->d_col_ptr, pk->col_ptr.data(), (size_t)(pk->Mb + 1) * 4, cudaMemcpyHostToDevice) != cudaSuccess ||
            cudaMemcpy(L->d_tile_parts, pk->tile_parts.data(), pk->tile_parts.size() * 4, cudaMemcpyHostToDevice) != cudaSuccess ||
            (L->n_tile_steps && cudaMemcpy(L->d_tile_steps, pk->tile_steps.data(), (size_t)L->n_tile_steps * sizeof(pp::TileStep),
                                           cudaMemcpyHostToDevice) != cudaSuccess) ||
            (pk->T && cudaMemcpy(L->d_tile_pos, pk->tile_pos.data(), (size_t)pk->T * 4, cudaMemcpyHostToDevice) != cudaSuccess) ||
            (tb && cudaMemcpy(L->d_tiles_rm, pk->tiles_rm.data(), tb, cudaMemcpyHostToDevice) != cudaSuccess))   // already swizzled by the packer
            return false;
    }
    if (!persist_setup(L)) return false;
    L->tile_ok = true;
    return true;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// How the persistent kernel stages x for this call (StreamArgs::stage_mode), or -1 when x does not fit shared memory.
int pick_stage_mode(const pp_layer* L, bool has_gather, bool own_gather, bool rows_aligned, int x_len, int batch) {
    const pp_packed* pk = L->pk;
    const bool has16 = has_gather && own_gather && L->d_gather16;
    // reading x through the index array inside the multiply loop: always for one input vector, for several
    // (fp16 layers) when tuning key 7 is 2
    const bool direct = pp::g_stage_direct && (batch == 1 || (pp::g_stage_direct == 2 && pk->wdtype == PP_F16));
    const int fast = has_gather ? (direct ? (has16 ? 4 : 3) : 1) : 2;
    if (rows_aligned && pp::stream_smem_bytes(pk->wdtype, pk->B, pk->Npad, x_len, L->stream_max_rows, batch, fast) <= pp::kStreamSmemLimit)
        return fast;
    if (pp::stream_smem_bytes(pk->wdtype, pk->B, pk->Npad, x_len, L->stream_max_rows, batch, 0) <= pp::kStreamSmemLimit)
        return 0;
    return -1;
}

// Arguments of one persistent-kernel launch over this layer.
pp::StreamArgs make_stream_args(const pp_layer* L, const int32_t* gather, const void* x, int ldx, int x_len, void* y, int ldy,
                                int out_mode, int batch, pp_act_t act, int x_limit, const int32_t* scatter, int stage_mode) {
    const pp_packed* pk = L->pk;
    pp::StreamArgs s{};
    s.stage_mode = stage_mode;
    s.values = L->d_values; s.xoff = L->d_xoff; s.strip_start = L->d_strip_start;
    s.cta_desc = L->d_cta_desc; s.strip_info = L->d_strip_info;
    s.gather_idx = gather; s.gather16 = L->d_gather16; s.scatter_idx = scatter; s.bias_piv = L->d_bias;
    s.x = x; s.y = y; s.partials = L->d_spartials; s.counters = L->d_scounters; s.status = L->d_status;
    s.ldx = ldx; s.ldy = ldy; s.x_limit = x_limit; s.n_pad = pk->Npad; s.x_len = x_len; s.max_rows = L->stream_max_rows; s.batch = batch;
    s.act = (int)act; s.out_mode = out_mode;
    return s;
}

// Enqueue one layer in groups of batch columns.
// Persistent kernel for up to kStreamMaxBatch columns; PP_ERR_UNSUPPORTED when x does not fit shared memory.
pp_status_t run_stream(pp_layer* L, const int32_t* gather, const void* x, int ldx, int x_len, int x_elt, void* y, int ldy,
                       int out_mode, int batch, pp_act_t act, cudaStream_t stream, int x_limit, const int32_t* scatter,
                       bool x_ready = false) {
    const pp_packed* pk = L->pk;
    const bool rows_aligned = aligned16(x) && (batch == 1 || ((size_t)ldx * x_elt) % 16 == 0);
    const int stage_mode = pick_stage_mode(L, gather != nullptr, gather == L->d_gather, rows_aligned, x_len, batch);
    if (stage_mode < 0) return PP_ERR_UNSUPPORTED;
    pp::StreamArgs s = make_stream_args(L, gather, x, ldx, x_len, y, ldy, out_mode, batch, act, x_limit, scatter, stage_mode);
    s.x_ready = x_ready ? 1 : 0;
    return pp::launch_stream(pk->wdtype, pk->B, s, pk->cta_desc.data(), L->stream_grid, stream) == cudaSuccess
               ? PP_OK : PP_ERR_CUDA;
}

// Enqueue one layer.  Batch <= 8: one launch of the persistent kernel.  Larger batches: the
// persistent kernel in groups of 8 columns when that takes no more passes over the weights than
// the chunked kernel would (fp32), else the chunked kernel in groups of up to 32 columns (fp16:
// at 8 columns the persistent kernel holds 16 KiB of x per column in shared memory, runs one CTA
// per SM and measured 60 us per pass against 85 us for one chunked pass over 16 columns).
pp_status_t run_layer(pp_layer* L, const int32_t* gather, const void* x, int ldx, int x_len, int x_elt, void* y, int ldy,
                      int out_mode, int batch, pp_act_t act, cudaStream_t stream, int x_limit = -1,
                      const int32_t* scatter = nullptr, bool x_ready = false) {
    const pp_packed* pk = L->pk;
    if (x_limit < 0) x_limit = pk->N;      // without a gather map: columns at or beyond x_limit read 0
    if (!scatter) scatter = L->d_scatter;  // a chain passes the map into its consumer's column order instead
    const int y_elt = (out_mode == pp::OUT_PIVOTED_F16 || out_mode == pp::OUT_SCATTER_F16) ? 2 : 4;
    const int chunk_group = pp::gemv_group_batch(pk->wdtype);
    const int stream_passes = (batch + pp::kStreamMaxBatch - 1) / pp::kStreamMaxBatch;
    const int chunk_passes = (batch + chunk_group - 1) / chunk_group;
    // Several batch columns with a gather map: unless the persistent kernel can hold x twice (as
    // given and permuted) in shared memory, permute x once in a pre-pass and let the layer kernel
    // read the pivoted rows without any index array.
    if (gather && batch > 1 && pp::g_prepass) {
        const bool stream_path = pp::g_use_stream && stream_passes <= chunk_passes;
        const int nb = batch < pp::kStreamMaxBatch ? batch : pp::kStreamMaxBatch;
        const bool fits = stream_path && aligned16(x) && ((size_t)ldx * x_elt) % 16 == 0 &&
                          pp::stream_smem_bytes(pk->wdtype, pk->B, pk->Npad, x_len, L->stream_max_rows, nb, 1) <= 113 * 1024;
        const bool direct_ok = stream_path && pp::g_stage_direct == 2 && pk->wdtype == PP_F16 && aligned16(x) &&
                               ((size_t)ldx * x_elt) % 16 == 0 && pp::g_prepass != 2 &&
                               pp::stream_smem_bytes(pk->wdtype, pk->B, pk->Npad, x_len, L->stream_max_rows, nb,
                                                     gather == L->d_gather && L->d_gather16 ? 4 : 3) <= pp::kStreamSmemLimit;
        if ((!fits && !direct_ok) || pp::g_prepass == 2) {
            const int group = stream_path ? pp::kStreamMaxBatch : chunk_group;
            for (int b0 = 0; b0 < batch; b0 += group) {
                const int gb = batch - b0 < group ? batch - b0 : group;
                if (pp::launch_pivot_x(pk->wdtype, static_cast<const char*>(x) + (size_t)b0 * ldx * x_elt, ldx, x_len, gather,
                                       pk->Npad, L->d_xstage, gb, stream) != cudaSuccess)
                    return PP_ERR_CUDA;
                const pp_status_t st = run_layer(L, nullptr, L->d_xstage, pk->Npad, pk->Npad, x_elt,
                                                 static_cast<char*>(y) + (size_t)b0 * ldy * y_elt, ldy, out_mode, gb, act,
                                                 stream, pk->Npad, scatter);
                if (st != PP_OK) return st;
            }
            return PP_OK;
        }
    }
    if (pp::g_use_stream && stream_passes <= chunk_passes) {
        bool done = true;
        for (int b0 = 0; b0 < batch; b0 += pp::kStreamMaxBatch) {
            const int nb = batch - b0 < pp::kStreamMaxBatch ? batch - b0 : pp::kStreamMaxBatch;
            const pp_status_t st = run_stream(L, gather, static_cast<const char*>(x) + (size_t)b0 * ldx * x_elt, ldx, x_len,
                                              x_elt, static_cast<char*>(y) + (size_t)b0 * ldy * y_elt, ldy, out_mode, nb, act,
                                              stream, x_limit, scatter, x_ready);
            if (st == PP_ERR_UNSUPPORTED && b0 == 0) { done = false; break; }   // x too large to stage: chunked kernel
            if (st != PP_OK) return st;
        }
        if (done) return PP_OK;
    }
    pp::GemvArgs a{};
    a.values = L->d_values; a.items = L->d_items; a.tile_col = L->d_tile_col;
    a.gather_idx = gather; a.scatter_idx = scatter; a.bias_piv = L->d_bias;
    a.partials = L->d_partials; a.counters = L->d_counters;
    a.ldx = ldx; a.ldy = ldy; a.x_limit = x_limit; a.act = (int)act; a.out_mode = out_mode;
    const int group = chunk_group;
    for (int b0 = 0; b0 < batch; b0 += group) {
        a.batch = batch - b0 < group ? batch - b0 : group;
        a.x = static_cast<const char*>(x) + (size_t)b0 * ldx * x_elt;
        a.y = static_cast<char*>(y) + (size_t)b0 * ldy * y_elt;
        if (pp::launch_gemv(pk->wdtype, pk->B, a, L->n_items, L->max_item_tiles, stream) != cudaSuccess)
            return PP_ERR_CUDA;
    }
    return PP_OK;
}

}  // namespace

namespace {
// Uploads a packed layer to the current device; takes ownership of pk (freed on failure).
pp_status_t layer_from_pack(pp_layer_t** out, pp_packed* pk);
void chain_plan_fused(pp_chain* C);
}

extern "C" {

pp_status_t pp_layer_create(pp_layer_t** out, int M, int N, int B, const int32_t* row_perm,
                            const int32_t* col_perm, const int32_t* tile_list, int64_t T,
                            const void* tile_values, pp_dtype_t wdtype, const float* bias) {
    if (!out) return PP_ERR_INVALID_ARG;
    *out = nullptr;
    pp_packed* pk = nullptr;
    pp_status_t st = pp_pack_create(&pk, M, N, B, row_perm, col_perm, tile_list, T, tile_values, wdtype, bias);
    if (st != PP_OK) return st;
    return layer_from_pack(out, pk);
}

pp_status_t pp_layer_create_blocks(pp_layer_t** out, int M, int N, int B, const int32_t* row_perm,
                                   const int32_t* col_perm, const int32_t* blocks, int64_t n_blocks,
                                   const void* block_values, pp_dtype_t wdtype, const float* bias) {
    if (!out) return PP_ERR_INVALID_ARG;
    *out = nullptr;
    pp_packed* pk = nullptr;
    pp_status_t st = pp_pack_create_blocks(&pk, M, N, B, row_perm, col_perm, blocks, n_blocks, block_values, wdtype, bias);
    if (st != PP_OK) return st;
    return layer_from_pack(out, pk);
}

}  // extern "C"

namespace {
pp_status_t layer_from_pack(pp_layer_t** out, pp_packed* pk) {
    const pp_dtype_t wdtype = pk->wdtype;
    const int B = pk->B;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { pp_pack_destroy(pk); cudaGetLastError(); return PP_ERR_CUDA; }
    pp_layer* L = new (std::nothrow) pp_layer();
    if (!L) { pp_pack_destroy(pk); return PP_ERR_ALLOC; }
    L->pk = pk;
    L->n_items = (int)pk->items.size();
    L->max_item_tiles = pk->max_item_tiles;
    L->stream_grid = (int)pk->cta_desc.size();
    for (const pp::CtaDesc& c : pk->cta_desc)
        L->stream_max_rows = std::max(L->stream_max_rows, c.s_count * pp::frag_geom(wdtype, B).rg_rows);
    const LayerLayout lo = layer_layout(pk);
    bool ok = alloc_layer(L, lo);
    if (ok) {
        const void* src[11] = {pk->cta_desc.data(), pk->strip_start.data(), pk->strip_info.data(),
                               pk->scatter_idx.data(), pk->bias_piv.data(), pk->gather_idx.data(),
                               pk->tile_col.data(), pk->items.data(), pk->xoff.data(), pk->values.data(), pk->gather16.data()};
        const size_t n[11] = {pk->cta_desc.size() * sizeof(pp::CtaDesc), pk->strip_start.size() * 4,
                              pk->strip_info.size() * sizeof(pp::StripInfo), pk->scatter_idx.size() * 4,
                              pk->bias_piv.size() * 4, pk->gather_idx.size() * 4, pk->tile_col.size() * 4,
                              pk->items.size() * sizeof(pp::WorkItem), pk->xoff.size() * 4, pk->values.size(),
                              pk->gather16.size() * 2};
        for (int i = 0; i < 11 && ok; ++i)
            ok = n[i] == 0 || cudaMemcpy(L->d_arena + lo.off[i], src[i], n[i], cudaMemcpyHostToDevice) == cudaSuccess;
    }
    ok = ok && tile_setup(L, nullptr);
    if (!ok) {
        const cudaError_t e = cudaGetLastError();
        free_layer(L);
        return e == cudaErrorMemoryAllocation ? PP_ERR_ALLOC : PP_ERR_CUDA;
    }
    // the tile values and per-fragment offsets now live on the device; drop the host copies
    std::vector<unsigned char>().swap(pk->values);
    std::vector<unsigned char>().swap(pk->tiles_rm);
    std::vector<int32_t>().swap(pk->xoff);
    *out = L;
    return PP_OK;
}
}  // namespace

extern "C" {

pp_status_t pp_layer_clone(pp_layer_t** out, const pp_layer_t* src) {
    if (!out) return PP_ERR_INVALID_ARG;
    *out = nullptr;
    if (!src) return PP_ERR_INVALID_ARG;
    pp_layer* L = new (std::nothrow) pp_layer();
    pp_packed* pk = new (std::nothrow) pp_packed(*src->pk);
    if (!L || !pk) { delete L; delete pk; return PP_ERR_ALLOC; }
    L->pk = pk;
    L->n_items = src->n_items;
    L->max_item_tiles = src->max_item_tiles;
    L->stream_grid = src->stream_grid;
    L->stream_max_rows = src->stream_max_rows;
    const LayerLayout lo = layer_layout(pk);
    const bool ok = lo.arena_bytes == src->arena_bytes && alloc_layer(L, lo) &&
                    cudaMemcpy(L->d_arena, src->d_arena, lo.arena_bytes, cudaMemcpyDeviceToDevice) == cudaSuccess &&
                    tile_setup(L, src);
    if (!ok) {
        const cudaError_t e = cudaGetLastError();
        free_layer(L);
        return e == cudaErrorMemoryAllocation ? PP_ERR_ALLOC : PP_ERR_CUDA;
    }
    *out = L;
    return PP_OK;
}

pp_status_t pp_layer_status(pp_layer_t* L, pp_status_t* status) {
    if (!L || !status) return PP_ERR_INVALID_ARG;
    *status = PP_OK;
    if (!L->d_status) return PP_OK;
    int flag = 0;
    if (cudaMemcpy(&flag, L->d_status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return PP_ERR_CUDA;
    if (flag) {
        *status = PP_ERR_TIMEOUT;
        if (cudaMemset(L->d_status, 0, sizeof(int)) != cudaSuccess) return PP_ERR_CUDA;
        // a persistent tile kernel that gave up may have left its group counters behind
        if (L->d_group_sync && cudaMemset(L->d_group_sync, 0, L->group_sync_bytes) != cudaSuccess) return PP_ERR_CUDA;
    }
    return PP_OK;
}

// Which tile kernel a batched call of this layer takes: 0 one block-row per CTA, 2 clustered, 3 persistent.
static int pick_tile_kernel(const pp_layer* L) {
    if (pp::g_tile_cluster == 3) return L->persist_ctas > 0 ? 3 : 0;
    if (pp::g_tile_cluster == 0 || pp::g_tile_cluster == 2) return pp::g_tile_cluster;
    if (L->persist_ctas > 0 && pp::g_tile_persist_auto) return 3;
    // Measured on 8192 x 8192 at every density from 6 % to 100 % and batch 16 ... 128: with several warps issuing
    // its tensor-core instructions the one-block-row kernel is the fastest of the three (26 / 36 us against 33 / 44 us
    // of the clustered kernel at density 1, batch 16 / 128), so the other two run only when asked for.
    return 0;
}

pp_status_t pp_layer_launch_info(const pp_layer_t* L, int batch, int32_t out[6]) {
    if (!L || !out || batch < 1) return PP_ERR_INVALID_ARG;
    const pp_packed* pk = L->pk;
    for (int i = 0; i < 6; ++i) out[i] = 0;
    if (L->tile_ok && pp::g_tile_min_batch > 0 && batch >= pp::g_tile_min_batch && (size_t)pk->N * 2 <= 48 * 1024) {
        const int kernel = pick_tile_kernel(L);
        out[0] = kernel == 3 ? 4 : kernel == 2 ? 3 : 2;
        out[1] = kernel == 3 ? L->persist_ctas : kernel == 2 ? (pk->Mb + pp::kTileRows - 1) / pp::kTileRows * pp::kTileRows : pk->Mb;
        return PP_OK;
    }
    const int nb = batch < pp::kStreamMaxBatch ? batch : pp::kStreamMaxBatch;
    const int stage = pp::g_use_stream ? pick_stage_mode(L, true, true, true, pk->N, nb) : -1;
    const int chunk_group = pp::gemv_group_batch(pk->wdtype);
    const bool stream_path = stage >= 0 && (batch + pp::kStreamMaxBatch - 1) / pp::kStreamMaxBatch <= (batch + chunk_group - 1) / chunk_group;
    if (!stream_path) { out[0] = 0; out[1] = L->n_items; return PP_OK; }
    out[0] = 1; out[1] = L->stream_grid; out[4] = stage;
    out[2] = pp::stream_pick_depth(pk->wdtype, pk->B, pk->Npad, pk->N, L->stream_max_rows, nb, stage, L->stream_grid,
                                   pp::stream_frags_per_warp(pk->cta_desc.data(), L->stream_grid));
    out[3] = (int32_t)pp::stream_launch_smem(pk->wdtype, pk->B, pk->Npad, pk->N, L->stream_max_rows, nb, stage, out[2]);
    out[5] = pp::g_stream_pdl;
    return PP_OK;
}

pp_status_t pp_layer_destroy(pp_layer_t* layer) {
    free_layer(layer);
    return PP_OK;
}

// One layer forward; pivoted: y is float[batch][M_pad] in pivoted row order (no output index array).
// x_ready: the caller's promise of tuning key 17 (only the persistent kernels act on it; a pre-pass or the copy of
// pp_forward_host produces x inside the stream, so those paths never pass it on).
static pp_status_t forward_impl(pp_layer* L, const void* x, void* y, int batch, pp_act_t act, cudaStream_t stream, bool pivoted,
                                bool x_ready = false) {
    const pp_packed* pk = L->pk;
    const int ldy = pivoted ? pk->Mpad : pk->M;
    if (L->tile_ok && pp::g_tile_min_batch > 0 && batch >= pp::g_tile_min_batch && (size_t)pk->N * 2 <= 48 * 1024) {
        // tensor-core tile path, 128 batch rows at a time
        pp::TileArgs t{};
        t.row_ptr = L->d_row_ptr; t.col_ptr = L->d_col_ptr; t.tile_col = L->d_tile_col;
        t.scatter_idx = L->d_scatter; t.bias_piv = L->d_bias; t.status = L->d_status;
        t.tiles_sw = static_cast<const unsigned char*>(L->d_tiles_rm); t.x_sw = static_cast<const unsigned char*>(L->d_x_piv);
        t.ldy = ldy; t.act = (int)act; t.pivoted = pivoted ? 1 : 0;
        t.steps = L->d_tile_steps; t.parts = L->d_tile_parts; t.Mb = pk->Mb; t.tile_pos = L->d_tile_pos;
        t.units = L->d_units; t.cta_unit = L->d_cta_unit; t.unit_partials = L->d_unit_partials;
        t.group_sync = L->d_group_sync; t.persist_ctas = L->persist_ctas;
        const int kernel = pick_tile_kernel(L);
        for (int b0 = 0; b0 < batch; b0 += pp::kTileBatch) {
            t.batch = batch - b0 < pp::kTileBatch ? batch - b0 : pp::kTileBatch;
            t.y = static_cast<float*>(y) + (size_t)b0 * ldy;
            const char* xc = static_cast<const char*>(x) + (size_t)b0 * pk->N * 2;
            if (pp::launch_tile(t, xc, pk->N, pk->N, L->d_gather, pk->Npad, pk->Mb, kernel, stream) != cudaSuccess)
                return PP_ERR_CUDA;
        }
        return PP_OK;
    }
    return run_layer(L, L->d_gather, x, pk->N, pk->N, pk->wdtype == PP_F16 ? 2 : 4, y, ldy,
                     pivoted ? pp::OUT_PIVOTED_F32 : pp::OUT_SCATTER_F32, batch, act, stream, -1, nullptr, x_ready);
}

pp_status_t pp_forward(pp_layer_t* L, const void* x, void* y, int batch, pp_act_t act, void* cuda_stream) {
    if (!L || !x || !y || batch < 1 || x == y) return PP_ERR_INVALID_ARG;
    if (act != PP_ACT_IDENTITY && act != PP_ACT_RELU) return PP_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(y)) return PP_ERR_INVALID_ARG;
    return forward_impl(L, x, y, batch, act, static_cast<cudaStream_t>(cuda_stream), false, pp::g_stream_x_ready != 0);
}

namespace {

// Copies between the layer's staging buffers and page-locked host memory that the device can address: a few CTAs
// move 16-byte words (bytes where a pointer or the length is not a multiple of 16), which costs one trip over the
// host link instead of the set-up of a copy engine transfer.  The kernel lets the next launch start at once and
// waits for the previous one itself (programmatic stream serialization; both are no-ops in a plain launch).
__global__ void __launch_bounds__(1024) host_link_copy_kernel(unsigned char* __restrict__ dst,
                                                              const unsigned char* __restrict__ src, size_t bytes) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const size_t tid = (size_t)blockIdx.x * blockDim.x + threadIdx.x, nthr = (size_t)gridDim.x * blockDim.x;
    if (((reinterpret_cast<uintptr_t>(dst) | reinterpret_cast<uintptr_t>(src)) & 15) == 0) {
        const size_t words = bytes / 16;
        for (size_t i = tid; i < words; i += nthr)
            reinterpret_cast<uint4*>(dst)[i] = reinterpret_cast<const uint4*>(src)[i];
        for (size_t i = words * 16 + tid; i < bytes; i += nthr) dst[i] = src[i];
    } else {
        for (size_t i = tid; i < bytes; i += nthr) dst[i] = src[i];
    }
}

// Device address of a host pointer if it lies in page-locked memory mapped into the device's address space
// (cudaHostAlloc, cudaHostRegister), nullptr otherwise (pageable memory, or the query failed).
void* device_view_of_host(const void* host) {
    cudaPointerAttributes attr{};
    if (cudaPointerGetAttributes(&attr, host) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    return attr.type == cudaMemoryTypeHost ? attr.devicePointer : nullptr;
}

cudaError_t launch_host_link_copy(void* dst, const void* src, size_t bytes, bool dependent, cudaStream_t stream) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)std::min<size_t>(64, (bytes + 16383) / 16384));
    cfg.blockDim = dim3(1024);
    cfg.stream = stream;
    cudaLaunchAttribute at{};
    at.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &at;
    cfg.numAttrs = dependent ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, host_link_copy_kernel, static_cast<unsigned char*>(dst),
                              static_cast<const unsigned char*>(src), bytes);
}

}  // namespace

pp_status_t pp_forward_host(pp_layer_t* L, const void* x_host, float* y_host, int batch, pp_act_t act, void* cuda_stream) {
    if (!L || !x_host || !y_host || batch < 1) return PP_ERR_INVALID_ARG;
    if (act != PP_ACT_IDENTITY && act != PP_ACT_RELU) return PP_ERR_INVALID_ARG;
    const pp_packed* pk = L->pk;
    const size_t esz = pk->wdtype == PP_F16 ? 2 : 4;
    if (batch > L->host_batch) {          // first call, or a larger batch than any before: (re)allocate the staging buffers
        cudaFree(L->d_host_x); cudaFree(L->d_host_y);
        L->d_host_x = nullptr; L->d_host_y = nullptr; L->host_batch = 0;
        if (cudaMalloc(reinterpret_cast<void**>(&L->d_host_x), (size_t)batch * pk->N * esz) != cudaSuccess ||
            cudaMalloc(reinterpret_cast<void**>(&L->d_host_y), (size_t)batch * pk->M * 4) != cudaSuccess) {
            cudaGetLastError();
            cudaFree(L->d_host_x); L->d_host_x = nullptr;
            return PP_ERR_ALLOC;
        }
        L->host_batch = batch;
    }
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const size_t xbytes = (size_t)batch * pk->N * esz, ybytes = (size_t)batch * pk->M * 4;
    // Page-locked buffers the device can address are moved by small kernels (no copy-engine set-up, and the layer
    // kernel's prologue runs under the inbound copy); anything else goes through cudaMemcpyAsync.
    void* xv = pp::g_host_link_kernels ? device_view_of_host(x_host) : nullptr;
    void* yv = xv ? device_view_of_host(y_host) : nullptr;
    if (xv && yv) {
        if (launch_host_link_copy(L->d_host_x, xv, xbytes, false, stream) != cudaSuccess) return PP_ERR_CUDA;
        const pp_status_t st = forward_impl(L, L->d_host_x, L->d_host_y, batch, act, stream, false);
        if (st != PP_OK) return st;
        if (launch_host_link_copy(yv, L->d_host_y, ybytes, pp::g_stream_pdl != 0, stream) != cudaSuccess ||
            cudaStreamSynchronize(stream) != cudaSuccess)
            return PP_ERR_CUDA;
        return PP_OK;
    }
    if (cudaMemcpyAsync(L->d_host_x, x_host, xbytes, cudaMemcpyHostToDevice, stream) != cudaSuccess)
        return PP_ERR_CUDA;
    const pp_status_t st = forward_impl(L, L->d_host_x, L->d_host_y, batch, act, stream, false);
    if (st != PP_OK) return st;
    if (cudaMemcpyAsync(y_host, L->d_host_y, ybytes, cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
        cudaStreamSynchronize(stream) != cudaSuccess)
        return PP_ERR_CUDA;
    return PP_OK;
}

pp_status_t pp_layer_output_map(const pp_layer_t* L, int32_t* map) {
    if (!L || !map) return PP_ERR_INVALID_ARG;
    const pp_packed* pk = L->pk;
    for (int i = 0; i < pk->Mpad; ++i) map[i] = pk->row_perm[(size_t)i] < pk->M ? pk->row_perm[(size_t)i] : -1;
    return PP_OK;
}

pp_status_t pp_forward_pivoted(pp_layer_t* L, const void* x, float* y_piv, int batch, pp_act_t act, void* cuda_stream) {
    if (!L || !x || !y_piv || batch < 1 || x == static_cast<const void*>(y_piv)) return PP_ERR_INVALID_ARG;
    if (act != PP_ACT_IDENTITY && act != PP_ACT_RELU) return PP_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(y_piv)) return PP_ERR_INVALID_ARG;
    return forward_impl(L, x, y_piv, batch, act, static_cast<cudaStream_t>(cuda_stream), true, pp::g_stream_x_ready != 0);
}

pp_status_t pp_chain_create(pp_chain_t** out, pp_layer_t* const* layers, const pp_act_t* acts, int n_layers,
                            int max_batch) {
    if (!out) return PP_ERR_INVALID_ARG;
    *out = nullptr;
    if (!layers || !acts || n_layers < 1 || max_batch < 1) return PP_ERR_INVALID_ARG;
    for (int l = 0; l < n_layers; ++l) {
        if (!layers[l]) return PP_ERR_INVALID_ARG;
        if (acts[l] != PP_ACT_IDENTITY && acts[l] != PP_ACT_RELU) return PP_ERR_INVALID_ARG;
        if (l > 0 && layers[l]->pk->N != layers[l - 1]->pk->M) return PP_ERR_INVALID_ARG;
    }
    pp_chain* C = new (std::nothrow) pp_chain();
    if (!C) return PP_ERR_ALLOC;
    C->layers.assign(layers, layers + n_layers);
    C->acts.assign(acts, acts + n_layers);
    C->max_batch = max_batch;
    C->d_q.assign((size_t)n_layers, nullptr);
    C->d_inter.assign((size_t)n_layers, nullptr);
    C->identity.assign((size_t)n_layers, 0);
    bool ok = true;
    pp_status_t st = PP_OK;
    for (int l = 1; l < n_layers && ok; ++l) {
        const pp_packed* A = layers[l - 1]->pk;
        const pp_packed* Bk = layers[l]->pk;
        std::vector<int32_t> q((size_t)Bk->Npad);
        st = pp_fold_perm(A->row_perm.data(), A->M, A->Mpad, Bk->col_perm.data(), Bk->N, Bk->Npad, q.data());
        if (st != PP_OK) { ok = false; break; }
        // q gathers (consumer column j <- producer row q[j]); the chain applies it on the store side:
        // producer row i -> consumer column j with q[j] == i.  The consumer then reads its input in
        // its own pivoted order with no index array at all; its padding columns stay zero.
        std::vector<int32_t> store((size_t)A->Mpad, -1);
        for (int j = 0; j < Bk->Npad; ++j)
            if (q[(size_t)j] >= 0) store[(size_t)q[(size_t)j]] = j;
        // Section 4.2.3: when every real producer row already sits at its consumer column (and the two
        // padded lengths agree), the producer stores its pivoted rows as they are -- no index array on
        // either side of the link.  Padding rows hold act(0) = 0 and land on padding columns.
        bool ident = A->Mpad == Bk->Npad;
        for (int i = 0; i < A->Mpad && ident; ++i) ident = store[(size_t)i] == i || store[(size_t)i] < 0;
        C->identity[(size_t)l] = ident ? 1 : 0;
        ok = upload(&C->d_q[(size_t)l], store.data(), store.size() * 4);
        const size_t elt = Bk->wdtype == PP_F16 ? 2 : 4;
        const size_t ibytes = (size_t)max_batch * Bk->Npad * elt;
        ok = ok && cudaMalloc(&C->d_inter[(size_t)l - 1], ibytes) == cudaSuccess &&
             cudaMemset(C->d_inter[(size_t)l - 1], 0, ibytes) == cudaSuccess;
        if (!ok) st = PP_ERR_ALLOC;
    }
    if (ok) {
        ok = cudaMalloc(reinterpret_cast<void**>(&C->d_fused_args), sizeof(pp::StreamArgs) * pp::kStreamMaxBatch * (size_t)n_layers) == cudaSuccess &&
             cudaMalloc(reinterpret_cast<void**>(&C->d_fused_grids), 4 * (size_t)n_layers) == cudaSuccess &&
             cudaMalloc(reinterpret_cast<void**>(&C->d_fused_sync), 256) == cudaSuccess &&
             cudaMemset(C->d_fused_sync, 0, 256) == cudaSuccess;
        if (!ok) st = PP_ERR_ALLOC;
    }
    if (!ok) {
        cudaGetLastError();
        pp_chain_destroy(C);
        return st;
    }
    chain_plan_fused(C);
    *out = C;
    return PP_OK;
}

pp_status_t pp_chain_destroy(pp_chain_t* C) {
    if (!C) return PP_OK;
    for (int32_t* q : C->d_q) cudaFree(q);
    for (void* b : C->d_inter) cudaFree(b);
    cudaFree(C->d_fused_args); cudaFree(C->d_fused_grids); cudaFree(C->d_fused_sync);
    delete C;
    return PP_OK;
}

}  // extern "C"

namespace {

// What layer l of a chain reads and writes: layer 0 gathers the call's x through its own column index array; every
// later layer finds its input already in its pivoted column order (written there by its producer's epilogue).
struct ChainLink {
    const int32_t* gather; const void* x; int ldx, x_len, x_limit;
    void* y; int ldy, out_mode; const int32_t* scatter;
};
ChainLink chain_link(const pp_chain* C, int l, const void* x, void* y) {
    const int n = (int)C->layers.size();
    const pp_layer* L = C->layers[(size_t)l];
    const pp_packed* pk = L->pk;
    ChainLink k{};
    k.gather = l == 0 ? L->d_gather : nullptr;
    k.x = l == 0 ? x : C->d_inter[(size_t)l - 1];
    k.ldx = k.x_len = k.x_limit = l == 0 ? pk->N : pk->Npad;
    k.scatter = L->d_scatter;
    if (l == n - 1) {
        k.y = y;
        k.ldy = C->out_pivoted ? pk->Mpad : pk->M;
        k.out_mode = C->out_pivoted ? pp::OUT_PIVOTED_F32 : pp::OUT_SCATTER_F32;
    } else {
        const pp_packed* nx = C->layers[(size_t)l + 1]->pk;
        const bool f16 = nx->wdtype == PP_F16;
        k.y = C->d_inter[(size_t)l];
        k.ldy = nx->Npad;
        if (C->identity[(size_t)l + 1] && pp::g_link_identity) {
            k.out_mode = f16 ? pp::OUT_PIVOTED_F16 : pp::OUT_PIVOTED_F32;
        } else {
            k.out_mode = f16 ? pp::OUT_SCATTER_F16 : pp::OUT_SCATTER_F32;
            k.scatter = C->d_q[(size_t)l + 1];
        }
    }
    return k;
}

// One-kernel execution of the chain: possible when every layer is fp16, its input fits the persistent kernel's
// bulk-copy staging for the batch, and the largest plan is resident at once.  (Re)builds the per-batch argument
// arrays; leaves fused_grid = 0 when the chain does not qualify.
void chain_plan_fused(pp_chain* C) {
    const int n = (int)C->layers.size();
    C->fused_grid = 0;
    for (size_t b = 0; b <= (size_t)pp::kStreamMaxBatch; ++b) { C->fused_region[b] = 0; C->fused_depth[b] = 0; }
    if (n < 2 || n > pp::kChainMaxLayers || !pp::g_chain_fused || !pp::g_use_stream) return;
    int grid = 0;
    std::vector<int> grids((size_t)n);
    for (int l = 0; l < n; ++l) {
        const pp_layer* L = C->layers[(size_t)l];
        if (L->pk->wdtype != PP_F16 || L->stream_grid < 1) return;
        grids[(size_t)l] = L->stream_grid;
        grid = std::max(grid, L->stream_grid);
    }
    std::vector<pp::StreamArgs> args((size_t)pp::kStreamMaxBatch * n);
    const int top = std::min(C->max_batch, pp::kStreamMaxBatch);
    bool any = false;
    for (int batch = 1; batch <= top; ++batch) {
        size_t region[2] = {0, 0};                            // at 4 and at 8 weight copies per warp
        bool ok = true;
        for (int l = 0; l < n && ok; ++l) {
            const pp_layer* L = C->layers[(size_t)l];
            const pp_packed* pk = L->pk;
            const ChainLink k = chain_link(C, l, nullptr, nullptr);
            const bool rows_aligned = batch == 1 || ((size_t)k.ldx * 2) % 16 == 0;
            const int stage = pick_stage_mode(L, k.gather != nullptr, true, rows_aligned, k.x_len, batch);
            if (stage < 1) { ok = false; break; }            // x must arrive by bulk copy
            pp::StreamArgs a = make_stream_args(L, k.gather, k.x, k.ldx, k.x_len, k.y, k.ldy, k.out_mode, batch,
                                                C->acts[(size_t)l], k.x_limit, k.scatter, stage);
            pp::stream_finish_args(PP_F16, a);
            a.status = reinterpret_cast<int*>(C->d_fused_sync + 1);
            args[(size_t)(batch - 1) * n + l] = a;
            for (int q = 0; q < 2; ++q)
                region[q] = std::max(region[q], pp::stream_launch_smem(PP_F16, pk->B, pk->Npad, k.x_len, L->stream_max_rows,
                                                                       batch, stage, q ? 8 : 4));
        }
        if (!ok) continue;
        // the deeper ring when two regions of it fit and the plans stay resident, else the shallow one
        for (int q = 1; q >= 0; --q) {
            const size_t r = (region[q] + 1023) / 1024 * 1024;
            if (2 * r <= pp::kStreamSmemLimit && pp::chain_resident_ctas(2 * r, q ? 8 : 4) >= grid) {
                C->fused_region[(size_t)batch] = r;
                C->fused_depth[(size_t)batch] = q ? 8 : 4;
                any = true;
                break;
            }
        }
    }
    if (!any) return;
    if (cudaMemcpy(C->d_fused_args, args.data(), args.size() * sizeof(pp::StreamArgs), cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMemcpy(C->d_fused_grids, grids.data(), (size_t)n * 4, cudaMemcpyHostToDevice) != cudaSuccess) {
        cudaGetLastError();
        return;
    }
    C->fused_grid = grid;
}

}  // namespace

extern "C" {

pp_status_t pp_chain_forward(pp_chain_t* C, const void* x, void* y, int batch, void* cuda_stream) {
    if (!C || !x || !y || batch < 1 || batch > C->max_batch || x == y) return PP_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(y)) return PP_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const int n = (int)C->layers.size();
    if (C->fused_grid > 0 && batch <= pp::kStreamMaxBatch && C->fused_region[(size_t)batch] > 0 && pp::g_chain_fused) {
        // all layers in one cooperative kernel, the grid meeting at a counter between layers
        pp::ChainLaunch P{};
        P.layers = C->d_fused_args + (size_t)(batch - 1) * n;
        P.grids = C->d_fused_grids;
        P.x = x; P.y = y;
        P.counter = C->d_fused_sync; P.status = reinterpret_cast<int*>(C->d_fused_sync + 1);
        P.n_layers = n; P.polls = 0; P.region_bytes = (int)C->fused_region[(size_t)batch];
        return pp::launch_chain_f16(P, C->fused_grid, 2 * C->fused_region[(size_t)batch], C->fused_depth[(size_t)batch], stream) == cudaSuccess
                   ? PP_OK : PP_ERR_CUDA;
    }
    for (int l = 0; l < n; ++l) {
        pp_layer* L = C->layers[(size_t)l];
        const ChainLink k = chain_link(C, l, x, y);
        const pp_status_t st = run_layer(L, k.gather, k.x, k.ldx, k.x_len, L->pk->wdtype == PP_F16 ? 2 : 4, k.y, k.ldy, k.out_mode,
                                         batch, C->acts[(size_t)l], stream, k.x_limit, k.scatter);
        if (st != PP_OK) return st;
    }
    return PP_OK;
}

pp_status_t pp_chain_status(pp_chain_t* C, pp_status_t* status) {
    if (!C || !status) return PP_ERR_INVALID_ARG;
    *status = PP_OK;
    unsigned words[2] = {0u, 0u};
    if (cudaDeviceSynchronize() != cudaSuccess ||
        cudaMemcpy(words, C->d_fused_sync, sizeof(words), cudaMemcpyDeviceToHost) != cudaSuccess) return PP_ERR_CUDA;
    if (words[1]) {
        *status = PP_ERR_TIMEOUT;        // the launch that gave up left its arrival counter behind: clear both
        if (cudaMemset(C->d_fused_sync, 0, sizeof(words)) != cudaSuccess) return PP_ERR_CUDA;
    }
    for (pp_layer* L : C->layers) {      // layer-by-layer execution raises the layers' own words
        pp_status_t st = PP_OK;
        const pp_status_t rc = pp_layer_status(L, &st);
        if (rc != PP_OK) return rc;
        if (st != PP_OK) *status = st;
    }
    return PP_OK;
}

pp_status_t pp_chain_set_output_pivoted(pp_chain_t* C, int enable) {
    if (!C || (enable != 0 && enable != 1)) return PP_ERR_INVALID_ARG;
    C->out_pivoted = enable != 0;
    chain_plan_fused(C);                 // the last layer's store mode is part of the one-kernel arguments
    return PP_OK;
}

pp_status_t pp_chain_output_map(const pp_chain_t* C, int32_t* map) {
    if (!C || !map) return PP_ERR_INVALID_ARG;
    return pp_layer_output_map(C->layers.back(), map);
}

pp_status_t pp_chain_link_info(const pp_chain_t* C, int32_t* identity) {
    if (!C || !identity) return PP_ERR_INVALID_ARG;
    for (size_t l = 0; l < C->layers.size(); ++l) identity[l] = C->identity[l];
    return PP_OK;
}

pp_status_t pp_lstm_status(pp_lstm_t* R, pp_status_t* status) {
    if (!R || !status) return PP_ERR_INVALID_ARG;
    unsigned int flag = 0;
    if (cudaDeviceSynchronize() != cudaSuccess) return PP_ERR_CUDA;
    if (cudaMemcpy(&flag, R->d_sync + 1, sizeof(flag), cudaMemcpyDeviceToHost) != cudaSuccess) return PP_ERR_CUDA;
    *status = flag ? PP_ERR_TIMEOUT : PP_OK;
    if (flag && cudaMemset(R->d_sync + 1, 0, sizeof(flag)) != cudaSuccess) return PP_ERR_CUDA;
    pp_status_t layer_st = PP_OK;                 // the per-step path raises the gate layer's own word
    const pp_status_t rc = pp_layer_status(R->gates, &layer_st);
    if (rc != PP_OK) return rc;
    if (layer_st != PP_OK) *status = layer_st;
    return PP_OK;
}

pp_status_t pp_lstm_create(pp_lstm_t** out, pp_layer_t* gates, int I, int H, int max_steps) {
    if (!out) return PP_ERR_INVALID_ARG;
    *out = nullptr;
    if (!gates || I < 1 || H < 1 || max_steps < 1) return PP_ERR_INVALID_ARG;
    const pp_packed* pk = gates->pk;
    if (pk->M != 4 * H || pk->N != I + H) return PP_ERR_INVALID_ARG;
    pp_lstm* R = new (std::nothrow) pp_lstm();
    if (!R) return PP_ERR_ALLOC;
    R->gates = gates; R->I = I; R->H = H; R->max_steps = max_steps;
    std::vector<int32_t> inv_col((size_t)pk->Npad);
    for (int j = 0; j < pk->Npad; ++j) inv_col[(size_t)pk->col_perm[(size_t)j]] = j;
    const size_t elt = pk->wdtype == PP_F16 ? 2 : 4;
    const bool ok = upload(&R->d_inv_row, pk->inv_row_perm.data(), pk->inv_row_perm.size() * 4) &&
                    upload(&R->d_inv_col, inv_col.data(), inv_col.size() * 4) &&
                    cudaMalloc(&R->d_z, (size_t)(max_steps + 1) * pk->Npad * elt) == cudaSuccess &&
                    cudaMalloc(reinterpret_cast<void**>(&R->d_g), 2 * (size_t)pk->Mpad * 8) == cudaSuccess &&
                    cudaMalloc(reinterpret_cast<void**>(&R->d_sync), 2 * sizeof(unsigned int)) == cudaSuccess &&
                    cudaMemset(R->d_sync, 0, 2 * sizeof(unsigned int)) == cudaSuccess;
    if (ok) lstm_plan_persistent(R);
    if (!ok) {
        const cudaError_t e = cudaGetLastError();
        pp_lstm_destroy(R);
        return e == cudaErrorMemoryAllocation ? PP_ERR_ALLOC : PP_ERR_CUDA;
    }
    *out = R;
    return PP_OK;
}

pp_status_t pp_lstm_destroy(pp_lstm_t* R) {
    if (!R) return PP_OK;
    cudaFree(R->d_inv_row); cudaFree(R->d_inv_col); cudaFree(R->d_z); cudaFree(R->d_g); cudaFree(R->d_sync);
    delete R;
    return PP_OK;
}

pp_status_t pp_lstm_forward(pp_lstm_t* R, const void* x_seq, void* h, float* c, int steps, void* cuda_stream) {
    if (!R || !x_seq || !h || !c || steps < 1 || steps > R->max_steps) return PP_ERR_INVALID_ARG;
    if (!aligned16(x_seq) || !aligned16(h) || !aligned16(c)) return PP_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    pp_layer* L = R->gates;
    const pp_packed* pk = L->pk;
    const int elt = pk->wdtype == PP_F16 ? 2 : 4;
    pp::LstmArgs a{};
    a.gather_idx = L->d_gather; a.inv_row = R->d_inv_row; a.inv_col = R->d_inv_col;
    a.z = R->d_z; a.x_seq = x_seq; a.h = h; a.c = c; a.g_piv = R->d_g;
    a.I = R->I; a.H = R->H; a.n_pad = pk->Npad; a.steps = steps; a.f16 = pk->wdtype == PP_F16;
    if (pp::launch_lstm_prepare(a, stream) != cudaSuccess) return PP_ERR_CUDA;
    if (pp::g_lstm_persist && R->persist_grid > 0) {
        // all steps in one cooperative kernel; no packet of an earlier call may be mistaken for a new one
        if (cudaMemsetAsync(R->d_g, 0, 2 * (size_t)pk->Mpad * 8, stream) != cudaSuccess) return PP_ERR_CUDA;
        pp::LstmPersistArgs q{};
        q.values = L->d_values; q.xoff = L->d_xoff; q.strip_start = L->d_strip_start; q.bias_piv = L->d_bias;
        q.inv_row = R->d_inv_row; q.inv_col = R->d_inv_col; q.z = R->d_z; q.g_pk = reinterpret_cast<uint2*>(R->d_g);
        q.status = reinterpret_cast<int*>(R->d_sync + 1); q.h = h; q.c = c;
        q.I = R->I; q.H = R->H; q.n_pad = pk->Npad; q.m_pad = pk->Mpad; q.steps = steps;
        q.n_strips = (int)pk->strip_start.size() - 1; q.strips_per_cta = R->persist_strips;
        return pp::launch_lstm_persist(q, R->persist_grid, R->persist_smem, stream) == cudaSuccess ? PP_OK : PP_ERR_CUDA;
    }
    for (int t = 0; t < steps; ++t) {
        const char* zt = static_cast<const char*>(R->d_z) + (size_t)t * pk->Npad * elt;
        // the input is already in pivoted order: no gather map, every pivoted column is real
        pp_status_t st = run_layer(L, nullptr, zt, pk->Npad, pk->Npad, elt, R->d_g, pk->Mpad, pp::OUT_PIVOTED_F32, 1,
                                   PP_ACT_IDENTITY, stream, pk->Npad);
        if (st != PP_OK) return st;
        if (pp::launch_lstm_gates(a, t, stream) != cudaSuccess) return PP_ERR_CUDA;
    }
    return PP_OK;
}

}  // extern "C"
