// Host-side pivot-format packer: validation, block-row-compressed index arrays,
// fragment-ordered tile values, pivoted bias, work list, permutation folding.
// Pure host code (no CUDA calls), so it can be exercised without a GPU.
#include <algorithm>
#include <cstring>
#include <new>
#include <numeric>

#include "pp_internal.h"
#include "pp_tile.cuh"

namespace pp {
int g_use_stream = 1;      // 0: the API never picks the persistent kernel
int g_tile_min_batch = 9;
int g_prepass = 1;
int g_lstm_persist = 1;
int g_tile_cluster = 1;
int g_tile_persist_auto = 0;
int g_link_identity = 1;
int g_host_link_kernels = 1;   // pp_forward_host: page-locked, device-addressable host buffers are moved by kernels
int g_chain_fused = 0;      // measured: one launch per layer (programmatic dependent launch) is the faster way through a chain
extern int g_stream_wait_polls;   // poll limit of the bounded device-side waits (pp_stream.cu)
int g_stage_direct = 2;    // 0: always materialise the pivoted x in shared memory; 1: one input vector is read through the
                           // index array in the multiply loop; 2: so are 2..8 vectors of fp16 layers
extern int g_stream_depth; // weight-ring slots per warp of the persistent kernel (pp_stream.cu)
extern int g_stream_pdl;   // programmatic dependent launch of the persistent kernel (pp_stream.cu)
extern int g_stream_x_ready;   // pp_forward fetches x before the dependency wait (pp_stream.cu)
}

namespace {

int g_target_kib = 32;     // tile-value kilobytes per work item
int g_min_items = 296;     // the splitter keeps halving the run length until it has this many items
int g_stream_ctas = 296;   // CTAs of the persistent kernel (2 per SM on a 148-SM part)
int g_stream_sms = 148;    // SMs the partition is balanced for
int g_stream_min_frags = 128;  // fewer CTAs are used rather than giving one less than this many fragments
int g_stream_snap_pct = -1;    // >= 0: manual partition, a CTA boundary within this % of a CTA's share of a
                               // strip boundary moves onto it; -1: the packer picks the partition itself

bool is_bijection(const int32_t* p, int64_t n) {
    std::vector<unsigned char> seen((size_t)n, 0);
    for (int64_t k = 0; k < n; ++k) {
        if (p[k] < 0 || p[k] >= n || seen[(size_t)p[k]]) return false;
        seen[(size_t)p[k]] = 1;
    }
    return true;
}

// Byte offset, inside a 512-byte fragment, of tile element (r, c) relative to the
// fragment's origin, plus which fragment (rg, f) it falls in.
struct ElemPos { int rg, f, byte; };

inline ElemPos elem_pos(pp_dtype_t dt, const pp::FragGeom& g, int r, int c) {
    ElemPos e;
    if (dt == PP_F16) {
        // 16x16 operand fragment of the warp-level matrix-multiply instruction: lane = 4*(row%8) + (col%8)/2,
        // element slot = (col%2) + 2*(row/8) + 4*(col/8)  -> 8 halves (16 bytes) per lane.
        e.rg = r / 16; e.f = c / 16;
        int rr = r % 16, cc = c % 16;
        int lane = 4 * (rr % 8) + (cc % 8) / 2;
        int slot = (cc % 2) + 2 * (rr / 8) + 4 * (cc / 8);
        e.byte = lane * 16 + slot * 2;
    } else {
        // lane = row (and, for 16-row tiles, which half of the 8 columns); 4 consecutive columns per lane.
        e.rg = r / g.rg_rows; e.f = c / g.kf;
        int rr = r % g.rg_rows, cc = c % g.kf;
        int lane = rr + g.rg_rows * (cc / 4);
        e.byte = lane * 16 + (cc % 4) * 4;
    }
    return e;
}

void build_items(pp_packed* p) {
    const pp::FragGeom g = pp::frag_geom(p->wdtype, p->B);
    const int esz = p->wdtype == PP_F16 ? 2 : 4;
    const int64_t tile_bytes = (int64_t)p->B * p->B * esz;
    int64_t run = std::max<int64_t>(1, (int64_t)g_target_kib * 1024 / tile_bytes);
    run = std::min<int64_t>(run, std::max(1, pp::kMaxRunColumns / p->B));   // staged x must fit shared memory
    auto count_items = [&](int64_t r) {
        int64_t n = 0;
        for (int br = 0; br < p->Mb; ++br) {
            int64_t k = p->row_ptr[br + 1] - p->row_ptr[br];
            n += std::max<int64_t>(1, (k + r - 1) / r);
        }
        return n;
    };
    while (run > 1 && count_items(run) < g_min_items) run = (run + 1) / 2;

    p->items.clear();
    p->max_item_tiles = 0;
    p->n_slots = 0;
    const int frags_per_tile = g.n_rg * g.fpt;
    for (int br = 0; br < p->Mb; ++br) {
        const int k = p->row_ptr[br + 1] - p->row_ptr[br];
        const int nparts = std::max<int>(1, (int)((k + run - 1) / run));
        const int slot_base = nparts > 1 ? p->n_slots : 0;
        if (nparts > 1) p->n_slots += nparts;
        for (int part = 0; part < nparts; ++part) {
            const int j0 = (int)((int64_t)k * part / nparts), j1 = (int)((int64_t)k * (part + 1) / nparts);
            pp::WorkItem it;
            it.frag_base = p->row_ptr[br] * frags_per_tile + j0 * g.fpt;
            it.rg_stride = k * g.fpt;
            it.nf = (j1 - j0) * g.fpt;
            it.col_off = p->col_ptr[br] + j0;
            it.ntiles = j1 - j0;
            it.br = br;
            it.part_nparts = part | (nparts << 16);
            it.slot_base = slot_base;
            p->items.push_back(it);
            p->max_item_tiles = std::max(p->max_item_tiles, j1 - j0);
        }
    }
}

// Plan of the persistent kernel: strips, per-fragment x offsets, one fragment range per CTA.
void build_stream_plan(pp_packed* p) {
    const pp::FragGeom g = pp::frag_geom(p->wdtype, p->B);
    const int S = p->Mb * g.n_rg;
    p->strip_start.assign((size_t)S + 1, 0);
    for (int s = 0; s < S; ++s) {
        const int br = s / g.n_rg;
        p->strip_start[(size_t)s + 1] = p->strip_start[(size_t)s] + (p->row_ptr[(size_t)br + 1] - p->row_ptr[(size_t)br]) * g.fpt;
    }
    const int64_t F = p->strip_start[(size_t)S];
    p->xoff.resize((size_t)F);
    for (int s = 0; s < S; ++s) {
        const int br = s / g.n_rg;
        const int k = p->row_ptr[(size_t)br + 1] - p->row_ptr[(size_t)br];
        for (int j = 0; j < k; ++j)
            for (int f = 0; f < g.fpt; ++f)
                p->xoff[(size_t)p->strip_start[(size_t)s] + (size_t)j * g.fpt + f] =
                    p->tile_col[(size_t)p->col_ptr[(size_t)br] + j] * p->B + f * g.kf;
    }

    // CTA boundaries as (strip, offset) pairs, offset in [0, len); (S, 0) is the end.
    struct Bnd { int s, off; };
    auto less = [](const Bnd& a, const Bnd& b) { return a.s < b.s || (a.s == b.s && a.off < b.off); };
    const Bnd end{S, 0};
    // Even split of the fragment sequence into G ranges; a boundary closer than tol_pct % of a
    // CTA's share to a strip boundary moves onto it (100: every boundary does -> no strip is shared).
    auto make_bounds = [&](int64_t G, int tol_pct) {
        const int64_t share = (F + G - 1) / G;
        const int64_t tol = tol_pct >= 100 ? F : share * tol_pct / 100;
        std::vector<Bnd> bnd;
        bnd.push_back({0, 0});
        for (int64_t c = 1; c < G; ++c) {
            const int64_t pos = F * c / G;
            int s = (int)(std::upper_bound(p->strip_start.begin(), p->strip_start.end(), (int32_t)pos) -
                          p->strip_start.begin()) - 1;      // non-empty strip containing pos
            if (s >= S) continue;
            const int64_t off = pos - p->strip_start[(size_t)s];
            const int64_t len = p->strip_start[(size_t)s + 1] - p->strip_start[(size_t)s];
            Bnd b;
            if (off <= tol && off <= len - off) b = {s, 0};
            else if (len - off <= tol) b = {s + 1, 0};
            else b = {s, (int)off};
            if (less(bnd.back(), b)) bnd.push_back(b);
        }
        while (bnd.size() > 1 && !less(bnd.back(), end)) bnd.pop_back();
        return bnd;
    };
    auto pos_of = [&](const Bnd& b) { return (int64_t)p->strip_start[(size_t)b.s] + b.off; };
    // Rough time of a partition.  CTAs are placed round-robin on the SMs, so SM i carries CTAs
    // i, i + n_sm, ...; the fullest SM at its share of the memory system sets the time.  A strip
    // shared by two CTAs costs one atomic exchange at the end, one shared by more a counter round.
    auto cost_us = [&](const std::vector<Bnd>& bnd) {
        const int n_sm = std::max(1, g_stream_sms);
        std::vector<int64_t> sm_load((size_t)n_sm, 0);
        bool shared = false, shared_many = false;
        for (size_t c = 0; c < bnd.size(); ++c) {
            const Bnd b1 = c + 1 < bnd.size() ? bnd[c + 1] : end;
            sm_load[c % (size_t)n_sm] += pos_of(b1) - pos_of(bnd[c]);
            shared = shared || bnd[c].off > 0;
            shared_many = shared_many || (bnd[c].off > 0 && b1.s == bnd[c].s && b1.off > 0);
        }
        const int64_t max_load = *std::max_element(sm_load.begin(), sm_load.end());
        const double bw_sm = std::min(100e9, 6.0e12 / (double)std::min<size_t>(bnd.size(), (size_t)n_sm));
        return (double)max_load * 512.0 / bw_sm * 1e6 + (shared_many ? 3.0 : shared ? 0.7 : 0.0);
    };
    std::vector<Bnd> bnd;
    if (g_stream_snap_pct >= 0) {       // manual partition (experiments, tests)
        const int64_t G = std::max<int64_t>(1, std::min<int64_t>(g_stream_ctas, F / std::max(1, g_stream_min_frags)));
        bnd = make_bounds(G, g_stream_snap_pct);
    } else {
        int nonempty = 0;
        for (int s = 0; s < S; ++s) nonempty += p->strip_start[(size_t)s + 1] > p->strip_start[(size_t)s];
        const int64_t g_even = std::max<int64_t>(1, std::min<int64_t>(g_stream_ctas, F / 32));
        bnd = make_bounds(g_even, 2);
        double best = cost_us(bnd);
        const int64_t g_hi = std::max<int64_t>(1, std::min<int64_t>(g_stream_ctas, nonempty));
        for (int64_t G = g_hi; G >= std::max<int64_t>(1, g_hi / 2); --G) {
            std::vector<Bnd> cand = make_bounds(G, 100);
            const double c = cost_us(cand);
            if (c < best - 1e-9) { best = c; bnd = std::move(cand); }
        }
    }
    // no CTA may list more than kStreamMaxStrips strips
    std::vector<Bnd> cut;
    for (size_t c = 0; c < bnd.size(); ++c) {
        const Bnd b0 = bnd[c], b1 = c + 1 < bnd.size() ? bnd[c + 1] : end;
        cut.push_back(b0);
        const int listed = b1.s - b0.s + (b1.off > 0 ? 1 : 0);
        for (int q = pp::kStreamMaxStrips; q < listed; q += pp::kStreamMaxStrips) cut.push_back({b0.s + q, 0});
    }
    p->cta_desc.clear();
    p->strip_info.assign((size_t)S, pp::StripInfo{-1, 0, 0, 0});
    for (size_t c = 0; c < cut.size(); ++c) {
        const Bnd b0 = cut[c], b1 = c + 1 < cut.size() ? cut[c + 1] : end;
        pp::CtaDesc d;
        d.p_begin = p->strip_start[(size_t)b0.s] + b0.off;
        d.p_end = p->strip_start[(size_t)b1.s] + b1.off;
        d.s_first = b0.s;
        d.s_count = b1.s - b0.s + (b1.off > 0 ? 1 : 0);
        for (int s = d.s_first; s < d.s_first + d.s_count; ++s) {
            pp::StripInfo& si = p->strip_info[(size_t)s];
            if (si.nparts == 0) si.first_cta = (int)c;
            si.nparts++;
        }
        p->cta_desc.push_back(d);
    }
    p->stream_slots = 0;
    for (int s = 0; s < S; ++s) {
        pp::StripInfo& si = p->strip_info[(size_t)s];
        if (si.nparts > 1) { si.slot_base = p->stream_slots; p->stream_slots += si.nparts; }
    }
}

}  // namespace

namespace pp {
// Plan of the persistent tile kernel for n_ctas CTAs: the step sequence of all groups cut into one contiguous
// range per CTA (equal shares of the cost: an X block counts as two tiles), and the units those ranges make with
// the groups, in (group, step) order.  Every group is covered: one without tiles gets an empty unit, so that its
// rows still receive act(bias).  A CTA's units are consecutive: cta_unit[c] .. cta_unit[c + 1].
void build_tile_units(const pp_packed* pk, int n_ctas, std::vector<TileUnit>& units, std::vector<int32_t>& cta_unit) {
    constexpr int R = kTileRows;
    const int groups = (pk->Mb + R - 1) / R;
    const std::vector<TileStep>& steps = pk->tile_steps;
    const int S = (int)steps.size();
    const int G = std::max(1, n_ctas);
    std::vector<int64_t> cum((size_t)S + 1, 0);
    for (int i = 0; i < S; ++i) cum[(size_t)i + 1] = cum[(size_t)i] + 2 + steps[(size_t)i].ntiles;
    std::vector<int> cta_step((size_t)G + 1, S);
    cta_step[0] = 0;
    for (int c = 1; c < G; ++c) {
        const int64_t want = cum[(size_t)S] * c / G;
        cta_step[(size_t)c] = (int)(std::lower_bound(cum.begin(), cum.end(), want) - cum.begin());
        cta_step[(size_t)c] = std::max(cta_step[(size_t)c], cta_step[(size_t)c - 1]);
    }
    auto owner_of = [&](int step) {                   // the CTA whose range holds this step position
        const int c = (int)(std::upper_bound(cta_step.begin(), cta_step.begin() + G, step) - cta_step.begin()) - 1;
        return std::min(std::max(c, 0), G - 1);
    };
    units.clear();
    std::vector<int> unit_cta;
    for (int g = 0; g < groups; ++g) {
        const int gs = pk->tile_parts[(size_t)g * (R + 1)], ge = pk->tile_parts[(size_t)g * (R + 1) + R];
        const size_t first = units.size();
        if (gs == ge) {
            units.push_back(TileUnit{gs, gs, g, 0, 1, (int32_t)first, {0, 0}});
            unit_cta.push_back(owner_of(std::min(gs, std::max(S - 1, 0))));
        } else {
            for (int s0 = gs; s0 < ge;) {
                const int c = owner_of(s0);
                const int s1 = std::min(ge, std::max(cta_step[(size_t)c + 1], s0 + 1));
                units.push_back(TileUnit{s0, s1, g, (int32_t)(units.size() - first), 0, (int32_t)first, {0, 0}});
                unit_cta.push_back(c);
                s0 = s1;
            }
        }
        for (size_t u = first; u < units.size(); ++u) units[u].n_parts = (int32_t)(units.size() - first);
    }
    cta_unit.assign((size_t)G + 1, (int32_t)units.size());
    size_t u = 0;
    for (int c = 0; c < G; ++c) {
        cta_unit[(size_t)c] = (int32_t)u;
        while (u < units.size() && unit_cta[u] <= c) ++u;      // owners never decrease along the sequence
    }
}
}  // namespace pp

extern "C" {

pp_status_t pp_pack_tile_units(const pp_packed_t* p, int n_ctas, int32_t* units_out, int64_t capacity_units,
                               int64_t* n_units_out, int32_t* cta_unit_out) {
    if (!p || n_ctas < 1 || !n_units_out) return PP_ERR_INVALID_ARG;
    if (p->wdtype != PP_F16 || p->B != 64) return PP_ERR_UNSUPPORTED;
    try {
        std::vector<pp::TileUnit> units;
        std::vector<int32_t> cta_unit;
        pp::build_tile_units(p, n_ctas, units, cta_unit);
        *n_units_out = (int64_t)units.size();
        if (!units_out && !cta_unit_out) return PP_OK;              // count only
        if (!units_out || !cta_unit_out || capacity_units < (int64_t)units.size()) return PP_ERR_INVALID_ARG;
        std::memcpy(units_out, units.data(), units.size() * sizeof(pp::TileUnit));
        std::memcpy(cta_unit_out, cta_unit.data(), cta_unit.size() * 4);
    } catch (const std::bad_alloc&) {
        return PP_ERR_ALLOC;
    }
    return PP_OK;
}

const char* pp_status_string(pp_status_t s) {
    switch (s) {
        case PP_OK: return "ok";
        case PP_ERR_INVALID_ARG: return "invalid argument";
        case PP_ERR_BAD_PERM: return "row_perm/col_perm is not a permutation of its padded range";
        case PP_ERR_BAD_TILE: return "tile out of range or listed twice";
        case PP_ERR_ALLOC: return "allocation failed";
        case PP_ERR_CUDA: return "CUDA runtime error";
        case PP_ERR_UNSUPPORTED: return "unsupported tile size, dtype or batch";
        case PP_ERR_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

// Plan of the clustered tile kernel: per group of kTileRows block-rows the union of their tile-columns
// in ascending order (one step each), cut into kTileRows contiguous parts of about equal bytes
// (16 KiB for the X block of a step + 8 KiB per tile).
static void build_tile_steps(pp_packed* p) {
    constexpr int R = pp::kTileRows;
    const int G = (p->Mb + R - 1) / R;
    p->tile_steps.clear();
    p->tile_parts.assign((size_t)G * (R + 1), 0);
    for (int g = 0; g < G; ++g) {
        const size_t first = p->tile_steps.size();
        std::vector<pp::TileStep> steps;
        std::vector<int32_t> slot_of_col((size_t)p->Nb, -1);
        std::vector<int32_t> cols;
        for (int j = 0; j < R; ++j) {
            const int br = g * R + j;
            if (br >= p->Mb) break;
            const int r0 = p->row_ptr[(size_t)br], k = p->row_ptr[(size_t)br + 1] - r0;
            for (int t = 0; t < k; ++t) {
                const int col = p->tile_col[(size_t)p->col_ptr[(size_t)br] + t];
                if (slot_of_col[(size_t)col] < 0) { slot_of_col[(size_t)col] = 0; cols.push_back(col); }
            }
        }
        std::sort(cols.begin(), cols.end());
        steps.resize(cols.size());
        for (size_t i = 0; i < cols.size(); ++i) {
            slot_of_col[(size_t)cols[i]] = (int32_t)i;
            steps[i].col = cols[i];
            for (int j = 0; j < R; ++j) steps[i].tile[j] = -1;
            steps[i].ntiles = 0; steps[i].pos = 0; steps[i].pad = 0;
        }
        for (int j = 0; j < R; ++j) {
            const int br = g * R + j;
            if (br >= p->Mb) break;
            const int r0 = p->row_ptr[(size_t)br], k = p->row_ptr[(size_t)br + 1] - r0;
            for (int t = 0; t < k; ++t) {
                pp::TileStep& st = steps[(size_t)slot_of_col[(size_t)p->tile_col[(size_t)p->col_ptr[(size_t)br] + t]]];
                st.tile[j] = r0 + t;
                st.ntiles++;
            }
        }
        int64_t total = 0;
        for (const pp::TileStep& st : steps) total += 2 + st.ntiles;
        int32_t* parts = &p->tile_parts[(size_t)g * (R + 1)];
        int64_t run = 0;
        int part = 1;
        parts[0] = (int32_t)first;
        for (size_t i = 0; i < steps.size(); ++i) {
            // the step goes to the part its centre of mass falls into
            while (part < R && (run + (2 + steps[i].ntiles) / 2) * R >= total * part) parts[part++] = (int32_t)(first + i);
            run += 2 + steps[i].ntiles;
        }
        while (part <= R) parts[part++] = (int32_t)(first + steps.size());
        p->tile_steps.insert(p->tile_steps.end(), steps.begin(), steps.end());
    }
    // the tiles of a step lie next to each other (block-rows ascending), steps one after the other
    p->tile_pos.assign((size_t)p->T, 0);
    int32_t pos = 0;
    for (pp::TileStep& st : p->tile_steps) {
        st.pos = pos;
        for (int j = 0; j < R; ++j)
            if (st.tile[j] >= 0) p->tile_pos[(size_t)st.tile[j]] = pos++;
    }
}

// Host-side self-check (no GPU): the per-device "done once" table keeps devices apart, ignores ordinals it has
// no slot for (the setting is then re-applied on every launch there) and starts empty.
pp_status_t pp_selftest_host(void) {
    pp::PerDeviceOnce t;
    for (int d = -1; d <= pp::PerDeviceOnce::kMaxDevices; ++d)
        if (t.is_done(d)) return PP_ERR_INVALID_ARG;
    t.mark(0);
    if (!t.is_done(0) || t.is_done(1)) return PP_ERR_INVALID_ARG;
    t.mark(3);
    t.mark(-1);
    t.mark(pp::PerDeviceOnce::kMaxDevices);
    for (int d = -1; d <= pp::PerDeviceOnce::kMaxDevices; ++d)
        if (t.is_done(d) != (d == 0 || d == 3)) return PP_ERR_INVALID_ARG;
    return PP_OK;
}

pp_status_t pp_set_tuning(int key, int value) {
    if (key == 0 && value >= 1) { g_target_kib = value; return PP_OK; }
    if (key == 1 && value >= 0) { g_min_items = value; return PP_OK; }
    if (key == 2 && value >= 1) { g_stream_ctas = value; return PP_OK; }
    if (key == 3 && value >= 1) { g_stream_min_frags = value; return PP_OK; }
    if (key == 4 && value >= -1 && value <= 100) { g_stream_snap_pct = value; return PP_OK; }
    if (key == 5 && (value == 0 || value == 1)) { pp::g_use_stream = value; return PP_OK; }
    if (key == 6 && (value == 0 || value == 4 || value == 6 || value == 8)) { pp::g_stream_depth = value; return PP_OK; }
    if (key == 7 && value >= 0 && value <= 2) { pp::g_stage_direct = value; return PP_OK; }
    if (key == 8 && (value == 0 || value == 1)) { pp::g_stream_pdl = value; return PP_OK; }
    if (key == 9 && value >= 0) { pp::g_tile_min_batch = value; return PP_OK; }
    if (key == 10 && value >= 0 && value <= 2) { pp::g_prepass = value; return PP_OK; }
    if (key == 11 && (value == 0 || value == 1)) { pp::g_lstm_persist = value; return PP_OK; }
    if (key == 12 && value >= 0 && value <= 3) { pp::g_tile_cluster = value; return PP_OK; }
    if (key == 13 && (value == 0 || value == 1)) { pp::g_link_identity = value; return PP_OK; }
    if (key == 14 && (value == 0 || value == 1)) { pp::g_chain_fused = value; return PP_OK; }
    if (key == 15 && value >= 0) { pp::g_stream_wait_polls = value; return PP_OK; }
    if (key == 16 && (value == 0 || value == 1)) { pp::g_host_link_kernels = value; return PP_OK; }
    if (key == 17 && (value == 0 || value == 1)) { pp::g_stream_x_ready = value; return PP_OK; }
    return PP_ERR_INVALID_ARG;
}

pp_status_t pp_pack_create(pp_packed_t** out, int M, int N, int B, const int32_t* row_perm,
                           const int32_t* col_perm, const int32_t* tile_list, int64_t T,
                           const void* tile_values, pp_dtype_t wdtype, const float* bias) {
    if (!out) return PP_ERR_INVALID_ARG;
    *out = nullptr;
    if (M <= 0 || N <= 0 || B <= 0 || T < 0 || !row_perm || !col_perm) return PP_ERR_INVALID_ARG;
    if (T > 0 && (!tile_list || !tile_values)) return PP_ERR_INVALID_ARG;
    if (wdtype != PP_F32 && wdtype != PP_F16) return PP_ERR_INVALID_ARG;
    if (B != 16 && B != 32 && B != 64) return PP_ERR_UNSUPPORTED;
    const int Mb = (M + B - 1) / B, Nb = (N + B - 1) / B;
    const int64_t Mpad = (int64_t)Mb * B, Npad = (int64_t)Nb * B;
    if (Mpad > INT32_MAX || Npad > INT32_MAX || T > (int64_t)Mb * Nb) {
        if (T > (int64_t)Mb * Nb) return PP_ERR_BAD_TILE;
        return PP_ERR_INVALID_ARG;
    }
    if (!is_bijection(row_perm, Mpad) || !is_bijection(col_perm, Npad)) return PP_ERR_BAD_PERM;

    pp_packed* p = new (std::nothrow) pp_packed();
    if (!p) return PP_ERR_ALLOC;
    try {
        p->M = M; p->N = N; p->B = B; p->Mb = Mb; p->Nb = Nb; p->Mpad = (int)Mpad; p->Npad = (int)Npad;
        p->T = T; p->wdtype = wdtype; p->has_bias = bias != nullptr;
        p->row_perm.assign(row_perm, row_perm + Mpad);
        p->col_perm.assign(col_perm, col_perm + Npad);
        p->inv_row_perm.resize((size_t)Mpad);
        for (int64_t i = 0; i < Mpad; ++i) p->inv_row_perm[(size_t)row_perm[i]] = (int32_t)i;

        // sort tiles by (block_row, block_col), rejecting out-of-range and duplicate tiles
        std::vector<int64_t> order((size_t)T);
        std::iota(order.begin(), order.end(), 0);
        for (int64_t t = 0; t < T; ++t) {
            const int32_t br = tile_list[2 * t], bc = tile_list[2 * t + 1];
            if (br < 0 || br >= Mb || bc < 0 || bc >= Nb) { delete p; return PP_ERR_BAD_TILE; }
        }
        std::sort(order.begin(), order.end(), [&](int64_t a, int64_t b) {
            const int64_t ka = (int64_t)tile_list[2 * a] * Nb + tile_list[2 * a + 1];
            const int64_t kb = (int64_t)tile_list[2 * b] * Nb + tile_list[2 * b + 1];
            return ka < kb;
        });
        for (int64_t s = 1; s < T; ++s) {
            const int64_t a = order[(size_t)s - 1], b = order[(size_t)s];
            if (tile_list[2 * a] == tile_list[2 * b] && tile_list[2 * a + 1] == tile_list[2 * b + 1]) {
                delete p; return PP_ERR_BAD_TILE;
            }
        }

        // block-row-compressed index arrays; each block-row's column list padded to 4 entries with -1
        p->row_ptr.assign((size_t)Mb + 1, 0);
        for (int64_t t = 0; t < T; ++t) p->row_ptr[(size_t)tile_list[2 * t] + 1]++;
        for (int br = 0; br < Mb; ++br) p->row_ptr[(size_t)br + 1] += p->row_ptr[(size_t)br];
        p->col_ptr.assign((size_t)Mb + 1, 0);
        for (int br = 0; br < Mb; ++br) {
            const int k = p->row_ptr[(size_t)br + 1] - p->row_ptr[(size_t)br];
            p->col_ptr[(size_t)br + 1] = p->col_ptr[(size_t)br] + (k + 3) / 4 * 4;
        }
        p->tile_col.assign((size_t)p->col_ptr[(size_t)Mb], -1);
        for (int br = 0; br < Mb; ++br)
            for (int s = p->row_ptr[(size_t)br]; s < p->row_ptr[(size_t)br + 1]; ++s)
                p->tile_col[(size_t)(p->col_ptr[(size_t)br] + s - p->row_ptr[(size_t)br])] =
                    tile_list[2 * order[(size_t)s] + 1];

        // tile values -> fragment order
        const pp::FragGeom g = pp::frag_geom(wdtype, B);
        const int esz = wdtype == PP_F16 ? 2 : 4;
        const int frags_per_tile = g.n_rg * g.fpt;
        p->values.assign((size_t)T * B * B * esz, 0);
        const unsigned char* src = static_cast<const unsigned char*>(tile_values);
        // Entries of a tile on padding rows or padding columns are not part of W (Eq. 1 pads in pivoted
        // space): they are stored as zero, so that padding rows of the pivoted output are exactly 0 and
        // whatever sits in the padding columns of a pivoted input never contributes.
        std::vector<unsigned char> clean((size_t)T * B * B * esz);
        for (int br = 0; br < Mb; ++br) {
            const int r0 = p->row_ptr[(size_t)br], k = p->row_ptr[(size_t)br + 1] - r0;
            for (int j = 0; j < k; ++j) {
                const unsigned char* tile = src + (size_t)order[(size_t)(r0 + j)] * B * B * esz;
                unsigned char* ctile = &clean[(size_t)(r0 + j) * B * B * esz];
                const int bc = p->tile_col[(size_t)p->col_ptr[(size_t)br] + j];
                for (int r = 0; r < B; ++r)
                    for (int c = 0; c < B; ++c) {
                        const bool real = row_perm[(int64_t)br * B + r] < M && col_perm[(int64_t)bc * B + c] < N;
                        if (real) std::memcpy(ctile + ((size_t)r * B + c) * esz, tile + ((size_t)r * B + c) * esz, esz);
                        const ElemPos e = elem_pos(wdtype, g, r, c);
                        const size_t frag = (size_t)r0 * frags_per_tile + ((size_t)e.rg * k + j) * g.fpt + e.f;
                        std::memcpy(&p->values[frag * 512 + e.byte], ctile + ((size_t)r * B + c) * esz, esz);
                    }
            }
        }

        if (wdtype == PP_F16 && B == 64) {       // second copy of the sorted tiles for the tensor-core path:
            build_tile_steps(p);
            p->tiles_rm.resize((size_t)T * B * B * 2);   // each tile as its swizzled shared-memory image, in step order
            for (int64_t s2 = 0; s2 < T; ++s2)
                pp::swizzle_tile_64x64(&clean[(size_t)s2 * B * B * 2], &p->tiles_rm[(size_t)p->tile_pos[(size_t)s2] * B * B * 2]);
        }

        p->gather_idx.resize((size_t)Npad);
        for (int64_t j = 0; j < Npad; ++j) p->gather_idx[(size_t)j] = col_perm[j] < N ? col_perm[j] : -1;
        if (Npad < 65536) {
            p->gather16.resize((size_t)Npad);
            for (int64_t j = 0; j < Npad; ++j) p->gather16[(size_t)j] = (uint16_t)(p->gather_idx[(size_t)j] + 1);
        }
        p->scatter_idx.resize((size_t)Mpad);
        p->bias_piv.assign((size_t)Mpad, 0.0f);
        for (int64_t i = 0; i < Mpad; ++i) {
            const bool real = row_perm[i] < M;
            p->scatter_idx[(size_t)i] = real ? row_perm[i] : -1;
            if (real && bias) p->bias_piv[(size_t)i] = bias[row_perm[i]];
        }
        build_items(p);
        build_stream_plan(p);
    } catch (const std::bad_alloc&) {
        delete p;
        return PP_ERR_ALLOC;
    }
    *out = p;
    return PP_OK;
}

// Irregular block structure (Section 4.1.5): blocks of any size and position are laid over the
// grid of B x B tiles the kernels work on.  Every tile a block touches is kept; the part of a tile no
// block covers is zero.  Several blocks may meet in one tile, but no element may belong to two.
pp_status_t pp_blocks_to_tiles(int M, int N, int B, const int32_t* blocks, int64_t n_blocks,
                               const void* block_values, pp_dtype_t wdtype, int64_t* T_out,
                               int32_t* tile_list_out, void* tile_values_out, int64_t capacity_tiles) {
    if (!T_out || M <= 0 || N <= 0 || B <= 0 || n_blocks < 0) return PP_ERR_INVALID_ARG;
    if (n_blocks > 0 && (!blocks || !block_values)) return PP_ERR_INVALID_ARG;
    if (wdtype != PP_F32 && wdtype != PP_F16) return PP_ERR_INVALID_ARG;
    const int64_t Mb = ((int64_t)M + B - 1) / B, Nb = ((int64_t)N + B - 1) / B;
    const int64_t Mpad = Mb * B, Npad = Nb * B;
    const size_t esz = wdtype == PP_F16 ? 2 : 4;
    try {
        std::vector<int64_t> keys;
        for (int64_t k = 0; k < n_blocks; ++k) {
            const int64_t r0 = blocks[4 * k], c0 = blocks[4 * k + 1], h = blocks[4 * k + 2], w = blocks[4 * k + 3];
            if (r0 < 0 || c0 < 0 || h <= 0 || w <= 0 || r0 + h > Mpad || c0 + w > Npad) return PP_ERR_BAD_TILE;
            for (int64_t br = r0 / B; br <= (r0 + h - 1) / B; ++br)
                for (int64_t bc = c0 / B; bc <= (c0 + w - 1) / B; ++bc) keys.push_back(br * Nb + bc);
        }
        std::sort(keys.begin(), keys.end());
        keys.erase(std::unique(keys.begin(), keys.end()), keys.end());
        const int64_t T = (int64_t)keys.size();
        *T_out = T;
        if (!tile_list_out && !tile_values_out) return PP_OK;          // count only
        if (!tile_list_out || !tile_values_out || capacity_tiles < T) return PP_ERR_INVALID_ARG;
        for (int64_t t = 0; t < T; ++t) {
            tile_list_out[2 * t] = (int32_t)(keys[(size_t)t] / Nb);
            tile_list_out[2 * t + 1] = (int32_t)(keys[(size_t)t] % Nb);
        }
        const size_t tile_elems = (size_t)B * B;
        unsigned char* dst = static_cast<unsigned char*>(tile_values_out);
        std::memset(dst, 0, (size_t)T * tile_elems * esz);
        std::vector<unsigned char> taken((size_t)T * tile_elems, 0);
        const unsigned char* src = static_cast<const unsigned char*>(block_values);
        for (int64_t k = 0; k < n_blocks; ++k) {
            const int64_t r0 = blocks[4 * k], c0 = blocks[4 * k + 1], h = blocks[4 * k + 2], w = blocks[4 * k + 3];
            for (int64_t r = 0; r < h; ++r) {
                const int64_t i = r0 + r;
                for (int64_t c = 0; c < w; ++c, src += esz) {
                    const int64_t j = c0 + c;
                    const int64_t key = (i / B) * Nb + j / B;
                    const size_t t = (size_t)(std::lower_bound(keys.begin(), keys.end(), key) - keys.begin());
                    const size_t e = t * tile_elems + (size_t)(i % B) * B + (size_t)(j % B);
                    if (taken[e]) return PP_ERR_BAD_TILE;               // two blocks overlap
                    taken[e] = 1;
                    std::memcpy(dst + e * esz, src, esz);
                }
            }
        }
    } catch (const std::bad_alloc&) {
        return PP_ERR_ALLOC;
    }
    return PP_OK;
}

pp_status_t pp_pack_create_blocks(pp_packed_t** out, int M, int N, int B, const int32_t* row_perm,
                                  const int32_t* col_perm, const int32_t* blocks, int64_t n_blocks,
                                  const void* block_values, pp_dtype_t wdtype, const float* bias) {
    if (!out) return PP_ERR_INVALID_ARG;
    *out = nullptr;
    int64_t T = 0;
    pp_status_t st = pp_blocks_to_tiles(M, N, B, blocks, n_blocks, block_values, wdtype, &T, nullptr, nullptr, 0);
    if (st != PP_OK) return st;
    try {
        std::vector<int32_t> tile_list((size_t)T * 2 + 2);
        std::vector<unsigned char> tile_values((size_t)T * B * B * (wdtype == PP_F16 ? 2 : 4) + 16);
        st = pp_blocks_to_tiles(M, N, B, blocks, n_blocks, block_values, wdtype, &T, tile_list.data(),
                                tile_values.data(), T);
        if (st != PP_OK) return st;
        return pp_pack_create(out, M, N, B, row_perm, col_perm, tile_list.data(), T, tile_values.data(), wdtype, bias);
    } catch (const std::bad_alloc&) {
        return PP_ERR_ALLOC;
    }
}

pp_status_t pp_pack_destroy(pp_packed_t* p) {
    delete p;
    return PP_OK;
}

pp_status_t pp_pack_info(const pp_packed_t* p, int64_t out[13]) {
    if (!p || !out) return PP_ERR_INVALID_ARG;
    out[8] = (int64_t)p->strip_start.size() - 1; out[9] = (int64_t)p->xoff.size();
    out[10] = (int64_t)p->cta_desc.size(); out[11] = p->stream_slots;
    out[12] = (int64_t)p->tile_steps.size();
    out[0] = p->Mb; out[1] = p->Nb; out[2] = p->T; out[3] = (int64_t)p->tile_col.size();
    out[4] = (int64_t)p->items.size(); out[5] = (int64_t)p->values.size();
    out[6] = p->max_item_tiles; out[7] = p->n_slots;
    return PP_OK;
}

pp_status_t pp_pack_get(const pp_packed_t* p, int which, void* dst, int64_t bytes) {
    if (!p || !dst || bytes < 0) return PP_ERR_INVALID_ARG;
    const void* src = nullptr;
    size_t n = 0;
    switch (which) {
        case 0: src = p->row_ptr.data(); n = p->row_ptr.size() * 4; break;
        case 1: src = p->col_ptr.data(); n = p->col_ptr.size() * 4; break;
        case 2: src = p->tile_col.data(); n = p->tile_col.size() * 4; break;
        case 3: src = p->gather_idx.data(); n = p->gather_idx.size() * 4; break;
        case 4: src = p->scatter_idx.data(); n = p->scatter_idx.size() * 4; break;
        case 5: src = p->bias_piv.data(); n = p->bias_piv.size() * 4; break;
        case 6: src = p->values.data(); n = p->values.size(); break;
        case 7: src = p->items.data(); n = p->items.size() * sizeof(pp::WorkItem); break;
        case 8: src = p->inv_row_perm.data(); n = p->inv_row_perm.size() * 4; break;
        case 9: src = p->strip_start.data(); n = p->strip_start.size() * 4; break;
        case 10: src = p->xoff.data(); n = p->xoff.size() * 4; break;
        case 11: src = p->cta_desc.data(); n = p->cta_desc.size() * sizeof(pp::CtaDesc); break;
        case 12: src = p->strip_info.data(); n = p->strip_info.size() * sizeof(pp::StripInfo); break;
        case 13: src = p->tile_steps.data(); n = p->tile_steps.size() * sizeof(pp::TileStep); break;
        case 14: src = p->tile_parts.data(); n = p->tile_parts.size() * 4; break;
        case 15: src = p->tile_pos.data(); n = p->tile_pos.size() * 4; break;
        default: return PP_ERR_INVALID_ARG;
    }
    if ((size_t)bytes < n) return PP_ERR_INVALID_ARG;
    if (n) std::memcpy(dst, src, n);
    return PP_OK;
}

pp_status_t pp_pack_unpack(const pp_packed_t* p, int32_t* tile_list_out, void* tile_values_out) {
    if (!p || (p->T > 0 && (!tile_list_out || !tile_values_out))) return PP_ERR_INVALID_ARG;
    const pp::FragGeom g = pp::frag_geom(p->wdtype, p->B);
    const int esz = p->wdtype == PP_F16 ? 2 : 4, B = p->B;
    const int frags_per_tile = g.n_rg * g.fpt;
    unsigned char* dst = static_cast<unsigned char*>(tile_values_out);
    for (int br = 0; br < p->Mb; ++br) {
        const int r0 = p->row_ptr[(size_t)br], k = p->row_ptr[(size_t)br + 1] - r0;
        for (int j = 0; j < k; ++j) {
            tile_list_out[2 * (r0 + j)] = br;
            tile_list_out[2 * (r0 + j) + 1] = p->tile_col[(size_t)(p->col_ptr[(size_t)br] + j)];
            unsigned char* tile = dst + (size_t)(r0 + j) * B * B * esz;
            for (int r = 0; r < B; ++r)
                for (int c = 0; c < B; ++c) {
                    const ElemPos e = elem_pos(p->wdtype, g, r, c);
                    const size_t frag = (size_t)r0 * frags_per_tile + ((size_t)e.rg * k + j) * g.fpt + e.f;
                    std::memcpy(tile + ((size_t)r * B + c) * esz, &p->values[frag * 512 + e.byte], esz);
                }
        }
    }
    return PP_OK;
}

pp_status_t pp_fold_perm(const int32_t* row_perm_A, int M_A, int M_pad_A, const int32_t* col_perm_B,
                         int N_B, int N_pad_B, int32_t* q_out) {
    if (!row_perm_A || !col_perm_B || !q_out || M_A <= 0 || N_B != M_A || M_pad_A < M_A || N_pad_B < N_B)
        return PP_ERR_INVALID_ARG;
    if (!is_bijection(row_perm_A, M_pad_A) || !is_bijection(col_perm_B, N_pad_B)) return PP_ERR_BAD_PERM;
    std::vector<int32_t> inv((size_t)M_pad_A);
    for (int i = 0; i < M_pad_A; ++i) inv[(size_t)row_perm_A[i]] = i;
    for (int j = 0; j < N_pad_B; ++j) q_out[j] = col_perm_B[j] < N_B ? inv[(size_t)col_perm_B[j]] : -1;
    return PP_OK;
}

}  // extern "C"
