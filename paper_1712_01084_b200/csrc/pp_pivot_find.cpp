// Feed-back search for the index arrays of a PBP layer (Section 3.2): given the absolute values of a
// trained layer matrix, pick row and column permutations that keep as much of their sum as possible
// in the diagonal sub-blocks, one bisection after the other.  Host code, run once per layer at
// "network implementation time"; its result goes to pp_layer_create_blocks.
//
// One bisection of a block: its first ceil(m/2) rows and ceil(n/2) columns form side 0, the rest side 1.
// Sweeps alternate between rows and columns: with the other axis fixed, a line's gain is the sum of its
// entries facing side 0 minus those facing side 1, and the ceil(half) lines of largest gain (ties: the
// line that comes first) take side 0 -- the best balanced choice for that axis, so the kept sum never
// drops and the sweeps end.  Lines keep their relative order inside a side.
#include <algorithm>
#include <cstdint>
#include <new>
#include <numeric>
#include <vector>

#include "pp.h"

namespace {

bool is_perm(const int32_t* p, int n) {
    std::vector<unsigned char> seen((size_t)n, 0);
    for (int k = 0; k < n; ++k) {
        if (p[k] < 0 || p[k] >= n || seen[(size_t)p[k]]) return false;
        seen[(size_t)p[k]] = 1;
    }
    return true;
}

struct Search {
    const float* a;      // |W|, [M][N]
    int N;
    std::vector<int32_t> rows, cols;      // original index of every pivoted row / column

    double at(int i, int j) const { return (double)a[(size_t)rows[(size_t)i] * N + cols[(size_t)j]]; }

    // Stable partition of order[first, first + count): the `half` lines of largest gain first.
    static bool regroup(std::vector<int32_t>& order, int first, int count, int half, const std::vector<double>& gain) {
        std::vector<int> idx((size_t)count);
        std::iota(idx.begin(), idx.end(), 0);
        std::stable_sort(idx.begin(), idx.end(), [&](int x, int y) { return gain[(size_t)x] > gain[(size_t)y]; });
        std::vector<unsigned char> top((size_t)count, 0);
        for (int k = 0; k < half; ++k) top[(size_t)idx[(size_t)k]] = 1;
        std::vector<int32_t> out;
        out.reserve((size_t)count);
        for (int k = 0; k < count; ++k) if (top[(size_t)k]) out.push_back(order[(size_t)(first + k)]);
        for (int k = 0; k < count; ++k) if (!top[(size_t)k]) out.push_back(order[(size_t)(first + k)]);
        bool changed = false;
        for (int k = 0; k < count; ++k) {
            changed = changed || out[(size_t)k] != order[(size_t)(first + k)];
            order[(size_t)(first + k)] = out[(size_t)k];
        }
        return changed;
    }

    void bisect(int r0, int c0, int h, int w, int max_sweeps) {
        const int hm = (h + 1) / 2, hn = (w + 1) / 2;
        std::vector<double> gain;
        for (int sweep = 0; sweep < max_sweeps; ++sweep) {
            gain.assign((size_t)h, 0.0);
            for (int i = 0; i < h; ++i) {
                double s0 = 0.0, s1 = 0.0;
                for (int j = 0; j < hn; ++j) s0 += at(r0 + i, c0 + j);
                for (int j = hn; j < w; ++j) s1 += at(r0 + i, c0 + j);
                gain[(size_t)i] = s0 - s1;
            }
            bool changed = regroup(rows, r0, h, hm, gain);
            gain.assign((size_t)w, 0.0);
            for (int j = 0; j < w; ++j) {
                double s0 = 0.0, s1 = 0.0;
                for (int i = 0; i < hm; ++i) s0 += at(r0 + i, c0 + j);
                for (int i = hm; i < h; ++i) s1 += at(r0 + i, c0 + j);
                gain[(size_t)j] = s0 - s1;
            }
            changed = regroup(cols, c0, w, hn, gain) || changed;
            if (!changed) break;
        }
    }
};

}  // namespace

extern "C" pp_status_t pp_pivot_find(int M, int N, const float* abs_w, int levels, int max_sweeps,
                                     const int32_t* row_init, const int32_t* col_init,
                                     int32_t* row_perm_out, int32_t* col_perm_out, int32_t* blocks_out,
                                     double* kept_sum_out) {
    if (M <= 0 || N <= 0 || !abs_w || levels < 0 || levels > 20 || max_sweeps < 1 || !row_perm_out || !col_perm_out || !blocks_out)
        return PP_ERR_INVALID_ARG;
    if (((int64_t)1 << levels) > std::min(M, N)) return PP_ERR_INVALID_ARG;      // a block must keep at least one row and column
    if ((row_init && !is_perm(row_init, M)) || (col_init && !is_perm(col_init, N))) return PP_ERR_BAD_PERM;
    try {
        Search s;
        s.a = abs_w; s.N = N;
        s.rows.resize((size_t)M); s.cols.resize((size_t)N);
        if (row_init) std::copy(row_init, row_init + M, s.rows.begin()); else std::iota(s.rows.begin(), s.rows.end(), 0);
        if (col_init) std::copy(col_init, col_init + N, s.cols.begin()); else std::iota(s.cols.begin(), s.cols.end(), 0);
        struct Blk { int r0, c0, h, w; };
        std::vector<Blk> blocks{{0, 0, M, N}};
        for (int l = 0; l < levels; ++l) {
            std::vector<Blk> next;
            for (const Blk& b : blocks) {
                s.bisect(b.r0, b.c0, b.h, b.w, max_sweeps);
                const int hm = (b.h + 1) / 2, hn = (b.w + 1) / 2;
                next.push_back({b.r0, b.c0, hm, hn});
                next.push_back({b.r0 + hm, b.c0 + hn, b.h - hm, b.w - hn});
            }
            blocks.swap(next);
        }
        double kept = 0.0;
        for (size_t k = 0; k < blocks.size(); ++k) {
            const Blk& b = blocks[k];
            blocks_out[4 * k] = b.r0; blocks_out[4 * k + 1] = b.c0; blocks_out[4 * k + 2] = b.h; blocks_out[4 * k + 3] = b.w;
            for (int i = 0; i < b.h; ++i)
                for (int j = 0; j < b.w; ++j) kept += s.at(b.r0 + i, b.c0 + j);
        }
        std::copy(s.rows.begin(), s.rows.end(), row_perm_out);
        std::copy(s.cols.begin(), s.cols.end(), col_perm_out);
        if (kept_sum_out) *kept_sum_out = kept;
    } catch (const std::bad_alloc&) {
        return PP_ERR_ALLOC;
    }
    return PP_OK;
}
