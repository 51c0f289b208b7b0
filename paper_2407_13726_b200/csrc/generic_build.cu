// Builds the index map of a structure outside the recognised classes (see generic.cuh): counts
// every slab by brute force, fits the piecewise polynomial S1 to those counts, fuses pieces that
// agree (Algorithm 2) and checks the result.  Host code.
#include <array>
#include <cstring>
#include <new>
#include <vector>

#include "common.cuh"
#include "generic.cuh"
#include "piecewise.cuh"

namespace dastac {
namespace {

constexpr int64_t kGMaxExtent = int64_t(1) << 20;
constexpr int64_t kGMaxOuter = int64_t(1) << 24;  // slabs (rank 2) or fibres (rank 3) counted at creation

// S1 of a piece in exact arithmetic
__int128 newton_at(const int64_t* nw, int64_t anchor, int64_t i) {
    const __int128 t = (__int128)i - anchor;
    return (__int128)nw[0] + (__int128)nw[1] * t + (__int128)nw[2] * (t * (t - 1) / 2) +
           (__int128)nw[3] * (t * (t - 1) * (t - 2) / 6);
}

}  // namespace

// rows: a0, a1, a2, c with "a . idx + c >= 0", the size symbols already folded in, equalities
// already split.  On success *out is a heap object the structure owns.
dastac_status build_generic_map(int rank, const int64_t* dims, const std::vector<std::array<int64_t, 4>>& user_rows,
                                GenericMap** out) {
    *out = nullptr;
    if (rank < 2 || rank > 3) return DASTAC_ERR_UNSUPPORTED_STRUCTURE;
    GenericMap g;
    std::memset(&g, 0, sizeof(g));
    g.rank = rank;
    for (int k = 0; k < rank; ++k) {
        if (dims[k] > kGMaxExtent) return DASTAC_ERR_UNSUPPORTED_STRUCTURE;
        g.dims[k] = dims[k];
    }
    if ((rank == 2 ? dims[0] : dims[0] * dims[1]) > kGMaxOuter) return DASTAC_ERR_UNSUPPORTED_STRUCTURE;
    auto add = [&](int64_t a0, int64_t a1, int64_t a2, int64_t c) {
        if (g.nrows >= kGMaxRows) return false;
        g.a[g.nrows][0] = a0, g.a[g.nrows][1] = a1, g.a[g.nrows][2] = a2, g.c[g.nrows] = c;
        ++g.nrows;
        return true;
    };
    for (int k = 0; k < rank; ++k) {  // the box
        int64_t e[3] = {0, 0, 0};
        e[k] = 1;
        if (!add(e[0], e[1], e[2], 0) || !add(-e[0], -e[1], -e[2], dims[k] - 1)) return DASTAC_ERR_UNSUPPORTED_STRUCTURE;
    }
    for (const auto& r : user_rows) {
        if (r[0] == 0 && r[1] == 0 && r[2] == 0) {
            if (r[3] < 0) return DASTAC_ERR_UNSUPPORTED_STRUCTURE;  // an empty set is recognised before this point
            continue;
        }
        if (!add(r[0], r[1], r[2], r[3])) return DASTAC_ERR_UNSUPPORTED_STRUCTURE;
    }
    // unit coefficients on the indices whose bounds are read off the rows
    int nl = 0, nu = 0;
    for (int r = 0; r < g.nrows; ++r) {
        const int64_t al = g.a[r][rank - 1];
        if (al < -1 || al > 1) return DASTAC_ERR_UNSUPPORTED_STRUCTURE;
        if (rank == 3) {
            if (g.a[r][1] < -1 || g.a[r][1] > 1) return DASTAC_ERR_UNSUPPORTED_STRUCTURE;
            nl += al > 0;
            nu += al < 0;
        }
        for (int k = 0; k < rank; ++k)
            if (g.a[r][k] > (int64_t(1) << 20) || g.a[r][k] < -(int64_t(1) << 20)) return DASTAC_ERR_UNSUPPORTED_STRUCTURE;
        if (g.c[r] > (int64_t(1) << 40) || g.c[r] < -(int64_t(1) << 40)) return DASTAC_ERR_UNSUPPORTED_STRUCTURE;
    }
    if (nl > kGMaxBounds || nu > kGMaxBounds) return DASTAC_ERR_UNSUPPORTED_STRUCTURE;

    // ---- brute-force count of every slab ----
    const int64_t n0 = dims[0];
    std::vector<int64_t> slab((size_t)n0, 0), before((size_t)n0 + 1, 0);
    for (int64_t i = 0; i < n0; ++i) {
        int64_t cnt = 0;
        if (rank == 2) {
            int64_t lo, hi;
            const int64_t outer[2] = {i, 0};
            if (g_last_bounds(g, outer, lo, hi) && hi >= lo) cnt = hi - lo + 1;
        } else {
            for (int64_t j = 0; j < dims[1]; ++j) {
                int64_t lo, hi;
                const int64_t outer[2] = {i, j};
                if (g_last_bounds(g, outer, lo, hi) && hi >= lo) cnt += hi - lo + 1;
            }
        }
        slab[(size_t)i] = cnt;
        before[(size_t)i + 1] = before[(size_t)i] + cnt;
        if (before[(size_t)i + 1] > (int64_t(1) << 62)) return DASTAC_ERR_OVERFLOW;
    }
    g.count = before[(size_t)n0];

    // ---- pieces: maximal runs on which the slab size is a polynomial of degree <= rank - 1 ----
    const int deg = rank - 1;
    struct Run {
        int64_t lo, hi;  // [lo, hi)
        int64_t nw[4];
    };
    std::vector<Run> runs;
    auto diff_zero = [&](int64_t at) {  // the (deg+1)-th forward difference of slab at `at`
        if (deg == 1) return slab[(size_t)at + 2] - 2 * slab[(size_t)at + 1] + slab[(size_t)at] == 0;
        return slab[(size_t)at + 3] - 3 * slab[(size_t)at + 2] + 3 * slab[(size_t)at + 1] - slab[(size_t)at] == 0;
    };
    for (int64_t a = 0; a < n0;) {
        int64_t b = a + 1;
        while (b < n0) {
            // extending to b is allowed when the run stays polynomial: all windows inside vanish
            const int64_t w = b - (deg + 1);
            if (w >= a && !diff_zero(w)) break;
            ++b;
        }
        Run r;
        r.lo = a;
        r.hi = b;
        r.nw[0] = before[(size_t)a];
        r.nw[1] = slab[(size_t)a];
        r.nw[2] = b - a >= 2 ? slab[(size_t)a + 1] - slab[(size_t)a] : 0;
        r.nw[3] = (deg == 2 && b - a >= 3) ? slab[(size_t)a + 2] - 2 * slab[(size_t)a + 1] + slab[(size_t)a] : 0;
        runs.push_back(r);
        if (runs.size() > 4096) return DASTAC_ERR_UNSUPPORTED_STRUCTURE;
        a = b;
    }
    if (runs.empty()) {
        Run r{0, 0, {0, 0, 0, 0}};
        runs.push_back(r);
    }
    // ---- Algorithm 2: a run whose counts another run's polynomial reproduces is absorbed by it ----
    std::vector<int> owner;
    pw_fuse_core((int)runs.size(),
                 [&](int k, int q) {
                     for (int64_t i = runs[(size_t)q].lo; i < runs[(size_t)q].hi; ++i)
                         if (newton_at(runs[(size_t)k].nw, runs[(size_t)k].lo, i) != (__int128)before[(size_t)i]) return false;
                     return true;
                 },
                 owner);
    // intervals in order, neighbours with the same polynomial merged
    g.npieces = 0;
    for (size_t q = 0; q < runs.size(); ++q) {
        const Run& src = runs[(size_t)owner[q]];
        if (g.npieces > 0 && g.anchor[g.npieces - 1] == src.lo && g.newton[g.npieces - 1][0] == src.nw[0] &&
            g.newton[g.npieces - 1][1] == src.nw[1] && g.newton[g.npieces - 1][2] == src.nw[2] &&
            g.newton[g.npieces - 1][3] == src.nw[3])
            continue;
        if (g.npieces >= kGMaxPieces) return DASTAC_ERR_UNSUPPORTED_STRUCTURE;
        g.piece_lo[g.npieces] = runs[q].lo;
        g.anchor[g.npieces] = src.lo;
        for (int e = 0; e < 4; ++e) g.newton[g.npieces][e] = src.nw[e];
        ++g.npieces;
    }
    g.piece_lo[g.npieces] = n0;
    // ---- checks: every term stays inside 63 bits, S1 reproduces the counts, S2 the fibre lengths ----
    for (int p = 0; p < g.npieces; ++p)
        for (int64_t i : {g.piece_lo[p], g.piece_lo[p + 1] - 1}) {
            const __int128 t = (__int128)i - g.anchor[p];
            const __int128 lim = (__int128)1 << 62;
            const __int128 terms[3] = {(__int128)g.newton[p][1] * t, (__int128)g.newton[p][2] * (t * (t - 1) / 2),
                                       (__int128)g.newton[p][3] * (t * (t - 1) * (t - 2) / 6)};
            for (const __int128 v : terms)
                if (v > lim || v < -lim) return DASTAC_ERR_OVERFLOW;
        }
    for (int64_t i = 0; i < n0; ++i)
        if (g_s1(g, i) != before[(size_t)i]) return DASTAC_ERR_UNSUPPORTED_STRUCTURE;
    if (rank == 3 && n0 > 0) {
        const int64_t step = n0 > 48 ? n0 / 48 : 1;
        for (int64_t i = 0; i < n0; i += step) {
            int64_t run = 0;
            for (int64_t j = 0; j < dims[1]; ++j) {
                if (g_s2(g, i, j) != run) return DASTAC_ERR_UNSUPPORTED_STRUCTURE;
                int64_t lo, hi;
                const int64_t outer[2] = {i, j};
                if (g_last_bounds(g, outer, lo, hi) && hi >= lo) run += hi - lo + 1;
            }
            if (run != slab[(size_t)i]) return DASTAC_ERR_UNSUPPORTED_STRUCTURE;
        }
    }
    GenericMap* heap = new (std::nothrow) GenericMap(g);
    if (!heap) return DASTAC_ERR_INVALID_ARG;
    *out = heap;
    return DASTAC_OK;
}

}  // namespace dastac
