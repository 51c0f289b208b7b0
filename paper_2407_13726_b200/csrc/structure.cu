// Host side of the structure object: descriptor analysis and the host rank / unrank calls.
//
// A descriptor row is an affine comparison over the indices and the size symbols (Section 2,
// "Unique set").  After the symbols are replaced by their values every supported row is a bound
// on one index or on the difference of two indices, so the whole set is a system of difference
// bounds.  Its closure under implication (all-pairs shortest paths) is a canonical form: two
// descriptors of the same set close to the same matrix, whatever rows they were written with.
// The closed matrix is matched against the classes whose counting polynomial is known.
#include <climits>
#include <cstring>
#include <array>
#include <new>
#include <vector>

#include "common.cuh"

namespace dastac {

dastac_status build_generic_map(int rank, const int64_t* dims, const std::vector<std::array<int64_t, 4>>& user_rows,
                                GenericMap** out);

std::atomic<int64_t> g_launches{0};

int sm_count() {
    static int cached[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
            n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}

namespace {

constexpr int64_t kInf = INT64_MAX / 4;
constexpr int64_t kMaxExtent = int64_t(1) << 30;
constexpr int64_t kMaxCount = int64_t(1) << 62;

int64_t floor_div(int64_t a, int64_t b) {  // b > 0
    int64_t q = a / b;
    return (a % b != 0 && a < 0) ? q - 1 : q;
}

// D[p][q] = upper bound of v_p - v_q, with v_rank == 0 (the origin).
struct Bounds {
    int n;  // rank + 1
    int64_t D[4][4];
    void tighten(int p, int q, int64_t c) {
        if (c < D[p][q]) D[p][q] = c;
    }
};

// Returns false when the system has no solution.
bool close_bounds(Bounds& b) {
    for (int k = 0; k < b.n; ++k)
        for (int p = 0; p < b.n; ++p)
            for (int q = 0; q < b.n; ++q)
                if (b.D[p][k] < kInf && b.D[k][q] < kInf && b.D[p][k] + b.D[k][q] < b.D[p][q])
                    b.D[p][q] = b.D[p][k] + b.D[k][q];
    for (int p = 0; p < b.n; ++p)
        if (b.D[p][p] < 0) return false;
    return true;
}

// Adds "sum a_k idx_k + c >= 0" to the system; false if the row has an unsupported shape.
bool add_row(Bounds& b, int rank, const int64_t* a, int64_t c) {
    int pos = -1, neg = -1, nz = 0;
    for (int k = 0; k < rank; ++k) {
        if (a[k] == 0) continue;
        ++nz;
        if (a[k] > 0) {
            if (pos >= 0) return false;
            pos = k;
        } else {
            if (neg >= 0) return false;
            neg = k;
        }
    }
    const int O = rank;
    if (nz == 0) {
        if (c < 0) b.tighten(O, O, -1);  // contradiction: 0 >= positive
        return true;
    }
    if (nz == 1) {
        if (pos >= 0) b.tighten(O, pos, floor_div(c, a[pos]));  // idx >= -c/a  <=>  0 - idx <= c/a
        else b.tighten(neg, O, floor_div(c, -a[neg]));          // idx <= c/a
        return true;
    }
    if (a[pos] != -a[neg]) return false;
    b.tighten(neg, pos, floor_div(c, a[pos]));  // a(idx_pos - idx_neg) + c >= 0
    return true;
}

}  // namespace
}  // namespace dastac

using namespace dastac;

static dastac_status create_recognised(const dastac_structure_desc* desc, dastac_structure** out);

// A descriptor that is none of the recognised classes gets a fitted map when it can (generic.cuh):
// exact lexicographic layout, no redundancy map, rank 2 or 3.
extern "C" dastac_status dastac_structure_create(const dastac_structure_desc* desc, dastac_structure** out) {
    const dastac_status st = create_recognised(desc, out);
    if (st != DASTAC_ERR_UNSUPPORTED_STRUCTURE) return st;
    if (desc->layout != DASTAC_LAYOUT_LEXICOGRAPHIC || desc->rank < 2) return st;
    if (desc->mirror)
        for (int k = 0; k < desc->rank; ++k)
            if (desc->mirror[k] != k) return st;
    const int rank = desc->rank, np = desc->nparams, width = rank + np + 1;
    std::vector<std::array<int64_t, 4>> rows;
    for (int r = 0; r < desc->nrows; ++r) {
        const int64_t* row = desc->rows + (size_t)r * width;
        std::array<int64_t, 4> a{0, 0, 0, row[width - 1]};
        for (int k = 0; k < rank; ++k) a[(size_t)k] = row[k];
        for (int p = 0; p < np; ++p) {
            if (desc->params[p] > (int64_t(1) << 40) || desc->params[p] < -(int64_t(1) << 40) || row[rank + p] > 1024 ||
                row[rank + p] < -1024)
                return st;
            a[3] += row[rank + p] * desc->params[p];
        }
        rows.push_back(a);
        if (desc->is_eq[r]) rows.push_back({-a[0], -a[1], -a[2], -a[3]});
    }
    GenericMap* g = nullptr;
    const dastac_status gs = build_generic_map(rank, desc->dims, rows, &g);
    if (gs != DASTAC_OK) return gs == DASTAC_ERR_OVERFLOW ? gs : st;
    dastac_structure* s = new (std::nothrow) dastac_structure;
    if (!s) {
        delete g;
        return DASTAC_ERR_INVALID_ARG;
    }
    std::memset(&s->map, 0, sizeof(s->map));
    s->map.kind = kGeneric;
    s->map.rank = rank;
    s->map.Q = 1;
    for (int k = 0; k < rank; ++k) s->map.dims[k] = desc->dims[k];
    s->map.count = s->map.slots = g->count;
    s->generic = g;
    *out = s;
    return DASTAC_OK;
}

static dastac_status create_recognised(const dastac_structure_desc* desc, dastac_structure** out) {
    if (!desc || !out) return DASTAC_ERR_INVALID_ARG;
    *out = nullptr;
    const int rank = desc->rank, np = desc->nparams, nr = desc->nrows;
    if (rank < 1 || rank > 3 || np < 0 || np > 8 || nr < 0 || nr > 64) return DASTAC_ERR_INVALID_ARG;
    if (!desc->dims || (nr > 0 && (!desc->rows || !desc->is_eq)) || (np > 0 && !desc->params))
        return DASTAC_ERR_INVALID_ARG;
    if (desc->layout != DASTAC_LAYOUT_LEXICOGRAPHIC && desc->layout != DASTAC_LAYOUT_PADDED_DIAGONALS)
        return DASTAC_ERR_INVALID_ARG;
    for (int k = 0; k < rank; ++k) {
        if (desc->dims[k] < 0) return DASTAC_ERR_INVALID_ARG;
        if (desc->dims[k] > kMaxExtent) return DASTAC_ERR_OVERFLOW;
    }
    if (desc->mirror) {
        bool seen[3] = {false, false, false};
        for (int k = 0; k < rank; ++k) {
            int v = desc->mirror[k];
            if (v < 0 || v >= rank || seen[v]) return DASTAC_ERR_INVALID_ARG;
            seen[v] = true;
        }
    }

    IndexMap m;
    std::memset(&m, 0, sizeof(m));
    m.rank = rank;
    m.Q = 1;
    for (int k = 0; k < rank; ++k) m.dims[k] = desc->dims[k];

    Bounds b;
    b.n = rank + 1;
    for (int p = 0; p < 4; ++p)
        for (int q = 0; q < 4; ++q) b.D[p][q] = (p == q) ? 0 : kInf;
    bool empty = false;
    for (int k = 0; k < rank; ++k) {
        if (desc->dims[k] == 0) empty = true;
        b.tighten(rank, k, 0);                  // idx_k >= 0
        b.tighten(k, rank, desc->dims[k] - 1);  // idx_k <= dims - 1
    }
    const int width = rank + np + 1;
    for (int r = 0; r < nr && !empty; ++r) {
        const int64_t* row = desc->rows + (size_t)r * width;
        int64_t c = row[width - 1];
        for (int p = 0; p < np; ++p) {
            // |coefficient * param| is kept far from overflow by the extent limits below
            if (desc->params[p] > kMaxCount / 4 || desc->params[p] < -kMaxCount / 4)
                return DASTAC_ERR_OVERFLOW;
            if (row[rank + p] > 4 || row[rank + p] < -4) return DASTAC_ERR_UNSUPPORTED_STRUCTURE;
            c += row[rank + p] * desc->params[p];
        }
        int64_t a[3] = {0, 0, 0}, na[3] = {0, 0, 0};
        for (int k = 0; k < rank; ++k) {
            a[k] = row[k];
            na[k] = -row[k];
        }
        if (!add_row(b, rank, a, c)) return DASTAC_ERR_UNSUPPORTED_STRUCTURE;
        if (desc->is_eq[r] && !add_row(b, rank, na, -c)) return DASTAC_ERR_UNSUPPORTED_STRUCTURE;
    }
    if (!empty && !close_bounds(b)) empty = true;

    auto finish = [&](void) -> dastac_status {
        if (m.count < 0 || m.count > kMaxCount || m.slots > kMaxCount) return DASTAC_ERR_OVERFLOW;
        dastac_structure* s = new (std::nothrow) dastac_structure;
        if (!s) return DASTAC_ERR_INVALID_ARG;
        s->map = m;
        *out = s;
        return DASTAC_OK;
    };

    if (empty) {
        m.kind = kEmpty;
        m.count = m.slots = 0;
        if (desc->mirror) m.symmetric = 0;
        return finish();
    }

    const int O = rank;
    int64_t lo[3], hi[3];
    for (int k = 0; k < rank; ++k) {
        lo[k] = -b.D[O][k];
        hi[k] = b.D[k][O];
    }
    // The sub-triangle j - i >= c (c >= 1) of a square box: its closure moves the lower bound of j
    // to c and the upper bound of i to N - 1 - c; nothing else relates the two indices.
    if (rank == 2 && desc->layout != DASTAC_LAYOUT_PADDED_DIAGONALS && m.dims[0] == m.dims[1] && b.D[0][1] < 0 &&
        lo[0] == 0 && lo[1] == -b.D[0][1] && hi[1] == m.dims[1] - 1 && hi[0] == m.dims[0] - 1 + b.D[0][1] &&
        b.D[1][0] == hi[1] - lo[0]) {
        if (desc->mirror && !(desc->mirror[0] == 0 && desc->mirror[1] == 1)) return DASTAC_ERR_UNSUPPORTED_STRUCTURE;
        m.kind = kUpperShifted;
        m.N = m.dims[1];
        m.w = -b.D[0][1];
        m.M = m.N - m.w;
        m.count = m.slots = tri(m.M);
        return finish();
    }
    // General offset band lo_off <= j - i <= hi_off of a square box, tried when none of the special
    // classes (which have faster kernels) applies: the closure must carry nothing but the two
    // difference bounds and the index ranges they imply.
    auto offset_band = [&]() -> bool {
        if (rank != 2 || desc->layout == DASTAC_LAYOUT_PADDED_DIAGONALS || m.dims[0] != m.dims[1]) return false;
        const int64_t N = m.dims[0], a = -b.D[0][1], c = b.D[1][0];
        if (a > c) return false;
        if (lo[0] != oband_first_row(c) || hi[0] != oband_last_row(N, a)) return false;
        if (lo[1] != (a > 0 ? a : 0) || hi[1] != (c < 0 ? N - 1 + c : N - 1)) return false;
        if (desc->mirror && !(desc->mirror[0] == 0 && desc->mirror[1] == 1)) return false;
        m.kind = kBandOffsets;
        m.N = N;
        m.lo_off = a;
        m.hi_off = c;
        m.count = m.slots = oband_row_start(N, a, c, oband_last_row(N, a) + 1);
        return true;
    };
    auto free_pair = [&](int p, int q) {  // no constraint between p and q beyond the box
        return b.D[p][q] == hi[p] - lo[q] && b.D[q][p] == hi[q] - lo[p];
    };
    // One index determined by the rest (fixed, or equal to an earlier index), the others dense: the
    // "Fixed i / Fixed j / Diagonal (plane)" structures of Table 1.
    auto plane = [&]() -> bool {
        if (rank < 2 || desc->layout == DASTAC_LAYOUT_PADDED_DIAGONALS) return false;
        if (desc->mirror)
            for (int k = 0; k < rank; ++k)
                if (desc->mirror[k] != k) return false;
        int dep = -1, src = -1;
        int64_t cval = 0;
        for (int a = 0; a < rank; ++a)  // a fixed index
            if (lo[a] == hi[a] && m.dims[a] > 1) {
                if (dep >= 0) return false;
                dep = a;
                cval = lo[a];
            }
        if (dep < 0) {  // an equality between two indices: the later one is the dependent one
            for (int a = 0; a < rank; ++a)
                for (int c = a + 1; c < rank; ++c)
                    if (b.D[a][c] == 0 && b.D[c][a] == 0) {
                        if (dep >= 0) return false;
                        dep = c;
                        src = a;
                    }
            if (dep < 0) return false;
        }
        int64_t ext[3] = {0, 0, 0};
        for (int k = 0; k < rank; ++k) {
            if (k == dep) continue;
            if (lo[k] != 0) return false;
            const int64_t full = (k == src) ? (m.dims[src] < m.dims[dep] ? m.dims[src] : m.dims[dep]) : m.dims[k];
            if (hi[k] != full - 1) return false;
            ext[k] = full;
        }
        if (src >= 0 && (lo[dep] != 0 || hi[dep] != hi[src])) return false;
        // nothing else relates the indices
        for (int p = 0; p < rank; ++p)
            for (int q = p + 1; q < rank; ++q) {
                if ((p == src && q == dep)) continue;
                if (!free_pair(p, q)) return false;
            }
        m.kind = kPlane;
        m.w = dep;
        m.lo_off = src;
        m.hi_off = cval;
        const int f0 = dep == 0 ? 1 : 0, f1 = dep == 2 ? 1 : 2;
        m.M = ext[f0];
        m.Q = rank == 3 ? ext[f1] : 1;
        m.N = m.dims[rank - 1];
        m.count = m.slots = m.M * m.Q;
        return true;
    };
    // Every class below starts at the origin of the box in every index.
    for (int k = 0; k < rank; ++k)
        if (lo[k] != 0) {
            if (offset_band()) return finish();
            if (plane()) return finish();
            return DASTAC_ERR_UNSUPPORTED_STRUCTURE;
        }
    // p <= q is the only relation between p and q:  D[p][q] == 0 and D[q][p] is the box value.
    auto ordered_pair = [&](int p, int q) { return b.D[p][q] == 0 && b.D[q][p] == hi[q] - lo[p]; };

    const bool padded = desc->layout == DASTAC_LAYOUT_PADDED_DIAGONALS;
    bool matched = false;
    if (rank == 1) {
        if (hi[0] == m.dims[0] - 1) {
            m.kind = kDense;
            m.count = m.dims[0];
            matched = true;
        }
    } else if (rank == 2) {
        const bool full0 = hi[0] == m.dims[0] - 1, full1 = hi[1] == m.dims[1] - 1;
        if (full1 && ordered_pair(0, 1) && hi[0] == (m.dims[0] < m.dims[1] ? m.dims[0] : m.dims[1]) - 1 &&
                   !padded) {
            m.kind = kUpper;
            m.N = m.dims[1];
            m.M = hi[0] + 1;
            m.count = upper_row_start(m.N, m.M);
            matched = true;
        } else if (full0 && ordered_pair(1, 0) && m.dims[0] == m.dims[1] && hi[1] == m.dims[1] - 1 &&
                   !padded) {
            m.kind = kLower;
            m.N = m.dims[0];
            m.count = tri(m.N);
            matched = true;
        } else if (full0 && full1 && free_pair(0, 1) && !padded) {
            m.kind = kDense;
            m.count = m.dims[0] * m.dims[1];
            matched = true;
        } else if (padded && full0 && full1 && m.dims[0] == m.dims[1] && b.D[0][1] == b.D[1][0] &&
                   b.D[0][1] >= 0) {
            m.kind = kBandDiagonals;
            m.N = m.dims[0];
            m.w = b.D[0][1];
            // A band as wide as the matrix closes to the dense box and its nominal half width,
            // which fixes the number of stored diagonals, can no longer be told: w <= N - 2.
            if (m.N > 1 && m.w >= m.N - 1) return DASTAC_ERR_UNSUPPORTED_STRUCTURE;
            m.count = (2 * m.w + 1) * m.N - m.w * (m.w + 1);
            m.slots = (2 * m.w + 1) * m.N;
            matched = true;
        } else if (!padded && full0 && full1 && m.dims[0] == m.dims[1] && b.D[0][1] == b.D[1][0] && b.D[0][1] >= 0 &&
                   2 * b.D[0][1] + 1 <= m.dims[0]) {
            // the same band packed row after row with nothing in between (three-piece polynomial)
            m.kind = kBandExact;
            m.N = m.dims[0];
            m.w = b.D[0][1];
            m.count = (2 * m.w + 1) * m.N - m.w * (m.w + 1);
            matched = true;
        }
    } else {  // rank 3
        const bool full = hi[0] == m.dims[0] - 1 && hi[1] == m.dims[1] - 1 && hi[2] == m.dims[2] - 1;
        if (padded) return DASTAC_ERR_UNSUPPORTED_STRUCTURE;
        if (false) {
        } else if (full && m.dims[0] == m.dims[1] && m.dims[1] == m.dims[2] && ordered_pair(0, 1) &&
                   ordered_pair(1, 2) && b.D[0][2] == 0 && b.D[2][0] == hi[2] - lo[0]) {
            if (m.dims[0] > (int64_t(1) << 20)) return DASTAC_ERR_OVERFLOW;
            m.kind = kTetrahedron;
            m.N = m.dims[0];
            m.count = tet(m.N);
            matched = true;
        } else if (hi[1] == m.dims[1] - 1 && hi[2] == m.dims[2] - 1 && ordered_pair(0, 1) &&
                   free_pair(0, 2) && free_pair(1, 2) &&
                   hi[0] == (m.dims[0] < m.dims[1] ? m.dims[0] : m.dims[1]) - 1) {
            m.kind = kUpper;
            m.N = m.dims[1];
            m.M = hi[0] + 1;
            m.Q = m.dims[2];
            // rows <= 2^59 points, Q <= 2^30: the product may not fit
            if (__builtin_mul_overflow(upper_row_start(m.N, m.M), m.Q, &m.count)) return DASTAC_ERR_OVERFLOW;
            matched = true;
        } else if (full && free_pair(0, 1) && free_pair(0, 2) && free_pair(1, 2)) {
            m.kind = kDense;
            // three extents of up to 2^30 each: checked product
            if (__builtin_mul_overflow(m.dims[0] * m.dims[1], m.dims[2], &m.count)) return DASTAC_ERR_OVERFLOW;
            matched = true;
        }
    }
    if (!matched && offset_band()) return finish();
    if (!matched && plane()) return finish();
    if (!matched) return DASTAC_ERR_UNSUPPORTED_STRUCTURE;
    if (m.kind != kBandDiagonals) m.slots = m.count;

    if (desc->mirror) {
        bool identity = true;
        for (int k = 0; k < rank; ++k) identity = identity && desc->mirror[k] == k;
        if (!identity) {
            if (!(m.kind == kUpper && rank == 2 && m.dims[0] == m.dims[1] && desc->mirror[0] == 1 &&
                  desc->mirror[1] == 0))
                return DASTAC_ERR_UNSUPPORTED_STRUCTURE;
            m.symmetric = 1;
        }
    }
    return finish();
}

extern "C" void dastac_structure_destroy(dastac_structure* s) { delete s; }

extern "C" dastac_status dastac_structure_count(const dastac_structure* s, int64_t* slots,
                                                int64_t* nnz) {
    if (!s) return DASTAC_ERR_INVALID_ARG;
    if (slots) *slots = s->map.slots;
    if (nnz) *nnz = s->map.count;
    return DASTAC_OK;
}

extern "C" dastac_status dastac_structure_kind(const dastac_structure* s, int32_t* kind,
                                               int32_t* symmetric) {
    if (!s) return DASTAC_ERR_INVALID_ARG;
    if (kind) *kind = s->map.kind;
    if (symmetric) *symmetric = s->map.symmetric;
    return DASTAC_OK;
}

extern "C" dastac_status dastac_rank(const dastac_structure* s, const int32_t* idx, int64_t* off) {
    if (!s || !idx || !off) return DASTAC_ERR_INVALID_ARG;
    if (s->map.kind == kGeneric) {
        const int64_t x[3] = {idx[0], s->map.rank > 1 ? idx[1] : 0, s->map.rank > 2 ? idx[2] : 0};
        if (!g_in_domain(*s->generic, x)) return DASTAC_ERR_INVALID_ARG;
        *off = g_rank(*s->generic, x);
        return DASTAC_OK;
    }
    if (!in_set(s->map, idx)) return DASTAC_ERR_INVALID_ARG;
    *off = rank_of(s->map, idx);
    return DASTAC_OK;
}

extern "C" dastac_status dastac_unrank(const dastac_structure* s, int64_t off, int32_t* idx) {
    if (!s || !idx) return DASTAC_ERR_INVALID_ARG;
    if (off < 0 || off >= s->map.slots) return DASTAC_ERR_INVALID_ARG;
    if (s->map.kind == kGeneric) {
        int64_t x[3] = {0, 0, 0};
        g_unrank(*s->generic, off, x);
        for (int k = 0; k < s->map.rank; ++k) idx[k] = (int32_t)x[k];
        return DASTAC_OK;
    }
    unrank_of(s->map, off, idx);
    return DASTAC_OK;
}

extern "C" const char* dastac_status_string(dastac_status st) {
    switch (st) {
        case DASTAC_OK: return "ok";
        case DASTAC_ERR_INVALID_ARG: return "invalid argument";
        case DASTAC_ERR_UNSUPPORTED_STRUCTURE: return "unsupported structure";
        case DASTAC_ERR_UNSUPPORTED_EXPR: return "unsupported expression";
        case DASTAC_ERR_SHAPE: return "shape mismatch";
        case DASTAC_ERR_ALIGNMENT: return "pointer not 16-byte aligned";
        case DASTAC_ERR_OVERFLOW: return "extent or count overflow";
        case DASTAC_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case DASTAC_ERR_CUDA: return "CUDA call failed";
        case DASTAC_ERR_TIMEOUT: return "bounded device wait expired";
        default: return "unknown status";
    }
}

extern "C" int64_t dastac_launch_count(void) { return g_launches.load(); }
