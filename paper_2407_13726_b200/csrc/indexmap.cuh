// Closed-form index maps of the recognised structure classes, evaluated in registers.
//
// rank  = number of points of the set that precede a point in lexicographic order, i.e. the value
//         of the counting polynomial of the preceding-access domain (Section 4, "Access domain
//         linearization").  Every polynomial is evaluated on its integer numerator with one exact
//         division at the end, the way the generated code of the paper's running example does
//         (all terms doubled, one final halving).
// unrank = the inverse map.  The paper never inverts the polynomial; it is needed here so that a
//         thread block can start in the middle of the packed stream.  A floating-point root gives
//         an estimate and integer comparisons against the polynomial correct it, so the result is
//         exact.
#pragma once
#include <cmath>
#include <cstdint>

#ifdef __CUDACC__
#define DASTAC_HD __host__ __device__ __forceinline__
#else
#define DASTAC_HD inline
#endif

namespace dastac {

enum Kind : int32_t {
    kEmpty = 0,
    kDense = 1,
    kUpper = 2,
    kLower = 3,
    kBandDiagonals = 4,
    kTetrahedron = 5,
    kBandExact = 6,  // |i - j| <= w packed row after row without padding (2w + 1 <= N)
    // j - i >= c in an N x N box (c >= 1): the upper triangle of size M = N - c sitting in the top
    // right corner (the sub-triangular structure of Section 6.4, "Density and Compression", with
    // c = N - k).  Row i < M holds columns i + c .. N-1; the shift c is kept in `w`.
    kUpperShifted = 7,
    // lo_off <= j - i <= hi_off inside an N x N box, any lo_off <= hi_off: rows packed back to back.
    // One diagonal at distance s (lo_off = hi_off = s) is the per-summand buffer of a strided band
    // (Section 6.4, "Distance of Elements and Compression"); asymmetric bands, strictly lower
    // triangles and the like fall out of the same counting function.
    kBandOffsets = 8,
    // One index is determined by the rest: idx[dep] = idx[src] (a diagonal plane such as i = j) or
    // idx[dep] = c (a fixed index), everything else dense: the structures "Diagonal (plane)",
    // "Fixed i", "Fixed j" of Table 1.  The packed layout is the dense box over the free indices
    // in their own order.  dep is kept in `w`, src (or -1) in `lo_off`, c in `hi_off`; M and Q hold
    // the extents of the first and second free index.
    kPlane = 9,
    // Any other conjunction of affine comparisons whose counting function could be fitted when the
    // structure was created; the map itself is a GenericMap (generic.cuh), not this struct.
    kGeneric = 10
};

// Plain data, passed to kernels by value.
struct IndexMap {
    int32_t kind;
    int32_t rank;
    int32_t symmetric;
    int32_t reserved;
    int64_t dims[3];  // logical extents
    int64_t M;        // kUpper: number of non-empty rows, min(dims[0], dims[1])
    int64_t N;        // kUpper/kLower/kBand: columns; kTetrahedron: n
    int64_t Q;        // kUpper: trailing dense extent (1 for a matrix)
    int64_t w;        // kBand: half width
    int64_t count;    // points of the set
    int64_t slots;    // elements of the packed vector (count, or (2w+1)N with padding)
    int64_t lo_off, hi_off;  // kBandOffsets: bounds of j - i
};

DASTAC_HD int64_t tri(int64_t m) { return (m * (m + 1)) >> 1; }
DASTAC_HD int64_t tet(int64_t m) { return (m * (m + 1)) / 2 * (m + 2) / 3; }  // m(m+1)(m+2)/6

// Largest r >= 0 with tri(r) <= q  (q >= 0).
DASTAC_HD int64_t tri_root(int64_t q) {
    int64_t r = (int64_t)((sqrt(8.0 * (double)q + 1.0) - 1.0) * 0.5);
    if (r < 0) r = 0;
    while (tri(r) > q) --r;
    while (tri(r + 1) <= q) ++r;
    return r;
}

// Largest a >= 0 with tet(a) <= q  (q >= 0).
DASTAC_HD int64_t tet_root(int64_t q) {
    int64_t a = (int64_t)cbrt(6.0 * (double)q);
    if (a > 0) --a;
    while (tet(a) > q) --a;
    while (tet(a + 1) <= q) ++a;
    return a;
}

// Exact band |i - j| <= w of an N x N matrix, 2w + 1 <= N, rows packed one after the other.  The
// counting polynomial has three pieces (rows clipped on the left, full rows, rows clipped on the
// right; Section 4, "Piecewise Polynomial Simplification" treats such piecewise results); written
// with clamps it is one expression: every row holds 2w + 1 points minus the w - i it loses on the
// left (rows i < w) and the i + w - (N - 1) it loses on the right (rows i > N - 1 - w).
DASTAC_HD int64_t band_row_start(int64_t N, int64_t w, int64_t i) {
    const int64_t a = i < w ? i : w;                      // rows before i that are clipped on the left
    const int64_t b = i > N - w ? i - (N - w) : 0;        // rows before i that are clipped on the right
    return i * (2 * w + 1) - (a * w - ((a * (a - 1)) >> 1)) - ((b * (b + 1)) >> 1);
}
DASTAC_HD int64_t band_jlo(int64_t w, int64_t i) { return i > w ? i - w : 0; }
DASTAC_HD int64_t band_jhi(int64_t N, int64_t w, int64_t i) { return i + w < N - 1 ? i + w : N - 1; }  // inclusive
// Row of position p (0 <= p < count): the clipped pieces are quadratic in i, the middle one linear.
DASTAC_HD int64_t band_row_of(int64_t N, int64_t w, int64_t p) {
    const int64_t top = band_row_start(N, w, w), mid_end = band_row_start(N, w, N - w);
    int64_t i;
    if (p < top) {  // rows 0 .. w-1: start(i) = i (w + 1) + i (i - 1) / 2
        const double f = 2.0 * (double)w + 1.0;
        i = (int64_t)((sqrt(f * f + 8.0 * (double)p) - f) * 0.5);
        if (i < 0) i = 0;
        while (i > 0 && band_row_start(N, w, i) > p) --i;
        while (i + 1 < w && band_row_start(N, w, i + 1) <= p) ++i;
    } else if (p < mid_end) {
        i = w + (p - top) / (2 * w + 1);
    } else {  // rows N-w .. N-1: the mirror image of the first piece
        const int64_t q = band_row_start(N, w, N) - 1 - p;
        const double f = 2.0 * (double)w + 1.0;
        int64_t r = (int64_t)((sqrt(f * f + 8.0 * (double)q) - f) * 0.5);
        if (r < 0) r = 0;
        while (r > 0 && band_row_start(N, w, r) > q) --r;
        while (r + 1 < w && band_row_start(N, w, r + 1) <= q) ++r;
        i = N - 1 - r;
    }
    return i;
}

// General offset band lo <= j - i <= hi of an N x N box.  Row t holds hi - lo + 1 points minus the
// max(0, -lo - t) it loses at column 0 and the max(0, t + hi - (N-1)) it loses at column N-1, for
// rows t in [first, last] = [max(0, -hi), min(N-1, N-1-lo)].  The points before row i are therefore
// a linear term minus two arithmetic series, each switched on by a clamp: a piecewise quadratic
// (Section 4, "Access domain linearization") written as one expression.
DASTAC_HD int64_t oband_first_row(int64_t hi) { return hi < 0 ? -hi : 0; }
DASTAC_HD int64_t oband_last_row(int64_t N, int64_t lo) { return lo > 0 ? N - 1 - lo : N - 1; }
DASTAC_HD int64_t oband_jlo(int64_t lo, int64_t i) { return i + lo > 0 ? i + lo : 0; }
DASTAC_HD int64_t oband_jhi(int64_t N, int64_t hi, int64_t i) { return i + hi < N - 1 ? i + hi : N - 1; }  // inclusive
// valid for first <= i <= last + 1
DASTAC_HD int64_t oband_row_start(int64_t N, int64_t lo, int64_t hi, int64_t i) {
    const int64_t f = oband_first_row(hi);
    int64_t total = (i - f) * (hi - lo + 1);
    const int64_t tl = i < -lo ? i : -lo;  // rows f .. tl-1 are clipped at column 0 by -lo - t
    if (tl > f) total -= (((-lo - f) + (-lo - (tl - 1))) * (tl - f)) >> 1;
    const int64_t tr = f > N - hi ? f : N - hi;  // rows tr .. i-1 are clipped at column N-1 by t + hi - N + 1
    if (i > tr) total -= (((tr + hi - N + 1) + (i + hi - N)) * (i - tr)) >> 1;
    return total;
}
// Row of position p: the starts are increasing in i, so bisection over the closed form is exact.
DASTAC_HD int64_t oband_row_of(int64_t N, int64_t lo, int64_t hi, int64_t p) {
    int64_t a = oband_first_row(hi), b = oband_last_row(N, lo);
    while (a < b) {
        const int64_t mid = (a + b + 1) >> 1;
        if (oband_row_start(N, lo, hi, mid) <= p) a = mid;
        else b = mid - 1;
    }
    return a;
}

// kPlane helpers: the k-th free index (k = 0, 1) of a map with dependent index dep.
DASTAC_HD int plane_free(int dep, int k) { return k + (k >= dep ? 1 : 0); }
// Element k of a 3-index array without a dynamically indexed access (keeps the array in registers).
DASTAC_HD int32_t pick3(const int32_t* v, int k) { return k == 0 ? v[0] : k == 1 ? v[1] : v[2]; }
DASTAC_HD void put3(int32_t* v, int k, int32_t x) {
    if (k == 0) v[0] = x;
    else if (k == 1) v[1] = x;
    else v[2] = x;
}

// Upper triangle / trapezoid: points before row i, in units of (j) positions.
DASTAC_HD int64_t upper_row_start(int64_t N, int64_t i) { return i * N - ((i * (i - 1)) >> 1); }

// rowbase(i) + j = position of (i, j): rowbase may be used with any j >= i.
DASTAC_HD int64_t upper_row_base(int64_t N, int64_t i) { return (i * (2 * N - i - 1)) >> 1; }

// Largest i with upper_row_start(N, i) <= t, for 0 <= t < tri-like count.
DASTAC_HD int64_t upper_row_of(int64_t N, int64_t t) {
    const double f = 2.0 * (double)N + 1.0;
    double disc = f * f - 8.0 * (double)t;
    if (disc < 0.0) disc = 0.0;
    int64_t i = (int64_t)((f - sqrt(disc)) * 0.5);
    if (i < 0) i = 0;
    if (i > N - 1) i = N - 1;
    while (i > 0 && upper_row_start(N, i) > t) --i;
    while (i + 1 < N && upper_row_start(N, i + 1) <= t) ++i;
    return i;
}

DASTAC_HD bool in_set(const IndexMap& m, const int32_t* idx) {
    // fixed trip counts with a guard keep idx and m in registers (no dynamically indexed arrays)
#pragma unroll
    for (int k = 0; k < 3; ++k)
        if (k < m.rank && (idx[k] < 0 || idx[k] >= m.dims[k])) return false;
    switch (m.kind) {
        case kDense: return true;
        case kUpper: return idx[0] <= idx[1];
        case kLower: return idx[1] <= idx[0];
        case kBandDiagonals: {
            int64_t d = (int64_t)idx[1] - idx[0];
            return d <= m.w && -d <= m.w;
        }
        case kTetrahedron: return idx[0] <= idx[1] && idx[1] <= idx[2];
        case kBandExact: {
            int64_t d = (int64_t)idx[1] - idx[0];
            return d <= m.w && -d <= m.w;
        }
        case kUpperShifted: return (int64_t)idx[1] - idx[0] >= m.w;
        case kBandOffsets: {
            int64_t d = (int64_t)idx[1] - idx[0];
            return d >= m.lo_off && d <= m.hi_off;
        }
        case kPlane: {
            const int dep = (int)m.w;
            const int64_t want = m.lo_off >= 0 ? (m.lo_off == 0 ? idx[0] : m.lo_off == 1 ? idx[1] : idx[2]) : m.hi_off;
            const int64_t have = dep == 0 ? idx[0] : dep == 1 ? idx[1] : idx[2];
            if (have != want) return false;
            // a free index that is the source of an equality is limited by the smaller extent
            const int64_t f0 = plane_free(dep, 0) == 0 ? idx[0] : idx[1];
            return f0 < m.M && (m.rank == 2 || (plane_free(dep, 1) == 1 ? idx[1] : idx[2]) < m.Q);
        }
        default: return false;
    }
}

// Position of a point of the set (caller guarantees membership).
DASTAC_HD int64_t rank_of(const IndexMap& m, const int32_t* idx) {
    switch (m.kind) {
        case kDense: {
            int64_t lin = 0;
#pragma unroll
            for (int k = 0; k < 3; ++k)
                if (k < m.rank) lin = lin * m.dims[k] + idx[k];
            return lin;
        }
        case kUpper: {
            int64_t p = upper_row_base(m.N, idx[0]) + idx[1];
            return m.rank == 3 ? p * m.Q + idx[2] : p;
        }
        case kLower: return tri(idx[0]) + idx[1];
        case kBandDiagonals: return ((int64_t)idx[1] - idx[0] + m.w) * m.N + idx[0];
        case kTetrahedron: {
            const int64_t n = m.N;
            return tet(n) - tet(n - idx[0]) + tri(n - idx[0]) - tri(n - idx[1]) +
                   ((int64_t)idx[2] - idx[1]);
        }
        case kBandExact: return band_row_start(m.N, m.w, idx[0]) + (idx[1] - band_jlo(m.w, idx[0]));
        case kUpperShifted: return upper_row_base(m.M, idx[0]) + (idx[1] - m.w);  // the size-M triangle at column j - c
        case kBandOffsets:
            return oband_row_start(m.N, m.lo_off, m.hi_off, idx[0]) + (idx[1] - oband_jlo(m.lo_off, idx[0]));
        case kPlane: {
            const int dep = (int)m.w;
            const int64_t f0 = plane_free(dep, 0) == 0 ? idx[0] : idx[1];
            if (m.rank == 2) return f0;
            const int64_t f1 = plane_free(dep, 1) == 1 ? idx[1] : idx[2];
            return f0 * m.Q + f1;
        }
        default: return -1;
    }
}

// Point stored at position p (0 <= p < slots).  Padding slots of the diagonal layout get column -1.
DASTAC_HD void unrank_of(const IndexMap& m, int64_t p, int32_t* idx) {
    switch (m.kind) {
        case kDense: {
#pragma unroll
            for (int k = 2; k >= 0; --k)
                if (k < m.rank) {
                    int64_t q = p / m.dims[k];
                    idx[k] = (int32_t)(p - q * m.dims[k]);
                    p = q;
                }
            return;
        }
        case kUpper: {
            int64_t t = p;
            if (m.rank == 3) {
                t = p / m.Q;
                idx[2] = (int32_t)(p - t * m.Q);
            }
            int64_t i = upper_row_of(m.N, t);
            idx[0] = (int32_t)i;
            idx[1] = (int32_t)(i + (t - upper_row_start(m.N, i)));
            return;
        }
        case kLower: {
            int64_t i = tri_root(p);
            idx[0] = (int32_t)i;
            idx[1] = (int32_t)(p - tri(i));
            return;
        }
        case kBandDiagonals: {
            int64_t d = p / m.N;
            int64_t i = p - d * m.N;
            int64_t j = i + d - m.w;
            idx[0] = (int32_t)i;
            idx[1] = (j < 0 || j >= m.N) ? -1 : (int32_t)j;
            return;
        }
        case kTetrahedron: {
            const int64_t n = m.N;
            int64_t q = m.count - 1 - p;
            int64_t a = tet_root(q);
            q -= tet(a);
            int64_t b = tri_root(q);
            int64_t c = q - tri(b);
            idx[0] = (int32_t)(n - 1 - a);
            idx[1] = (int32_t)(n - 1 - b);
            idx[2] = (int32_t)(n - 1 - c);
            return;
        }
        case kBandExact: {
            const int64_t i = band_row_of(m.N, m.w, p);
            idx[0] = (int32_t)i;
            idx[1] = (int32_t)(band_jlo(m.w, i) + (p - band_row_start(m.N, m.w, i)));
            return;
        }
        case kUpperShifted: {
            const int64_t i = upper_row_of(m.M, p);
            idx[0] = (int32_t)i;
            idx[1] = (int32_t)(m.w + i + (p - upper_row_start(m.M, i)));
            return;
        }
        case kBandOffsets: {
            const int64_t i = oband_row_of(m.N, m.lo_off, m.hi_off, p);
            idx[0] = (int32_t)i;
            idx[1] = (int32_t)(oband_jlo(m.lo_off, i) + (p - oband_row_start(m.N, m.lo_off, m.hi_off, i)));
            return;
        }
        case kPlane: {
            const int dep = (int)m.w;
            int64_t f0 = p, f1 = 0;
            if (m.rank == 3) {
                f0 = p / m.Q;
                f1 = p - f0 * m.Q;
            }
            int32_t v[3] = {0, 0, 0};
            put3(v, plane_free(dep, 0), (int32_t)f0);
            if (m.rank == 3) put3(v, plane_free(dep, 1), (int32_t)f1);
            put3(v, dep, m.lo_off >= 0 ? pick3(v, (int)m.lo_off) : (int32_t)m.hi_off);
#pragma unroll
            for (int k = 0; k < 3; ++k)
                if (k < m.rank) idx[k] = v[k];
            return;
        }
        default: return;
    }
}

// For fixed outer indices idx[0 .. rank-2], the innermost indices of the set form one interval
// [jlo, jhi) and the point (outer, j) is stored at pbase + j: pbase is the loop-invariant part of
// the ranking polynomial, hoisted out of the innermost loop.  Returns false when the interval is
// empty or the layout is not contiguous along the innermost index (padded diagonals).
DASTAC_HD bool row_span(const IndexMap& m, const int32_t* idx, int64_t& jlo, int64_t& jhi, int64_t& pbase) {
    switch (m.kind) {
        case kDense: {
            int64_t lin = 0;
#pragma unroll
            for (int k = 0; k < 2; ++k)
                if (k + 1 < m.rank) lin = lin * m.dims[k] + idx[k];
            jlo = 0;
            jhi = m.rank == 3 ? m.dims[2] : m.rank == 2 ? m.dims[1] : m.dims[0];
            pbase = lin * jhi;
            return jhi > 0;
        }
        case kUpper: {
            // Q > 1 with rank 2: the half cube seen as a matrix of rows i and columns j Q + l (used by
            // the copy kernels when the two inner dense strides are compact)
            if (m.rank == 3) {  // half cube: the trailing index of fibre (i, j), j >= i
                if (idx[0] >= m.M || idx[1] < idx[0]) return false;
                jlo = 0;
                jhi = m.Q;
                pbase = (upper_row_base(m.N, idx[0]) + idx[1]) * m.Q;
                return jhi > 0;
            }
            if (idx[0] >= m.M) return false;
            jlo = idx[0] * m.Q;
            jhi = m.N * m.Q;
            pbase = upper_row_base(m.N, idx[0]) * m.Q;
            return true;
        }
        case kLower: {
            jlo = 0;
            jhi = (int64_t)idx[0] + 1;
            pbase = tri(idx[0]);
            return true;
        }
        case kTetrahedron: {
            if (idx[1] < idx[0]) return false;
            const int64_t n = m.N;
            jlo = idx[1];
            jhi = n;
            pbase = tet(n) - tet(n - idx[0]) + tri(n - idx[0]) - tri(n - idx[1]) - idx[1];
            return true;
        }
        case kBandExact: {
            jlo = band_jlo(m.w, idx[0]);
            jhi = band_jhi(m.N, m.w, idx[0]) + 1;
            pbase = band_row_start(m.N, m.w, idx[0]) - jlo;
            return true;
        }
        case kUpperShifted: {
            if (idx[0] >= m.M) return false;
            jlo = idx[0] + m.w;
            jhi = m.N;
            pbase = upper_row_base(m.M, idx[0]) - m.w;
            return true;
        }
        case kPlane: {
            // contiguous along the innermost index only when that index is free
            const int dep = (int)m.w, last = m.rank - 1;
            if (dep == last) return false;
            const int64_t want = m.lo_off >= 0 ? (m.lo_off == 0 ? idx[0] : idx[1]) : m.hi_off;
            if ((dep == 0 ? idx[0] : idx[1]) != want) return false;
            jlo = 0;
            if (m.rank == 2) {  // dep = 0: the single stored row
                jhi = m.M;
                pbase = 0;
            } else {
                const int64_t f0 = plane_free(dep, 0) == 0 ? idx[0] : idx[1];
                if (f0 >= m.M) return false;
                jhi = m.Q;
                pbase = f0 * m.Q;
            }
            return jhi > 0;
        }
        case kBandOffsets: {
            if (idx[0] < oband_first_row(m.hi_off) || idx[0] > oband_last_row(m.N, m.lo_off)) return false;
            jlo = oband_jlo(m.lo_off, idx[0]);
            jhi = oband_jhi(m.N, m.hi_off, idx[0]) + 1;
            pbase = oband_row_start(m.N, m.lo_off, m.hi_off, idx[0]) - jlo;
            return true;
        }
        default: return false;
    }
}

// Step idx to the point stored at the next position (valid while that position exists).
// Not defined for the padded-diagonal layout, whose slots are walked by position.
DASTAC_HD void advance(const IndexMap& m, int32_t* idx) {
    switch (m.kind) {
        case kDense: {
#pragma unroll
            for (int k = 2; k >= 0; --k)
                if (k < m.rank) {
                    if (++idx[k] < m.dims[k]) return;
                    idx[k] = 0;
                }
            return;
        }
        case kUpper: {
            if (m.rank == 3) {
                if (++idx[2] < m.Q) return;
                idx[2] = 0;
            }
            if (++idx[1] < m.N) return;
            ++idx[0];
            idx[1] = idx[0];
            return;
        }
        case kLower: {
            if (++idx[1] <= idx[0]) return;
            ++idx[0];
            idx[1] = 0;
            return;
        }
        case kTetrahedron: {
            if (++idx[2] < m.N) return;
            if (++idx[1] >= m.N) {
                ++idx[0];
                idx[1] = idx[0];
            }
            idx[2] = idx[1];
            return;
        }
        case kBandExact: {
            if (idx[1] < band_jhi(m.N, m.w, idx[0])) {
                ++idx[1];
                return;
            }
            ++idx[0];
            idx[1] = (int32_t)band_jlo(m.w, idx[0]);
            return;
        }
        case kUpperShifted: {
            if (++idx[1] < m.N) return;
            ++idx[0];
            idx[1] = (int32_t)(idx[0] + m.w);
            return;
        }
        case kPlane: {
            const int dep = (int)m.w;
            const int a = plane_free(dep, 0), b = plane_free(dep, 1);
            int32_t v[3] = {idx[0], m.rank > 1 ? idx[1] : 0, m.rank > 2 ? idx[2] : 0};
            bool carry = true;
            if (m.rank == 3) {
                const int32_t nb = pick3(v, b) + 1;
                carry = nb >= m.Q;
                put3(v, b, carry ? 0 : nb);
            }
            if (carry) put3(v, a, pick3(v, a) + 1);
            if (m.lo_off >= 0) put3(v, dep, pick3(v, (int)m.lo_off));
#pragma unroll
            for (int k = 0; k < 3; ++k)
                if (k < m.rank) idx[k] = v[k];
            return;
        }
        case kBandOffsets: {
            if (idx[1] < oband_jhi(m.N, m.hi_off, idx[0])) {
                ++idx[1];
                return;
            }
            ++idx[0];
            idx[1] = (int32_t)oband_jlo(m.lo_off, idx[0]);
            return;
        }
        default: return;
    }
}

}  // namespace dastac
