// Index map of a structure that is none of the recognised classes: any conjunction of affine
// comparisons over up to three indices whose innermost bounded indices carry unit coefficients.
//
// The packed position of a point is the number of points that precede it (Section 4, "Preceding
// Accesses" and "Access domain linearization"), split by the level at which the predecessor
// differs:
//
//   P(i, j, k) = S1(i) + S2(i, j) + (k - klo(i, j))
//
//   S1(i)    = points in the slabs before i.  A piecewise polynomial in i of degree <= rank; its
//              pieces and coefficients are fitted on the host, when the structure is created, to
//              the library's own brute-force count of every slab (the stand-in for the symbolic
//              counting step of Algorithm 1), pieces that agree are fused (Algorithm 2), and the
//              result is checked against the enumeration.  Stored in Newton form on integer
//              differences, so its evaluation is exact integer arithmetic with exact divisions
//              by 2 and 6 only.
//   S2(i, j) = points of slab i in the fibres before j (rank 3 only): the sum over j' < j of the
//              fibre length max(0, min_u U_u(i,j') - max_l L_l(i,j') + 1), where the U_u, L_l are the
//              bounds on k read off the comparison rows.  The sum of this piecewise linear
//              function is taken in closed form, segment by segment between the points where the
//              binding bound changes (an arithmetic series per segment): no loop over j'.
//   klo      = the largest lower bound on the last index, read off the rows.
//
// No table indexed by a tensor index is kept: the map is the comparison rows, at most kGMaxPieces
// intervals of i and one cubic per interval.  It is slower than the closed forms of the recognised
// classes and is used by the element-wise kernels only.
#pragma once
#include <cstdint>

#ifndef DASTAC_HD
#ifdef __CUDACC__
#define DASTAC_HD __host__ __device__ __forceinline__
#else
#define DASTAC_HD inline
#endif
#endif

namespace dastac {

constexpr int kGMaxRows = 24;     // comparison rows, the box included
constexpr int kGMaxPieces = 12;   // intervals of i with their own cubic
constexpr int kGMaxBounds = 4;    // lower (and upper) bounds on the last index of a rank-3 set

struct GenericMap {
    int32_t rank, nrows, npieces, reserved;
    int64_t dims[3];
    int64_t count;
    int64_t a[kGMaxRows][3];  // row r:  a[r][0] i + a[r][1] j + a[r][2] k + c[r] >= 0
    int64_t c[kGMaxRows];
    // interval p covers piece_lo[p] <= i < piece_lo[p + 1]; on it
    //   S1(i) = n0 + n1 t + n2 C(t,2) + n3 C(t,3),   t = i - anchor[p]
    int64_t piece_lo[kGMaxPieces + 1];
    int64_t anchor[kGMaxPieces];
    int64_t newton[kGMaxPieces][4];
};

DASTAC_HD int64_t g_floor_div(int64_t x, int64_t d) {  // d > 0
    int64_t q = x / d;
    return (x % d != 0 && x < 0) ? q - 1 : q;
}

DASTAC_HD bool g_in_domain(const GenericMap& g, const int64_t* idx) {
    for (int r = 0; r < g.nrows; ++r) {
        int64_t v = g.c[r];
        for (int k = 0; k < g.rank; ++k) v += g.a[r][k] * idx[k];
        if (v < 0) return false;
    }
    return true;
}

// Interval [lo, hi] of the last index for fixed outer indices; false when a row that does not
// involve the last index fails (the fibre is empty whatever the interval says).
DASTAC_HD bool g_last_bounds(const GenericMap& g, const int64_t* outer, int64_t& lo, int64_t& hi) {
    const int last = g.rank - 1;
    lo = INT64_MIN / 4;
    hi = INT64_MAX / 4;
    bool ok = true;
    for (int r = 0; r < g.nrows; ++r) {
        int64_t rest = g.c[r];
        for (int k = 0; k < last; ++k) rest += g.a[r][k] * outer[k];
        const int64_t al = g.a[r][last];
        if (al == 0) {
            ok = ok && rest >= 0;
        } else if (al > 0) {  // x >= -rest  (|al| == 1)
            if (-rest > lo) lo = -rest;
        } else {  // x <= rest
            if (rest < hi) hi = rest;
        }
    }
    return ok;
}

DASTAC_HD int64_t g_s1(const GenericMap& g, int64_t i) {
    int p = 0;
    while (p + 1 < g.npieces && i >= g.piece_lo[p + 1]) ++p;
    const int64_t t = i - g.anchor[p];
    const int64_t c2 = (t * (t - 1)) / 2;            // exact: a product of two consecutive integers
    const int64_t c3 = (t * (t - 1)) / 2 * (t - 2) / 3;  // exact: C(t,3) = C(t,2) (t-2) / 3
    return g.newton[p][0] + g.newton[p][1] * t + g.newton[p][2] * c2 + g.newton[p][3] * c3;
}

// Points of slab i in the fibres j' < j (rank 3).
DASTAC_HD int64_t g_s2(const GenericMap& g, int64_t i, int64_t j) {
    // bounds on k as functions of j':  alpha j' + beta, and the range of j' that the rows without k allow
    int64_t la[kGMaxBounds], lb[kGMaxBounds], ua[kGMaxBounds], ub[kGMaxBounds];
    int nl = 0, nu = 0;
    int64_t jlo = 0, jhi = j - 1;
    for (int r = 0; r < g.nrows; ++r) {
        const int64_t rest = g.a[r][0] * i + g.c[r];
        const int64_t a1 = g.a[r][1], a2 = g.a[r][2];
        if (a2 > 0) {  // k >= -(a1 j' + rest)
            if (nl < kGMaxBounds) la[nl] = -a1, lb[nl] = -rest, ++nl;
        } else if (a2 < 0) {  // k <= a1 j' + rest
            if (nu < kGMaxBounds) ua[nu] = a1, ub[nu] = rest, ++nu;
        } else if (a1 > 0) {  // j' >= -rest
            if (-rest > jlo) jlo = -rest;
        } else if (a1 < 0) {  // j' <= rest
            if (rest < jhi) jhi = rest;
        } else if (rest < 0) {
            return 0;  // the slab is empty
        }
    }
    if (jhi < jlo) return 0;
    auto fibre = [&](int64_t x) {  // min U - max L + 1 at j' = x (may be negative)
        int64_t L = la[0] * x + lb[0], U = ua[0] * x + ub[0];
        for (int q = 1; q < nl; ++q) {
            const int64_t v = la[q] * x + lb[q];
            if (v > L) L = v;
        }
        for (int q = 1; q < nu; ++q) {
            const int64_t v = ua[q] * x + ub[q];
            if (v < U) U = v;
        }
        return U - L + 1;
    };
    // Walk [jlo, jhi] segment by segment: the next segment starts at the smallest point > x where two
    // of the affine functions involved (two lower bounds, two upper bounds, or an upper and a lower
    // bound shifted by one) cross.  Inside a segment the fibre length is one affine function of j'
    // with one sign, so its sum is an arithmetic series.
    int64_t total = 0, x = jlo;
    while (x <= jhi) {
        int64_t next = jhi + 1;
        auto cross = [&](int64_t a_, int64_t b_, int64_t c_, int64_t d_) {
            // a_ x + b_ = c_ x + d_  at  x* = (d_ - b_) / (a_ - c_): candidates floor(x*), floor(x*) + 1
            const int64_t den = a_ - c_;
            if (den == 0) return;
            int64_t num = d_ - b_, dd = den;
            if (dd < 0) num = -num, dd = -dd;
            const int64_t f = g_floor_div(num, dd);
            if (f > x && f < next) next = f;
            if (f + 1 > x && f + 1 < next) next = f + 1;
        };
        for (int p = 0; p < nl; ++p)
            for (int q = p + 1; q < nl; ++q) cross(la[p], lb[p], la[q], lb[q]);
        for (int p = 0; p < nu; ++p)
            for (int q = p + 1; q < nu; ++q) cross(ua[p], ub[p], ua[q], ub[q]);
        for (int p = 0; p < nu; ++p)
            for (int q = 0; q < nl; ++q) cross(ua[p], ub[p] + 1, la[q], lb[q]);
        const int64_t y = next - 1;  // the segment is [x, y]
        int64_t v0 = fibre(x), v1 = fibre(y);
        if (v0 < 0) v0 = 0;
        if (v1 < 0) v1 = 0;
        total += ((v0 + v1) * (y - x + 1)) / 2;
        x = next;
    }
    return total;
}

DASTAC_HD int64_t g_rank(const GenericMap& g, const int64_t* idx) {
    int64_t lo, hi;
    g_last_bounds(g, idx, lo, hi);
    if (g.rank == 1) return idx[0] - lo;
    int64_t p = g_s1(g, idx[0]);
    if (g.rank == 3) p += g_s2(g, idx[0], idx[1]);
    return p + (idx[g.rank - 1] - lo);
}

// Inverse by bisection on the monotone partial counts.
DASTAC_HD void g_unrank(const GenericMap& g, int64_t p, int64_t* idx) {
    if (g.rank == 1) {
        int64_t lo, hi;
        g_last_bounds(g, idx, lo, hi);
        idx[0] = lo + p;
        return;
    }
    int64_t a = 0, b = g.dims[0] - 1;  // largest i with S1(i) <= p
    while (a < b) {
        const int64_t mid = (a + b + 1) >> 1;
        if (g_s1(g, mid) <= p) a = mid;
        else b = mid - 1;
    }
    idx[0] = a;
    int64_t r = p - g_s1(g, a);
    if (g.rank == 3) {
        int64_t ja = 0, jb = g.dims[1] - 1;  // largest j with S2(i, j) <= r
        while (ja < jb) {
            const int64_t mid = (ja + jb + 1) >> 1;
            if (g_s2(g, a, mid) <= r) ja = mid;
            else jb = mid - 1;
        }
        idx[1] = ja;
        r -= g_s2(g, a, ja);
    }
    int64_t lo, hi;
    g_last_bounds(g, idx, lo, hi);
    idx[g.rank - 1] = lo + r;
}

}  // namespace dastac
