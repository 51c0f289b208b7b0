// Algorithm 2 ("Piecewise QuasiPolynomial Fusion", Section 4, "Piecewise Polynomial
// Simplification"): the counting step yields one polynomial per piece of the counted set, often
// with special cases on boundaries; a piece whose polynomial is reproduced by another piece's
// polynomial on its own domain is dropped and the other piece's domain grows by it.
//
// Host code only.  Polynomials have rational coefficients with a common denominator and are
// compared exactly (128-bit numerators).
#include <cstring>

#include "../../include/dastac.h"
#include "piecewise.cuh"

namespace dastac {
namespace {

using Key = std::array<int32_t, 3>;
using Terms = std::map<Key, __int128>;

// numerators of P * Q.den - Q * P.den (the common denominator P.den * Q.den is positive)
Terms difference(const PwPoly& P, const PwPoly& Q) {
    Terms t;
    for (size_t k = 0; k < P.num.size(); ++k) t[P.exps[k]] += (__int128)P.num[k] * Q.den;
    for (size_t k = 0; k < Q.num.size(); ++k) t[Q.exps[k]] -= (__int128)Q.num[k] * P.den;
    return t;
}

bool all_zero(const Terms& t) {
    for (const auto& kv : t)
        if (kv.second != 0) return false;
    return true;
}

// x_v := x_w + c (w < 0: x_v := c) in every term
Terms substitute(const Terms& t, int v, int w, int64_t c) {
    Terms out;
    for (const auto& kv : t) {
        const int e = kv.first[v];
        Key base = kv.first;
        base[v] = 0;
        // (x_w + c)^e = sum_u C(e,u) x_w^u c^(e-u)
        __int128 binom = 1;
        for (int u = 0; u <= e; ++u) {
            __int128 pw = 1;
            for (int q = 0; q < e - u; ++q) pw *= c;
            if (w < 0) {
                if (u == 0) out[base] += kv.second * pw;
            } else {
                Key k2 = base;
                k2[w] += u;
                out[k2] += kv.second * binom * pw;
            }
            binom = binom * (e - u) / (u + 1);
        }
    }
    return out;
}

__int128 evaluate(const Terms& t, const int64_t* x) {
    __int128 s = 0;
    for (const auto& kv : t) {
        __int128 m = kv.second;
        for (int v = 0; v < 3; ++v)
            for (int q = 0; q < kv.first[v]; ++q) m *= x[v];
        s += m;
    }
    return s;
}

bool in_domain(const PwDomain& D, const int64_t* x) {
    for (size_t r = 0; r < D.rows.size(); ++r) {
        int64_t v = D.rows[r][3];
        for (int k = 0; k < D.nvars; ++k) v += D.rows[r][k] * x[k];
        if (D.is_eq[r] ? v != 0 : v < 0) return false;
    }
    return true;
}

}  // namespace

bool pw_difference_vanishes_on(const PwPoly& P, const PwPoly& Q, const PwDomain& D, int64_t max_points, bool& decided) {
    decided = true;
    Terms diff = difference(P, Q);
    if (all_zero(diff)) return true;
    // the equalities of D that fix a variable, or tie it to another one with unit coefficients
    for (size_t r = 0; r < D.rows.size(); ++r) {
        if (!D.is_eq[r]) continue;
        int nz = 0, v = -1, w = -1;
        for (int k = 0; k < D.nvars; ++k)
            if (D.rows[r][k] != 0) {
                ++nz;
                if (v < 0) v = k;
                else w = k;
            }
        const int64_t c = D.rows[r][3];
        if (nz == 1 && (D.rows[r][v] == 1 || D.rows[r][v] == -1)) {
            diff = substitute(diff, v, -1, D.rows[r][v] == 1 ? -c : c);  // a x + c = 0
        } else if (nz == 2 && D.rows[r][v] == -D.rows[r][w] && (D.rows[r][v] == 1 || D.rows[r][v] == -1)) {
            // x_v - x_w + c = 0 (or its negative): the later variable is replaced
            const int64_t shift = D.rows[r][w] == 1 ? -c : c;  // x_w = x_v + shift
            diff = substitute(diff, w, v, shift);
        }
    }
    if (all_zero(diff)) return true;
    // exact check on the integer points of D
    __int128 box = 1;
    for (int k = 0; k < D.nvars; ++k) {
        if (D.hi[k] < D.lo[k]) return true;  // empty domain
        box *= (__int128)(D.hi[k] - D.lo[k] + 1);
        if (box > max_points) {
            decided = false;
            return false;
        }
    }
    const Terms full = difference(P, Q);
    int64_t x[3] = {D.lo[0], D.nvars > 1 ? D.lo[1] : 0, D.nvars > 2 ? D.lo[2] : 0};
    for (;;) {
        if (in_domain(D, x) && evaluate(full, x) != 0) return false;
        int k = D.nvars - 1;
        for (; k >= 0; --k) {
            if (++x[k] <= D.hi[k]) break;
            x[k] = D.lo[k];
        }
        if (k < 0) break;
    }
    return true;
}

void pw_fuse_core(int n, const std::function<bool(int, int)>& agrees, std::vector<int>& owner) {
    owner.resize((size_t)n);
    for (int k = 0; k < n; ++k) owner[(size_t)k] = k;
    for (int k = 0; k < n; ++k) {
        if (owner[(size_t)k] != k) continue;  // removed earlier
        for (int other = 0; other < n; ++other) {
            if (other == k || owner[(size_t)other] != other) continue;
            // D' is everything `other` stands for by now
            bool all = true;
            for (int q = 0; q < n && all; ++q)
                if (owner[(size_t)q] == other) all = agrees(k, q);
            if (!all) continue;
            for (int q = 0; q < n; ++q)
                if (owner[(size_t)q] == other) owner[(size_t)q] = k;
        }
    }
}

void pw_fuse(const std::vector<PwPiece>& pieces, std::vector<int>& owner, int64_t max_points) {
    pw_fuse_core((int)pieces.size(),
                 [&](int k, int q) {
                     bool decided = true;
                     return pw_difference_vanishes_on(pieces[(size_t)k].poly, pieces[(size_t)q].poly,
                                                      pieces[(size_t)q].domain, max_points, decided);
                 },
                 owner);
}

}  // namespace dastac

using namespace dastac;

extern "C" dastac_status dastac_piecewise_fuse(const dastac_piece* pieces, int32_t n, int32_t* owner) {
    if (n < 0 || (n > 0 && (!pieces || !owner))) return DASTAC_ERR_INVALID_ARG;
    std::vector<PwPiece> ps((size_t)n);
    for (int k = 0; k < n; ++k) {
        const dastac_structure_desc& d = pieces[k].domain;
        const dastac_poly& p = pieces[k].poly;
        if (d.rank < 1 || d.rank > 3 || p.nvars != d.rank || p.nterms < 0 || p.den <= 0 || d.nparams < 0 ||
            d.nparams > 8 || d.nrows < 0 || d.nrows > 64 || !d.dims || (d.nrows > 0 && (!d.rows || !d.is_eq)) ||
            (d.nparams > 0 && !d.params) || (p.nterms > 0 && (!p.exps || !p.num)))
            return DASTAC_ERR_INVALID_ARG;
        PwPiece& q = ps[(size_t)k];
        q.domain.nvars = d.rank;
        for (int v = 0; v < d.rank; ++v) {
            if (d.dims[v] < 0) return DASTAC_ERR_INVALID_ARG;
            q.domain.lo[v] = 0;
            q.domain.hi[v] = d.dims[v] - 1;
        }
        const int width = d.rank + d.nparams + 1;
        for (int r = 0; r < d.nrows; ++r) {
            const int64_t* row = d.rows + (size_t)r * width;
            std::array<int64_t, 4> a{0, 0, 0, row[width - 1]};
            for (int v = 0; v < d.rank; ++v) a[v] = row[v];
            for (int s = 0; s < d.nparams; ++s) a[3] += row[d.rank + s] * d.params[s];
            q.domain.rows.push_back(a);
            q.domain.is_eq.push_back(d.is_eq[r] ? 1 : 0);
        }
        q.poly.nvars = p.nvars;
        q.poly.den = p.den;
        for (int t = 0; t < p.nterms; ++t) {
            std::array<int32_t, 3> e{0, 0, 0};
            for (int v = 0; v < p.nvars; ++v) {
                e[v] = p.exps[(size_t)t * p.nvars + v];
                if (e[v] < 0 || e[v] > 6) return DASTAC_ERR_INVALID_ARG;
            }
            q.poly.exps.push_back(e);
            q.poly.num.push_back(p.num[t]);
        }
    }
    std::vector<int> own;
    pw_fuse(ps, own);
    for (int k = 0; k < n; ++k) owner[k] = own[(size_t)k];
    return DASTAC_OK;
}
