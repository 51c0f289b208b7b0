// Piecewise polynomials over polyhedral domains and their fusion (Algorithm 2, "Piecewise
// QuasiPolynomial Fusion"): host-side objects, exact rational arithmetic.
#pragma once
#include <array>
#include <cstdint>
#include <functional>
#include <map>
#include <vector>

namespace dastac {

// sum_t num[t] / den * prod_v x_v ^ exps[t][v]
struct PwPoly {
    int nvars = 0;
    std::vector<std::array<int32_t, 3>> exps;
    std::vector<int64_t> num;
    int64_t den = 1;
};

// { x in box : a[r] . x + c[r] >= 0 (or == 0) for every row r }
struct PwDomain {
    int nvars = 0;
    int64_t lo[3] = {0, 0, 0}, hi[3] = {-1, -1, -1};  // inclusive box
    std::vector<std::array<int64_t, 4>> rows;         // a0, a1, a2, c
    std::vector<uint8_t> is_eq;
};

struct PwPiece {
    PwDomain domain;
    PwPoly poly;
};

// (P - Q) restricted to D is identically zero.  Decided symbolically when the equalities of D alone
// make the difference vanish, else by evaluating it at every integer point of D when D has at most
// `max_points` box points; `decided` is false when neither applies (the answer is then "no").
bool pw_difference_vanishes_on(const PwPoly& P, const PwPoly& Q, const PwDomain& D, int64_t max_points, bool& decided);

// Algorithm 2: for every piece (D, P), every other piece (D', P') with (P - P')|_D' = 0 is removed
// and D grows by D'.  owner[k] = the piece whose polynomial holds on piece k afterwards
// (owner[k] == k for the pieces that remain).
void pw_fuse(const std::vector<PwPiece>& pieces, std::vector<int>& owner, int64_t max_points = int64_t(1) << 22);

// The same procedure over any representation of the pieces: agrees(k, q) answers whether piece k's
// polynomial equals piece q's on the (original) domain of piece q.
void pw_fuse_core(int n, const std::function<bool(int, int)>& agrees, std::vector<int>& owner);

}  // namespace dastac
