/*
 * CPU oracle for structured tensor algebra on packed layouts.  TEST INFRASTRUCTURE ONLY: it is
 * called by the tests, by the smoke check and by the benchmark's CPU-baseline leg, never by the
 * CUDA library, and it shares no code with it.
 *
 * Everything here is the plain definition written out, with no closed-form index polynomial:
 *
 *  - A structure is a set of integer points inside the box [0, dims) that satisfy every row of a
 *    list of affine comparisons over the indices and the size symbols (Section 2, "Unique set";
 *    Section 4, "Iteration space extraction").
 *  - The packed position of a point is the number of points of the set that precede it in
 *    lexicographic order, first index slowest, last index contiguous (Section 4, "Iteration
 *    space extraction", "Preceding Accesses" and "Access domain linearization":
 *    P = #{preceding accesses}).  Here that number is a counter advanced while enumerating.
 *  - Compress / decompress copy values between the dense tensor and the packed vector while
 *    walking the accessed indices (Section 3, "Data Layout Compression"); a redundancy map sends a
 *    redundant index to its unique representative (Section 2, "Redundancy map").
 *  - A contraction is the sum-of-products rule evaluated over the full dense index ranges with the
 *    body guarded by the structure predicate, each product added to the output element
 *    (Section 5.2, "Uncompressed Compute Code Generation"), accumulated in double.
 *
 * Parallelism: OpenMP static schedule over the outermost output index, which is the
 * parallelisation the paper itself applies (Section 5.2, "Parallelization").
 */
#include <math.h>
#ifdef _OPENMP
#include <omp.h>
#endif
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_MAX_RANK 4

/* rows: nrows x (rank + nparams + 1), row-major.  Row r holds
 *   sum_k rows[r][k] * idx[k] + sum_p rows[r][rank+p] * params[p] + rows[r][rank+nparams]
 * which must be >= 0 (is_eq[r] == 0) or == 0 (is_eq[r] != 0). */
typedef struct {
    int32_t rank, nparams, nrows;
    const int64_t* dims;
    const int64_t* rows;
    const uint8_t* is_eq;
    const int64_t* params;
} orc_desc;

static int in_domain(const orc_desc* d, const int64_t* idx) {
    const int w = d->rank + d->nparams + 1;
    for (int r = 0; r < d->nrows; ++r) {
        const int64_t* row = d->rows + (size_t)r * w;
        int64_t v = row[w - 1];
        for (int k = 0; k < d->rank; ++k) v += row[k] * idx[k];
        for (int p = 0; p < d->nparams; ++p) v += row[d->rank + p] * d->params[p];
        if (d->is_eq[r] ? (v != 0) : (v < 0)) return 0;
    }
    return 1;
}

/* Advance idx to the next point of the box in lexicographic order; 0 when the box is exhausted. */
static int box_next(const orc_desc* d, int64_t* idx) {
    for (int k = d->rank - 1; k >= 0; --k) {
        if (++idx[k] < d->dims[k]) return 1;
        idx[k] = 0;
    }
    return 0;
}

static int box_empty(const orc_desc* d) {
    for (int k = 0; k < d->rank; ++k)
        if (d->dims[k] <= 0) return 1;
    return d->rank <= 0;
}

static int64_t dense_linear(const orc_desc* d, const int64_t* idx) {
    int64_t lin = 0;
    for (int k = 0; k < d->rank; ++k) lin = lin * d->dims[k] + idx[k];
    return lin;
}

/* Number of points of the set. */
int64_t orc_count(const orc_desc* d) {
    if (box_empty(d)) return 0;
    int64_t idx[ORC_MAX_RANK] = {0, 0, 0, 0}, counter = 0;
    do {
        if (in_domain(d, idx)) ++counter;
    } while (box_next(d, idx));
    return counter;
}

/* table[dense linear index] = packed position of that point, or -1 outside the set. */
void orc_rank_table(const orc_desc* d, int64_t* table) {
    if (box_empty(d)) return;
    int64_t idx[ORC_MAX_RANK] = {0, 0, 0, 0}, counter = 0;
    do {
        table[dense_linear(d, idx)] = in_domain(d, idx) ? counter++ : -1;
    } while (box_next(d, idx));
}

/* idx_out[p * rank + k] = k-th index of the point stored at packed position p. */
void orc_unrank_table(const orc_desc* d, int32_t* idx_out) {
    if (box_empty(d)) return;
    int64_t idx[ORC_MAX_RANK] = {0, 0, 0, 0}, counter = 0;
    do {
        if (in_domain(d, idx)) {
            for (int k = 0; k < d->rank; ++k) idx_out[counter * d->rank + k] = (int32_t)idx[k];
            ++counter;
        }
    } while (box_next(d, idx));
}

/* Packed position of one point: the points preceding it are counted one by one.
 * Returns -1 if the point is not in the set. */
int64_t orc_rank_point(const orc_desc* d, const int64_t* point) {
    if (box_empty(d)) return -1;
    for (int k = 0; k < d->rank; ++k)
        if (point[k] < 0 || point[k] >= d->dims[k]) return -1;
    if (!in_domain(d, point)) return -1;
    int64_t idx[ORC_MAX_RANK] = {0, 0, 0, 0}, counter = 0;
    do {
        if (memcmp(idx, point, sizeof(int64_t) * (size_t)d->rank) == 0) return counter;
        if (in_domain(d, idx)) ++counter;
    } while (box_next(d, idx));
    return -1;
}

/* Compress: packed[counter] = dense[idx] over the set, elements moved as raw bytes. */
void orc_pack(const orc_desc* d, int64_t elt_size, const void* dense, void* packed) {
    if (box_empty(d)) return;
    int64_t idx[ORC_MAX_RANK] = {0, 0, 0, 0}, counter = 0;
    do {
        if (in_domain(d, idx)) {
            memcpy((char*)packed + counter * elt_size,
                   (const char*)dense + dense_linear(d, idx) * elt_size, (size_t)elt_size);
            ++counter;
        }
    } while (box_next(d, idx));
}

/* Decompress: dense = 0; dense[idx] = packed[counter]; with a redundancy map given as an index
 * permutation (mirror[k] = which source index lands in position k), the permuted point receives
 * the same value when it differs from the point itself. */
void orc_unpack(const orc_desc* d, const int32_t* mirror, int64_t elt_size, const void* packed,
                void* dense) {
    if (box_empty(d)) return;
    int64_t total = 1;
    for (int k = 0; k < d->rank; ++k) total *= d->dims[k];
    memset(dense, 0, (size_t)(total * elt_size));
    int64_t idx[ORC_MAX_RANK] = {0, 0, 0, 0}, counter = 0;
    do {
        if (in_domain(d, idx)) {
            const char* src = (const char*)packed + counter * elt_size;
            memcpy((char*)dense + dense_linear(d, idx) * elt_size, src, (size_t)elt_size);
            if (mirror) {
                int64_t m[ORC_MAX_RANK];
                int ok = 1;
                for (int k = 0; k < d->rank; ++k) {
                    m[k] = idx[mirror[k]];
                    if (m[k] >= d->dims[k]) ok = 0;
                }
                if (ok && memcmp(m, idx, sizeof(int64_t) * (size_t)d->rank) != 0)
                    memcpy((char*)dense + dense_linear(d, m) * elt_size, src, (size_t)elt_size);
            }
            ++counter;
        }
    } while (box_next(d, idx));
}

/* ---- band stored as padded diagonals -------------------------------------------------------
 * Layout: 2w+1 diagonals of N slots; slot (d, i), d outer, holds A[i][i + d - w] when that
 * column exists and +0.0f otherwise.  The enumeration runs over slots. */
void orc_band_pack(int64_t N, int64_t w, const float* dense, float* packed) {
    int64_t counter = 0;
    for (int64_t d = 0; d <= 2 * w; ++d)
        for (int64_t i = 0; i < N; ++i) {
            int64_t j = i + d - w;
            packed[counter++] = (j >= 0 && j < N) ? dense[i * N + j] : 0.0f;
        }
}

void orc_band_unpack(int64_t N, int64_t w, const float* packed, float* dense) {
    memset(dense, 0, (size_t)(N * N) * sizeof(float));
    int64_t counter = 0;
    for (int64_t d = 0; d <= 2 * w; ++d)
        for (int64_t i = 0; i < N; ++i) {
            int64_t j = i + d - w;
            if (j >= 0 && j < N) dense[i * N + j] = packed[counter];
            ++counter;
        }
}

/* slot_table[i * N + j] = slot of (i, j), or -1 outside the band. */
void orc_band_slot_table(int64_t N, int64_t w, int64_t* slot_table) {
    for (int64_t t = 0; t < N * N; ++t) slot_table[t] = -1;
    int64_t counter = 0;
    for (int64_t d = 0; d <= 2 * w; ++d)
        for (int64_t i = 0; i < N; ++i) {
            int64_t j = i + d - w;
            if (j >= 0 && j < N) slot_table[i * N + j] = counter;
            ++counter;
        }
}

/* ---- contractions ---------------------------------------------------------------------------
 * Inputs are fp32 arrays, or bf16 bit patterns (is_bf16 != 0) widened exactly to double.
 * Outputs: `out` = the sum in double, `out_abs` = the sum of the absolute values of the same
 * products (the denominator of the forward-error bound), both may be computed for a subset of the
 * outermost output index: sel[s] is the logical index i of the s-th supplied slice of the
 * structured operand. */
static inline double widen(const void* p, int64_t at, int is_bf16) {
    if (is_bf16) {
        union { uint32_t u; float f; } c;
        c.u = (uint32_t)((const uint16_t*)p)[at] << 16;
        return (double)c.f;
    }
    return (double)((const float*)p)[at];
}

/* y[i] = sum_j [ (i, j) in set ] A[i][j] * x[j]           (A(i) := B(i,j) * C(j), Table 1 "SpMV")
 * A_rows[s] is the dense row sel[s] of A (N values). */
void orc_matvec(const orc_desc* d, int64_t nsel, const int64_t* sel, const float* A_rows,
                const float* x, double* out, double* out_abs) {
    const int64_t N = d->dims[1];
#pragma omp parallel for schedule(static)
    for (int64_t s = 0; s < nsel; ++s) {
        double acc = 0.0, acc_abs = 0.0;
        for (int64_t j = 0; j < N; ++j) {
            int64_t idx[2] = {sel[s], j};
            if (in_domain(d, idx)) {
                double p = (double)A_rows[s * N + j] * (double)x[j];
                acc += p;
                acc_abs += fabs(p);
            }
        }
        out[s] = acc;
        out_abs[s] = acc_abs;
    }
}

/* Symmetric product from the unique upper part:  Sfull[i][j] = U[min(i,j)][max(i,j)],
 * y[i] = sum_j Sfull[i][j] * x[j]  (Section 2, "Redundancy map": redundant (x, y) with x > y reads
 * the unique element (y, x)).  U is a dense N x N array; entries below the diagonal are ignored. */
void orc_symv(int64_t N, const float* U, const float* x, double* out, double* out_abs) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < N; ++i) {
        double acc = 0.0, acc_abs = 0.0;
        for (int64_t j = 0; j < N; ++j) {
            int64_t lo = i < j ? i : j, hi = i < j ? j : i;
            double p = (double)U[lo * N + hi] * (double)x[j];
            acc += p;
            acc_abs += fabs(p);
        }
        out[i] = acc;
        out_abs[i] = acc_abs;
    }
}

/* C[i][c] = sum_j [ (i, j) in set ] A[i][j] * B[j][c];  B is N x ncols row-major. */
void orc_matmat(const orc_desc* d, int is_bf16, int64_t nsel, const int64_t* sel,
                const void* A_rows, const void* B, int64_t ncols, double* out, double* out_abs) {
    const int64_t N = d->dims[1];
#pragma omp parallel for schedule(static)
    for (int64_t s = 0; s < nsel; ++s) {
        for (int64_t c = 0; c < ncols; ++c) {
            double acc = 0.0, acc_abs = 0.0;
            for (int64_t j = 0; j < N; ++j) {
                int64_t idx[2] = {sel[s], j};
                if (in_domain(d, idx)) {
                    double p = widen(A_rows, s * N + j, is_bf16) * widen(B, j * ncols + c, is_bf16);
                    acc += p;
                    acc_abs += fabs(p);
                }
            }
            out[s * ncols + c] = acc;
            out_abs[s * ncols + c] = acc_abs;
        }
    }
}

/* M[i][r] = sum_j sum_k [ (i, j, k) in set ] T[i][j][k] * B[j][r] * C[k][r]
 * (A(i,j) := B(i,k,l) * C(k,j) * D(l,j), Table 1 "MTTKRP", with the indices renamed).
 * T_slabs[s] is the dense n x n slab sel[s] of T. */
void orc_mttkrp(const orc_desc* d, int64_t nsel, const int64_t* sel, const float* T_slabs,
                const float* B, const float* C, int64_t R, double* out, double* out_abs) {
    const int64_t nj = d->dims[1], nk = d->dims[2];
#pragma omp parallel for schedule(static)
    for (int64_t s = 0; s < nsel; ++s) {
        for (int64_t r = 0; r < R; ++r) {
            double acc = 0.0, acc_abs = 0.0;
            for (int64_t j = 0; j < nj; ++j)
                for (int64_t k = 0; k < nk; ++k) {
                    int64_t idx[3] = {sel[s], j, k};
                    if (in_domain(d, idx)) {
                        double p = (double)T_slabs[(s * nj + j) * nk + k] * (double)B[j * R + r] *
                                   (double)C[k * R + r];
                        acc += p;
                        acc_abs += fabs(p);
                    }
                }
            out[s * R + r] = acc;
            out_abs[s * R + r] = acc_abs;
        }
    }
}

/* A[i][j][k] = sum_l [ (i, j, l) in set ] B[i][j][l] * C[k][l]
 * (A(i,j,k) := B(i,j,l) * C(k,l), the tensor-times-matrix rule of the running example, Section 3).
 * B_slabs[s] is the dense N x Q slab sel[s] of B; C is K x Q row-major; out[s] is the N x K slab. */
void orc_ttm(const orc_desc* d, int64_t nsel, const int64_t* sel, const float* B_slabs, const float* C,
             int64_t K, double* out, double* out_abs) {
    const int64_t N = d->dims[1], Q = d->dims[2];
#pragma omp parallel for schedule(static)
    for (int64_t s = 0; s < nsel; ++s) {
        for (int64_t j = 0; j < N; ++j)
            for (int64_t k = 0; k < K; ++k) {
                double acc = 0.0, acc_abs = 0.0;
                for (int64_t l = 0; l < Q; ++l) {
                    int64_t idx[3] = {sel[s], j, l};
                    if (in_domain(d, idx)) {
                        double p = (double)B_slabs[(s * N + j) * Q + l] * (double)C[k * Q + l];
                        acc += p;
                        acc_abs += fabs(p);
                    }
                }
                out[(s * N + j) * K + k] = acc;
                out_abs[(s * N + j) * K + k] = acc_abs;
            }
    }
}

/* A2[i1][i2] = sum_x [ (i1, i2) in set ] B[x][i1] * B[x][i2]
 * (A^k(i_1..i_k) := B(x,i_1) * ... * B(x,i_k) with k = 2, Table 1 "Polynomial Regression"; the set is
 * the unique part i1 <= i2 of the symmetric result, Section 2 "Redundancy map", and the output is
 * stored compressed over it, Section 4 "Iteration space extraction").  B is M x n row-major, fp32 or
 * bf16 bit patterns; out[s] is row sel[s] of the result as a dense row of n values, entries outside
 * the set are 0. */
void orc_moment2(const orc_desc* d, int is_bf16, int64_t nsel, const int64_t* sel, const void* B,
                 int64_t M, double* out, double* out_abs) {
    const int64_t n = d->dims[1];
#pragma omp parallel for collapse(2) schedule(static)
    for (int64_t s = 0; s < nsel; ++s) {
        for (int64_t i2 = 0; i2 < n; ++i2) {
            double acc = 0.0, acc_abs = 0.0;
            int64_t idx[2] = {sel[s], i2};
            if (in_domain(d, idx)) {
                for (int64_t x = 0; x < M; ++x) {
                    double p = widen(B, x * n + sel[s], is_bf16) * widen(B, x * n + i2, is_bf16);
                    acc += p;
                    acc_abs += fabs(p);
                }
            }
            out[s * n + i2] = acc;
            out_abs[s * n + i2] = acc_abs;
        }
    }
}

/* A3[i1][i2][i3] = sum_x [ (i1, i2, i3) in set ] B[x][i1] * B[x][i2] * B[x][i3]
 * (A^k(i_1..i_k) := B(x,i_1) * ... * B(x,i_k) with k = 3, Table 1 "Polynomial Regression"; the set is
 * the unique part i1 <= i2 <= i3 of the fully symmetric result, the hyper-triangular domain of
 * Section 1).  out[s] is slab sel[s] of the result as a dense n x n array, zero outside the set. */
void orc_moment3(const orc_desc* d, int is_bf16, int64_t nsel, const int64_t* sel, const void* B,
                 int64_t M, double* out, double* out_abs) {
    const int64_t n = d->dims[1];
#pragma omp parallel for collapse(2) schedule(static)
    for (int64_t s = 0; s < nsel; ++s) {
        for (int64_t i2 = 0; i2 < n; ++i2) {
            for (int64_t i3 = 0; i3 < n; ++i3) {
                double acc = 0.0, acc_abs = 0.0;
                int64_t idx[3] = {sel[s], i2, i3};
                if (in_domain(d, idx)) {
                    for (int64_t x = 0; x < M; ++x) {
                        double p = widen(B, x * n + sel[s], is_bf16) * widen(B, x * n + i2, is_bf16) *
                                   widen(B, x * n + i3, is_bf16);
                        acc += p;
                        acc_abs += fabs(p);
                    }
                }
                out[(s * n + i2) * n + i3] = acc;
                out_abs[(s * n + i2) * n + i3] = acc_abs;
            }
        }
    }
}

/* A[idx] = [ idx in set ] B[idx] * C[idx]   (A(i,j,k) := B(i,j,k) * C(i,j,k), Table 1 "THP", the tensor
 * Hadamard product with a structured B and a dense C; any rank up to 3).  B, C and out are dense
 * arrays over the box; outside the set the result is 0. */
void orc_hadamard(const orc_desc* d, const float* B, const float* C, double* out, double* out_abs) {
    int64_t total = 1;
    for (int k = 0; k < d->rank; ++k) total *= d->dims[k];
    for (int64_t t = 0; t < total; ++t) out[t] = out_abs[t] = 0.0;
    if (box_empty(d)) return;
    int64_t idx[ORC_MAX_RANK] = {0, 0, 0, 0};
    do {
        if (in_domain(d, idx)) {
            const int64_t lin = dense_linear(d, idx);
            const double p = (double)B[lin] * (double)C[lin];
            out[lin] = p;
            out_abs[lin] = fabs(p);
        }
    } while (box_next(d, idx));
}

/* ---- timed variants: loops clipped to the domain ---------------------------------------------
 * The same products as the masked forms above, but the loops run over the stored elements only
 * (Section 5.3, "Compressed Compute Code Generation": the generated loops visit the accessed
 * indices, and the operand is read from its compressed buffer).  The operand is the packed vector
 * in the enumeration order of the masked oracle; the position of a row's first element is a
 * counter advanced by the trip count of the clipped inner loop, never a ranking polynomial.
 * These exist to be timed as the CPU baseline (1 thread, or `threads` OpenMP threads with a static
 * schedule over the outermost output index, the paper's own parallelisation); a test checks them
 * against the masked forms on small sizes.  Results are double. */

/* y[i] = sum_{j >= i} A[i][j] x[j], A packed row after row (upper triangle). */
void orc_clip_matvec_upper(int64_t N, const float* packed, const float* x, double* y, int threads) {
    int64_t* start = (int64_t*)malloc(sizeof(int64_t) * (size_t)(N + 1));
    int64_t counter = 0;
    for (int64_t i = 0; i < N; ++i) {
        start[i] = counter;
        for (int64_t j = i; j < N; ++j) ++counter;
    }
#pragma omp parallel for schedule(static) num_threads(threads)
    for (int64_t i = 0; i < N; ++i) {
        const float* row = packed + start[i];
        double acc = 0.0;
        for (int64_t j = i; j < N; ++j) acc += (double)row[j - i] * (double)x[j];
        y[i] = acc;
    }
    free(start);
}

/* y = Sfull x from the packed upper triangle: every stored off-diagonal element is used for the two
 * outputs it contributes to.  Threads own blocks of rows of the stored triangle and private copies
 * of y, summed at the end. */
void orc_clip_symv(int64_t N, const float* packed, const float* x, double* y, int threads) {
    int64_t* start = (int64_t*)malloc(sizeof(int64_t) * (size_t)(N + 1));
    int64_t counter = 0;
    for (int64_t i = 0; i < N; ++i) {
        start[i] = counter;
        counter += N - i; /* trip count of j = i .. N-1 */
    }
    if (threads < 1) threads = 1;
    double* priv = (double*)calloc((size_t)threads * (size_t)N, sizeof(double));
#pragma omp parallel num_threads(threads)
    {
        int t = 0, nt = 1;
#ifdef _OPENMP
        t = omp_get_thread_num();
        nt = omp_get_num_threads();
#endif
        double* mine = priv + (size_t)t * (size_t)N;
        /* rows dealt round-robin so that every thread gets long and short rows */
        for (int64_t i = t; i < N; i += nt) {
            const float* row = packed + start[i];
            double acc = (double)row[0] * (double)x[i];
            const double xi = (double)x[i];
            for (int64_t j = i + 1; j < N; ++j) {
                const double v = (double)row[j - i];
                acc += v * (double)x[j];
                mine[j] += v * xi;
            }
            mine[i] += acc;
        }
    }
    for (int64_t i = 0; i < N; ++i) {
        double acc = 0.0;
        for (int t = 0; t < threads; ++t) acc += priv[(size_t)t * (size_t)N + i];
        y[i] = acc;
    }
    free(priv);
    free(start);
}

/* C[i][c] = sum_{|i-j| <= w} A[i][j] B[j][c], A as 2w+1 padded diagonals of N slots (slot (d, i)). */
void orc_clip_band_matmat(int64_t N, int64_t w, const float* diags, const float* B, int64_t ncols,
                          double* out, int threads) {
#pragma omp parallel for schedule(static) num_threads(threads)
    for (int64_t i = 0; i < N; ++i) {
        double* o = out + i * ncols;
        for (int64_t c = 0; c < ncols; ++c) o[c] = 0.0;
        const int64_t jlo = i - w < 0 ? 0 : i - w, jhi = i + w > N - 1 ? N - 1 : i + w;
        for (int64_t j = jlo; j <= jhi; ++j) {
            const double a = (double)diags[(j - i + w) * N + i];
            const float* b = B + j * ncols;
            for (int64_t c = 0; c < ncols; ++c) o[c] += a * (double)b[c];
        }
    }
}

/* M[i][r] = sum_{i <= j <= k} T[i][j][k] B[j][r] C[k][r], T packed in lexicographic order. */
void orc_clip_mttkrp_tetra(int64_t n, const float* packed, const float* B, const float* C, int64_t R,
                           double* M, int threads) {
    int64_t* start = (int64_t*)malloc(sizeof(int64_t) * (size_t)(n + 1));
    int64_t counter = 0;
    for (int64_t i = 0; i < n; ++i) {
        start[i] = counter;
        for (int64_t j = i; j < n; ++j) counter += n - j; /* trip count of k = j .. n-1 */
    }
#pragma omp parallel for schedule(dynamic, 1) num_threads(threads)
    for (int64_t i = 0; i < n; ++i) {
        double* m = M + i * R;
        for (int64_t r = 0; r < R; ++r) m[r] = 0.0;
        const float* t = packed + start[i];
        for (int64_t j = i; j < n; ++j) {
            const float* b = B + j * R;
            for (int64_t k = j; k < n; ++k) {
                const double v = (double)*t++;
                const float* c = C + k * R;
                for (int64_t r = 0; r < R; ++r) m[r] += v * (double)b[r] * (double)c[r];
            }
        }
    }
    free(start);
}

/* C[i][c] = sum_{j >= i} A[i][j] B[j][c] for the rows i in sel, bf16 bit patterns, A packed. */
void orc_clip_matmat_upper_bf16(int64_t N, int64_t nsel, const int64_t* sel, const uint16_t* packed,
                                const uint16_t* B, int64_t ncols, double* out, int threads) {
    int64_t* start = (int64_t*)malloc(sizeof(int64_t) * (size_t)(N + 1));
    int64_t counter = 0;
    for (int64_t i = 0; i < N; ++i) {
        start[i] = counter;
        counter += N - i;
    }
#pragma omp parallel for schedule(dynamic, 1) num_threads(threads)
    for (int64_t s = 0; s < nsel; ++s) {
        const int64_t i = sel[s];
        double* o = out + s * ncols;
        for (int64_t c = 0; c < ncols; ++c) o[c] = 0.0;
        const uint16_t* row = packed + start[i];
        for (int64_t j = i; j < N; ++j) {
            const double a = widen(row, j - i, 1);
            const uint16_t* b = B + j * ncols;
            for (int64_t c = 0; c < ncols; ++c) o[c] += a * widen(b, c, 1);
        }
    }
    free(start);
}

/* Thread count the contractions above will use. */
#ifdef _OPENMP
int orc_num_threads(void) { return omp_get_max_threads(); }
#else
int orc_num_threads(void) { return 1; }
#endif
