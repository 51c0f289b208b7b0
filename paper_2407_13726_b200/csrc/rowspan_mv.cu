// y = A x for any packed matrix whose rows are stored contiguously (A(i) := B(i,j) * C(j), Table 1
// "SpMV"), fp32, optionally batched: dense boxes, lower triangles, exact and offset bands (a single
// off-diagonal is the per-summand buffer of the strided band of Section 6.4, the first row plus the
// sub-diagonal make a Leslie matrix).  For a fixed row the stored columns are one interval
// [jlo, jhi) at positions pbase + j, pbase being the hoisted part of the ranking polynomial
// (Section 4, last paragraph): a group of L lanes walks the interval and reduces with shuffles.
// The upper-triangular classes have their own kernels; this one is bound by HBM for long rows and
// by the index arithmetic per row for very short ones.
#include "common.cuh"

namespace dastac {
namespace {

template <int L>
__global__ void __launch_bounds__(256)
rowspan_mv_kernel(const IndexMap m, const float* __restrict__ A, const float* __restrict__ x, float* __restrict__ y,
                  const int64_t rows, const int64_t a_stride, const int64_t x_stride, const int64_t y_stride,
                  const int accumulate) {
    const int sub = threadIdx.x & (L - 1);
    const int64_t row = (blockIdx.x * (int64_t)blockDim.x + threadIdx.x) / L;
    A += blockIdx.y * a_stride;
    x += blockIdx.y * x_stride;
    y += blockIdx.y * y_stride;
    float acc0 = 0.f, acc1 = 0.f;
    if (row < rows) {
        int32_t idx[3] = {(int32_t)row, 0, 0};
        int64_t jlo = 0, jhi = 0, pbase = 0;
        if (row_span(m, idx, jlo, jhi, pbase)) {
            const float* a = A + pbase;  // a[j] = A(row, j)
            int64_t j = jlo + sub;
            // eight independent loads of each operand per lane keep enough bytes in flight for long rows
            for (; j + 7 * L < jhi; j += 8 * L) {
                float av[8], xv[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    av[u] = __ldg(a + j + u * L);
                    xv[u] = __ldg(x + j + u * L);
                }
#pragma unroll
                for (int u = 0; u < 8; u += 2) {
                    acc0 = fmaf(av[u], xv[u], acc0);
                    acc1 = fmaf(av[u + 1], xv[u + 1], acc1);
                }
            }
            for (; j < jhi; j += L) acc0 = fmaf(__ldg(a + j), __ldg(x + j), acc0);
        }
    }
    float acc = acc0 + acc1;
#pragma unroll
    for (int o = L / 2; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (row < rows && sub == 0) y[row] = accumulate ? y[row] + acc : acc;
}

// C = A B with a dense row-major B for the same classes: a warp owns a row of A and 32 columns of C at
// a time; the row's elements are read coalesced and broadcast by shuffles, the rows of B coalesced.
// One multiply-add per lane and stored element: bound by the reads of B from cache, well below the
// symmetric band's tiled kernel; it covers the classes that kernel does not take.
__global__ void __launch_bounds__(256)
rowspan_mm_kernel(const IndexMap m, const float* __restrict__ A, const float* __restrict__ B, const int64_t ldb,
                  float* __restrict__ C, const int64_t ldc, const int64_t ncols, const int64_t rows, const int accumulate) {
    const int lane = threadIdx.x & 31;
    const int64_t col_blocks = (ncols + 31) / 32;
    const int64_t items = rows * col_blocks;
    const int64_t warps = (int64_t)gridDim.x * (blockDim.x >> 5);
    for (int64_t it = blockIdx.x * (int64_t)(blockDim.x >> 5) + (threadIdx.x >> 5); it < items; it += warps) {
        const int64_t row = it / col_blocks, c = (it - row * col_blocks) * 32 + lane;
        int32_t idx[3] = {(int32_t)row, 0, 0};
        int64_t jlo = 0, jhi = 0, pbase = 0;
        float acc = 0.f;
        if (row_span(m, idx, jlo, jhi, pbase)) {
            const float* a = A + pbase;
            for (int64_t j0 = jlo; j0 < jhi; j0 += 32) {
                const float t = (j0 + lane < jhi) ? __ldg(a + j0 + lane) : 0.f;
                const int nj = (int)(jhi - j0 < 32 ? jhi - j0 : 32);
                for (int jj = 0; jj < nj; ++jj) {
                    const float tj = __shfl_sync(0xffffffffu, t, jj);
                    if (c < ncols) acc = fmaf(tj, __ldg(B + (j0 + jj) * ldb + c), acc);
                }
            }
        }
        if (c < ncols) C[row * ldc + c] = accumulate ? C[row * ldc + c] + acc : acc;
    }
}

}  // namespace

// Longest stored row of a structure whose rows are contiguous, or -1 when the class has none.
static int64_t longest_row(const IndexMap& m) {
    if (m.rank != 2) return -1;
    switch (m.kind) {
        case kDense: return m.dims[1];
        case kUpper: return m.dims[0] != m.dims[1] ? m.N : -1;  // trapezoids (a box of one row closes to this class)
        case kLower: return m.N;
        case kBandExact: return 2 * m.w + 1;
        case kPlane: return m.w == 0 ? m.M : -1;  // one stored row (a fixed first index)
        case kBandOffsets: {
            const int64_t len = m.hi_off - m.lo_off + 1;
            return len < m.N ? len : m.N;
        }
        default: return -1;
    }
}

bool rowspan_mv_supports(const IndexMap& m) { return longest_row(m) >= 0 && !m.symmetric; }

dastac_status launch_rowspan_mv(const IndexMap& m, const float* A, const float* x, float* y, int batch,
                                int64_t a_stride, int64_t x_stride, int64_t y_stride, int accumulate,
                                cudaStream_t st) {
    const int64_t rows = m.dims[0];
    if (rows == 0 || batch == 0) return DASTAC_OK;
    const int64_t len = longest_row(m);
    const int L = len <= 4 ? 1 : len <= 256 ? 8 : 32;
    const int64_t blocks = (rows * L + 255) / 256;
    if (blocks > 0x7fffffffLL) return DASTAC_ERR_OVERFLOW;
    dastac_status last = DASTAC_OK;
    for (int b0 = 0; b0 < batch; b0 += 65535) {  // gridDim.y limit
        const int nb = batch - b0 < 65535 ? batch - b0 : 65535;
        const dim3 grid((unsigned)blocks, (unsigned)nb);
        const float* Ab = A + b0 * a_stride;
        const float* xb = x + b0 * x_stride;
        float* yb = y + b0 * y_stride;
        if (L == 1)
            rowspan_mv_kernel<1><<<grid, 256, 0, st>>>(m, Ab, xb, yb, rows, a_stride, x_stride, y_stride, accumulate);
        else if (L == 8)
            rowspan_mv_kernel<8><<<grid, 256, 0, st>>>(m, Ab, xb, yb, rows, a_stride, x_stride, y_stride, accumulate);
        else
            rowspan_mv_kernel<32><<<grid, 256, 0, st>>>(m, Ab, xb, yb, rows, a_stride, x_stride, y_stride, accumulate);
        last = launch_status();
        if (last != DASTAC_OK) return last;
    }
    return last;
}

dastac_status launch_rowspan_mm(const IndexMap& m, const float* A, const float* B, int64_t ldb, float* C,
                                int64_t ldc, int64_t ncols, int accumulate, cudaStream_t st) {
    const int64_t rows = m.dims[0];
    if (rows == 0 || ncols == 0) return DASTAC_OK;
    const int64_t items = rows * ((ncols + 31) / 32);
    int64_t blocks = (items + 7) / 8;
    const int64_t cap = (int64_t)sm_count() * 8;
    if (blocks > cap) blocks = cap;
    rowspan_mm_kernel<<<(unsigned)blocks, 256, 0, st>>>(m, A, B, ldb, C, ldc, ncols, rows, accumulate);
    return launch_status();
}

}  // namespace dastac
