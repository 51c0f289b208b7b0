// C = A B for a banded A (|i - j| <= w) stored as 2w+1 padded diagonals of N slots, B and C dense
// row-major, fp32.  Slot (d, i) holds A(i, i + d - w): for a fixed diagonal consecutive rows are
// consecutive in memory and the position is the affine map d*N + i.  Padding slots are never read
// into a result: a slot whose column i + d - w falls outside [0, N) is replaced by zero while the
// band is staged, whatever it contains.
//
// A CTA computes 64 rows x 256 columns.  Its slice of the band (all diagonals of its 64 rows) is
// staged in shared memory in the packed layout itself, Ad[d][row], with coalesced loads along
// each diagonal.  A lane owns 8 rows x 8 columns and walks the diagonals: for diagonal d its
// eight rows need B rows i+d-w .. i+7+d-w, a window that slides down by one row per diagonal, so
// each step loads the eight A values (two broadcast 128-bit shared loads), one new B row segment
// (two 128-bit loads served by L1) and issues 64 multiply-adds.  The window is kept in registers,
// 16 slots deep so that a row is requested eight steps before its first use, and rotates with
// period 16; the loop is unrolled by 16 so every register index is static.  Only the band is
// visited: the executed work is the diagonal count rounded up to a multiple of 16.
#include "common.cuh"

namespace dastac {
namespace {

constexpr int kRows = 64, kCols = 256, kThreads = 256;
constexpr int kMaxChunkDiagonals = 128;  // diagonals staged at a time (32 KiB of shared memory)

__device__ __forceinline__ void load_row8(float (&dst)[8], const float* __restrict__ B, int64_t ldb,
                                          int64_t jj, int64_t N, int64_t c0, int64_t ncols, bool vec) {
    if (jj < 0 || jj >= N) {
#pragma unroll
        for (int e = 0; e < 8; ++e) dst[e] = 0.f;
        return;
    }
    const float* src = B + jj * ldb + c0;
    if (vec && c0 + 8 <= ncols) {
        const float4 lo = __ldg(reinterpret_cast<const float4*>(src));
        const float4 hi = __ldg(reinterpret_cast<const float4*>(src) + 1);
        dst[0] = lo.x; dst[1] = lo.y; dst[2] = lo.z; dst[3] = lo.w;
        dst[4] = hi.x; dst[5] = hi.y; dst[6] = hi.z; dst[7] = hi.w;
    } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) dst[e] = (c0 + e < ncols) ? __ldg(src + e) : 0.f;
    }
}

__global__ void __launch_bounds__(kThreads)
bandmm_kernel(int64_t N, int64_t w, int64_t row_tile0, const float* __restrict__ A,
              const float* __restrict__ B, int64_t ldb, float* __restrict__ C, int64_t ldc,
              int64_t ncols, int accumulate, int chunk_diagonals, int vec_b, int vec_c) {
    extern __shared__ __align__(16) float Ad[];  // [chunk_diagonals][kRows]
    const int64_t i0 = (row_tile0 + blockIdx.y) * (int64_t)kRows;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // warp = (16-row pair, 128-column half); lane = (8-row group, 8-column group)
    const int il = 16 * (warp >> 1) + 8 * (lane >> 4);
    const int64_t c0 = blockIdx.x * (int64_t)kCols + 128 * (warp & 1) + 8 * (lane & 15);
    const int64_t i_f = i0 + il;
    const int64_t diagonals = 2 * w + 1;
    const bool vb = vec_b != 0;

    float acc[8][8];
#pragma unroll
    for (int q = 0; q < 8; ++q)
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[q][e] = 0.f;

    for (int64_t dc = 0; dc < diagonals; dc += chunk_diagonals) {
        __syncthreads();
        // stage diagonals dc .. dc+chunk-1 of rows i0 .. i0+63; zero outside the band / matrix
        for (int t = tid; t < chunk_diagonals * kRows; t += kThreads) {
            const int dl = t / kRows, r = t - dl * kRows;
            const int64_t d = dc + dl, i = i0 + r, jj = i + d - w;
            Ad[t] = (d < diagonals && i < N && jj >= 0 && jj < N) ? __ldg(A + d * N + i) : 0.f;
        }
        __syncthreads();
        if (c0 >= ncols || i_f >= N) continue;  // lane has no output; it still helped staging

        // Window of B rows in registers: 16 slots, row (i_f + d - w + q) sits in slot (d - dc + q) mod 16.
        // Step d uses rows q = 0..7 and loads the row that step d + 8 will need last (q = 15 from here),
        // so every load has eight steps of multiply-adds to complete behind it.
        float win[16][8];
        {
            const int64_t J = i_f + dc - w;
#pragma unroll
            for (int q = 0; q < 15; ++q) load_row8(win[q], B, ldb, J + q, N, c0, ncols, vb);
        }
        const int64_t d_end = (diagonals - dc < chunk_diagonals) ? diagonals - dc : chunk_diagonals;
        for (int64_t db = 0; db < d_end; db += 16) {
#pragma unroll
            for (int u = 0; u < 16; ++u) {
                const int64_t d = dc + db + u;
                load_row8(win[(u + 15) & 15], B, ldb, i_f + d - w + 15, N, c0, ncols, vb);
                const float4 a_lo = *reinterpret_cast<const float4*>(&Ad[(db + u) * kRows + il]);
                const float4 a_hi = *reinterpret_cast<const float4*>(&Ad[(db + u) * kRows + il + 4]);
                const float a[8] = {a_lo.x, a_lo.y, a_lo.z, a_lo.w, a_hi.x, a_hi.y, a_hi.z, a_hi.w};
#pragma unroll
                for (int q = 0; q < 8; ++q)
#pragma unroll
                    for (int e = 0; e < 8; ++e) acc[q][e] = fmaf(a[q], win[(u + q) & 15][e], acc[q][e]);
            }
        }
    }
    if (c0 >= ncols || i_f >= N) return;
#pragma unroll
    for (int q = 0; q < 8; ++q) {
        const int64_t i = i_f + q;
        if (i >= N) break;
        float* dst = C + i * ldc + c0;
        if (vec_c && c0 + 8 <= ncols) {
            float4 lo = make_float4(acc[q][0], acc[q][1], acc[q][2], acc[q][3]);
            float4 hi = make_float4(acc[q][4], acc[q][5], acc[q][6], acc[q][7]);
            if (accumulate) {
                const float4 o0 = *reinterpret_cast<const float4*>(dst);
                const float4 o1 = *(reinterpret_cast<const float4*>(dst) + 1);
                lo.x += o0.x; lo.y += o0.y; lo.z += o0.z; lo.w += o0.w;
                hi.x += o1.x; hi.y += o1.y; hi.z += o1.z; hi.w += o1.w;
            }
            *reinterpret_cast<float4*>(dst) = lo;
            *(reinterpret_cast<float4*>(dst) + 1) = hi;
        } else {
#pragma unroll
            for (int e = 0; e < 8; ++e)
                if (c0 + e < ncols) dst[e] = accumulate ? dst[e] + acc[q][e] : acc[q][e];
        }
    }
}

}  // namespace

dastac_status launch_bandmm(const IndexMap& m, const float* A, const float* B, int64_t ldb, float* C,
                            int64_t ldc, int64_t ncols, int accumulate, cudaStream_t st) {
    const int64_t N = m.N;
    if (N == 0 || ncols == 0) return DASTAC_OK;
    const int64_t diagonals = 2 * m.w + 1;
    // The staged chunk holds a multiple of 16 diagonals (the lane loop is unrolled by 16).
    int64_t chunk = round_up(diagonals, 16);
    if (chunk > kMaxChunkDiagonals) chunk = kMaxChunkDiagonals;
    const size_t smem = (size_t)chunk * kRows * sizeof(float);
    const int64_t gx = (ncols + kCols - 1) / kCols, gy = (N + kRows - 1) / kRows;
    if (gx > 0x7fffffffLL) return DASTAC_ERR_OVERFLOW;
    const int vec_b = ((ldb & 3) == 0) && aligned16(B), vec_c = ((ldc & 3) == 0) && aligned16(C);
    for (int64_t y0 = 0; y0 < gy; y0 += 65535) {  // gridDim.y is limited to 65535
        const int64_t ny = gy - y0 < 65535 ? gy - y0 : 65535;
        bandmm_kernel<<<dim3((unsigned)gx, (unsigned)ny), kThreads, smem, st>>>(
            N, m.w, y0, A, B, ldb, C, ldc, ncols, accumulate, (int)chunk, vec_b, vec_c);
        dastac_status s = launch_status();
        if (s != DASTAC_OK) return s;
    }
    return DASTAC_OK;
}

}  // namespace dastac
