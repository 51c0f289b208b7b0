// y = A x for a packed upper-triangular A (the paper's SpMV_UT rule A(i) := B(i,j) * C(j), Table 1),
// fp32, optionally batched over independent instances that share one structure.
//
// Work balance over the uneven rows: row i has N - i stored elements, so rows i and N-1-i together
// always hold N + 1.  One warp owns one such pair; every warp therefore streams the same number
// of packed elements.  Inside a row the position is rowbase(i) + j with rowbase hoisted, the
// loop-invariant part of the ranking polynomial (Section 4, last paragraph; Section 5.3, "Loop
// Invariant Code Motion").
//
// Two kernels.  For N <= kQuadMaxN the packed rows are read with aligned 128-bit loads: rowbase(i)
// mod 4 = r shifts the columns an aligned quad holds (quad q of the row = columns 4q-r .. 4q-r+3),
// so the block keeps four copies of x in shared memory, copy r shifted by r elements, and a quad of
// A meets its four x values in one aligned 128-bit shared load.  Only the first and last quad of a
// row need masking.  Rows this short cannot amortise a whole warp's per-row work, so eight lanes
// share a pair and a warp runs four neighbouring pairs at once.  Larger N uses one warp per pair,
// 32-bit loads and x read through the cache.
#include "common.cuh"

namespace dastac {
namespace {

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Dot product of packed row i (columns i..N-1) with x, distributed over the lanes of a warp.
__device__ __forceinline__ float row_dot(const float* __restrict__ A, const float* __restrict__ x,
                                         int64_t N, int64_t i, int lane) {
    const float* row = A + upper_row_base(N, i);  // row[j] = A(i, j)
    float acc0 = 0.f, acc1 = 0.f, acc2 = 0.f, acc3 = 0.f;
    int64_t j = i + lane;
    for (; j + 96 < N; j += 128) {
        acc0 = fmaf(row[j], x[j], acc0);
        acc1 = fmaf(row[j + 32], x[j + 32], acc1);
        acc2 = fmaf(row[j + 64], x[j + 64], acc2);
        acc3 = fmaf(row[j + 96], x[j + 96], acc3);
    }
    for (; j < N; j += 32) acc0 = fmaf(row[j], x[j], acc0);
    return warp_sum((acc0 + acc1) + (acc2 + acc3));
}

constexpr int kQuadMaxN = 2048;  // 4 shifted copies of x: 4 * (N + 8) floats of shared memory

struct QuadRow {
    const float4* row;  // row[q] = columns 4q - r .. 4q - r + 3
    const float4* xr;   // copy r of x
    int i, r, q_lo, q_hi;
};

__device__ __forceinline__ QuadRow quad_row(const float4* __restrict__ A4, const float4* __restrict__ xs4,
                                            const int copy_quads, const int N, const int i) {
    const int64_t base = upper_row_base(N, i);
    QuadRow R;
    R.i = i;
    R.r = (int)(base & 3);
    R.row = A4 + (base >> 2);
    R.xr = xs4 + R.r * copy_quads;
    R.q_lo = (i + R.r) >> 2;
    R.q_hi = (N - 1 + R.r) >> 2;
    return R;
}

constexpr int kQuadUnroll = 4;  // quads in flight per lane

// Partial dot product of one packed row with x over the quads q_lo + sub, + kGroup, ...
// kGroup = lanes that share one row pair.
template <int kGroup>
__device__ __forceinline__ float row_dot_quads(const QuadRow& R, const int N, const int sub) {
    float acc0 = 0.f, acc1 = 0.f;
    for (int q0 = R.q_lo + sub; q0 <= R.q_hi; q0 += kGroup * kQuadUnroll) {
        float4 a[kQuadUnroll];
#pragma unroll
        for (int k = 0; k < kQuadUnroll; ++k) {
            const int q = q0 + kGroup * k;
            a[k] = q <= R.q_hi ? __ldg(R.row + q) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int k = 0; k < kQuadUnroll; ++k) {
            const int q = q0 + kGroup * k;
            if (q > R.q_hi) break;
            float4 xv = R.xr[q];
            if (q == R.q_lo || q == R.q_hi) {
                // first and last quad of a row: columns outside [i, N) belong to the neighbouring rows
                // (or to the padding behind the last row): select them away, do not multiply by zero
                const int j = 4 * q - R.r;
                const bool k0 = j >= R.i && j < N, k1 = j + 1 >= R.i && j + 1 < N, k2 = j + 2 >= R.i && j + 2 < N,
                           k3 = j + 3 >= R.i && j + 3 < N;
                a[k].x = k0 ? a[k].x : 0.f;
                a[k].y = k1 ? a[k].y : 0.f;
                a[k].z = k2 ? a[k].z : 0.f;
                a[k].w = k3 ? a[k].w : 0.f;
            }
            acc0 = fmaf(a[k].x, xv.x, acc0);
            acc1 = fmaf(a[k].y, xv.y, acc1);
            acc0 = fmaf(a[k].z, xv.z, acc0);
            acc1 = fmaf(a[k].w, xv.w, acc1);
        }
    }
    return acc0 + acc1;
}

template <int kGroup>
__device__ __forceinline__ float group_sum(float v) {
#pragma unroll
    for (int o = kGroup / 2; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

template <int kGroup>
__global__ void __launch_bounds__(256)
trmv_quad_kernel(const int N, const float* __restrict__ A, const float* __restrict__ x, float* __restrict__ y,
                 int64_t a_stride, int64_t x_stride, int64_t y_stride, int accumulate) {
    extern __shared__ float4 xs_raw[];  // four copies of N4 floats: copy r holds x[c - r] at c
    const int N4 = (N + 8) & ~3;
    float* xs = reinterpret_cast<float*>(xs_raw);
    A += blockIdx.y * a_stride;
    x += blockIdx.y * x_stride;
    y += blockIdx.y * y_stride;
    for (int c = threadIdx.x; c < N4; c += blockDim.x) {
#pragma unroll
        for (int r = 0; r < 4; ++r) xs[r * N4 + c] = (c - r >= 0 && c - r < N) ? __ldg(x + c - r) : 0.f;
    }
    __syncthreads();
    const float4* A4 = reinterpret_cast<const float4*>(A);
    const int sub = threadIdx.x & (kGroup - 1), group = threadIdx.x / kGroup, groups = blockDim.x / kGroup;
    const int pairs = (N + 1) >> 1;
    // a warp's groups take neighbouring pairs, whose rows differ by one element: no divergence to speak of
    for (int pair0 = blockIdx.x * groups; pair0 < pairs; pair0 += gridDim.x * groups) {
        const int pair = pair0 + group;
        const bool live = pair < pairs;
        const int i0 = live ? pair : 0, i1 = live ? N - 1 - pair : 0;
        float s0 = 0.f, s1 = 0.f;
        if (live) {
            s0 = row_dot_quads<kGroup>(quad_row(A4, xs_raw, N4 / 4, N, i0), N, sub);
            if (i1 != i0) s1 = row_dot_quads<kGroup>(quad_row(A4, xs_raw, N4 / 4, N, i1), N, sub);
        }
        s0 = group_sum<kGroup>(s0);
        s1 = group_sum<kGroup>(s1);
        if (live && sub == 0) {
            y[i0] = accumulate ? y[i0] + s0 : s0;
            if (i1 != i0) y[i1] = accumulate ? y[i1] + s1 : s1;
        }
    }
}

__global__ void __launch_bounds__(256)
trmv_pair_kernel(int64_t N, const float* __restrict__ A, const float* __restrict__ x,
                 float* __restrict__ y, int64_t a_stride, int64_t x_stride, int64_t y_stride,
                 int accumulate) {
    const int lane = threadIdx.x & 31;
    const int64_t pair = blockIdx.x * (int64_t)(blockDim.x >> 5) + (threadIdx.x >> 5);
    const int64_t pairs = (N + 1) >> 1;
    if (pair >= pairs) return;
    A += blockIdx.y * a_stride;
    x += blockIdx.y * x_stride;
    y += blockIdx.y * y_stride;
    const int64_t i0 = pair, i1 = N - 1 - pair;
    float s0 = row_dot(A, x, N, i0, lane);
    if (lane == 0) y[i0] = accumulate ? y[i0] + s0 : s0;
    if (i1 != i0) {
        float s1 = row_dot(A, x, N, i1, lane);
        if (lane == 0) y[i1] = accumulate ? y[i1] + s1 : s1;
    }
}

}  // namespace

dastac_status launch_trmv(const IndexMap& m, const float* A, const float* x, float* y, int batch,
                          int64_t a_stride, int64_t x_stride, int64_t y_stride, int accumulate,
                          cudaStream_t st) {
    const int64_t N = m.N;
    if (N == 0 || batch == 0) return DASTAC_OK;
    const int64_t pairs = (N + 1) >> 1;
    const int warps = 8;
    dastac_status last = DASTAC_OK;
    if (N <= kQuadMaxN && (a_stride & 3) == 0) {
        // Few pairs in all (a single small instance): a whole warp per pair keeps the launch short.
        const bool wide = (int64_t)batch * pairs <= (int64_t)sm_count() * 64;
        // parts per instance: enough blocks to fill the GPU; one pass of a block = 32 (or 8) row pairs
        int64_t parts = wide ? (pairs + 7) / 8 : (pairs + 31) / 32;
        const int64_t want = ((int64_t)sm_count() * 16 + batch - 1) / batch;
        if (parts > want) parts = want;
        if (parts < 1) parts = 1;
        const size_t smem = (size_t)4 * ((N + 8) & ~3) * sizeof(float);
        for (int b0 = 0; b0 < batch; b0 += 65535) {
            int nb = batch - b0 < 65535 ? batch - b0 : 65535;
            if (wide)
                trmv_quad_kernel<32><<<dim3((unsigned)parts, (unsigned)nb), warps * 32, smem, st>>>(
                    (int)N, A + b0 * a_stride, x + b0 * x_stride, y + b0 * y_stride, a_stride, x_stride, y_stride,
                    accumulate);
            else
                trmv_quad_kernel<8><<<dim3((unsigned)parts, (unsigned)nb), warps * 32, smem, st>>>(
                    (int)N, A + b0 * a_stride, x + b0 * x_stride, y + b0 * y_stride, a_stride, x_stride, y_stride,
                    accumulate);
            last = launch_status();
            if (last != DASTAC_OK) return last;
        }
        return last;
    }
    // Large matrices, few instances, 16-byte aligned instances: the streaming kernel of the symmetric
    // product without its mirrored half (aligned 128-bit loads; x windows in registers).
    // (measured: 6.65 against 6.36 TB/s at N = 65536; below that the kernel after this one is as fast or faster)
    if (batch <= 4 && N >= 65536 && N < (int64_t(1) << 30) && (a_stride & 3) == 0 && aligned16(A)) {
        for (int b0 = 0; b0 < batch; ++b0) {
            last = launch_symv(m, A + b0 * a_stride, x + b0 * x_stride, y + b0 * y_stride, accumulate, nullptr, st, 0);
            if (last != DASTAC_OK) return last;
        }
        return last;
    }
    for (int b0 = 0; b0 < batch; b0 += 65535) {  // gridDim.y limit
        int nb = batch - b0 < 65535 ? batch - b0 : 65535;
        dim3 grid((unsigned)((pairs + warps - 1) / warps), (unsigned)nb);
        trmv_pair_kernel<<<grid, warps * 32, 0, st>>>(N, A + b0 * a_stride, x + b0 * x_stride,
                                                      y + b0 * y_stride, a_stride, x_stride,
                                                      y_stride, accumulate);
        last = launch_status();
        if (last != DASTAC_OK) return last;
    }
    return last;
}

}  // namespace dastac
