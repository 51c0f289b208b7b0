// M(i,r) = sum_{j,k} T(i,j,k) B(j,r) C(k,r) over the tetrahedron i <= j <= k (the paper's MTTKRP
// rule A(i,j) := B(i,k,l) * C(k,j) * D(l,j), Table 1, with the hyper-triangular domain), fp32.
//
// Factored evaluation: for a fixed fibre (i, j) the packed values T(i,j,j..n-1) are contiguous;
// u(r) = sum_k T(i,j,k) C(k,r) is formed first and M(i,r) += B(j,r) u(r) once per fibre, which
// needs one multiply-add per stored element and rank column instead of two multiplies and an add.
// The fibre start is the ranking polynomial evaluated once, then advanced by the fibre length.
#include "common.cuh"

namespace dastac {
namespace {

constexpr int kWarps = 8;

// Block = one slab i; warp = fibres j = i + warp, i + warp + kWarps, ...; lane = rank column r.
__global__ void __launch_bounds__(kWarps * 32)
mttkrp_kernel(IndexMap m, const float* __restrict__ T, const float* __restrict__ B, int64_t ldb,
              const float* __restrict__ C, int64_t ldc, float* __restrict__ M, int64_t ldm,
              int64_t R) {
    const int64_t n = m.N;
    const int64_t i = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int64_t r0 = 0; r0 < R; r0 += 32) {
        const int64_t r = r0 + lane;
        float acc = 0.f;
        for (int64_t j = i + warp; j < n; j += kWarps) {
            int32_t idx[3] = {(int32_t)i, (int32_t)j, (int32_t)j};
            const float* fibre = T + rank_of(m, idx) - j;  // fibre[k] = T(i, j, k)
            float u = 0.f;
            if (r < R)
                for (int64_t k = j; k < n; ++k) u = fmaf(fibre[k], C[k * ldc + r], u);
            if (r < R) acc = fmaf(B[j * ldb + r], u, acc);
        }
        if (r < R) atomicAdd(&M[i * ldm + r], acc);
    }
}

__global__ void zero_rows_kernel(float* __restrict__ M, int64_t ldm, int64_t rows, int64_t R) {
    for (int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; t < rows * R;
         t += (int64_t)gridDim.x * blockDim.x)
        M[(t / R) * ldm + (t % R)] = 0.f;
}

}  // namespace

dastac_status launch_mttkrp(const IndexMap& m, const float* T, const float* B, int64_t ldb,
                            const float* C, int64_t ldc, float* M, int64_t ldm, int64_t R,
                            int accumulate, cudaStream_t st) {
    const int64_t n = m.N;
    if (n == 0 || R == 0) return DASTAC_OK;
    if (!accumulate) {
        int64_t blocks = (n * R + 255) / 256;
        if (blocks > 4096) blocks = 4096;
        zero_rows_kernel<<<(unsigned)blocks, 256, 0, st>>>(M, ldm, n, R);
        dastac_status s = launch_status();
        if (s != DASTAC_OK) return s;
    }
    mttkrp_kernel<<<(unsigned)n, kWarps * 32, 0, st>>>(m, T, B, ldb, C, ldc, M, ldm, R);
    return launch_status();
}

}  // namespace dastac
