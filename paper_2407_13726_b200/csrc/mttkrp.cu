// M(i,r) = sum_{j,k} T(i,j,k) B(j,r) C(k,r) over the tetrahedron i <= j <= k (the paper's MTTKRP
// rule A(i,j) := B(i,k,l) * C(k,j) * D(l,j), Table 1, with the hyper-triangular domain), fp32.
//
// Factored evaluation: for a fixed slab i, U(j,r) = sum_{k>=j} T(i,j,k) C(k,r) is a triangular
// matrix times the tall matrix C, and M(i,r) = sum_j B(j,r) U(j,r): one multiply-add per stored
// element and rank column instead of two multiplies and an add.
//
// Work unit = (slab i, 32 consecutive fibres j0..j0+31), owned by one warp; its K range is
// [j0, n).  The warp walks K in chunks of 32: the 32x32 chunk of T (rows are contiguous packed
// fibres, position rowbase(i,j) + k with rowbase advanced by n-j-1 per fibre, never re-ranked) is
// loaded coalesced, transposed through registers into shared memory, and multiplied with the
// matching 32 rows of C by a 4(j) x 8(r) register tile per lane.  Shared memory is private to the
// warp, so only warp-level synchronisation is used.
//
// Balance over the uneven fibre lengths: a unit's cost depends on j0 only (n - j0 columns), and
// the number of units sharing a j0 is floor(j0/32)+1, so the list of units sorted by decreasing
// cost has a closed-form position -> (i, j0) map (a triangular root).  Persistent warps take
// units from that list in boustrophedon order, which deals every warp the same mix of long and
// short units without any counter in memory.
#include "common.cuh"

namespace dastac {
namespace {

constexpr int kWarps = 8;
constexpr int kTile = 32;        // fibres per unit and K elements per chunk
constexpr int kTsPitch = 36;     // floats; 16-byte aligned rows, conflict-free 128-bit stores
constexpr int kRTile = 32;       // rank columns per pass

// Two fp32 multiply-adds per instruction (packed pair in a 64-bit register): d = a * b + d.
__device__ __forceinline__ unsigned long long pack2(float lo, float hi) {
    unsigned long long r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(unsigned long long v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ void fma2(unsigned long long& d, unsigned long long a, unsigned long long b) {
    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(d) : "l"(a), "l"(b));
}

struct WarpSmem {
    float Ts[kTile][kTsPitch];   // Ts[k][j] chunk of T, transposed
    float Cs[kTile][kRTile];     // Cs[k][r] chunk of C
};

__global__ void __launch_bounds__(kWarps * 32, 2)
mttkrp_kernel(IndexMap m, const float* __restrict__ T, const float* __restrict__ B, int64_t ldb,
              const float* __restrict__ C, int64_t ldc, float* __restrict__ M, int64_t ldm,
              int64_t R, int64_t units) {
    extern __shared__ __align__(16) uint8_t smem_raw[];
    WarpSmem* smem = reinterpret_cast<WarpSmem*>(smem_raw);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    WarpSmem& sm = smem[warp];
    const int64_t n = m.N;
    const int jg = lane >> 2, rg = lane & 3;  // lane's 4 fibres and 8 rank columns inside the tile
    const int64_t W = (int64_t)gridDim.x * kWarps;
    const int64_t w = (int64_t)blockIdx.x * kWarps + warp;
    const int64_t g_full = n / kTile;

    for (int64_t round = 0;; ++round) {
        const int64_t p = round * W + ((round & 1) ? (W - 1 - w) : w);
        if (round * W >= units) break;
        if (p >= units) continue;
        // position in the cost-sorted list -> (j0, i): block g = j0/32 holds 32 (g+1) units
        int64_t g = tri_root(p / kTile);
        if (g > g_full) g = g_full;
        const int64_t pp = p - kTile * tri(g);
        const int64_t j0 = kTile * g + pp / (g + 1);
        const int64_t i = j0 - kTile * (pp % (g + 1));

        // rowbase(i, j0): position of T(i, j0, k) is rowbase + k
        int32_t idx[3] = {(int32_t)i, (int32_t)j0, (int32_t)j0};
        const int64_t rowbase0 = rank_of(m, idx) - j0;

        for (int64_t r0 = 0; r0 < R; r0 += kRTile) {
            unsigned long long acc2[4][4];  // [fibre][pair of rank columns]
#pragma unroll
            for (int q = 0; q < 4; ++q)
#pragma unroll
                for (int e = 0; e < 4; ++e) acc2[q][e] = 0ull;

            float v[kTile];  // lane's column of the next chunk: T(i, j0+jj, kc+lane)
            const float* Tu = T + rowbase0;  // Tu[roff(jj) + k] = T(i, j0+jj, k), roff advanced by n-j-1
            const uint32_t n32 = (uint32_t)n, j032 = (uint32_t)j0;
            auto load_chunk = [&](int64_t kc) {
                const uint32_t k = (uint32_t)kc + lane;
                uint32_t roff = 0;
                if (kc > j0 && kc + kTile <= n && j0 + kTile <= n) {
                    // interior chunk: every element is inside the tetrahedron
#pragma unroll
                    for (int jj = 0; jj < kTile; ++jj) {
                        v[jj] = __ldg(Tu + (roff + k));
                        roff += n32 - (j032 + jj) - 1;
                    }
                } else {
#pragma unroll
                    for (int jj = 0; jj < kTile; ++jj) {
                        const uint32_t j = j032 + jj;
                        v[jj] = (j < n32 && k >= j && k < n32) ? __ldg(Tu + (roff + k)) : 0.f;
                        roff += n32 - j - 1;
                    }
                }
            };
            const bool c_fast = (r0 + kRTile <= R) && ((ldc & 3) == 0);
            load_chunk(j0);
            for (int64_t kc = j0; kc < n; kc += kTile) {
                __syncwarp();
#pragma unroll
                for (int q = 0; q < kTile / 4; ++q)
                    *reinterpret_cast<float4*>(&sm.Ts[lane][4 * q]) =
                        make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
                // rows kc..kc+31 of C, columns r0..r0+31: lane = (row within 4, 16-byte chunk)
                if (c_fast && kc + kTile <= n) {
                    const float4* src = reinterpret_cast<const float4*>(C + (kc + (lane >> 3)) * ldc + r0) + (lane & 7);
#pragma unroll
                    for (int q = 0; q < kTile / 4; ++q)
                        *reinterpret_cast<float4*>(&sm.Cs[4 * q + (lane >> 3)][4 * (lane & 7)]) = __ldg(src + q * ldc);
                } else {
#pragma unroll
                    for (int q = 0; q < kTile / 4; ++q) {
                        const int kk = 4 * q + (lane >> 3);
                        const int64_t k = kc + kk, r = r0 + 4 * (lane & 7);
                        float4 c4 = make_float4(0.f, 0.f, 0.f, 0.f);
                        if (k < n) {
                            const float* src = C + k * ldc + r;
                            if (r + 4 <= R && (ldc & 3) == 0) {
                                c4 = __ldg(reinterpret_cast<const float4*>(src));
                            } else {
                                if (r < R) c4.x = __ldg(src);
                                if (r + 1 < R) c4.y = __ldg(src + 1);
                                if (r + 2 < R) c4.z = __ldg(src + 2);
                                if (r + 3 < R) c4.w = __ldg(src + 3);
                            }
                        }
                        *reinterpret_cast<float4*>(&sm.Cs[kk][4 * (lane & 7)]) = c4;
                    }
                }
                __syncwarp();
                if (kc + kTile < n) load_chunk(kc + kTile);  // prefetch into registers
#pragma unroll 8
                for (int kk = 0; kk < kTile; ++kk) {
                    const float4 t4 = *reinterpret_cast<const float4*>(&sm.Ts[kk][4 * jg]);
                    const ulonglong2 ca = *reinterpret_cast<const ulonglong2*>(&sm.Cs[kk][8 * rg]);
                    const ulonglong2 cb = *reinterpret_cast<const ulonglong2*>(&sm.Cs[kk][8 * rg + 4]);
                    const unsigned long long t2[4] = {pack2(t4.x, t4.x), pack2(t4.y, t4.y), pack2(t4.z, t4.z),
                                                      pack2(t4.w, t4.w)};
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        fma2(acc2[q][0], t2[q], ca.x);
                        fma2(acc2[q][1], t2[q], ca.y);
                        fma2(acc2[q][2], t2[q], cb.x);
                        fma2(acc2[q][3], t2[q], cb.y);
                    }
                }
            }
            float acc[4][8];
#pragma unroll
            for (int q = 0; q < 4; ++q)
#pragma unroll
                for (int e = 0; e < 4; ++e) unpack2(acc2[q][e], acc[q][2 * e], acc[q][2 * e + 1]);
            // M(i, r) += sum_j B(j, r) U(j, r): the lane's 4 fibres, then the 8 fibre groups
            float s[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) s[e] = 0.f;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int64_t j = j0 + 4 * jg + q;
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const int64_t r = r0 + 8 * rg + e;
                    const float b = (j < n && r < R) ? __ldg(B + j * ldb + r) : 0.f;
                    s[e] = fmaf(b, acc[q][e], s[e]);
                }
            }
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                s[e] += __shfl_xor_sync(0xffffffffu, s[e], 4);
                s[e] += __shfl_xor_sync(0xffffffffu, s[e], 8);
                s[e] += __shfl_xor_sync(0xffffffffu, s[e], 16);
            }
            if (jg == 0) {
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const int64_t r = r0 + 8 * rg + e;
                    if (r < R) atomicAdd(&M[i * ldm + r], s[e]);
                }
            }
        }
    }
}

__global__ void zero_rows_kernel(float* __restrict__ M, int64_t ldm, int64_t rows, int64_t R) {
    for (int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; t < rows * R;
         t += (int64_t)gridDim.x * blockDim.x)
        M[(t / R) * ldm + (t % R)] = 0.f;
}

// The same rule over any rank-3 structure whose fibres (i, j, :) are stored contiguously (dense box,
// upper half cube, planes with a free trailing index: the other MTTKRP structures of Table 1 are of
// this kind).  A warp owns a fibre: the stored interval of k comes from the hoisted row base, lane r
// accumulates U(r) = sum_k T(i,j,k) C(k,r) with T read coalesced and broadcast by shuffles, and
// B(j,r) U(r) is added to M(i,r) atomically.  One multiply-add per lane and element: bound by the
// loads of C from cache, far from the tetrahedral kernel's rate; it exists for coverage.
__global__ void __launch_bounds__(256)
mttkrp_fibre_kernel(IndexMap m, const float* __restrict__ T, const float* __restrict__ B, int64_t ldb,
                    const float* __restrict__ C, int64_t ldc, float* __restrict__ M, int64_t ldm, int64_t R) {
    const int lane = threadIdx.x & 31;
    const int64_t fibres = m.dims[0] * m.dims[1];
    const int64_t warps = (int64_t)gridDim.x * (blockDim.x >> 5);
    for (int64_t f = blockIdx.x * (int64_t)(blockDim.x >> 5) + (threadIdx.x >> 5); f < fibres; f += warps) {
        const int64_t i = f / m.dims[1], j = f - i * m.dims[1];
        int32_t idx[3] = {(int32_t)i, (int32_t)j, 0};
        int64_t klo = 0, khi = 0, pbase = 0;
        if (!row_span(m, idx, klo, khi, pbase)) continue;
        const float* row = T + pbase;  // row[k] = T(i, j, k)
        for (int64_t r0 = 0; r0 < R; r0 += 32) {
            const int64_t r = r0 + lane;
            float acc = 0.f;
            for (int64_t k0 = klo; k0 < khi; k0 += 32) {
                const float t = (k0 + lane < khi) ? __ldg(row + k0 + lane) : 0.f;
                const int nk = (int)(khi - k0 < 32 ? khi - k0 : 32);
                for (int kk = 0; kk < nk; ++kk) {
                    const float tk = __shfl_sync(0xffffffffu, t, kk);
                    if (r < R) acc = fmaf(tk, __ldg(C + (k0 + kk) * ldc + r), acc);
                }
            }
            if (r < R) atomicAdd(&M[i * ldm + r], __ldg(B + j * ldb + r) * acc);
        }
    }
}

}  // namespace

bool mttkrp_supports(const IndexMap& m) {
    if (m.rank != 3) return false;
    return m.kind == kTetrahedron || m.kind == kDense || m.kind == kUpper || (m.kind == kPlane && m.w != 2);
}

dastac_status launch_mttkrp(const IndexMap& m, const float* T, const float* B, int64_t ldb,
                            const float* C, int64_t ldc, float* M, int64_t ldm, int64_t R,
                            int accumulate, int32_t* err_word, cudaStream_t st) {
    (void)err_word;  // no kernel of this rule has a bounded wait
    const int64_t n = m.dims[0];  // rows of the result
    if (n == 0 || R == 0) return DASTAC_OK;
    if (!accumulate) {
        int64_t blocks = (n * R + 255) / 256;
        if (blocks > 4096) blocks = 4096;
        zero_rows_kernel<<<(unsigned)blocks, 256, 0, st>>>(M, ldm, n, R);
        dastac_status s = launch_status();
        if (s != DASTAC_OK) return s;
    }
    if (m.kind != kTetrahedron) {
        const int64_t fibres = m.dims[0] * m.dims[1];
        if (fibres == 0 || m.dims[2] == 0) return DASTAC_OK;
        int64_t blocks = (fibres + 7) / 8;
        const int64_t capf = (int64_t)sm_count() * 8;
        if (blocks > capf) blocks = capf;
        mttkrp_fibre_kernel<<<(unsigned)blocks, 256, 0, st>>>(m, T, B, ldb, C, ldc, M, ldm, R);
        return launch_status();
    }
    // units = sum over j0 of (floor(j0/32) + 1)
    const int64_t g_full = n / kTile;
    const int64_t units = kTile * tri(g_full) + (n - kTile * g_full) * (g_full + 1);
    int64_t blocks = (units + kWarps - 1) / kWarps;
    const int64_t cap = (int64_t)sm_count() * 2;
    if (blocks > cap) blocks = cap;
    constexpr size_t kSmem = sizeof(WarpSmem) * kWarps;
    static bool attr_set[64];
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        if (cudaFuncSetAttribute(mttkrp_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmem) !=
            cudaSuccess)
            return DASTAC_ERR_CUDA;
        attr_set[dev] = true;
    }
    mttkrp_kernel<<<(unsigned)blocks, kWarps * 32, kSmem, st>>>(m, T, B, ldb, C, ldc, M, ldm, R, units);
    return launch_status();
}

}  // namespace dastac
