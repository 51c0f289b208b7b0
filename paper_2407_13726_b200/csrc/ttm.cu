// A(i,j,k) = sum_l B(i,j,l) C(k,l) with B nonzero only for i <= j (the paper's running example,
// Section 3: the tensor-times-matrix rule over the upper half cube), fp32, packed input AND packed
// output.  The ranking polynomial of the half cube, P(i,j,l) = rowbase(i,j) Q + l, keeps the
// trailing index contiguous, and the output has the same (i,j) set with trailing extent K, so in
// packed form the rule is one dense product with no index arithmetic left in it at all:
//     Y[p][k] = sum_l X[p][l] C[k][l],   p = 0 .. count/Q - 1,
// X the packed input viewed as a [p][Q] matrix, Y the packed output viewed as [p][K].  The zero
// region is never touched.
//
// CTA = 256 packed rows x 32 output columns, l in chunks of 32 through shared memory; a lane owns
// 8 rows x 4 columns (packed fp32x2 multiply-adds, the pair runs along k).
#include "common.cuh"

namespace dastac {
namespace {

constexpr int kThreads = 256;
constexpr int kRowsT = 256;   // packed rows per CTA
constexpr int kKT = 32;       // output columns per CTA
constexpr int kLc = 32;       // l per chunk
constexpr int kXPitch = 36;   // floats: 16-byte aligned rows; the rows of a quarter warp fall in distinct banks

typedef unsigned long long pair_t;
__device__ __forceinline__ pair_t pack2(float lo, float hi) {
    pair_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(pair_t v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ void fma2(pair_t& d, pair_t a, pair_t b) {
    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(d) : "l"(a), "l"(b));
}

__global__ void __launch_bounds__(kThreads, 2)
ttm_kernel(int64_t P, int64_t Q, int64_t K, const float* __restrict__ X, const float* __restrict__ C, int64_t ldc,
           float* __restrict__ Y, int accumulate, int vec_x, int vec_y) {
    __shared__ __align__(16) float Xs[kRowsT][kXPitch];  // Xs[r][l]
    __shared__ __align__(16) float Cs[kLc][kKT];         // Cs[l][k]: k contiguous, so a pair is (k, k+1)
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int rg = warp * 4 + (lane >> 3), kg = lane & 7;  // lane's rows 8 rg .. 8 rg + 7, columns 4 kg .. 4 kg + 3
    const int64_t p0 = (int64_t)blockIdx.x * kRowsT, k0 = (int64_t)blockIdx.y * kKT;

    pair_t acc2[8][2];
#pragma unroll
    for (int q = 0; q < 8; ++q) acc2[q][0] = acc2[q][1] = 0ull;

    for (int64_t l0 = 0; l0 < Q; l0 += kLc) {
        __syncthreads();  // the previous chunk's readers are done
        // X tile: 256 rows x 32 l, rows of the packed input are contiguous
        if (vec_x && l0 + kLc <= Q) {
#pragma unroll
            for (int e = 0; e < kRowsT * (kLc / 4) / kThreads; ++e) {
                const int item = tid + e * kThreads, r = item >> 3, c4 = item & 7;
                const int64_t p = p0 + r;
                const float4 v = p < P ? __ldg(reinterpret_cast<const float4*>(X + p * Q + l0) + c4)
                                       : make_float4(0.f, 0.f, 0.f, 0.f);
                *reinterpret_cast<float4*>(&Xs[r][4 * c4]) = v;
            }
        } else {
            for (int item = tid; item < kRowsT * kLc; item += kThreads) {
                const int r = item >> 5, l = item & 31;
                const int64_t p = p0 + r;
                Xs[r][l] = (p < P && l0 + l < Q) ? __ldg(X + p * Q + l0 + l) : 0.f;
            }
        }
        // C tile transposed: Cs[l][k] = C(k0 + k, l0 + l); lanes run along k so that the shared stores of a
        // warp fall in 32 different banks (the tile is 4 KiB: the strided global reads do not matter)
        for (int item = tid; item < kKT * kLc; item += kThreads) {
            const int k = item & 31, l = item >> 5;
            Cs[l][k] = (k0 + k < K && l0 + l < Q) ? __ldg(C + (k0 + k) * ldc + l0 + l) : 0.f;
        }
        __syncthreads();
#pragma unroll 2
        for (int l4 = 0; l4 < kLc / 4; ++l4) {
            float4 x[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) x[q] = *reinterpret_cast<const float4*>(&Xs[8 * rg + q][4 * l4]);
#pragma unroll
            for (int dl = 0; dl < 4; ++dl) {
                const ulonglong2 c = *reinterpret_cast<const ulonglong2*>(&Cs[4 * l4 + dl][4 * kg]);
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    const float xv = dl == 0 ? x[q].x : dl == 1 ? x[q].y : dl == 2 ? x[q].z : x[q].w;
                    const pair_t x2 = pack2(xv, xv);
                    fma2(acc2[q][0], x2, c.x);
                    fma2(acc2[q][1], x2, c.y);
                }
            }
        }
    }
#pragma unroll
    for (int q = 0; q < 8; ++q) {
        const int64_t p = p0 + 8 * rg + q, k = k0 + 4 * kg;
        if (p >= P || k >= K) continue;
        float o[4];
        unpack2(acc2[q][0], o[0], o[1]);
        unpack2(acc2[q][1], o[2], o[3]);
        float* dst = Y + p * K + k;
        if (vec_y && k + 4 <= K) {
            float4 v = make_float4(o[0], o[1], o[2], o[3]);
            if (accumulate) {
                const float4 old = *reinterpret_cast<const float4*>(dst);
                v.x += old.x; v.y += old.y; v.z += old.z; v.w += old.w;
            }
            *reinterpret_cast<float4*>(dst) = v;
        } else {
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if (k + e < K) dst[e] = accumulate ? dst[e] + o[e] : o[e];
        }
    }
}

// ---- persistent form ---------------------------------------------------------------------------------
// When the rows of X are 16-byte aligned and Q is a multiple of 32, a CTA walks a list of row tiles
// and asks for the next (tile, l-chunk) item with cp.async while it computes the current one, so the
// copies of a CTA overlap its own arithmetic instead of relying on the other CTAs of the SM being
// in a different phase.
struct TtmStage {
    float Xs[kRowsT][kXPitch];
    float Cs[kLc][kKT];
};

__device__ __forceinline__ void cp_async16(void* dst, const void* src, int src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"((uint32_t)__cvta_generic_to_shared(dst)), "l"(src),
                 "r"(src_bytes)
                 : "memory");
}

__global__ void __launch_bounds__(kThreads, 2)
ttm_stream_kernel(int64_t P, int64_t Q, int64_t K, int64_t row_tiles, const float* __restrict__ X,
                  const float* __restrict__ C, int64_t ldc, float* __restrict__ Y, int accumulate, int vec_y) {
    extern __shared__ __align__(16) uint8_t ttm_smem[];
    TtmStage* stage = reinterpret_cast<TtmStage*>(ttm_smem);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int rg = warp * 4 + (lane >> 3), kg = lane & 7;
    const int64_t k0 = (int64_t)blockIdx.y * kKT;
    const int64_t chunks = Q / kLc;
    const int64_t my_tiles = (row_tiles - blockIdx.x + gridDim.x - 1) / gridDim.x;
    const int64_t items = my_tiles * chunks;

    auto request = [&](int64_t n) {  // copies of item n into stage n & 1
        TtmStage& sg = stage[n & 1];
        const int64_t p0 = (blockIdx.x + (n / chunks) * gridDim.x) * kRowsT, l0 = (n % chunks) * kLc;
#pragma unroll
        for (int e = 0; e < kRowsT * (kLc / 4) / kThreads; ++e) {
            const int item = tid + e * kThreads, r = item >> 3, c4 = item & 7;
            const int64_t p = p0 + r;
            cp_async16(&sg.Xs[r][4 * c4], p < P ? X + p * Q + l0 + 4 * c4 : X, p < P ? 16 : 0);
        }
        if (chunks > 1 || n < 2)  // with a single chunk the C tile never changes: fill each stage once
            for (int item = tid; item < kKT * kLc; item += kThreads) {
                const int k = item & 31, l = item >> 5;
                sg.Cs[l][k] = (k0 + k < K) ? __ldg(C + (k0 + k) * ldc + l0 + l) : 0.f;
            }
    };

    if (items > 0) request(0);
    pair_t acc2[8][2];
    for (int64_t n = 0; n < items; ++n) {
        asm volatile("cp.async.wait_all;" ::: "memory");
        __syncthreads();  // item n has landed; everybody is done with the other stage
        if (n + 1 < items) request(n + 1);
        const TtmStage& sg = stage[n & 1];
        const int64_t chunk = n % chunks;
        if (chunk == 0) {
#pragma unroll
            for (int q = 0; q < 8; ++q) acc2[q][0] = acc2[q][1] = 0ull;
        }
#pragma unroll 2
        for (int l4 = 0; l4 < kLc / 4; ++l4) {
            float4 x[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) x[q] = *reinterpret_cast<const float4*>(&sg.Xs[8 * rg + q][4 * l4]);
#pragma unroll
            for (int dl = 0; dl < 4; ++dl) {
                const ulonglong2 c = *reinterpret_cast<const ulonglong2*>(&sg.Cs[4 * l4 + dl][4 * kg]);
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    const float xv = dl == 0 ? x[q].x : dl == 1 ? x[q].y : dl == 2 ? x[q].z : x[q].w;
                    const pair_t x2 = pack2(xv, xv);
                    fma2(acc2[q][0], x2, c.x);
                    fma2(acc2[q][1], x2, c.y);
                }
            }
        }
        if (chunk == chunks - 1) {
            const int64_t p0 = (blockIdx.x + (n / chunks) * gridDim.x) * kRowsT;
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                const int64_t p = p0 + 8 * rg + q, k = k0 + 4 * kg;
                if (p >= P || k >= K) continue;
                float o[4];
                unpack2(acc2[q][0], o[0], o[1]);
                unpack2(acc2[q][1], o[2], o[3]);
                float* dst = Y + p * K + k;
                if (vec_y && k + 4 <= K) {
                    float4 v = make_float4(o[0], o[1], o[2], o[3]);
                    if (accumulate) {
                        const float4 old = *reinterpret_cast<const float4*>(dst);
                        v.x += old.x; v.y += old.y; v.z += old.z; v.w += old.w;
                    }
                    *reinterpret_cast<float4*>(dst) = v;
                } else {
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        if (k + e < K) dst[e] = accumulate ? dst[e] + o[e] : o[e];
                }
            }
        }
    }
}

}  // namespace

// P = packed (i, j) pairs, Q and K = trailing extents of the input and of the output.
dastac_status launch_ttm(int64_t P, int64_t Q, int64_t K, const float* X, const float* C, int64_t ldc, float* Y,
                         int accumulate, cudaStream_t st) {
    if (P == 0 || K == 0 || Q == 0) return DASTAC_OK;
    const int64_t gx = (P + kRowsT - 1) / kRowsT, gy = (K + kKT - 1) / kKT;
    if (gx > 0x7fffffffLL || gy > 65535) return DASTAC_ERR_OVERFLOW;
    const int vec_x = (Q % 4 == 0) && aligned16(X), vec_y = (K % 4 == 0) && aligned16(Y);
    if (vec_x && Q % kLc == 0) {
        static bool attr_set[64];
        int dev = 0;
        cudaGetDevice(&dev);
        if (dev >= 0 && dev < 64 && !attr_set[dev]) {
            if (cudaFuncSetAttribute(ttm_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)(2 * sizeof(TtmStage))) != cudaSuccess)
                return DASTAC_ERR_CUDA;
            attr_set[dev] = true;
        }
        int64_t bx = ((int64_t)sm_count() * 2 + gy - 1) / gy;  // two CTAs per SM in all
        if (bx > gx) bx = gx;
        ttm_stream_kernel<<<dim3((unsigned)bx, (unsigned)gy), kThreads, 2 * sizeof(TtmStage), st>>>(P, Q, K, gx, X, C, ldc, Y,
                                                                                             accumulate, vec_y);
        return launch_status();
    }
    ttm_kernel<<<dim3((unsigned)gx, (unsigned)gy), kThreads, 0, st>>>(P, Q, K, X, C, ldc, Y, accumulate, vec_x, vec_y);
    return launch_status();
}

}  // namespace dastac
