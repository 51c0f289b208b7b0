// Split-precision tensor-core form of the tetrahedral MTTKRP (opt-in, its own entry point).
//
// M(i,r) = sum_{i<=j<=k} T(i,j,k) B(j,r) C(k,r) (Table 1 "MTTKRP" over the hyper-triangular domain of
// Section 1), factored as in mttkrp.cu: for a slab i, U = T_i C is a triangular matrix times the
// tall matrix C, and M(i,:) = sum_j B(j,:) o U(j,:).  Here U is computed on the tensor cores in
// TF32 with every fp32 operand split into a high and a low part (hi = the value with its low 13
// mantissa bits cleared, lo = value - hi, exact in fp32, of which the tensor core reads the upper 19 bits):
//     T C  ~  Thi Chi + Thi Clo + Tlo Chi        (the dropped Tlo Clo is 2^-22 relative)
// accumulated in fp32 in tensor memory; the error per product is about 2^-21, far inside the 1e-5
// bound of the fp32 kernels, which a single TF32 pass (2^-11) would break.
//
// Tile = (slab i, 128 fibres j0 .. j0+127), K blocks of 32 from the block that holds j0 to n.
//   producer warps   read the packed fibres with aligned 128-bit loads (a row starts at
//                    rowbase + j, aligned only by accident, so a lane combines the two quads that
//                    cover an aligned group of four k), zero what lies outside j <= k < n, split
//                    into hi / lo and store both as K-major, 128-byte-swizzled 128 x 32 tiles
//   MMA thread       per K block: four tcgen05.mma kind::tf32 M128 N64 K8 with A = Thi and
//                    B = [Chi ; Clo] (columns 0..31 get Thi Chi, 32..63 get Thi Clo), then four
//                    M128 N32 K8 with A = Tlo, B = Chi into columns 0..31
//   epilogue warps   tcgen05.ld, U = D[:,0:32] + D[:,32:64], times B(j,:), summed over the 128
//                    rows by a shuffle reduce-scatter, one atomic add per column and warp
// The factor C is staged once per CTA as hi / lo K-major tiles (n x 32 x 4 bytes each), so the
// form needs n <= 512 (128 KiB for both parts beside the A stages).  Accumulators are double
// buffered in tensor memory (2 x 64 columns).  Every wait is bounded.
#include <mutex>

#include "common.cuh"
#include "tf32_mma.cuh"
#include "waits.cuh"

namespace dastac {
namespace {

constexpr int kTcRows = 128;             // fibres per tile
constexpr int kTcBlockK = 32;            // k per K block: one 128-byte swizzle row
constexpr int kTcTileBytes = kTcRows * 128;          // 16 KiB: a 128 x 32 fp32 tile
constexpr int kTcStageBytes = 2 * kTcTileBytes;      // hi + lo
constexpr int kTcMaxN = 512;
constexpr int kTcProducerWarps = 8;                  // warps that fill one stage
constexpr int kTcProducerGroups = 2;                 // groups of such warps, taking the items in turn
constexpr int kTcWarpMma = 4;                        // warps 0-3 epilogue, 4 MMA, 5.. producers
constexpr int kTcThreads = (5 + kTcProducerWarps * kTcProducerGroups) * 32;
constexpr int kTcAhead = 2;                         // items whose loads are in flight per producer thread
constexpr int kTcTmemCols = 128;                     // two accumulators of 64 columns
constexpr long long kTcWaitBudget = 2000000000LL;
constexpr int32_t kErrWordMttkrpTc = 0x4d43;         // "MC"

constexpr uint32_t tc_idesc(int n_cols) { return tc_idesc_mn(kTcRows, n_cols); }

struct TcParams {
    const float* T;
    const float* B;
    const float* C;
    float* M;
    int64_t ldb, ldc, ldm;
    int64_t tetn;      // tet(n)
    int64_t cap_quads; // 16-byte quads of the packed buffer (count rounded up to 4 elements)
    int32_t n, R, n_kb, stages, tiles;
    int32_t* err_word;
};

// Tiles sorted by their first fibre j0 = i + 128 t (cost falls as j0 grows): block g = j0 / 128
// holds 128 (g + 1) tiles, tile q of the block is (j0 = 128 g + q / (g + 1), t = q mod (g + 1)).
__host__ __device__ inline int tc_tile_count(int n) {
    int total = 0;
    for (int g = 0; 128 * g < n; ++g) {
        const int rows = n - 128 * g < 128 ? n - 128 * g : 128;
        total += rows * (g + 1);
    }
    return total;
}
__device__ __forceinline__ void tc_decode(int q, int& i, int& j0) {
    int g = 0;
    while (q >= 128 * (g + 1)) {
        q -= 128 * (g + 1);
        ++g;
    }
    j0 = 128 * g + q / (g + 1);
    i = j0 - 128 * (q % (g + 1));
}

// Bounded wait shared by the roles: false when the budget ran out here or elsewhere in the CTA.
__device__ __forceinline__ bool tc_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* err_word) {
    return tc_wait_coded(bar, parity, abort_flag, err_word, kErrWordMttkrpTc, kTcWaitBudget);
}

// Writes a thread's 16 values of k (element k0 + x is v[x + SH]) as hi / lo parts into its row of the
// two swizzled tiles; outside j <= k < n (or for a fibre beyond n) zeros are written.
template <int SH>
__device__ __forceinline__ void tc_store_item(const float (&v)[20], uint8_t* row_hi, int h, int m, int k0, int j, int n,
                                              bool live, bool interior) {
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        float hi[4], lo[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int x = 4 * c + e;
            float val = v[x + SH];
            if (!interior) {
                const int k = k0 + x;
                if (!(live && k >= j && k < n)) val = 0.f;
            }
            tc_split(val, hi[e], lo[e]);
        }
        const uint32_t off = (uint32_t)(((h * 4 + c) ^ (m & 7)) << 4);
        *reinterpret_cast<float4*>(row_hi + off) = make_float4(hi[0], hi[1], hi[2], hi[3]);
        *reinterpret_cast<float4*>(row_hi + kTcTileBytes + off) = make_float4(lo[0], lo[1], lo[2], lo[3]);
    }
}

__global__ void __launch_bounds__(kTcThreads, 1) mttkrp_tc_kernel(const TcParams p) {
    extern __shared__ uint8_t tc_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(tc_raw) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint8_t* const Cb = smem;                                      // n_kb blocks of 8 KiB: [Chi ; Clo]
    uint8_t* const stage0 = smem + (size_t)p.n_kb * 8192;          // A stages: hi tile, lo tile
    uint64_t* const bars = reinterpret_cast<uint64_t*>(stage0 + (size_t)p.stages * kTcStageBytes);
    const int S = p.stages;
    auto full = [&](int s) { return tc_smem(&bars[s]); };
    auto empty = [&](int s) { return tc_smem(&bars[S + s]); };
    auto tmem_full = [&](int a) { return tc_smem(&bars[2 * S + a]); };
    auto tmem_empty = [&](int a) { return tc_smem(&bars[2 * S + 2 + a]); };
    uint32_t* const tmem_slot = reinterpret_cast<uint32_t*>(&bars[2 * S + 4]);
    volatile int* const abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            tc_mbar_init(full(s), kTcProducerWarps);
            tc_mbar_init(empty(s), 1);
        }
        for (int a = 0; a < 2; ++a) {
            tc_mbar_init(tmem_full(a), 1);
            tc_mbar_init(tmem_empty(a), 4);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tc_smem(tmem_slot)),
                     "r"((uint32_t)kTcTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // C(:, 0..31) as hi / lo K-major tiles: element (k, r) -> block k / 32, rows r (hi) and 32 + r (lo)
    for (int base = threadIdx.x; base < p.n_kb * 32 * 32; base += 8 * blockDim.x) {
        float cv[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {  // eight independent loads in flight per thread
            const int idx = base + u * blockDim.x, k = idx >> 5, r = idx & 31;
            cv[u] = (idx < p.n_kb * 32 * 32 && k < p.n && r < p.R) ? __ldg(p.C + (int64_t)k * p.ldc + r) : 0.f;
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int idx = base + u * blockDim.x, k = idx >> 5, r = idx & 31;
            if (idx >= p.n_kb * 32 * 32) break;
            float hi, lo;
            tc_split(cv[u], hi, lo);
            const int kk = k & 31;
            uint8_t* blk = Cb + (size_t)(k >> 5) * 8192;
            const uint32_t in_row = (uint32_t)((((kk >> 2) ^ (r & 7)) << 4) + (kk & 3) * 4);
            *reinterpret_cast<float*>(blk + (r >> 3) * 1024 + (r & 7) * 128 + in_row) = hi;
            *reinterpret_cast<float*>(blk + 4096 + (r >> 3) * 1024 + (r & 7) * 128 + in_row) = lo;
        }
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;

    const int G = gridDim.x;
    auto tile_of = [&](int round) { return round * G + ((round & 1) ? (G - 1 - (int)blockIdx.x) : (int)blockIdx.x); };
    const int rounds = (p.tiles + G - 1) / G;
    const int n = p.n;

    if (warp > kTcWarpMma) {
        // ---- producers: thread = (row m, half h) of the 128 x 32 tile ----
        // The loads of an item (tile, K block) are issued kTcAhead items before its tile is written,
        // so that several K blocks of packed data are in flight per thread.
        // Warp w owns the rows m = w + 8 r (r = 0..15): fibres eight apart share their misalignment
        // (the row base advances by n-j-1 per fibre, eight steps sum to a multiple of 4), so the
        // realignment shift is uniform in the warp and is resolved by one switch, not per element.
        // Two groups of eight warps take the items in turn, so that the dependent chain of one item
        // (wait, realign, split, store, fence, arrive) overlaps with the other group's.
        const int pw = (warp - (kTcWarpMma + 1)) % kTcProducerWarps, grp = (warp - (kTcWarpMma + 1)) / kTcProducerWarps;
        const int m = pw + 8 * (lane >> 1), h = lane & 1;
        const float4* Tq = reinterpret_cast<const float4*>(p.T);
        struct Item {
            int j, k0, s;       // fibre of this thread, first of its 16 values of k, misalignment
            bool valid, live;   // an item exists; the fibre exists
            bool interior;      // every (row, k) of the tile's K block lies inside the set
        };
        // iterator over this CTA's items
        int round = -1, kb = 0, kb_end = 0, cur_j = 0, cur_s = 0, cur_j0 = 0;
        bool cur_live = false;
        int64_t cur_rb = 0;
        auto next_item = [&](Item& itx, int64_t& q0) {
            while (kb >= kb_end) {  // next tile
                ++round;
                if (round >= rounds) {
                    itx.valid = false;
                    return;
                }
                const int q = tile_of(round);
                if (q >= p.tiles) continue;
                int i, j0;
                tc_decode(q, i, j0);
                cur_j = j0 + m;
                cur_j0 = j0;
                cur_live = cur_j < n;
                cur_rb = cur_live ? p.tetn - tet((int64_t)(n - i)) + tri((int64_t)(n - i)) - tri((int64_t)(n - cur_j)) - cur_j : 0;
                cur_s = (int)(cur_rb & 3);
                kb = j0 >> 5;
                kb_end = p.n_kb;
            }
            itx.valid = true;
            itx.live = cur_live;
            itx.j = cur_j;
            itx.s = cur_s;
            itx.k0 = kb * 32 + h * 16;
            itx.interior = kb * 32 >= cur_j0 + kTcRows - 1 && kb * 32 + 31 < n && cur_j0 + kTcRows - 1 < n;
            q0 = (cur_rb + itx.k0) >> 2;  // memory quad that holds element k0
            ++kb;
        };
        auto load_item = [&](const Item& itx, int64_t q0, float (&v)[20]) {
#pragma unroll
            for (int e = 0; e < 20; ++e) v[e] = 0.f;
            if (itx.valid && itx.live && itx.k0 + 15 >= itx.j && itx.k0 < n) {
#pragma unroll
                for (int c = 0; c < 5; ++c) {
                    // quad c holds k = k0 - s + 4c .. +3: loaded when it holds an element of the row
                    const int klo = itx.k0 - itx.s + 4 * c;
                    if (klo + 3 >= itx.j && klo < n && q0 + c < p.cap_quads) {
                        const float4 t4 = __ldg(Tq + q0 + c);
                        v[4 * c] = t4.x, v[4 * c + 1] = t4.y, v[4 * c + 2] = t4.z, v[4 * c + 3] = t4.w;
                    }
                }
            }
        };
        auto next_own_item = [&](Item& itx, int64_t& q0) {  // this group's next item: every kTcProducerGroups-th
            next_item(itx, q0);
#pragma unroll
            for (int g = 1; g < kTcProducerGroups; ++g) {
                Item skip;
                int64_t qs = 0;
                next_item(skip, qs);
            }
        };
        Item items[kTcAhead];
        float vals[kTcAhead][20];
        for (int g = 0; g < grp; ++g) {  // items 0 .. grp-1 belong to the groups before this one
            Item skip;
            int64_t qs = 0;
            next_item(skip, qs);
        }
#pragma unroll
        for (int d = 0; d < kTcAhead; ++d) {
            int64_t q0 = 0;
            next_own_item(items[d], q0);
            load_item(items[d], q0, vals[d]);
        }
        uint32_t it = (uint32_t)grp;
        bool ok = true;
        while (ok) {
#pragma unroll
            for (int d = 0; d < kTcAhead; ++d) {
                if (!ok) break;
                const Item itx = items[d];
                if (!itx.valid) {
                    ok = false;
                    break;
                }
                const int st = it % S;
                if (it >= (uint32_t)S && !tc_wait(empty(st), ((it / S) & 1) ^ 1, abort_flag, p.err_word)) {
                    ok = false;
                    break;
                }
                uint8_t* row_hi = stage0 + (size_t)st * kTcStageBytes + (m >> 3) * 1024 + (m & 7) * 128;
                // lane 0 holds the warp's first row: if that fibre does not exist none of the warp's does
                const int s_warp = __shfl_sync(0xffffffffu, itx.s, 0);
                switch (s_warp) {
                    case 0: tc_store_item<0>(vals[d], row_hi, h, m, itx.k0, itx.j, n, itx.live, itx.interior); break;
                    case 1: tc_store_item<1>(vals[d], row_hi, h, m, itx.k0, itx.j, n, itx.live, itx.interior); break;
                    case 2: tc_store_item<2>(vals[d], row_hi, h, m, itx.k0, itx.j, n, itx.live, itx.interior); break;
                    default: tc_store_item<3>(vals[d], row_hi, h, m, itx.k0, itx.j, n, itx.live, itx.interior); break;
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0) tc_mbar_arrive(full(st));
                it += kTcProducerGroups;
                int64_t q0 = 0;
                next_own_item(items[d], q0);
                load_item(items[d], q0, vals[d]);
            }
        }
    }
    else if (warp == kTcWarpMma) {
        // ---- MMA issuer: one thread ----
        if (lane == 0) {
            constexpr uint32_t kIdesc64 = tc_idesc(64), kIdesc32 = tc_idesc(32);
            uint32_t it = 0, tile_n = 0;
            bool ok = true;
            for (int round = 0; round < rounds && ok; ++round) {
                const int q = tile_of(round);
                if (q >= p.tiles) continue;
                int i, j0;
                tc_decode(q, i, j0);
                const int acc = tile_n & 1;
                const uint32_t use = tile_n >> 1;  // earlier uses of this accumulator
                if (use >= 1 && !tc_wait(tmem_empty(acc), (use - 1) & 1, abort_flag, p.err_word)) {
                    ok = false;
                    break;
                }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t d_tmem = tmem_base + acc * 64;
                const int kb_first = j0 >> 5;
                for (int kb = kb_first; kb < p.n_kb; ++kb, ++it) {
                    const int st = it % S;
                    if (!tc_wait(full(st), (it / S) & 1, abort_flag, p.err_word)) {
                        ok = false;
                        break;
                    }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t a_hi = tc_smem(stage0 + (size_t)st * kTcStageBytes);
                    const uint32_t a_lo = a_hi + kTcTileBytes;
                    const uint32_t b_blk = tc_smem(Cb + (size_t)kb * 8192);
#pragma unroll
                    for (int k8 = 0; k8 < 4; ++k8)  // Thi [Chi ; Clo] -> columns 0..63
                        tc_mma_tf32(d_tmem, tc_desc(a_hi + k8 * 32), tc_desc(b_blk + k8 * 32), kIdesc64,
                                    (kb > kb_first || k8 > 0) ? 1u : 0u);
#pragma unroll
                    for (int k8 = 0; k8 < 4; ++k8)  // Tlo Chi -> columns 0..31
                        tc_mma_tf32(d_tmem, tc_desc(a_lo + k8 * 32), tc_desc(b_blk + k8 * 32), kIdesc32, 1u);
                    tc_commit(empty(st));
                }
                if (ok) tc_commit(tmem_full(acc));
                ++tile_n;
            }
        }
    } else {
        // ---- epilogue: thread = row of the tile = lane of tensor memory ----
        uint32_t tile_n = 0;
        bool ok = true;
        for (int round = 0; round < rounds && ok; ++round) {
            const int q = tile_of(round);
            if (q >= p.tiles) continue;
            int i, j0;
            tc_decode(q, i, j0);
            const int acc = tile_n & 1;
            const uint32_t use = tile_n >> 1;
            int got = 1;
            if (lane == 0) got = tc_wait(tmem_full(acc), use & 1, abort_flag, p.err_word) ? 1 : 0;
            got = __shfl_sync(0xffffffffu, got, 0);
            if (!got) {
                ok = false;
                break;
            }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16) + acc * 64;
            uint32_t d0[32], d1[32];
            tc_ld32(taddr, d0);
            tc_ld32(taddr + 32, d1);
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) tc_mbar_arrive(tmem_empty(acc));  // the accumulator may be overwritten
            // v(r) = B(j, r) (Thi Chi + Tlo Chi + Thi Clo)(j, r)
            const int j = j0 + warp * 32 + lane;
            float v[32];
            const bool bvec = (p.ldb & 3) == 0 && p.R == 32 && (reinterpret_cast<uintptr_t>(p.B) & 15u) == 0;
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                float4 b4 = make_float4(0.f, 0.f, 0.f, 0.f);
                if (j < n) {
                    const float* src = p.B + (int64_t)j * p.ldb + 4 * c;
                    if (bvec) {
                        b4 = __ldg(reinterpret_cast<const float4*>(src));
                    } else {
                        if (4 * c < p.R) b4.x = __ldg(src);
                        if (4 * c + 1 < p.R) b4.y = __ldg(src + 1);
                        if (4 * c + 2 < p.R) b4.z = __ldg(src + 2);
                        if (4 * c + 3 < p.R) b4.w = __ldg(src + 3);
                    }
                }
                v[4 * c] = b4.x * (__uint_as_float(d0[4 * c]) + __uint_as_float(d1[4 * c]));
                v[4 * c + 1] = b4.y * (__uint_as_float(d0[4 * c + 1]) + __uint_as_float(d1[4 * c + 1]));
                v[4 * c + 2] = b4.z * (__uint_as_float(d0[4 * c + 2]) + __uint_as_float(d1[4 * c + 2]));
                v[4 * c + 3] = b4.w * (__uint_as_float(d0[4 * c + 3]) + __uint_as_float(d1[4 * c + 3]));
            }
            // sum over the warp's 32 rows: reduce-scatter, lane r ends with column r
#pragma unroll
            for (int w = 16; w >= 1; w >>= 1) {
                const bool upper = (lane & w) != 0;
#pragma unroll
                for (int e = 0; e < w; ++e) {
                    const float mine = upper ? v[e + w] : v[e];
                    const float other = upper ? v[e] : v[e + w];
                    v[e] = mine + __shfl_xor_sync(0xffffffffu, other, w);
                }
            }
            if (lane < p.R) atomicAdd(p.M + (int64_t)i * p.ldm + lane, v[0]);
            ++tile_n;
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)kTcTmemCols) : "memory");
    }
}

__global__ void tc_zero_rows_kernel(float* __restrict__ M, int64_t ldm, int64_t rows, int64_t R) {
    for (int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; t < rows * R; t += (int64_t)gridDim.x * blockDim.x)
        M[(t / R) * ldm + (t % R)] = 0.f;
}

}  // namespace
}  // namespace dastac

using namespace dastac;

extern "C" dastac_status dastac_mttkrp_split_tf32(const dastac_structure* s, const float* T, const float* B, int64_t ldb,
                                                  const float* C, int64_t ldc, float* M, int64_t ldm, int64_t R,
                                                  int32_t accumulate, int32_t* err_word, void* stream) {
    if (!s) return DASTAC_ERR_INVALID_ARG;
    const IndexMap& m = s->map;
    if (m.kind == kEmpty) return DASTAC_OK;
    if (m.kind != kTetrahedron) return DASTAC_ERR_UNSUPPORTED_EXPR;
    const int64_t n = m.N;
    if (n > kTcMaxN || R > 32) return DASTAC_ERR_UNSUPPORTED_EXPR;
    if (n == 0 || R == 0) return DASTAC_OK;
    if (R < 0 || !T || !B || !C || !M || ldb < R || ldc < R || ldm < R) return DASTAC_ERR_INVALID_ARG;
    if (!aligned16(T)) return DASTAC_ERR_ALIGNMENT;
    cudaStream_t cs = (cudaStream_t)stream;
    TcParams p;
    p.T = T, p.B = B, p.C = C, p.M = M;
    p.ldb = ldb, p.ldc = ldc, p.ldm = ldm;
    p.tetn = tet(n);
    p.cap_quads = (m.count + 3) / 4;
    p.n = (int32_t)n, p.R = (int32_t)R;
    p.n_kb = (int32_t)((n + kTcBlockK - 1) / kTcBlockK);
    p.tiles = tc_tile_count((int)n);
    p.err_word = err_word;
    const size_t fixed = (size_t)p.n_kb * 8192 + 1024 /*alignment*/ + 256 /*barriers*/;
    p.stages = (int32_t)((227 * 1024 - fixed) / kTcStageBytes);
    if (p.stages > 4) p.stages = 4;
    if (p.stages < 2) return DASTAC_ERR_UNSUPPORTED_EXPR;
    const size_t smem = fixed + (size_t)p.stages * kTcStageBytes;
    static bool attr_set[64];
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        if (cudaFuncSetAttribute(mttkrp_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess)
            return DASTAC_ERR_CUDA;
        attr_set[dev] = true;
    }
    if (!accumulate) {
        int64_t blocks = (n * R + 255) / 256;
        if (blocks > 1024) blocks = 1024;
        tc_zero_rows_kernel<<<(unsigned)blocks, 256, 0, cs>>>(M, ldm, n, R);
        const dastac_status st = launch_status();
        if (st != DASTAC_OK) return st;
    }
    int grid = sm_count();
    if (grid > p.tiles) grid = p.tiles;
    mttkrp_tc_kernel<<<grid, kTcThreads, smem, cs>>>(p);
    return launch_status();
}
