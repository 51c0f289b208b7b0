// Split-precision tensor-core form of band x dense (opt-in, its own entry point).
//
// C = A B with A banded, |i - j| <= w (Section 1, the banded motivation; Section 6.4), stored as
// padded diagonals or packed exactly row after row; B and C dense row-major fp32.  A tile of 128
// rows i0 .. i0+127 touches the B rows i0-w .. i0+127+w only, so the product of the tile is the
// dense product of a 128 x (128 + 2w) slice of A (the band inside it, zeros elsewhere) with that
// window of B.  It runs on the tensor cores in TF32 with both operands split into a high and a low
// part (tf32_mma.cuh): A B ~ Ahi Bhi + Ahi Blo + Alo Bhi, accumulated in fp32 in tensor memory,
// about 2^-21 per product, inside the 1e-5 bound of the fp32 kernels.
//
// Tile = (128 rows, 256 columns); K blocks of 32 rows of the B window.
//   producer warps   two groups of eight, taking the K blocks in turn, one stage each.  The K block of
//                    B arrives by bulk tensor copies (eight 32 x 32 boxes) straight into the N-major
//                    operand layout of 4-byte types (rows of 128 bytes, 32-byte pieces swizzled with
//                    the row); the block itself serves as Bhi, since the tensor core reads only the
//                    upper 19 bits of a value, and the warps write Blo = B - trunc(B) beside it.  (A B
//                    whose rows are not 16-byte aligned is read column by column with plain loads
//                    and stored in the same layout.)  The slice of A is K-major: it is zeroed and the
//                    band written into it diagonal by diagonal: for diagonal d the 32 rows whose
//                    entry falls into this K block are consecutive in memory in the padded layout
//                    (one coalesced load) and land on 32 different banks of the swizzled tile.
//   MMA thread       per K block and k-step of 8: three tcgen05.mma kind::tf32 M128 N256 K8
//                    (Ahi Bhi, Ahi Blo, Alo Bhi) into one accumulator
//   epilogue warps   one per lane quarter of tensor memory: tcgen05.ld, then 32 x 32 chunks leave
//                    through shared memory by bulk tensor stores (reduce-add when accumulating);
//                    a C whose rows are not 16-byte aligned is written with plain stores
// Two stages of operands (96 KiB each), two accumulators of 256 columns (all of tensor memory).
// K blocks that lie outside the matrix (first and last tiles) are skipped.  Every wait is bounded.
#include <cuda.h>

#include <cstring>

#include "common.cuh"
#include "tf32_mma.cuh"
#include "waits.cuh"

namespace dastac {
namespace {

constexpr int kBtRows = 128;                 // rows of C per tile
constexpr int kBtCols = 256;                 // columns of C per tile
constexpr int kBtATile = kBtRows * 128;      // 16 KiB: 128 x 32 fp32
constexpr int kBtBTile = kBtCols * 128;      // 32 KiB: 256 x 32 fp32
constexpr int kBtStageBytes = 2 * kBtATile + 2 * kBtBTile;  // Ahi, Alo, Bhi, Blo
constexpr int kBtStages = 2;
constexpr int kBtEpiWarps = 4, kBtWarpMma = 4, kBtProducerWarps = 8;  // warps 0-3 epilogue, 4 MMA, 5.. producers
constexpr int kBtEpiCols = kBtCols / (kBtEpiWarps / 4);  // columns of the tile per epilogue warp
constexpr int kBtProducerGroups = 2;         // = kBtStages: group g fills stage g
constexpr int kBtThreads = (kBtEpiWarps + 1 + kBtProducerWarps * kBtProducerGroups) * 32;
// diagonals of one K block per producer warp: at most ceil(min(2w + 1, 159) / 8), a template parameter
// of the kernel (10 for 2w + 1 <= 80, else 20) so that narrow bands hold fewer values in registers
constexpr int kBtTmemCols = 512;
constexpr long long kBtWaitBudget = 2000000000LL;
constexpr int32_t kErrWordBandTc = 0x4254;   // "BT"
constexpr int kBtEpiBufBytes = 32 * 128;     // a 32 x 32 fp32 chunk of C on its way out
constexpr int kBtEpiBytes = kBtEpiWarps * 2 * kBtEpiBufBytes;  // two buffers per epilogue warp
constexpr size_t kBtSmemBytes = (size_t)kBtStages * kBtStageBytes + kBtEpiBytes + 1024 /*alignment*/ + 256 /*barriers*/;

struct BtParams {
    const float* A;
    const float* B;
    float* C;
    int64_t N, w, ldb, ldc, ncols;
    int32_t row_tiles, col_tiles, tiles;
    int32_t exact;       // A packed row after row instead of padded diagonals
    int32_t accumulate;
    int32_t vec_c;       // C allows 128-bit accesses
    int32_t tma_b;       // B is described by a tensor map: its K blocks arrive by bulk tensor copies
    int32_t tma_c;       // C is described by the tensor map: chunks leave through shared memory by bulk stores
    int32_t* err_word;
};

// K blocks of a tile that intersect the matrix: window row kk of the tile is B row i0 - w + kk
__device__ __forceinline__ void bt_k_range(const BtParams& p, int64_t i0, int& kb_lo, int& kb_hi) {
    const int64_t row0 = i0 - p.w;
    const int64_t rows_live = p.N - i0 < kBtRows ? p.N - i0 : kBtRows;
    int64_t kk_end = rows_live + 2 * p.w;          // one past the last window row any live row reads
    if (p.N - row0 < kk_end) kk_end = p.N - row0;  // ... that exists
    kb_lo = row0 < 0 ? (int)((-row0) >> 5) : 0;
    kb_hi = (int)((kk_end + 31) >> 5);
}

// N-major B operand of a 4-byte type: rows (one k, 32 consecutive n) of 128 bytes whose 32-byte
// pieces are swizzled with the row; groups of four rows 512 bytes apart, blocks of 32 columns one
// 32 x 32 box (4096 bytes) apart.
__device__ __forceinline__ uint64_t bt_desc_b(uint32_t addr) {
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3FFF);
    d |= (uint64_t)(4096 >> 4) << 16;  // leading byte offset: next block of 32 columns
    d |= (uint64_t)(512 >> 4) << 32;   // stride byte offset: next group of four rows
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)1 << 61;            // 128-byte swizzle of 32-byte pieces
    return d;
}
__device__ __forceinline__ bool bt_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* err_word) {
    return tc_wait_coded(bar, parity, abort_flag, err_word, kErrWordBandTc, kBtWaitBudget);
}
// Barrier of the eight warps of a producer group (barrier 1 + group) that also tells every one of them whether any thread raised
// `flag`: the warps leave their loop together, so none is left waiting at this barrier.
template <int ID>
__device__ __forceinline__ bool bt_bar_or(bool flag) {
    uint32_t any;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.b32 p, %1, 0;\n\t"
        "bar.red.or.pred q, %2, %3, p;\n\t"
        "selp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(any)
        : "r"((uint32_t)flag), "n"(ID), "n"(kBtProducerWarps * 32)
        : "memory");
    return any != 0;
}
__device__ __forceinline__ bool bt_producer_sync_any(bool flag, int group) {
    return group == 0 ? bt_bar_or<1>(flag) : bt_bar_or<2>(flag);
}

template <int kBtSegs>
__global__ void __launch_bounds__(kBtThreads, 1) bandmm_tc_kernel(const __grid_constant__ CUtensorMap tmap_b, const __grid_constant__ CUtensorMap tmap_c, const BtParams p) {
    extern __shared__ uint8_t bt_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(bt_raw) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint8_t* const epi0 = smem + (size_t)kBtStages * kBtStageBytes;
    uint64_t* const bars = reinterpret_cast<uint64_t*>(epi0 + kBtEpiBytes);
    constexpr int S = kBtStages;
    auto full = [&](int s) { return tc_smem(&bars[s]); };
    auto empty = [&](int s) { return tc_smem(&bars[S + s]); };
    auto tmem_full = [&](int a) { return tc_smem(&bars[2 * S + a]); };
    auto tmem_empty = [&](int a) { return tc_smem(&bars[2 * S + 2 + a]); };
    auto raw = [&](int s) { return tc_smem(&bars[2 * S + 4 + s]); };  // the stage's block of B has landed
    uint32_t* const tmem_slot = reinterpret_cast<uint32_t*>(&bars[3 * S + 4]);
    volatile int* const abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            tc_mbar_init(full(s), kBtProducerWarps);
            tc_mbar_init(empty(s), 1);
            tc_mbar_init(raw(s), 1);
        }
        for (int a = 0; a < 2; ++a) {
            tc_mbar_init(tmem_full(a), 1);
            tc_mbar_init(tmem_empty(a), kBtEpiWarps);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tc_smem(tmem_slot)),
                     "r"((uint32_t)kBtTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;

    const int G = gridDim.x;
    const int rounds = (p.tiles + G - 1) / G;
    auto tile_of = [&](int round) { return round * G + (int)blockIdx.x; };
    const int64_t N = p.N, w = p.w;

    if (warp > kBtWarpMma) {
        // ---- producers: two groups of eight warps take the items (tile, K block) in turn, group g
        // fills stage g.  A group issues the loads of its next item right after it has published the
        // current one, so they are in flight while the tensor core works on the other group's stage.
        const int pw = (warp - (kBtWarpMma + 1)) % kBtProducerWarps, grp = (warp - (kBtWarpMma + 1)) / kBtProducerWarps;
        const int t = pw * 32 + lane;  // column of the tile whose B values this thread splits
        int round = -1, kb = -1, kb_end = 0;
        int64_t i0 = 0, cb = 0;
        bool valid = true;
        auto next_item = [&]() {  // advances to the next (tile, K block) of this CTA
            if (!valid) return;
            ++kb;
            while (kb >= kb_end) {
                ++round;
                if (round >= rounds || tile_of(round) >= p.tiles) {
                    valid = false;
                    return;
                }
                const int q = tile_of(round);
                i0 = (int64_t)(q / p.col_tiles) * kBtRows;
                cb = (int64_t)(q % p.col_tiles) * kBtCols;
                bt_k_range(p, i0, kb, kb_end);
            }
        };
        float av[kBtSegs];
        auto load_item = [&]() {
            const int64_t j0 = i0 - w + 32 * (int64_t)kb;  // B row of the block's first window row
            // Diagonals d whose entries fall into this K block for some row of the tile: row r holds
            // diagonal d at window row kk = r + d, so d in [32 kb - 127, 32 kb + 31].  This warp takes
            // d = d_lo + pw + 8u; its lane reads row r0 - 8u, always column j of A.
            const int d0 = (32 * kb - (kBtRows - 1) > 0 ? 32 * kb - (kBtRows - 1) : 0) + pw;
            const int d_hi = (int)(32 * (int64_t)kb + 31 < 2 * w ? 32 * (int64_t)kb + 31 : 2 * w);
            const int r0 = 32 * kb - d0 + lane;
            const int r_lim = (int)(N - i0 < kBtRows ? N - i0 : kBtRows);  // rows of the tile that exist
            const int64_t j = j0 + lane;
            const bool j_ok = j >= 0 && j < N;
            if (!p.exact) {
                int64_t aoff = (int64_t)d0 * N + i0 + r0;  // slot (d, i) = d N + i; next segment: + 8 (N - 1)
                const int64_t astep = 8 * (N - 1);
#pragma unroll
                for (int u = 0; u < kBtSegs; ++u, aoff += astep) {
                    const int r = r0 - 8 * u;
                    av[u] = (d0 + 8 * u <= d_hi && j_ok && r >= 0 && r < r_lim) ? __ldg(p.A + aoff) : 0.f;
                }
            } else {
#pragma unroll
                for (int u = 0; u < kBtSegs; ++u) {
                    const int r = r0 - 8 * u;
                    const int64_t i = i0 + r;
                    av[u] = (d0 + 8 * u <= d_hi && j_ok && r >= 0 && r < r_lim) ? __ldg(p.A + (band_row_start(N, w, i) - band_jlo(w, i) + j)) : 0.f;
                }
            }
        };
        for (int g = 0; g <= grp; ++g) next_item();  // group g starts at item g
        if (valid) load_item();
        const int st = grp;
        uint8_t* const a_hi = smem + (size_t)st * kBtStageBytes;
        uint8_t* const b_hi = a_hi + 2 * kBtATile;
        uint32_t use = 0;  // items this group has written into its stage
        while (valid) {
            // one lane per warp waits for the stage; the group's barrier below spreads the outcome
            bool ok = true;
            if (use >= 1 && lane == 0) ok = bt_wait(empty(st), (use - 1) & 1, abort_flag, p.err_word);
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            if (ok) {
                if (p.tma_b) {
                    // The K block of B, 32 rows x 256 columns, as eight 32 x 32 boxes: rows of 128 bytes
                    // whose 32-byte pieces are swizzled with the row (the N-major operand layout of
                    // 4-byte types).  Rows and columns outside B arrive as zeros.  The block itself is
                    // the high part: the tensor core reads the upper 19 bits of every value.
                    if (pw == 0 && lane == 0) {
                        const int64_t j0 = i0 - w + 32 * (int64_t)kb;
                        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(raw(st)), "r"((uint32_t)kBtBTile)
                                     : "memory");
#pragma unroll
                        for (int a = 0; a < kBtCols / 32; ++a)
                            asm volatile(
                                "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                                ::"r"(tc_smem(b_hi + a * 4096)), "l"(&tmap_b), "r"((int)(cb + 32 * a)), "r"((int)j0), "r"(raw(st))
                                : "memory");
                    }
                } else {
                    // column t of the block with plain loads (issued here, when the stage is free: this
                    // path holds no values across K blocks)
                    float bv[32];
                    const int64_t j0 = i0 - w + 32 * (int64_t)kb;
                    const int64_t col = cb + t;
                    const bool col_ok = col < p.ncols;
                    int64_t boff = j0 * p.ldb + col;  // used only where the row and column exist
                    if (j0 >= 0 && j0 + 31 < N) {  // block-uniform: every row of the K block exists
#pragma unroll
                        for (int e = 0; e < 32; ++e, boff += p.ldb) bv[e] = col_ok ? __ldg(p.B + boff) : 0.f;
                    } else {
#pragma unroll
                        for (int e = 0; e < 32; ++e, boff += p.ldb) {
                            const int64_t j = j0 + e;
                            bv[e] = (col_ok && j >= 0 && j < N) ? __ldg(p.B + boff) : 0.f;
                        }
                    }
                    // element (k, n) of the N-major layout sits at
                    // (n / 32) * 4096 + k * 128 + (((n % 32) / 8) ^ (k % 4)) * 32 + (n % 8) * 4
                    uint8_t* const colp = b_hi + (t >> 5) * 4096 + (t & 7) * 4;
#pragma unroll
                    for (int e = 0; e < 32; ++e) {
                        float hi, lo;
                        tc_split(bv[e], hi, lo);
                        const uint32_t off = (uint32_t)(e * 128 + ((((t & 31) >> 3) ^ (e & 3)) << 5));
                        *reinterpret_cast<float*>(colp + off) = hi;
                        *reinterpret_cast<float*>(colp + kBtBTile + off) = lo;
                    }
                }
                // the slice of A: zeros, then the band
#pragma unroll
                for (int u = 0; u < 2 * kBtATile / (16 * kBtProducerWarps * 32); ++u)
                    *reinterpret_cast<float4*>(a_hi + (size_t)(u * kBtProducerWarps * 32 + t) * 16) =
                        make_float4(0.f, 0.f, 0.f, 0.f);
                if (p.tma_b) {  // the block of B has landed (every warp's lane 0 looks for itself)
                    if (lane == 0) ok = bt_wait(raw(st), use & 1, abort_flag, p.err_word);
                    ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
                }
            }
            if (bt_producer_sync_any(!ok, grp)) break;  // a wait ran out somewhere: all eight warps stop here
            {
                // segment u lands in row r0 - 8u, column lane of the K block: eight rows up is 1024 bytes back
                const int d0 = (32 * kb - (kBtRows - 1) > 0 ? 32 * kb - (kBtRows - 1) : 0) + pw;
                const int d_hi = (int)(32 * (int64_t)kb + 31 < 2 * w ? 32 * (int64_t)kb + 31 : 2 * w);
                const int r0 = 32 * kb - d0 + lane;
                const int off0 = (r0 >> 3) * 1024 + (r0 & 7) * 128 + (((lane >> 2) ^ (r0 & 7)) << 4) + (lane & 3) * 4;
#pragma unroll
                for (int u = 0; u < kBtSegs; ++u) {
                    const int r = r0 - 8 * u;
                    if (d0 + 8 * u <= d_hi && r >= 0 && r < kBtRows) {
                        float hi, lo;
                        tc_split(av[u], hi, lo);
                        *reinterpret_cast<float*>(a_hi + off0 - 1024 * u) = hi;
                        *reinterpret_cast<float*>(a_hi + kBtATile + off0 - 1024 * u) = lo;
                    }
                }
            }
            if (p.tma_b) {
                // low parts of the block: same layout, element by element
                constexpr int kPer = kBtBTile / (16 * kBtProducerWarps * 32);
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    float4 v[kPer / 2];  // loads first: the stores below must not wait on them one by one
#pragma unroll
                    for (int u = 0; u < kPer / 2; ++u)
                        v[u] = *reinterpret_cast<const float4*>(b_hi + (size_t)((half * (kPer / 2) + u) * kBtProducerWarps * 32 + t) * 16);
#pragma unroll
                    for (int u = 0; u < kPer / 2; ++u) {
                        float4 h, l;
                        tc_split(v[u].x, h.x, l.x), tc_split(v[u].y, h.y, l.y), tc_split(v[u].z, h.z, l.z), tc_split(v[u].w, h.w, l.w);
                        *reinterpret_cast<float4*>(b_hi + kBtBTile + (size_t)((half * (kPer / 2) + u) * kBtProducerWarps * 32 + t) * 16) = l;
                    }
                }
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) tc_mbar_arrive(full(st));
            ++use;
            next_item();
            next_item();
            if (valid) load_item();
        }
    }
    else if (warp == kBtWarpMma) {
        // ---- MMA issuer: one thread ----
        if (lane == 0) {
            constexpr uint32_t kIdesc = tc_idesc_mn(kBtRows, kBtCols) | (1u << 16);  // B operand N-major
            uint32_t it = 0, tile_n = 0;
            bool ok = true;
            for (int round = 0; round < rounds && ok; ++round) {
                const int q = tile_of(round);
                if (q >= p.tiles) break;
                const int64_t i0 = (int64_t)(q / p.col_tiles) * kBtRows;
                int kb_lo, kb_hi;
                bt_k_range(p, i0, kb_lo, kb_hi);
                const int acc = tile_n & 1;
                const uint32_t use = tile_n >> 1;  // earlier uses of this accumulator
                if (use >= 1 && !bt_wait(tmem_empty(acc), (use - 1) & 1, abort_flag, p.err_word)) {
                    ok = false;
                    break;
                }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t d_tmem = tmem_base + acc * kBtCols;
                for (int kb = kb_lo; kb < kb_hi; ++kb, ++it) {
                    const int st = it % S;
                    if (!bt_wait(full(st), (it / S) & 1, abort_flag, p.err_word)) {
                        ok = false;
                        break;
                    }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t a_hi = tc_smem(smem + (size_t)st * kBtStageBytes);
                    const uint32_t a_lo = a_hi + kBtATile;
                    const uint32_t b_hi = a_hi + 2 * kBtATile;
                    const uint32_t b_lo = b_hi + kBtBTile;
#pragma unroll
                    for (int k8 = 0; k8 < 4; ++k8) {
                        tc_mma_tf32(d_tmem, tc_desc(a_hi + k8 * 32), bt_desc_b(b_hi + k8 * 1024), kIdesc,
                                    (kb > kb_lo || k8 > 0) ? 1u : 0u);
                        tc_mma_tf32(d_tmem, tc_desc(a_hi + k8 * 32), bt_desc_b(b_lo + k8 * 1024), kIdesc, 1u);
                        tc_mma_tf32(d_tmem, tc_desc(a_lo + k8 * 32), bt_desc_b(b_hi + k8 * 1024), kIdesc, 1u);
                    }
                    tc_commit(empty(st));
                }
                if (ok) tc_commit(tmem_full(acc));
                ++tile_n;
            }
        }
    } else {
        // ---- epilogue: warp = (lane quarter of tensor memory, column half); thread = row ----
        const int quarter = warp & 3, half = warp >> 2;
        uint32_t tile_n = 0, chunk_n = 0;
        for (int round = 0; round < rounds; ++round) {
            const int q = tile_of(round);
            if (q >= p.tiles) break;
            const int64_t i0 = (int64_t)(q / p.col_tiles) * kBtRows;
            const int64_t cb = (int64_t)(q % p.col_tiles) * kBtCols + half * kBtEpiCols;
            const int acc = tile_n & 1;
            const uint32_t use = tile_n >> 1;
            int got = 1;
            if (lane == 0) got = bt_wait(tmem_full(acc), use & 1, abort_flag, p.err_word) ? 1 : 0;
            got = __shfl_sync(0xffffffffu, got, 0);
            if (!got) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const int64_t i = i0 + quarter * 32 + lane;
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * kBtCols + half * kBtEpiCols;
            float* crow = p.C + i * p.ldc + cb;
            if (p.tma_c) {
                // A 32 x 32 chunk goes to one of the warp's two buffers (rows of 128 bytes, 16-byte
                // pieces swizzled like the tensor map's 128-byte mode, so the lanes' stores spread
                // over the banks) and leaves by one bulk tensor store, or reduce-add when
                // accumulating; rows and columns outside C are clipped by the copy.
#pragma unroll 1
                for (int cc = 0; cc < kBtEpiCols / 32; ++cc, ++chunk_n) {
                    uint8_t* const buf = epi0 + (size_t)(warp * 2 + (chunk_n & 1)) * kBtEpiBufBytes;
                    if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");  // its last store has read it
                    __syncwarp();
                    uint32_t r[32];
                    tc_ld32(taddr + cc * 32, r);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                    for (int v = 0; v < 8; ++v)
                        *reinterpret_cast<float4*>(buf + lane * 128 + ((v ^ (lane & 7)) << 4)) =
                            make_float4(__uint_as_float(r[4 * v]), __uint_as_float(r[4 * v + 1]),
                                        __uint_as_float(r[4 * v + 2]), __uint_as_float(r[4 * v + 3]));
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    const int64_t col0 = cb + cc * 32, row0 = i0 + quarter * 32;
                    if (lane == 0 && col0 < p.ncols && row0 < N) {
                        if (p.accumulate)
                            asm volatile(
                                "cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%1, %2}], [%3];"
                                ::"l"(&tmap_c), "r"((int)col0), "r"((int)row0), "r"(tc_smem(buf))
                                : "memory");
                        else
                            asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%1, %2}], [%3];"
                                         ::"l"(&tmap_c), "r"((int)col0), "r"((int)row0), "r"(tc_smem(buf))
                                         : "memory");
                    }
                    if (lane == 0) asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                }
            } else {
#pragma unroll 1
            for (int cc = 0; cc < kBtEpiCols / 32; ++cc) {
                uint32_t r[32];
                tc_ld32(taddr + cc * 32, r);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                const int64_t col0 = cb + cc * 32;
                if (i < N) {
                    if (p.vec_c && col0 + 32 <= p.ncols) {
                        float4* dst = reinterpret_cast<float4*>(crow + cc * 32);
#pragma unroll
                        for (int v = 0; v < 8; ++v) {
                            float4 o = make_float4(__uint_as_float(r[4 * v]), __uint_as_float(r[4 * v + 1]),
                                                   __uint_as_float(r[4 * v + 2]), __uint_as_float(r[4 * v + 3]));
                            if (p.accumulate) {
                                const float4 old = dst[v];
                                o.x += old.x, o.y += old.y, o.z += old.z, o.w += old.w;
                            }
                            dst[v] = o;
                        }
                    } else {
#pragma unroll
                        for (int v = 0; v < 32; ++v)
                            if (col0 + v < p.ncols) {
                                float o = __uint_as_float(r[v]);
                                if (p.accumulate) o += crow[cc * 32 + v];
                                crow[cc * 32 + v] = o;
                            }
                    }
                }
            }
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) tc_mbar_arrive(tmem_empty(acc));  // the accumulator may be overwritten
            ++tile_n;
        }
        // shared memory stays allocated until the bulk stores have read it and written C
        if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)kBtTmemCols) : "memory");
    }
}

typedef CUresult (*BtEncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                    const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                    CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

BtEncodeTiledFn bt_encode_fn() {
    static BtEncodeTiledFn fn = nullptr;
    if (!fn) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = (BtEncodeTiledFn)ptr;
    }
    return fn;
}

}  // namespace
}  // namespace dastac

using namespace dastac;

extern "C" dastac_status dastac_bandmm_split_tf32(const dastac_structure* s, const float* A, const float* B, int64_t ldb,
                                                  float* C, int64_t ldc, int64_t ncols, int32_t accumulate,
                                                  int32_t* err_word, void* stream) {
    if (!s) return DASTAC_ERR_INVALID_ARG;
    const IndexMap& m = s->map;
    if (m.kind == kEmpty) return DASTAC_OK;
    if (m.kind != kBandDiagonals && m.kind != kBandExact) return DASTAC_ERR_UNSUPPORTED_EXPR;
    const int64_t N = m.N;
    if (ncols < 0) return DASTAC_ERR_INVALID_ARG;
    if (N == 0 || ncols == 0) return DASTAC_OK;
    if (!A || !B || !C || ldb < ncols || ldc < ncols) return DASTAC_ERR_INVALID_ARG;
    // window rows and diagonals are counted in 32-bit integers inside the kernel
    if (m.w > (int64_t)1 << 24 || N > (int64_t)1 << 40) return DASTAC_ERR_OVERFLOW;
    BtParams p;
    p.A = A, p.B = B, p.C = C;
    p.N = N, p.w = m.w, p.ldb = ldb, p.ldc = ldc, p.ncols = ncols;
    const int64_t row_tiles = (N + kBtRows - 1) / kBtRows, col_tiles = (ncols + kBtCols - 1) / kBtCols;
    if (row_tiles * col_tiles > 0x7fffffffLL) return DASTAC_ERR_OVERFLOW;
    p.row_tiles = (int32_t)row_tiles, p.col_tiles = (int32_t)col_tiles, p.tiles = (int32_t)(row_tiles * col_tiles);
    p.exact = m.kind == kBandExact;
    p.accumulate = accumulate;
    p.vec_c = ((ldc & 3) == 0) && aligned16(C);
    p.err_word = err_word;
    // C as a 2-D tensor of 32 x 32 boxes in the 128-byte swizzle, when its rows are 16-byte aligned
    CUtensorMap tmap_c;
    std::memset(&tmap_c, 0, sizeof(tmap_c));
    p.tma_c = 0;
    if (p.vec_c && N < ((int64_t)1 << 31) && ncols < ((int64_t)1 << 31)) {
        BtEncodeTiledFn enc = bt_encode_fn();
        if (!enc) return DASTAC_ERR_CUDA;
        const cuuint64_t dims[2] = {(cuuint64_t)ncols, (cuuint64_t)N};
        const cuuint64_t strides[1] = {(cuuint64_t)ldc * 4};
        const cuuint32_t box[2] = {32, 32};
        const cuuint32_t estr[2] = {1, 1};
        if (enc(&tmap_c, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, C, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return DASTAC_ERR_CUDA;
        p.tma_c = 1;
    }
    // B as a 2-D tensor of 32 x 32 boxes, 32-byte pieces swizzled within 128 bytes, under the same conditions
    CUtensorMap tmap_b;
    std::memset(&tmap_b, 0, sizeof(tmap_b));
    p.tma_b = 0;
    if ((ldb & 3) == 0 && aligned16(B) && N < ((int64_t)1 << 31) && ncols < ((int64_t)1 << 31)) {
        BtEncodeTiledFn enc = bt_encode_fn();
        if (!enc) return DASTAC_ERR_CUDA;
        const cuuint64_t dims[2] = {(cuuint64_t)ncols, (cuuint64_t)N};
        const cuuint64_t strides[1] = {(cuuint64_t)ldb * 4};
        const cuuint32_t box[2] = {32, 32};
        const cuuint32_t estr[2] = {1, 1};
        if (enc(&tmap_b, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(B), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return DASTAC_ERR_CUDA;
        p.tma_b = 1;
    }
    static bool attr_set[64];
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        if (cudaFuncSetAttribute(bandmm_tc_kernel<10>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kBtSmemBytes) != cudaSuccess ||
            cudaFuncSetAttribute(bandmm_tc_kernel<20>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kBtSmemBytes) != cudaSuccess)
            return DASTAC_ERR_CUDA;
        attr_set[dev] = true;
    }
    int grid = sm_count();
    if (grid > p.tiles) grid = p.tiles;
    if (2 * m.w + 1 <= 80)
        bandmm_tc_kernel<10><<<grid, kBtThreads, kBtSmemBytes, (cudaStream_t)stream>>>(tmap_b, tmap_c, p);
    else
        bandmm_tc_kernel<20><<<grid, kBtThreads, kBtSmemBytes, (cudaStream_t)stream>>>(tmap_b, tmap_c, p);
    return launch_status();
}
