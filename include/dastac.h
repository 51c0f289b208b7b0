/*
 * dastac.h - structured tensor algebra on densely packed layouts, CUDA (sm_100a) library, C ABI.
 *
 * A tensor whose nonzero, non-redundant region is a polyhedron is stored as a packed vector: the
 * position of a logical index is the number of points of the region that precede it in
 * lexicographic order, computed from a closed-form ranking polynomial in registers, with no index
 * arrays in memory.  Contractions read the packed operands directly.
 *
 * General conventions
 *   - Every function returns a dastac_status; nothing throws or aborts across this boundary.
 *     Argument errors are detected before any device work is enqueued.
 *   - Device work is only enqueued on `stream` (a cudaStream_t passed as void*, NULL = default
 *     stream); no call synchronises unless stated.  The current CUDA device must be the one that
 *     owns the buffers.
 *   - The caller owns every buffer.  Pointers are device pointers unless marked "host".  The
 *     library allocates no device memory; scratch space is passed in as `workspace`.
 *   - Indices are int32 per dimension (extents up to 2^30); packed positions are int64.
 *   - Dense operands are described by element strides; packed operands are contiguous.
 *   - State kept by the library in the calling process, none of it visible in results: a launch
 *     counter (dastac_launch_count), per-device caches of attribute set-up and of work partitions,
 *     and, on every GPU that loads it, one device error word (dastac_device_error) and the
 *     scratch array of dastac_trimm_bf16_noalloc.
 *   - fp32 arithmetic flushes subnormal inputs and results to zero (the kernels are compiled
 *     that way); pack and unpack copy bits and are not affected.
 *   - Packed buffers must be 16-byte aligned and have a capacity of `slots` elements as reported
 *     by dastac_structure_count (the point count rounded up to a multiple of 16 bytes); the
 *     library never reads element values beyond `count` into a result, but it may load the
 *     padding bytes.
 */
#ifndef DASTAC_H_
#define DASTAC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    DASTAC_OK = 0,
    DASTAC_ERR_INVALID_ARG = 1,           /* NULL pointer, negative size, malformed descriptor     */
    DASTAC_ERR_UNSUPPORTED_STRUCTURE = 2, /* descriptor is valid but is not a recognised class     */
    DASTAC_ERR_UNSUPPORTED_EXPR = 3,      /* expression x structure x dtype has no kernel          */
    DASTAC_ERR_SHAPE = 4,                 /* operand extents disagree                              */
    DASTAC_ERR_ALIGNMENT = 5,             /* a data pointer is not 16-byte aligned                 */
    DASTAC_ERR_OVERFLOW = 6,              /* an extent exceeds 2^30 or a count exceeds 2^62        */
    DASTAC_ERR_WORKSPACE = 7,             /* workspace missing, misaligned or too small            */
    DASTAC_ERR_CUDA = 8,                  /* a CUDA runtime/driver call failed                     */
    DASTAC_ERR_TIMEOUT = 9                /* a bounded device-side wait expired (dastac_device_error) */
} dastac_status;

typedef enum { DASTAC_F32 = 0, DASTAC_BF16 = 1 } dastac_dtype;
typedef enum { DASTAC_MEM_DEVICE = 0, DASTAC_MEM_HOST = 1 } dastac_memspace;

/* Recognised structure classes (result of descriptor analysis). */
typedef enum {
    DASTAC_KIND_EMPTY = 0,
    DASTAC_KIND_DENSE = 1,          /* the whole box, row-major                                    */
    DASTAC_KIND_UPPER = 2,          /* 0<=i<M, i<=j<N, optional trailing dense extent Q (rank 3)   */
    DASTAC_KIND_LOWER = 3,          /* 0<=j<=i<N                                                   */
    DASTAC_KIND_BAND_DIAGONALS = 4, /* |i-j|<=w stored as 2w+1 diagonals of N slots                */
    DASTAC_KIND_TETRAHEDRON = 5,    /* 0<=i<=j<=k<n                                                */
    DASTAC_KIND_BAND_EXACT = 6,     /* |i-j|<=w, 2w+1<=N, rows packed back to back (no padding)    */
    DASTAC_KIND_UPPER_SHIFTED = 7,  /* j-i>=c, c>=1, square: the size N-c triangle in the top right corner
                                       (the sub-triangular structure of Section 6.4)               */
    DASTAC_KIND_BAND_OFFSETS = 8,   /* lo<=j-i<=hi, square, any lo<=hi: rows packed back to back.  One
                                       off-diagonal (lo=hi=s) is a per-summand buffer of the strided band
                                       of Section 6.4; chosen when no class above applies           */
    DASTAC_KIND_PLANE = 9,          /* one index fixed (idx_a = c) or equal to an earlier one (idx_b = idx_a),
                                       everything else dense: "Fixed i", "Fixed j", "Diagonal (plane)" of
                                       Table 1; packed as the dense box over the free indices        */
    DASTAC_KIND_GENERIC = 10        /* any other conjunction of affine comparisons (rank 2 or 3, unit
                                       coefficients on the inner indices) whose counting function the
                                       library could fit when the structure was created: index maps, pack
                                       and unpack only, through slower element-wise kernels           */
} dastac_kind;

#define DASTAC_LAYOUT_LEXICOGRAPHIC 0 /* exact pack in lexicographic order                         */
#define DASTAC_LAYOUT_PADDED_DIAGONALS 1 /* band only: diagonal-major, N slots per diagonal        */

/*
 * Structure descriptor: the unique set of a tensor as a conjunction of affine comparisons over the
 * indices and size symbols (paper Section 2, "Unique set"; Section 4, "Iteration space
 * extraction"), an optional redundancy map (Section 2, "Redundancy map") and the requested layout.
 *
 *   rows    host, nrows x (rank + nparams + 1), row-major.  Row r states
 *             sum_k rows[r][k]*idx[k] + sum_p rows[r][rank+p]*params[p] + rows[r][rank+nparams] >= 0
 *           or "== 0" when is_eq[r] != 0.  The box 0 <= idx[k] < dims[k] is always implied.
 *   mirror  host, NULL or a permutation of 0..rank-1: the redundant point (idx[mirror[0]], ...)
 *           holds the same value as idx.  Only the swap {1,0} on a square upper triangle (a
 *           symmetric matrix stored as its upper part) is supported.
 *   layout  DASTAC_LAYOUT_*.
 * All arrays are read during dastac_structure_create only.
 */
typedef struct {
    int32_t rank;     /* 1..3 */
    int32_t nparams;  /* 0..8 */
    int32_t nrows;    /* 0..64 */
    const int64_t* dims;
    const int64_t* rows;
    const uint8_t* is_eq;
    const int64_t* params;
    const int32_t* mirror;
    int32_t layout;
} dastac_structure_desc;

/* Immutable host object: recognised class plus the coefficients of its ranking polynomial. */
typedef struct dastac_structure dastac_structure;

/*
 * Analyse a descriptor (Algorithm 1, "Symbolic Indexing").  The comparisons are normalised to
 * difference bounds, closed under implication, and matched against the classes whose counting
 * polynomial is known in closed form, so redundant or re-ordered rows do not matter.
 * A set that is none of those classes (or has rows that are not difference bounds, such as
 * i + j <= N - 1 or 2 i <= j) gets DASTAC_KIND_GENERIC when it can: the library counts every slab
 * of the set by brute force, fits the piecewise polynomial "points before slab i" to those counts
 * (the stand-in for the symbolic counting step of Algorithm 1), fuses pieces that agree
 * (Algorithm 2) and verifies the map.  Conditions: lexicographic layout, no redundancy map, rank 2
 * or 3, coefficients -1, 0 or 1 on the last index (rank 3: on the last two), extents up to 2^20
 * and at most 2^24 slabs (rank 2) or fibres (rank 3), at most 12 polynomial pieces; creation
 * costs time proportional to the number of fibres.
 * Errors: INVALID_ARG, OVERFLOW, UNSUPPORTED_STRUCTURE (none of the above applies).
 */
dastac_status dastac_structure_create(const dastac_structure_desc* desc, dastac_structure** out);
void dastac_structure_destroy(dastac_structure* s);

/* slots = elements a packed buffer must hold (count, or (2w+1)*N for padded diagonals; the
 * buffer capacity must be slots rounded up to 16 bytes); nnz = points of the set. */
dastac_status dastac_structure_count(const dastac_structure* s, int64_t* slots, int64_t* nnz);
/* kind = dastac_kind; symmetric = 1 if a redundancy swap is attached. */
dastac_status dastac_structure_kind(const dastac_structure* s, int32_t* kind, int32_t* symmetric);

/*
 * Ranking polynomial P(idx) = number of preceding points (Section 4, "Access domain
 * linearization"), evaluated in exact 64-bit integer arithmetic with a single final division
 * (Section 3, figure of the generated loop nest).  Host versions; idx and the result are host
 * pointers.  dastac_rank returns INVALID_ARG for a point outside the set.  dastac_unrank is the
 * inverse; for a padding slot of the padded-diagonal layout it sets the column to -1.
 */
dastac_status dastac_rank(const dastac_structure* s, const int32_t* idx, int64_t* off);
dastac_status dastac_unrank(const dastac_structure* s, int64_t off, int32_t* idx);

/*
 * Device versions over n points: idx is n x rank int32 (device), off is n int64 (device).  A point
 * outside the set ranks to -1.  These run the same in-register maps the kernels use.
 */
dastac_status dastac_rank_batch(const dastac_structure* s, const int32_t* idx, int64_t n,
                                int64_t* off, void* stream);
dastac_status dastac_unrank_batch(const dastac_structure* s, const int64_t* off, int64_t n,
                                  int32_t* idx, void* stream);

/*
 * Compress / decompress (Section 3, "Data Layout Compression": copy over the accessed indices).
 *   pack    packed[P(idx)] = dense[idx] for every point of the set; padded-diagonal padding
 *           slots receive +0.  Bit-exact copy.
 *   unpack  dense = 0 everywhere in the box, then dense[idx] = packed[P(idx)]; with a redundancy
 *           swap the mirrored element receives the same bits.  Padding slots are ignored.
 * dense_strides: host array of `rank` element strides of the dense tensor.
 * The row-wise kernels fetch windows of a row by bulk copies and wait for them with a budget; a
 * wait that runs out (never expected) leaves the rest of the launch's output unwritten and sets
 * the device error word, which dastac_device_error reports as DASTAC_ERR_TIMEOUT.
 */
dastac_status dastac_pack(const dastac_structure* s, dastac_dtype dtype, const void* dense,
                          const int64_t* dense_strides, void* packed, void* stream);
dastac_status dastac_unpack(const dastac_structure* s, dastac_dtype dtype, const void* packed,
                            void* dense, const int64_t* dense_strides, void* stream);

/*
 * Contraction operand.
 *   structure == NULL: dense tensor, `rank` extents in dims, element strides in strides.
 *   structure != NULL: packed tensor of that structure (dims/strides ignored except that
 *                      batch instances are batch_stride elements apart).  Outputs are dense except
 *                      where the table of dastac_contract says otherwise.
 *   space: where `data` lives.  Host operands are staged through the workspace with asynchronous
 *          copies on `stream` (pinned memory recommended); a host output is valid after the
 *          caller synchronises the stream.
 *   batch: number of independent instances sharing the structure (0 or 1 = single).  Dense
 *          operands of a batched call are batch_stride elements apart as well.
 */
typedef struct {
    void* data;
    int32_t dtype; /* dastac_dtype */
    int32_t space; /* dastac_memspace */
    const dastac_structure* structure;
    int32_t rank;
    int32_t batch;
    int64_t batch_stride;
    int64_t dims[4];
    int64_t strides[4];
} dastac_operand;

/*
 * Evaluate a sum-of-products rule (Section 3, "Input"; Table 1) whose first operand is packed
 * (the last two rules of the table have dense inputs and pack their output instead).
 * Supported (expression, structure of in[0], dtypes):
 *   "ij,j->i"       upper triangle (square)             f32        y = A x         (batched)
 *   "ij,j->i"       upper triangle + swap (symmetric)   f32        y = S x
 *   "ij,j->i"       dense box, trapezoid, lower         f32        y = A x         (batched); rows without a
 *                   triangle, exact band, offset band,                stored element give 0.  A rule with
 *                   single stored row
 *                   several summands (strided band: three diagonals; Leslie matrix: first row +
 *                   sub-diagonal) is evaluated summand by summand, each with its own packed buffer
 *                   (Section 4, one buffer per summand), the later calls with accumulate = 1
 *   "ij,j->i"       sub-triangle j - i >= c             f32        y = A x         (batched); rows N-c .. N-1 of
 *                   y have no stored element and are set to 0 (left unchanged when accumulating)
 *   "ij,jc->ic"     band, padded diagonals or exact     f32        C = A B
 *   "ij,jc->ic"     dense box, trapezoid, lower         f32        C = A B for the other row-contiguous classes
 *                   triangle, offset band, single row                 (row-wise kernel, slower than the band's)
 *   "ij,jc->ic"     upper triangle (square)             bf16 -> f32 output, fp32 accumulation
 *   "ijk,jr,kr->ir" tetrahedron                         f32        M = T x_2 B x_3 C (MTTKRP)
 *   "ijk,jr,kr->ir" dense box, upper half cube, plane   f32        the same rule over the other rank-3 structures
 *                   with a free trailing index                         whose fibres (i, j, :) are contiguous (slower kernel)
 *   "ijl,kl->ijk"   upper half cube (i <= j, dense l)   f32        A = B x_3 C (tensor times matrix, the
 *                   running example of Section 3); `out` is PACKED too: out->structure must be the
 *                   upper half cube with the same first two extents and trailing extent K = rows of C.
 *                   The same rule runs on the plane structures whose trailing index is dense
 *                   (i = j, fixed i, fixed j: TTM_DP, TTM_J of Table 1), `out` being the same plane
 *   "ij,ij->ij"     any structure (also "i,i->i",       f32        A = B o C, the tensor Hadamard product (Table 1,
 *                   "ijk,ijk->ijk" by rank)                            THP) of a packed structured B and a dense C of the
 *                   same box; `out` is PACKED with the same structure as B (a structure created from the
 *                   same descriptor): out[P(idx)] = B[P(idx)] * C[idx]
 *   "xi,xj->ij"     in[0] = in[1] = dense B (M x n)     bf16 -> f32  A2 = B^T B, the degree-2 moments of
 *                   polynomial regression (Table 1, A^k(i_1..i_k) := B(x,i_1) ... B(x,i_k), k = 2).  This
 *                   rule has no packed input: both inputs must be the same dense tensor (same data,
 *                   extents and strides, unit stride along i) and `out` is PACKED: out->structure is the
 *                   n x n upper triangle (the unique part i <= j of the symmetric result, Section 2;
 *                   with or without the redundancy swap), fp32 accumulation.  Positions of the packed
 *                   buffer beyond the set's count are not written.
 *   "xi,xj,xk->ijk" in[0] = in[1] = in[2] = dense B     bf16 -> f32  A3, the degree-3 moments (k = 3 of the same
 *                   rule); `out` is PACKED: out->structure is the n x n x n tetrahedron i <= j <= k (the
 *                   hyper-triangular domain of Section 1).  The pairwise products B(x,i) B(x,j) are
 *                   rounded to bf16 once before they meet the third factor on the tensor cores
 *                   (relative error 2^-9 per term); accumulation is fp32.  Needs workspace (a transposed
 *                   copy of B).
 * accumulate: 0 -> out = result (the library zero-fills where it needs to), 1 -> out += result.
 * workspace: device scratch of at least dastac_contract_workspace bytes, 256-byte aligned; may be
 *            NULL when that size is 0.  Its contents are undefined afterwards.
 * err_word: optional device int32; a kernel whose bounded wait expires stores a non-zero code
 *           there and drains instead of hanging.  The caller zeroes and reads it.
 * Floating-point sums are re-associated freely (the paper generates fast-math code), so results
 * agree with a reference to rounding, not bit for bit.
 */
dastac_status dastac_contract_workspace(const char* expr, const dastac_operand* in, int32_t n_in,
                                        const dastac_operand* out, size_t* bytes);
dastac_status dastac_contract(const char* expr, const dastac_operand* in, int32_t n_in,
                              const dastac_operand* out, int32_t accumulate, void* workspace,
                              size_t workspace_bytes, int32_t* err_word, void* stream);

const char* dastac_status_string(dastac_status st);

/*
 * The bf16 triangular x dense contraction ("ij,jc->ic", upper triangle, bf16 -> f32) without any
 * workspace argument and without any memory allocation.  The paper has no counterpart: this entry
 * point exists for callers that must not, or cannot, obtain device memory around the call - code
 * running inside a region where allocation is forbidden (a real-time loop, a callback that holds a
 * lock the allocator also takes, a process whose memory pool was handed out in full at start-up).
 * dastac_contract needs about N*N bytes of caller-provided scratch for this expression; here that
 * scratch is a fixed array inside the library image, DASTAC_NOALLOC_SCRATCH_BYTES per GPU that
 * loads the library, held until the process exits.
 *
 *   s        square upper triangle, N <= DASTAC_NOALLOC_MAX_N; larger N returns DASTAC_ERR_WORKSPACE
 *   A        device, packed bf16 rows of s (capacity as for every packed buffer), 16-byte aligned
 *   B        device, N x ncols bf16, row pitch ldb elements; ldb must be a multiple of 8 (a pitch
 *            that is not a multiple of 16 bytes returns DASTAC_ERR_ALIGNMENT), 16-byte aligned
 *   C        device, N x ncols f32, row pitch ldc elements, 16-byte aligned
 *   accumulate, err_word, stream   as for dastac_contract
 *
 * Results are those of dastac_contract on the same operands.  The call itself calls no cudaMalloc,
 * cudaFree or other allocating routine.  The first call on a device looks up the array's device
 * address (cudaGetSymbolAddress); make that first call before starting any stream capture.
 * Every call on a device uses the same array and rewrites all of it that it needs, so nothing has
 * to be cleared between calls, but two calls whose kernels may run at the same time (different
 * streams, or different host threads on different streams) race on it: serialise them.
 */
#define DASTAC_NOALLOC_MAX_N 2048
#define DASTAC_NOALLOC_SCRATCH_BYTES (288 * 16384)
dastac_status dastac_trimm_bf16_noalloc(const dastac_structure* s, const void* A, const void* B,
                                        int64_t ldb, int64_t ncols, float* C, int64_t ldc,
                                        int32_t accumulate, int32_t* err_word, void* stream);

/*
 * Split-precision tensor-core form of the tetrahedral MTTKRP (opt-in; dastac_contract keeps the
 * plain fp32 multiply-add kernel).  The same rule M(i,r) = sum_{i<=j<=k} T(i,j,k) B(j,r) C(k,r)
 * (Table 1 "MTTKRP" over the hyper-triangular domain of Section 1) with the product T_i C of
 * every slab evaluated on the tensor cores in TF32: each fp32 value is split into a high and a
 * low part and the three products hi*hi, hi*lo, lo*hi are accumulated in fp32, which keeps the
 * error per product near 2^-21 (a single TF32 pass would be 2^-11); the multiplication by B and
 * the sum over j are fp32.  Results agree with dastac_contract's within the same 1e-5 bound.
 *   s         tetrahedron, n <= 512 (the factor C is kept in shared memory as hi / lo tiles);
 *             anything else returns DASTAC_ERR_UNSUPPORTED_EXPR
 *   T         device, packed fp32 tensor of s, 16-byte aligned
 *   B, C      device, n x R fp32, row pitches ldb, ldc elements; R <= 32
 *   M         device, n x R fp32, row pitch ldm; accumulate as for dastac_contract
 *   err_word  optional device int32, set when a bounded wait inside the kernel expires
 * Needs no workspace.
 */
dastac_status dastac_mttkrp_split_tf32(const dastac_structure* s, const float* T, const float* B, int64_t ldb,
                                       const float* C, int64_t ldc, float* M, int64_t ldm, int64_t R,
                                       int32_t accumulate, int32_t* err_word, void* stream);

/*
 * Split-precision tensor-core form of band x dense (opt-in; dastac_contract keeps the plain fp32
 * multiply-add kernel).  C = A B (or C += A B) for a band |i - j| <= w (Section 1, the banded
 * motivation; Section 6.4): a tile of 128 rows of C is the dense product of the 128 x (128 + 2w)
 * slice of A that holds its band with the B rows i0-w .. i0+127+w, taken on the tensor cores in
 * TF32 with both operands split into a high and a low part and the three products hi*hi, hi*lo,
 * lo*hi accumulated in fp32 (about 2^-21 per product).  Results agree with dastac_contract's
 * within the same 1e-5 bound.  Padding slots of the diagonal layout are never read.
 *   s         band as padded diagonals or packed exactly; anything else returns
 *             DASTAC_ERR_UNSUPPORTED_EXPR
 *   A         device, packed fp32 values of s (no alignment requirement)
 *   B         device, N x ncols fp32, row pitch ldb elements (no alignment requirement)
 *   C         device, N x ncols fp32, row pitch ldc elements; 128-bit stores when C is 16-byte
 *             aligned and ldc is a multiple of 4, scalar stores otherwise
 *   accumulate, stream   as for dastac_contract
 *   err_word  optional device int32, set when a bounded wait inside the kernel expires
 * Needs no workspace.  Unlike dastac_contract, which visits the band only, a row of B meets every
 * row of the 128-row tile whose window holds it, with a zero factor outside the band: an infinity
 * or NaN in B therefore reaches rows of C that the band does not connect it to.
 */
dastac_status dastac_bandmm_split_tf32(const dastac_structure* s, const float* A, const float* B, int64_t ldb,
                                       float* C, int64_t ldc, int64_t ncols, int32_t accumulate,
                                       int32_t* err_word, void* stream);

/*
 * Split-precision tensor-core form of tensor times matrix with packed input and output (opt-in;
 * dastac_contract keeps the plain fp32 multiply-add kernel).  A(i,j,k) = sum_l B(i,j,l) C(k,l) (the
 * running example of Section 3) over a rank-3 structure whose trailing index is dense: in packed
 * form the rule is the dense product Y[p][k] = sum_l X[p][l] C[k][l] of the packed input, viewed as
 * a [count / Q][Q] matrix, with C.  It is taken on the tensor cores in TF32 with both operands
 * split into a high and a low part and the three products hi*hi, hi*lo, lo*hi accumulated in fp32
 * (about 2^-21 per product); results agree with dastac_contract's within the same 1e-5 bound.
 *   s         rank-3 structure with a dense trailing index of extent Q (upper half cube, dense
 *             box, planes with a free last index); anything else returns DASTAC_ERR_UNSUPPORTED_EXPR,
 *             as does Q > 256
 *   X         device, packed fp32 values of s, 16-byte aligned, Q a multiple of 4
 *             (DASTAC_ERR_ALIGNMENT otherwise: a packed row must be a row of a tensor map)
 *   C         device, K x Q fp32, row pitch ldc elements
 *   Y         device, packed fp32 output over the same leading index set with trailing extent K
 *             (count / Q * K values); bulk tensor stores when Y is 16-byte aligned and K is a
 *             multiple of 4, plain stores otherwise
 *   accumulate, stream   as for dastac_contract
 *   err_word  optional device int32, set when a bounded wait inside the kernel expires
 * Needs no workspace.
 */
dastac_status dastac_ttm_split_tf32(const dastac_structure* s, const float* X, const float* C, int64_t ldc,
                                    int64_t K, float* Y, int32_t accumulate, int32_t* err_word, void* stream);

/*
 * A structured operand given as several summands (Section 4: the method works on the individual
 * summands of a rule; every summand's region has its own compressed buffer, and a summand whose
 * region equals an earlier one reuses that buffer instead of getting a second copy).  Examples:
 * the strided band of Section 6.4 (three diagonals), the Leslie matrix of Table 1 (first row and
 * sub-diagonal).
 *   dastac_rule_create   one structure per summand descriptor (each as for
 *                        dastac_structure_create, all over the same box) and the buffer index of
 *                        each; summands with equal regions get the same index.  n = 1..64.
 *   dastac_rule_size     number of summands and of distinct buffers.
 *   dastac_rule_summand  structure (owned by the rule) and buffer index of summand k.
 *   dastac_rule_pack     fills every distinct buffer from the dense tensor: `packed` is a host
 *                        array of n_buffers device pointers, buffer b sized and aligned for the
 *                        structure of the first summand that uses it.
 *   dastac_rule_contract the rule `expr` with the summed operand in first place:
 *                        out = sum_k contract(expr, summand k, rest...), enqueued in one call; the
 *                        first summand overwrites `out` (adds to it when accumulate != 0), the
 *                        others add.  `rest` holds the remaining inputs (in[1..] of
 *                        dastac_contract), `packed` the device buffers as for dastac_rule_pack,
 *                        `packed_batch_strides` (host, may be NULL) their batch strides.  Every
 *                        summand must be a supported (expression, structure) pair; all are
 *                        checked before anything is enqueued.  Workspace: the largest need of any
 *                        summand (dastac_rule_contract_workspace).
 * Regions of different summands that overlap without being equal are stored twice and counted
 * twice, as the summed rule says.
 */
typedef struct dastac_rule dastac_rule;
dastac_status dastac_rule_create(const dastac_structure_desc* summands, int32_t n, dastac_rule** out);
void dastac_rule_destroy(dastac_rule* r);
dastac_status dastac_rule_size(const dastac_rule* r, int32_t* n_summands, int32_t* n_buffers);
dastac_status dastac_rule_summand(const dastac_rule* r, int32_t k, const dastac_structure** s, int32_t* buffer);
dastac_status dastac_rule_pack(const dastac_rule* r, dastac_dtype dtype, const void* dense,
                               const int64_t* dense_strides, void* const* packed, void* stream);
dastac_status dastac_rule_contract_workspace(const char* expr, const dastac_rule* r, dastac_dtype dtype,
                                             const dastac_operand* rest, int32_t n_rest,
                                             const dastac_operand* out, size_t* bytes);
dastac_status dastac_rule_contract(const char* expr, const dastac_rule* r, dastac_dtype dtype,
                                   void* const* packed, const int64_t* packed_batch_strides,
                                   const dastac_operand* rest, int32_t n_rest, const dastac_operand* out,
                                   int32_t accumulate, void* workspace, size_t workspace_bytes,
                                   int32_t* err_word, void* stream);

/*
 * Algorithm 2, "Piecewise QuasiPolynomial Fusion" (Section 4, "Piecewise Polynomial
 * Simplification"), as a host procedure.  The counting step returns one polynomial per piece of
 * the counted set; a piece (D', P') is dropped when another piece's polynomial P equals P' on D',
 * and that piece's domain grows by D'.
 *   poly     sum_t num[t] / den * prod_v x_v ^ exps[t * nvars + v]   (host arrays; den > 0;
 *            exponents 0..6; nvars = the domain's rank)
 *   domain   a descriptor as for dastac_structure_create (rows may be equalities; mirror and
 *            layout are ignored); the box 0 <= x_v < dims[v] is implied
 *   owner    host, n entries out: owner[k] = index of the piece whose polynomial holds on piece k
 *            after fusion (owner[k] == k for the pieces that remain)
 * "(P - P') restricted to D' is zero" is decided exactly: symbolically when the equalities of D'
 * make the difference vanish, else at every integer point of D' when its box has at most 2^22
 * points; a larger domain that is not decided symbolically is left alone.
 */
typedef struct {
    int32_t nvars;
    int32_t nterms;
    const int32_t* exps;
    const int64_t* num;
    int64_t den;
} dastac_poly;
typedef struct {
    dastac_structure_desc domain;
    dastac_poly poly;
} dastac_piece;
dastac_status dastac_piecewise_fuse(const dastac_piece* pieces, int32_t n, int32_t* owner);

/*
 * Device error word (no counterpart in the paper: it belongs to the execution model, not to the
 * method).  Kernels whose entry points take no `err_word` (pack, unpack) record an expired bounded
 * wait in a device int32 owned by the library, one per GPU.  dastac_device_error copies the current
 * device's word to *word (host, may be NULL), clears it on the device when `clear` != 0, and
 * returns DASTAC_OK when it was 0 and DASTAC_ERR_TIMEOUT otherwise.  Unlike the other device
 * calls it SYNCHRONISES `stream`, so it reports everything enqueued on that stream before it.
 */
dastac_status dastac_device_error(int32_t* word, int32_t clear, void* stream);
/*
 * Self-test of the expiry path: enqueues one warp that waits `budget_cycles` SM clock cycles
 * (0 .. 2e9) on a shared-memory barrier that nothing arrives on, then records a code in the
 * device error word and returns normally.  Afterwards dastac_device_error reports
 * DASTAC_ERR_TIMEOUT and the device is as usable as before: no trap, no fault, no unbounded loop.
 */
dastac_status dastac_selftest_wait_expiry(int64_t budget_cycles, void* stream);

/* Number of kernels this library has launched in the calling process (for launch accounting). */
int64_t dastac_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* DASTAC_H_ */
