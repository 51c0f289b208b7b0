// dastac_contract: validates a sum-of-products rule over a packed first operand, stages host
// operands through the caller's workspace and enqueues the kernel of the matching class.
#include <cstring>

#include "common.cuh"

namespace dastac {
namespace {

enum ExprClass { kMatVec, kMatMat, kMttkrp, kTtm, kMoment2, kMoment3, kHadamard, kNoExpr };

ExprClass parse_expr(const char* e) {
    if (!e) return kNoExpr;
    if (!std::strcmp(e, "ij,j->i")) return kMatVec;
    if (!std::strcmp(e, "ij,jc->ic")) return kMatMat;
    if (!std::strcmp(e, "ijk,jr,kr->ir")) return kMttkrp;
    if (!std::strcmp(e, "ijl,kl->ijk")) return kTtm;
    if (!std::strcmp(e, "xi,xj->ij")) return kMoment2;
    if (!std::strcmp(e, "xi,xj,xk->ijk")) return kMoment3;
    if (!std::strcmp(e, "i,i->i") || !std::strcmp(e, "ij,ij->ij") || !std::strcmp(e, "ijk,ijk->ijk")) return kHadamard;
    return kNoExpr;
}

int batch_of(const dastac_operand& o) { return o.batch > 1 ? o.batch : 1; }

// Elements spanned by one instance of an operand.
int64_t span_elems(const dastac_operand& o) {
    if (o.structure) {
        const int per16 = 16 / elt_size(o.dtype);
        return round_up(o.structure->map.slots, per16);
    }
    int64_t span = 1;
    for (int k = 0; k < o.rank; ++k) {
        if (o.dims[k] == 0) return 0;
        span += (o.dims[k] - 1) * o.strides[k];
    }
    return span;
}

int64_t total_bytes(const dastac_operand& o) {
    const int64_t one = span_elems(o);
    if (one == 0) return 0;
    return ((batch_of(o) - 1) * o.batch_stride + one) * elt_size(o.dtype);
}

struct Plan {
    ExprClass cls = kNoExpr;
    const IndexMap* map = nullptr;
    bool symmetric = false;
    int batch = 1;
    int64_t N = 0, ncols = 0, R = 0;
    size_t scratch = 0;          // kernel scratch bytes (start of the workspace)
    size_t stage_off[4] = {0, 0, 0, 0};  // in[0..2], out
    size_t total = 0;
};

bool dense_ok(const dastac_operand& o, int rank) {
    if (o.structure || o.rank != rank || !(o.space == DASTAC_MEM_DEVICE || o.space == DASTAC_MEM_HOST))
        return false;
    for (int k = 0; k < rank; ++k)
        if (o.dims[k] < 0 || o.strides[k] < 0) return false;
    return true;
}

dastac_status make_plan(const char* expr, const dastac_operand* in, int32_t n_in,
                        const dastac_operand* out, Plan& p) {
    p.cls = parse_expr(expr);
    if (!in || !out || n_in < 1) return DASTAC_ERR_INVALID_ARG;
    if (p.cls == kNoExpr) return DASTAC_ERR_UNSUPPORTED_EXPR;
    const int want_in = (p.cls == kMttkrp || p.cls == kMoment3) ? 3 : 2;  // the tensor-times-matrix rule has two inputs as well
    if (n_in != want_in) return DASTAC_ERR_INVALID_ARG;
    // fitted maps have element-wise kernels only (index maps, pack, unpack)
    for (int k = 0; k < n_in; ++k)
        if (in[k].structure && in[k].structure->map.kind == kGeneric) return DASTAC_ERR_UNSUPPORTED_EXPR;
    if (out->structure && out->structure->map.kind == kGeneric) return DASTAC_ERR_UNSUPPORTED_EXPR;
    if (p.cls == kMoment2 || p.cls == kMoment3) {
        // dense B (samples x features) as every factor, packed unique part of the symmetric result out
        for (int k = 0; k < n_in; ++k)
            if (!dense_ok(in[k], 2)) return DASTAC_ERR_INVALID_ARG;
        if (!out->structure) return DASTAC_ERR_UNSUPPORTED_EXPR;
        // all factors are the same tensor: only then is the result symmetric
        for (int k = 1; k < n_in; ++k)
            if (in[0].data != in[k].data || in[0].space != in[k].space || in[0].dtype != in[k].dtype ||
                in[0].dims[0] != in[k].dims[0] || in[0].dims[1] != in[k].dims[1] ||
                in[0].strides[0] != in[k].strides[0] || in[0].strides[1] != in[k].strides[1])
                return DASTAC_ERR_UNSUPPORTED_EXPR;
        const IndexMap& mo = out->structure->map;
        if (p.cls == kMoment2 && !(mo.kind == kUpper && mo.rank == 2 && mo.dims[0] == mo.dims[1]) && mo.kind != kEmpty)
            return DASTAC_ERR_UNSUPPORTED_EXPR;
        if (p.cls == kMoment3 && mo.kind != kTetrahedron && mo.kind != kEmpty) return DASTAC_ERR_UNSUPPORTED_EXPR;
        if (in[0].dtype != DASTAC_BF16 || out->dtype != DASTAC_F32) return DASTAC_ERR_UNSUPPORTED_EXPR;
        if (batch_of(in[0]) != 1 || batch_of(*out) != 1) return DASTAC_ERR_UNSUPPORTED_EXPR;
        if (!(out->space == DASTAC_MEM_DEVICE || out->space == DASTAC_MEM_HOST)) return DASTAC_ERR_INVALID_ARG;
        if (in[0].dims[1] != mo.dims[0] || in[0].dims[1] != mo.dims[1]) return DASTAC_ERR_SHAPE;
        if (in[0].dims[1] > 1 && in[0].strides[1] != 1) return DASTAC_ERR_SHAPE;
        p.map = &mo;
        p.N = mo.dims[0];
        p.R = in[0].dims[0];  // samples
        p.scratch = p.cls == kMoment3 ? moment3_workspace_bytes(p.R, p.N, in[0].strides[0])
                                      : moment2_workspace_bytes(p.R, p.N, in[0].strides[0]);
        size_t off = (size_t)round_up((int64_t)p.scratch, 256);
        p.stage_off[0] = p.stage_off[1] = p.stage_off[2] = off;  // one staged copy serves every factor
        if (in[0].space == DASTAC_MEM_HOST) off += (size_t)round_up(total_bytes(in[0]), 256);
        p.stage_off[3] = off;
        if (out->space == DASTAC_MEM_HOST) off += (size_t)round_up(total_bytes(*out), 256);
        p.total = off;
        return DASTAC_OK;
    }
    if (!in[0].structure) return DASTAC_ERR_UNSUPPORTED_EXPR;
    if (!(in[0].space == DASTAC_MEM_DEVICE || in[0].space == DASTAC_MEM_HOST))
        return DASTAC_ERR_INVALID_ARG;
    const IndexMap& m = in[0].structure->map;
    p.map = &m;
    p.batch = batch_of(in[0]);

    if (p.cls == kHadamard) {
        // packed structured operand times a dense one of the same box; the result has the same structure
        const int want_rank = (int)(std::strchr(expr, ',') - expr);
        if (m.rank != want_rank && m.kind != kEmpty) return DASTAC_ERR_UNSUPPORTED_EXPR;
        if (!out->structure) return DASTAC_ERR_UNSUPPORTED_EXPR;
        const IndexMap& mo = out->structure->map;
        if (std::memcmp(&mo, &m, sizeof(IndexMap)) != 0) return DASTAC_ERR_SHAPE;  // the same structure on both sides
        if (in[0].dtype != DASTAC_F32 || in[1].dtype != DASTAC_F32 || out->dtype != DASTAC_F32)
            return DASTAC_ERR_UNSUPPORTED_EXPR;
        if (p.batch != 1 || batch_of(in[1]) != 1 || batch_of(*out) != 1) return DASTAC_ERR_UNSUPPORTED_EXPR;
        if (!dense_ok(in[1], m.rank)) return DASTAC_ERR_INVALID_ARG;
        if (!(out->space == DASTAC_MEM_DEVICE || out->space == DASTAC_MEM_HOST)) return DASTAC_ERR_INVALID_ARG;
        for (int k = 0; k < m.rank; ++k)
            if (in[1].dims[k] != m.dims[k]) return DASTAC_ERR_SHAPE;
    } else if (out->structure && p.cls != kTtm) {
        return DASTAC_ERR_UNSUPPORTED_EXPR;  // no other rule with a packed first operand packs its output
    }
    if (p.cls == kHadamard) {
    } else if (p.cls == kTtm) {
        // packed upper half cube in, packed upper half cube out: same (i, j) set, trailing extents Q and K
        if (!out->structure) return DASTAC_ERR_UNSUPPORTED_EXPR;
        const IndexMap& mo = out->structure->map;
        if (p.batch != 1 || batch_of(in[1]) != 1 || batch_of(*out) != 1) return DASTAC_ERR_UNSUPPORTED_EXPR;
        // classes whose trailing index is dense and contiguous (extents of 1 can close a half cube to
        // the dense box or to the one-point tetrahedron: the same set, the same layout)
        auto trailing_dense = [](const IndexMap& x) {
            return x.kind == kEmpty || (x.rank == 3 && (x.kind == kUpper || x.kind == kDense ||
                                                        (x.kind == kPlane && x.w != 2) ||
                                                        (x.kind == kTetrahedron && x.dims[0] == 1)));
        };
        if (!trailing_dense(m) || !trailing_dense(mo)) return DASTAC_ERR_UNSUPPORTED_EXPR;
        if (in[0].dtype != DASTAC_F32 || in[1].dtype != DASTAC_F32 || out->dtype != DASTAC_F32)
            return DASTAC_ERR_UNSUPPORTED_EXPR;
        if (!dense_ok(in[1], 2)) return DASTAC_ERR_INVALID_ARG;
        if (!(out->space == DASTAC_MEM_DEVICE || out->space == DASTAC_MEM_HOST)) return DASTAC_ERR_INVALID_ARG;
        if (mo.dims[0] != m.dims[0] || mo.dims[1] != m.dims[1] || in[1].dims[0] != mo.dims[2] ||
            in[1].dims[1] != m.dims[2])
            return DASTAC_ERR_SHAPE;
        if (m.dims[2] > 1 && in[1].strides[1] != 1) return DASTAC_ERR_SHAPE;
        // the same (i, j) set on both sides
        if ((m.dims[2] > 0 ? m.count / m.dims[2] : 0) != (mo.dims[2] > 0 ? mo.count / mo.dims[2] : 0) &&
            m.dims[2] > 0 && mo.dims[2] > 0)
            return DASTAC_ERR_SHAPE;
        // planes: the same determined index on both sides
        if ((m.kind == kPlane || mo.kind == kPlane) &&
            !(m.kind == mo.kind && m.w == mo.w && m.lo_off == mo.lo_off && m.hi_off == mo.hi_off))
            return DASTAC_ERR_SHAPE;
        p.N = m.dims[2];   // Q
        p.R = mo.dims[2];  // K
    } else if (p.cls == kMatVec) {
        if (!(m.kind == kUpper && m.rank == 2 && m.dims[0] == m.dims[1]) && m.kind != kEmpty &&
            m.kind != kUpperShifted && !rowspan_mv_supports(m))
            return DASTAC_ERR_UNSUPPORTED_EXPR;
        if (in[0].dtype != DASTAC_F32 || in[1].dtype != DASTAC_F32 || out->dtype != DASTAC_F32)
            return DASTAC_ERR_UNSUPPORTED_EXPR;
        if (!dense_ok(in[1], 1) || !dense_ok(*out, 1)) return DASTAC_ERR_INVALID_ARG;
        p.N = m.dims[1];
        if (in[1].dims[0] != p.N || out->dims[0] != m.dims[0]) return DASTAC_ERR_SHAPE;
        if (p.N > 1 && (in[1].strides[0] != 1 || out->strides[0] != 1)) return DASTAC_ERR_SHAPE;
        p.symmetric = m.symmetric != 0;
        if (batch_of(in[1]) != p.batch || batch_of(*out) != p.batch) return DASTAC_ERR_SHAPE;
        if (p.symmetric && p.batch != 1) return DASTAC_ERR_UNSUPPORTED_EXPR;
        if (p.symmetric) p.scratch = symv_workspace_bytes(m);
    } else if (p.cls == kMatMat) {
        if (p.batch != 1 || batch_of(in[1]) != 1 || batch_of(*out) != 1)
            return DASTAC_ERR_UNSUPPORTED_EXPR;
        if (!dense_ok(in[1], 2) || !dense_ok(*out, 2)) return DASTAC_ERR_INVALID_ARG;
        const bool band = (m.kind == kBandDiagonals || m.kind == kBandExact) && in[0].dtype == DASTAC_F32 &&
                          in[1].dtype == DASTAC_F32 && out->dtype == DASTAC_F32;
        const bool tri_bf16 = m.kind == kUpper && m.rank == 2 && m.dims[0] == m.dims[1] &&
                              !m.symmetric && in[0].dtype == DASTAC_BF16 &&
                              in[1].dtype == DASTAC_BF16 && out->dtype == DASTAC_F32;
        const bool rowwise = rowspan_mv_supports(m) && in[0].dtype == DASTAC_F32 && in[1].dtype == DASTAC_F32 &&
                             out->dtype == DASTAC_F32;
        if (!band && !tri_bf16 && !rowwise && m.kind != kEmpty) return DASTAC_ERR_UNSUPPORTED_EXPR;
        p.N = m.dims[1];
        p.ncols = in[1].dims[1];
        if (in[1].dims[0] != p.N || out->dims[0] != m.dims[0] || out->dims[1] != p.ncols)
            return DASTAC_ERR_SHAPE;
        if (p.ncols > 1 && (in[1].strides[1] != 1 || out->strides[1] != 1)) return DASTAC_ERR_SHAPE;
        if (tri_bf16) p.scratch = trimm_workspace_bytes(m, p.ncols, in[1].strides[0]);
    } else {
        if (p.batch != 1 || batch_of(in[1]) != 1 || batch_of(in[2]) != 1 || batch_of(*out) != 1)
            return DASTAC_ERR_UNSUPPORTED_EXPR;
        if (!mttkrp_supports(m) && m.kind != kEmpty) return DASTAC_ERR_UNSUPPORTED_EXPR;
        if (in[0].dtype != DASTAC_F32 || in[1].dtype != DASTAC_F32 || in[2].dtype != DASTAC_F32 ||
            out->dtype != DASTAC_F32)
            return DASTAC_ERR_UNSUPPORTED_EXPR;
        if (!dense_ok(in[1], 2) || !dense_ok(in[2], 2) || !dense_ok(*out, 2))
            return DASTAC_ERR_INVALID_ARG;
        p.N = m.dims[0];
        p.R = in[1].dims[1];
        if (in[1].dims[0] != m.dims[1] || in[2].dims[0] != m.dims[2] || in[2].dims[1] != p.R ||
            out->dims[0] != m.dims[0] || out->dims[1] != p.R)
            return DASTAC_ERR_SHAPE;
        if (p.R > 1 && (in[1].strides[1] != 1 || in[2].strides[1] != 1 || out->strides[1] != 1))
            return DASTAC_ERR_SHAPE;
    }

    // Workspace layout: kernel scratch, then one staging area per host operand.
    size_t off = (size_t)round_up((int64_t)p.scratch, 256);
    for (int k = 0; k < n_in; ++k) {
        p.stage_off[k] = off;
        if (in[k].space == DASTAC_MEM_HOST) off += (size_t)round_up(total_bytes(in[k]), 256);
    }
    p.stage_off[3] = off;
    if (out->space == DASTAC_MEM_HOST) off += (size_t)round_up(total_bytes(*out), 256);
    p.total = off;
    return DASTAC_OK;
}

}  // namespace
}  // namespace dastac

using namespace dastac;

extern "C" dastac_status dastac_contract_workspace(const char* expr, const dastac_operand* in,
                                                   int32_t n_in, const dastac_operand* out,
                                                   size_t* bytes) {
    if (!bytes) return DASTAC_ERR_INVALID_ARG;
    Plan p;
    dastac_status st = make_plan(expr, in, n_in, out, p);
    if (st != DASTAC_OK) return st;
    *bytes = p.total;
    return DASTAC_OK;
}

extern "C" dastac_status dastac_contract(const char* expr, const dastac_operand* in, int32_t n_in,
                                         const dastac_operand* out, int32_t accumulate,
                                         void* workspace, size_t workspace_bytes, int32_t* err_word,
                                         void* stream) {
    Plan p;
    dastac_status st = make_plan(expr, in, n_in, out, p);
    if (st != DASTAC_OK) return st;
    if (p.total > 0) {
        if (!workspace || workspace_bytes < p.total ||
            (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0)
            return DASTAC_ERR_WORKSPACE;
    }
    cudaStream_t cs = (cudaStream_t)stream;
    const IndexMap& m = *p.map;

    // Resolve device pointers (staging host operands).
    const void* dev_in[3] = {nullptr, nullptr, nullptr};
    for (int k = 0; k < n_in; ++k) {
        if ((p.cls == kMoment2 || p.cls == kMoment3) && k >= 1) {  // the same tensor as in[0]
            dev_in[k] = dev_in[0];
            continue;
        }
        const int64_t bytes = total_bytes(in[k]);
        if (bytes > 0 && !in[k].data) return DASTAC_ERR_INVALID_ARG;
        if (in[k].space == DASTAC_MEM_HOST && bytes > 0) {
            void* d = static_cast<char*>(workspace) + p.stage_off[k];
            if (cudaMemcpyAsync(d, in[k].data, (size_t)bytes, cudaMemcpyHostToDevice, cs) != cudaSuccess)
                return DASTAC_ERR_CUDA;
            dev_in[k] = d;
        } else {
            dev_in[k] = in[k].data;
        }
        if (bytes > 0 && !aligned16(dev_in[k])) return DASTAC_ERR_ALIGNMENT;
    }
    const int64_t out_bytes = total_bytes(*out);
    if (out_bytes > 0 && !out->data) return DASTAC_ERR_INVALID_ARG;
    void* dev_out = out->data;
    if (out->space == DASTAC_MEM_HOST && out_bytes > 0) {
        dev_out = static_cast<char*>(workspace) + p.stage_off[3];
        if (accumulate &&
            cudaMemcpyAsync(dev_out, out->data, (size_t)out_bytes, cudaMemcpyHostToDevice, cs) != cudaSuccess)
            return DASTAC_ERR_CUDA;
    }
    if (out_bytes > 0 && !aligned16(dev_out)) return DASTAC_ERR_ALIGNMENT;
    void* scratch = p.scratch ? workspace : nullptr;

    if (p.cls == kHadamard) {
        st = (m.kind == kEmpty || out_bytes == 0)
                 ? DASTAC_OK
                 : launch_hadamard(m, (const float*)dev_in[0], (const float*)dev_in[1], in[1].strides, (float*)dev_out,
                                   accumulate, cs);
    } else if (p.cls == kMoment3) {
        st = (m.kind == kEmpty || out_bytes == 0)
                 ? DASTAC_OK
                 : launch_moment3_bf16(m, dev_in[0], in[0].strides[0], p.R, (float*)dev_out, accumulate, scratch,
                                       err_word, cs);
    } else if (p.cls == kMoment2) {
        st = (m.kind == kEmpty || out_bytes == 0)
                 ? DASTAC_OK
                 : launch_moment2_bf16(m, dev_in[0], in[0].strides[0], p.R, (float*)dev_out, accumulate, scratch,
                                       err_word, cs);
    } else if (m.kind == kEmpty || out_bytes == 0) {
        st = DASTAC_OK;
        // an empty sum over l (Q = 0) still defines the packed output: zero
        if (p.cls == kTtm && out_bytes > 0 && !accumulate &&
            cudaMemsetAsync(dev_out, 0, (size_t)out_bytes, cs) != cudaSuccess)
            st = DASTAC_ERR_CUDA;
    } else if (p.cls == kTtm) {
        st = launch_ttm(m.count / p.N, p.N, p.R, (const float*)dev_in[0], (const float*)dev_in[1], in[1].strides[0],
                        (float*)dev_out, accumulate, cs);
    } else if (p.cls == kMatVec && m.kind == kUpperShifted) {
        // The sub-triangle is the size-M upper triangle applied to x shifted by c; rows M .. N-1 of y
        // have no stored element: they are zero (or left alone when accumulating).
        IndexMap t = m;
        t.kind = kUpper;
        t.N = t.dims[0] = t.dims[1] = m.M;
        t.w = 0;
        st = launch_trmv(t, (const float*)dev_in[0], (const float*)dev_in[1] + m.w, (float*)dev_out, p.batch,
                         in[0].batch_stride, in[1].batch_stride, out->batch_stride, accumulate, cs);
        if (st == DASTAC_OK && !accumulate &&
            cudaMemset2DAsync((float*)dev_out + m.M, (size_t)(p.batch > 1 ? out->batch_stride : m.N) * sizeof(float), 0,
                              (size_t)m.w * sizeof(float), (size_t)p.batch, cs) != cudaSuccess)
            st = DASTAC_ERR_CUDA;
    } else if (p.cls == kMatVec && rowspan_mv_supports(m)) {
        st = launch_rowspan_mv(m, (const float*)dev_in[0], (const float*)dev_in[1], (float*)dev_out, p.batch,
                               in[0].batch_stride, in[1].batch_stride, out->batch_stride, accumulate, cs);
    } else if (p.cls == kMatVec && !p.symmetric) {
        st = launch_trmv(m, (const float*)dev_in[0], (const float*)dev_in[1], (float*)dev_out,
                         p.batch, in[0].batch_stride, in[1].batch_stride, out->batch_stride,
                         accumulate, cs);
    } else if (p.cls == kMatVec) {
        st = launch_symv(m, (const float*)dev_in[0], (const float*)dev_in[1], (float*)dev_out,
                         accumulate, scratch, cs);
    } else if (p.cls == kMatMat && (m.kind == kBandDiagonals || m.kind == kBandExact)) {
        st = launch_bandmm(m, (const float*)dev_in[0], (const float*)dev_in[1], in[1].strides[0],
                           (float*)dev_out, out->strides[0], p.ncols, accumulate, err_word, cs);
    } else if (p.cls == kMatMat && in[0].dtype == DASTAC_F32) {
        st = launch_rowspan_mm(m, (const float*)dev_in[0], (const float*)dev_in[1], in[1].strides[0], (float*)dev_out,
                               out->strides[0], p.ncols, accumulate, cs);
    } else if (p.cls == kMatMat) {
        st = launch_trimm_bf16(m, dev_in[0], dev_in[1], in[1].strides[0], (float*)dev_out,
                               out->strides[0], p.ncols, accumulate, scratch, err_word, cs);
    } else {
        st = launch_mttkrp(m, (const float*)dev_in[0], (const float*)dev_in[1], in[1].strides[0],
                           (const float*)dev_in[2], in[2].strides[0], (float*)dev_out,
                           out->strides[0], p.R, accumulate, err_word, cs);
    }
    if (st != DASTAC_OK) return st;
    if (out->space == DASTAC_MEM_HOST && out_bytes > 0 &&
        cudaMemcpyAsync(out->data, dev_out, (size_t)out_bytes, cudaMemcpyDeviceToHost, cs) != cudaSuccess)
        return DASTAC_ERR_CUDA;
    return DASTAC_OK;
}
