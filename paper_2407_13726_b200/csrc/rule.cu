// A structured operand given as a sum of summands (Section 4: the method "only works with
// individual summands of a rule"; every summand's region gets its own compressed buffer, and a
// region that equals an earlier one reuses that buffer).  A rule object holds one structure per
// summand and the buffer each one reads; packing fills every distinct buffer, and a contraction
// over the rule is the sum of the contractions over its summands, evaluated in one call.
#include <cstring>
#include <new>
#include <vector>

#include "common.cuh"

struct dastac_rule {
    std::vector<dastac_structure*> summand;
    std::vector<int32_t> buffer;  // summand k reads packed buffer buffer[k]
    int32_t n_buffers = 0;
    ~dastac_rule() {
        for (dastac_structure* s : summand) dastac_structure_destroy(s);
    }
};

namespace {

// Two summands cover the same region when their maps are equal (the maps are canonical: a class
// and its coefficients, or the normalised rows and fitted pieces).
bool same_region(const dastac_structure* a, const dastac_structure* b) {
    if (std::memcmp(&a->map, &b->map, sizeof(a->map)) != 0) return false;
    if ((a->generic == nullptr) != (b->generic == nullptr)) return false;
    return !a->generic || std::memcmp(a->generic, b->generic, sizeof(*a->generic)) == 0;
}

}  // namespace

extern "C" dastac_status dastac_rule_create(const dastac_structure_desc* summands, int32_t n, dastac_rule** out) {
    if (!summands || !out || n < 1 || n > 64) return DASTAC_ERR_INVALID_ARG;
    *out = nullptr;
    dastac_rule* r = new (std::nothrow) dastac_rule;
    if (!r) return DASTAC_ERR_INVALID_ARG;
    for (int k = 0; k < n; ++k) {
        dastac_structure* s = nullptr;
        const dastac_status st = dastac_structure_create(&summands[k], &s);
        if (st != DASTAC_OK) {
            delete r;
            return st;
        }
        // all summands describe parts of the same tensor
        if (k > 0 && (s->map.rank != r->summand[0]->map.rank ||
                      std::memcmp(s->map.dims, r->summand[0]->map.dims, sizeof(s->map.dims)) != 0)) {
            dastac_structure_destroy(s);
            delete r;
            return DASTAC_ERR_SHAPE;
        }
        int32_t buf = r->n_buffers;
        for (int q = 0; q < k; ++q)
            if (same_region(s, r->summand[(size_t)q])) {
                buf = r->buffer[(size_t)q];
                break;
            }
        if (buf == r->n_buffers) ++r->n_buffers;
        r->summand.push_back(s);
        r->buffer.push_back(buf);
    }
    *out = r;
    return DASTAC_OK;
}

extern "C" void dastac_rule_destroy(dastac_rule* r) { delete r; }

extern "C" dastac_status dastac_rule_size(const dastac_rule* r, int32_t* n_summands, int32_t* n_buffers) {
    if (!r) return DASTAC_ERR_INVALID_ARG;
    if (n_summands) *n_summands = (int32_t)r->summand.size();
    if (n_buffers) *n_buffers = r->n_buffers;
    return DASTAC_OK;
}

extern "C" dastac_status dastac_rule_summand(const dastac_rule* r, int32_t k, const dastac_structure** s, int32_t* buffer) {
    if (!r || k < 0 || k >= (int32_t)r->summand.size()) return DASTAC_ERR_INVALID_ARG;
    if (s) *s = r->summand[(size_t)k];
    if (buffer) *buffer = r->buffer[(size_t)k];
    return DASTAC_OK;
}

extern "C" dastac_status dastac_rule_pack(const dastac_rule* r, dastac_dtype dtype, const void* dense,
                                          const int64_t* dense_strides, void* const* packed, void* stream) {
    if (!r || !packed) return DASTAC_ERR_INVALID_ARG;
    std::vector<char> done((size_t)r->n_buffers, 0);
    for (size_t k = 0; k < r->summand.size(); ++k) {
        const int32_t b = r->buffer[k];
        if (done[(size_t)b]) continue;  // an equal region: already packed
        done[(size_t)b] = 1;
        const dastac_status st = dastac_pack(r->summand[k], dtype, dense, dense_strides, packed[b], stream);
        if (st != DASTAC_OK) return st;
    }
    return DASTAC_OK;
}

namespace {

dastac_status check_rule_args(const dastac_rule* r, const dastac_operand* rest, int32_t n_rest, const dastac_operand* out) {
    if (!r || !out || n_rest < 1 || n_rest > 2 || !rest) return DASTAC_ERR_INVALID_ARG;
    return DASTAC_OK;
}

void first_operand(const dastac_rule* r, size_t k, void* data, dastac_dtype dtype, int32_t batch, int64_t batch_stride,
                   dastac_operand& op) {
    std::memset(&op, 0, sizeof(op));
    op.data = data;
    op.dtype = dtype;
    op.space = DASTAC_MEM_DEVICE;
    op.structure = r->summand[k];
    op.rank = r->summand[k]->map.rank;
    op.batch = batch;
    op.batch_stride = batch_stride;
    for (int d = 0; d < op.rank; ++d) op.dims[d] = r->summand[k]->map.dims[d];
}

}  // namespace

extern "C" dastac_status dastac_rule_contract_workspace(const char* expr, const dastac_rule* r, dastac_dtype dtype,
                                                        const dastac_operand* rest, int32_t n_rest,
                                                        const dastac_operand* out, size_t* bytes) {
    if (!bytes) return DASTAC_ERR_INVALID_ARG;
    dastac_status st = check_rule_args(r, rest, n_rest, out);
    if (st != DASTAC_OK) return st;
    size_t need = 0;
    for (size_t k = 0; k < r->summand.size(); ++k) {
        dastac_operand in[3];
        first_operand(r, k, nullptr, dtype, out->batch, 0, in[0]);
        for (int q = 0; q < n_rest; ++q) in[q + 1] = rest[q];
        size_t b = 0;
        st = dastac_contract_workspace(expr, in, n_rest + 1, out, &b);
        if (st != DASTAC_OK) return st;
        if (b > need) need = b;
    }
    *bytes = need;
    return DASTAC_OK;
}

extern "C" dastac_status dastac_rule_contract(const char* expr, const dastac_rule* r, dastac_dtype dtype,
                                              void* const* packed, const int64_t* packed_batch_strides,
                                              const dastac_operand* rest, int32_t n_rest, const dastac_operand* out,
                                              int32_t accumulate, void* workspace, size_t workspace_bytes,
                                              int32_t* err_word, void* stream) {
    dastac_status st = check_rule_args(r, rest, n_rest, out);
    if (st != DASTAC_OK) return st;
    if (!packed) return DASTAC_ERR_INVALID_ARG;
    // every summand is checked before the first one is enqueued
    size_t need = 0;
    st = dastac_rule_contract_workspace(expr, r, dtype, rest, n_rest, out, &need);
    if (st != DASTAC_OK) return st;
    if (need > 0 && (!workspace || workspace_bytes < need)) return DASTAC_ERR_WORKSPACE;
    for (size_t k = 0; k < r->summand.size(); ++k) {
        dastac_operand in[3];
        const int32_t b = r->buffer[k];
        first_operand(r, k, packed[b], dtype, out->batch, packed_batch_strides ? packed_batch_strides[b] : 0, in[0]);
        for (int q = 0; q < n_rest; ++q) in[q + 1] = rest[q];
        // the first summand overwrites (unless the caller accumulates), the others add to it
        st = dastac_contract(expr, in, n_rest + 1, out, (accumulate || k > 0) ? 1 : 0, workspace, workspace_bytes, err_word,
                             stream);
        if (st != DASTAC_OK) return st;
    }
    return DASTAC_OK;
}
