// CPU oracle for the delta-extract / remap / apply path.
//
// THIS IS TEST INFRASTRUCTURE, NOT PRODUCT CODE.  It is a plain, slow,
// single-threaded restatement of what the path computes, written from the
// paper's equations so that a reader can check it by eye.  Only the tests,
// the smoke check and the benchmark's CPU-baseline leg may load it; the CUDA
// library never does, and the two share no source, header, table or helper.
//
// Build: g++ -O2 -std=c++17 -ffp-contract=off -fno-fast-math -shared -fPIC
// (no FTZ/DAZ, default rounding mode).  -ffp-contract=off matters: every fp32
// operation below must round on its own.
//
// Parity pins (tests marked "not gpu"): constants against exact rational
// arithmetic; the inverse against hand-worked exactly-representable cases and
// against a forward AdamW step (Eq. 9) within a stated ulp bound; the BF16
// cast against a nearest-neighbour formulation in fp64 and a library cast;
// the changed set against an unfused array-at-a-time evaluation; the remap
// against coverage / reassembly invariants and dense slicing; apply against
// idempotence, untouched positions and the end-state identity; the destination-side mapping
// against dense slicing of the changed positions and against extract-then-apply.
//
// Passages followed:
//   Eq. 2  (AdamW inverse, Section 4.1; derivation Eq. 9-11, Appendix A)
//   Eq. 4  (BF16 cast, 16-bit pattern compare, nonzero, target values; Section 4.2.1)
//   Eq. 5-6 and the membership test between them (unravel - remap - ravel; Section 4.2.2)
//   Eq. 7  (direct sparse apply; Section 4.3)
//   Section 4.4 (destination-side mapping of canonical entries: Eq. 5-7 per received entry)

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <string>
#include <vector>

namespace {

inline uint32_t f32_bits(float x) {
    uint32_t u;
    std::memcpy(&u, &x, sizeof u);
    return u;
}

// Call-uniform constants, Eq. 2: the two bias corrections 1-beta^t and the
// decay factor 1-eta*lambda are evaluated once in double and rounded once to
// fp32; eta and epsilon are rounded to fp32.
struct Consts {
    float bc1, bc2, decay, lr, eps;
};

// Eq. 2, transcribed literally.  Every operation is a separate fp32 operation
// rounded to nearest-even; divisions are divisions; epsilon sits outside the
// square root, as printed.
inline float invert_one(float theta, float m, float v, const Consts& c) {
    float mhat = m / c.bc1;              // m_t / (1 - beta1^t)
    float vhat = v / c.bc2;              // v_t / (1 - beta2^t)
    float root = std::sqrt(vhat);        // sqrt(vhat)
    float den = root + c.eps;            // sqrt(vhat) + eps
    float u = mhat / den;                // adaptive update direction
    float step = c.lr * u;               // eta_t * u
    float num = theta + step;            // theta_t + eta_t * u
    float prev = num / c.decay;          // / (1 - eta_t * lambda)
    return prev;
}

// Q_BF16 of Eq. 4: round-to-nearest-even on the upper 16 bits of the fp32
// pattern.  NaN maps to the quiet pattern 0x7FC0; overflow to +-Inf and
// subnormals fall out of the integer rounding.
inline uint16_t bf16_rne(float x) {
    uint32_t u = f32_bits(x);
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) return 0x7FC0;
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7FFFu + lsb;
    return (uint16_t)(u >> 16);
}

struct Result {
    std::vector<uint64_t> op_count;   // n_ops: c_o = |I_o| (Section 4.3), zeros included
    std::vector<uint64_t> list_ptr;   // n_shards + 1
    std::vector<uint32_t> offsets;
    std::vector<uint16_t> values;
    uint64_t nonfinite = 0;           // scanned slots whose reconstruction broke: NaN, or +-Inf from a finite theta_t
    std::string error;
};

struct Entry {
    uint64_t j;
    uint16_t v;
};

}  // namespace

extern "C" {

// out5 = {bc1, bc2, decay, lr_f, eps_f}
void oracle_derive_constants(int64_t step, double lr, double beta1, double beta2, double eps,
                             double wd, float* out5) {
    double t = (double)step;
    out5[0] = (float)(1.0 - std::pow(beta1, t));
    out5[1] = (float)(1.0 - std::pow(beta2, t));
    out5[2] = (float)(1.0 - lr * wd);
    out5[3] = (float)lr;
    out5[4] = (float)eps;
}

// prev[i] = reconstructed theta_{t-1}[i], Eq. 2.
void oracle_invert(const float* theta, const float* m, const float* v, uint64_t n,
                   const float* c5, float* prev) {
    Consts c{c5[0], c5[1], c5[2], c5[3], c5[4]};
    for (uint64_t i = 0; i < n; ++i) prev[i] = invert_one(theta[i], m[i], v[i], c);
}

void oracle_bf16_rne(const float* x, uint64_t n, uint16_t* out) {
    for (uint64_t i = 0; i < n; ++i) out[i] = bf16_rne(x[i]);
}

// Eq. 4 on one tensor: mask[i] = 1 where the stored BF16 patterns of theta_t
// and of the reconstruction differ; value[i] = BF16(theta_t)[i] (always
// written).  Returns the number of changed elements.
uint64_t oracle_changed_mask(const float* theta, const float* m, const float* v, uint64_t n,
                             const float* c5, uint8_t* mask, uint16_t* value) {
    Consts c{c5[0], c5[1], c5[2], c5[3], c5[4]};
    uint64_t cnt = 0;
    for (uint64_t i = 0; i < n; ++i) {
        float prev = invert_one(theta[i], m[i], v[i], c);
        uint16_t bt = bf16_rne(theta[i]);
        uint16_t bp = bf16_rne(prev);
        mask[i] = (uint8_t)(bt != bp);
        value[i] = bt;
        cnt += mask[i];
    }
    return cnt;
}

// Full extract over a transfer plan.
//   tensor_shape : n_tensors x 2  (n_s; 1-D tensors as [n, 1])
//   shard_numel  : n_shards       (flattened receiver-local tensor sizes)
//   ops          : n_ops x 10 = {src_tensor, dst_shard, a_s0, a_s1, e0, e1,
//                                dst_base, dst_ld, a_r0, a_r1}
//                  receiver flat index j = dst_base + (u0-a_s0+a_r0)*dst_ld + (u1-a_s1+a_r1)
//   theta/m/v    : n_tensors host pointers
// Source-major, exactly the order of Eq. 4-6: for each tensor, for each flat
// index in ascending order that changed, for each operation on that tensor in
// plan order: unravel, test membership, ravel in receiver coordinates, append
// (j, value) to the operation's receiver list.  Each list is then put in
// ascending j (Section 4.2.2: a payload keeps its entries in order); a repeated j within one list is
// a plan error.  Lists are concatenated in shard order; empty lists keep
// their slot (list_ptr[k] == list_ptr[k+1]).
// `consts` holds 5 scalars per source tensor (n_tensors x 5): eta_t and lambda of Eq. 2 belong
// to the element's parameter group, so tensors of different groups carry different scalars.
void* oracle_extract(uint64_t n_tensors, const int64_t* tensor_shape, uint64_t n_shards,
                     const int64_t* shard_numel, uint64_t n_ops, const int64_t* ops,
                     const float* const* theta, const float* const* m, const float* const* v,
                     const float* consts) {
    Result* res = new Result();
    res->op_count.assign(n_ops, 0);
    std::vector<std::vector<uint64_t>> ops_of(n_tensors);
    for (uint64_t o = 0; o < n_ops; ++o) {
        const int64_t* op = ops + 10 * o;
        if (op[0] < 0 || (uint64_t)op[0] >= n_tensors || op[1] < 0 || (uint64_t)op[1] >= n_shards) {
            res->error = "operation names a tensor or shard that does not exist";
            return res;
        }
        ops_of[(uint64_t)op[0]].push_back(o);
    }
    std::vector<std::vector<Entry>> lists(n_shards);
    for (uint64_t p = 0; p < n_tensors; ++p) {
        const uint64_t n0 = (uint64_t)tensor_shape[2 * p], n1 = (uint64_t)tensor_shape[2 * p + 1];
        const uint64_t n = n0 * n1;
        if (ops_of[p].empty()) continue;
        const float* c5 = consts + 5 * p;
        const Consts c{c5[0], c5[1], c5[2], c5[3], c5[4]};
        for (uint64_t i = 0; i < n; ++i) {
            float prev = invert_one(theta[p][i], m[p][i], v[p][i], c);
            uint16_t bt = bf16_rne(theta[p][i]);
            uint16_t bp = bf16_rne(prev);
            // The paper says nothing about NaN or Inf; they are compared like any other pattern.
            // Reconstructions that broke - NaN (a NaN theta_t or moment, a negative v, 0/0), or an
            // overflow to +-Inf from a finite theta_t - are counted, once per receiver slot the
            // element maps to, so that a caller can notice; an infinite theta_t that stays
            // infinite is a value the model already held and is not.
            const bool odd = std::isnan(prev) || (std::isinf(prev) && std::isfinite(theta[p][i]));
            if (bt == bp && !odd) continue;
            // Eq. 5: u = unravel(i, n_s)
            const uint64_t u0 = i / n1, u1 = i % n1;
            for (uint64_t o : ops_of[p]) {
                const int64_t* op = ops + 10 * o;
                const uint64_t as0 = (uint64_t)op[2], as1 = (uint64_t)op[3];
                const uint64_t e0 = (uint64_t)op[4], e1 = (uint64_t)op[5];
                // a_s <= u < a_s + e, component-wise
                if (u0 < as0 || u0 >= as0 + e0 || u1 < as1 || u1 >= as1 + e1) continue;
                if (odd) res->nonfinite += 1;
                if (bt == bp) continue;
                // Eq. 6: j = ravel(u - a_s + a_r, n_r)
                const uint64_t j = (uint64_t)op[6] + (u0 - as0 + (uint64_t)op[8]) * (uint64_t)op[7] +
                                   (u1 - as1 + (uint64_t)op[9]);
                const uint64_t k = (uint64_t)op[1];
                if (j >= (uint64_t)shard_numel[k]) {
                    res->error = "receiver index outside its shard";
                    return res;
                }
                lists[k].push_back(Entry{j, bt});
                res->op_count[o] += 1;
            }
        }
    }
    res->list_ptr.assign(n_shards + 1, 0);
    for (uint64_t k = 0; k < n_shards; ++k) {
        auto& L = lists[k];
        std::stable_sort(L.begin(), L.end(), [](const Entry& a, const Entry& b) { return a.j < b.j; });
        for (size_t q = 1; q < L.size(); ++q)
            if (L[q].j == L[q - 1].j) {
                res->error = "two operations write the same receiver slot";
                return res;
            }
        res->list_ptr[k + 1] = res->list_ptr[k] + L.size();
    }
    res->offsets.reserve(res->list_ptr[n_shards]);
    res->values.reserve(res->list_ptr[n_shards]);
    for (uint64_t k = 0; k < n_shards; ++k)
        for (const Entry& e : lists[k]) {
            res->offsets.push_back((uint32_t)e.j);
            res->values.push_back(e.v);
        }
    return res;
}

const char* oracle_result_error(void* h) {
    Result* r = (Result*)h;
    return r->error.empty() ? nullptr : r->error.c_str();
}

uint64_t oracle_result_total(void* h) { return ((Result*)h)->offsets.size(); }

void oracle_result_copy(void* h, uint64_t* list_ptr, uint32_t* offsets, uint16_t* values) {
    Result* r = (Result*)h;
    std::copy(r->list_ptr.begin(), r->list_ptr.end(), list_ptr);
    std::copy(r->offsets.begin(), r->offsets.end(), offsets);
    std::copy(r->values.begin(), r->values.end(), values);
}

// c_o for every operation of the plan, in plan order (round 1 of the two-round transfer).
void oracle_result_op_counts(void* h, uint64_t* out) {
    Result* r = (Result*)h;
    std::copy(r->op_count.begin(), r->op_count.end(), out);
}

// Scanned receiver slots whose reconstructed theta_{t-1} is NaN, or infinite from a finite theta_t.
uint64_t oracle_result_nonfinite(void* h) { return ((Result*)h)->nonfinite; }

void oracle_result_free(void* h) { delete (Result*)h; }

// Eq. 7: vec(W_r)[I] <- V for every list.  Returns 0, or 1 if an index lies
// outside its shard (nothing further is written after the first such entry).
int oracle_apply(uint64_t n_shards, const int64_t* shard_numel, const uint64_t* list_ptr,
                 const uint32_t* offsets, const uint16_t* values, uint16_t* const* shards) {
    for (uint64_t k = 0; k < n_shards; ++k)
        for (uint64_t q = list_ptr[k]; q < list_ptr[k + 1]; ++q) {
            if ((int64_t)offsets[q] >= shard_numel[k]) return 1;
            shards[k][offsets[q]] = values[q];
        }
    return 0;
}

}  // extern "C"

// Destination-side mapping of canonical entries (Section 4.4: the storage-mediated path ships
// canonical changes and leaves the mapping into the inference layout to the destination).
// list p = changed flat indices i of canonical tensor p with their target values.  Literally
// Eq. 5-7: for every entry, u = unravel(i, n_s); for every operation on tensor p in plan order
// with a_s <= u < a_s + e: j = ravel(u - a_s + a_r, n_r) and shard[dst][j] <- value.  Operations
// whose shard pointer is NULL belong to other receivers and are skipped.  Returns 0, 1 if a j
// lies outside its shard, 2 if an index lies outside its tensor (nothing further is written).
extern "C" int oracle_apply_canonical(uint64_t n_tensors, const int64_t* tensor_shape, uint64_t n_shards,
                                      const int64_t* shard_numel, uint64_t n_ops, const int64_t* ops,
                                      const uint64_t* list_ptr, const uint32_t* indices,
                                      const uint16_t* values, uint16_t* const* shards) {
    (void)n_shards;
    for (uint64_t p = 0; p < n_tensors; ++p) {
        const uint64_t n0 = (uint64_t)tensor_shape[2 * p], n1 = (uint64_t)tensor_shape[2 * p + 1];
        for (uint64_t q = list_ptr[p]; q < list_ptr[p + 1]; ++q) {
            const uint64_t i = indices[q];
            if (i >= n0 * n1) return 2;
            const uint64_t u0 = i / n1, u1 = i % n1;                       // Eq. 5
            for (uint64_t o = 0; o < n_ops; ++o) {
                const int64_t* op = ops + 10 * o;
                if ((uint64_t)op[0] != p) continue;
                const uint64_t as0 = (uint64_t)op[2], as1 = (uint64_t)op[3];
                const uint64_t e0 = (uint64_t)op[4], e1 = (uint64_t)op[5];
                if (u0 < as0 || u0 >= as0 + e0 || u1 < as1 || u1 >= as1 + e1) continue;
                uint16_t* dst = shards[(uint64_t)op[1]];
                if (!dst) continue;
                const uint64_t j = (uint64_t)op[6] + (u0 - as0 + (uint64_t)op[8]) * (uint64_t)op[7] +
                                   (u1 - as1 + (uint64_t)op[9]);                // Eq. 6
                if (j >= (uint64_t)shard_numel[(uint64_t)op[1]]) return 1;
                dst[j] = values[q];                                          // Eq. 7
            }
        }
    }
    return 0;
}
