// Test oracle for the fused star-join query: TEST INFRASTRUCTURE ONLY.
//
// A plain, slow, single-threaded restatement of what the query means
// (Section 4.2.2 of the paper: the fact table is the spine; a selection
// narrows the surviving rows, a join probe drops rows without a matching
// dimension key, a gather pulls a dimension attribute into the row, and the
// terminal aggregates the survivors; Section 3.3 for the star-join SQL shape;
// Section 2.2 for the bit-for-bit integer acceptance rule).  Because the fused
// GPU pipeline reaches exactly the SQL result, this file is that definition
// written out: a row-at-a-time nested filter, a std::unordered_map per
// filtered dimension, and a std::map for the groups.  It shares no code,
// headers or tables with the CUDA path, and nothing outside tests, the smoke
// check and the benchmark's CPU-baseline leg may call it.
//
// Integer semantics: column values are sign-extended to 64 bits before any
// arithmetic (the 64-bit product of Listing 2); sums wrap modulo 2^64; `%`
// truncates toward zero as in C.  Every function here is pinned by the CPU
// tests (brute-force nested loops, hand-computed examples, closed forms and
// invariants); nothing is "parity unpinned".

#include <chrono>
#include <cstdint>
#include <map>
#include <new>
#include <unordered_map>
#include <vector>

namespace {

enum { ORC_OK = 0, ORC_DUP_KEY = 1, ORC_GROUP_RANGE = 2, ORC_INVALID = 3 };
enum { OP_EQ = 0, OP_NE, OP_LT, OP_LE, OP_GT, OP_GE, OP_BETWEEN, OP_IN };
enum { AGG_COL = 0, AGG_MUL, AGG_SUB, AGG_ADD };
enum { SRC_FACT = 0, SRC_PAYLOAD = 1 };
enum { MODE_SCALAR = 0, MODE_DENSE = 1, MODE_HASHED = 2 };

} // namespace

extern "C" {

struct orc_col {
    const void *data;
    int32_t is64;
    int64_t n;
};
struct orc_pred {
    int32_t col;
    int32_t op;
    int64_t lo, hi;
    const int64_t *set;
    int32_t nset;
};
struct orc_term {
    int32_t src, a, b;
    int64_t mult;
};
struct orc_key {
    orc_term t[4];
    int32_t nterms;
    int64_t offset, modulo;
};
struct orc_agg {
    int32_t op;
    orc_term x, y;
    int32_t want_count;
};
struct orc_dim {
    std::unordered_map<int64_t, std::vector<int64_t>> rows; // key -> payload tuple
};
struct orc_join {
    int32_t fk_col;
    const orc_dim *dim;
};
struct orc_group {
    int64_t sum, count;
};
struct orc_result {
    std::map<int64_t, orc_group> groups;
};

} // extern "C"

namespace {

inline int64_t cell(const orc_col &c, int64_t i)
{
    return c.is64 ? static_cast<const int64_t *>(c.data)[i]
                  : static_cast<int64_t>(static_cast<const int32_t *>(c.data)[i]);
}

inline bool holds(const orc_pred &p, int64_t v)
{
    switch (p.op) {
    case OP_EQ: return v == p.lo;
    case OP_NE: return v != p.lo;
    case OP_LT: return v < p.lo;
    case OP_LE: return v <= p.lo;
    case OP_GT: return v > p.lo;
    case OP_GE: return v >= p.lo;
    case OP_BETWEEN: return v >= p.lo && v <= p.hi; // inclusive both ends
    case OP_IN:
        for (int k = 0; k < p.nset; ++k)
            if (v == p.set[k]) return true;
        return false;
    }
    return false;
}

// wrap-around helpers (two's complement, no signed-overflow UB)
inline int64_t wadd(int64_t a, int64_t b) { return (int64_t)((uint64_t)a + (uint64_t)b); }
inline int64_t wsub(int64_t a, int64_t b) { return (int64_t)((uint64_t)a - (uint64_t)b); }
inline int64_t wmul(int64_t a, int64_t b) { return (int64_t)((uint64_t)a * (uint64_t)b); }

} // namespace

extern "C" {

// Filtered dimension: every row passing all predicates is entered under its
// key with its payload tuple.  A repeated key among the passing rows is an
// error (the paper's tables are indexed by primary key, Section 3.3).
orc_dim *orc_dim_build(const orc_col *cols, int ncols, const orc_pred *preds, int npreds, int key_col,
                       const int *payload_cols, int npayload, int *status)
{
    *status = ORC_OK;
    if (ncols <= 0 || key_col < 0 || key_col >= ncols) {
        *status = ORC_INVALID;
        return nullptr;
    }
    orc_dim *d = new (std::nothrow) orc_dim();
    if (!d) {
        *status = ORC_INVALID;
        return nullptr;
    }
    const int64_t n = cols[key_col].n;
    for (int64_t r = 0; r < n; ++r) {
        bool ok = true;
        for (int k = 0; k < npreds && ok; ++k) ok = holds(preds[k], cell(cols[preds[k].col], r));
        if (!ok) continue;
        std::vector<int64_t> pay(npayload);
        for (int k = 0; k < npayload; ++k) pay[k] = cell(cols[payload_cols[k]], r);
        auto ins = d->rows.emplace(cell(cols[key_col], r), std::move(pay));
        if (!ins.second) *status = ORC_DUP_KEY;
    }
    return d;
}

int64_t orc_dim_size(const orc_dim *d) { return d ? (int64_t)d->rows.size() : 0; }
void orc_dim_free(orc_dim *d) { delete d; }

// The query over fact rows [row_begin, row_end).
orc_result *orc_run(const orc_col *fact, int nfact, int64_t row_begin, int64_t row_end, const orc_pred *preds,
                    int npreds, const orc_join *joins, int njoins, const orc_key *key, const orc_agg *agg, int mode,
                    int64_t num_groups, int *status, double *seconds)
{
    *status = ORC_OK;
    orc_result *res = new (std::nothrow) orc_result();
    if (!res || nfact <= 0 || njoins > 16 || (mode != MODE_SCALAR && !key)) {
        *status = ORC_INVALID;
        return res;
    }
    const std::vector<int64_t> *hit[16];
    auto term = [&](const orc_term &t, int64_t i) -> int64_t {
        int64_t raw = (t.src == SRC_FACT) ? cell(fact[t.a], i) : (*hit[t.a])[t.b];
        return wmul(t.mult, raw);
    };
    const auto t0 = std::chrono::steady_clock::now();
    for (int64_t i = row_begin; i < row_end; ++i) {
        bool ok = true;
        for (int k = 0; k < npreds && ok; ++k) ok = holds(preds[k], cell(fact[preds[k].col], i));
        if (!ok) continue;
        for (int j = 0; j < njoins && ok; ++j) {
            auto it = joins[j].dim->rows.find(cell(fact[joins[j].fk_col], i));
            if (it == joins[j].dim->rows.end()) ok = false;
            else hit[j] = &it->second;
        }
        if (!ok) continue;
        int64_t g = 0;
        if (mode != MODE_SCALAR) {
            g = key->offset;
            for (int t = 0; t < key->nterms; ++t) g = wadd(g, term(key->t[t], i));
            if (key->modulo != 0) g = g % key->modulo;
            if (mode == MODE_DENSE && (g < 0 || g >= num_groups)) {
                *status = ORC_GROUP_RANGE;
                continue;
            }
        }
        int64_t v = term(agg->x, i);
        switch (agg->op) {
        case AGG_COL: break;
        case AGG_MUL: v = wmul(v, term(agg->y, i)); break;
        case AGG_SUB: v = wsub(v, term(agg->y, i)); break;
        case AGG_ADD: v = wadd(v, term(agg->y, i)); break;
        }
        orc_group &slot = res->groups[g];
        slot.sum = wadd(slot.sum, v);
        slot.count += 1;
    }
    const auto t1 = std::chrono::steady_clock::now();
    if (seconds) *seconds = std::chrono::duration<double>(t1 - t0).count();
    return res;
}

int64_t orc_result_groups(const orc_result *r) { return r ? (int64_t)r->groups.size() : 0; }

// Groups in ascending key order.
void orc_result_copy(const orc_result *r, int64_t *keys, int64_t *sums, int64_t *counts)
{
    int64_t k = 0;
    for (const auto &kv : r->groups) {
        keys[k] = kv.first;
        sums[k] = kv.second.sum;
        counts[k] = kv.second.count;
        ++k;
    }
}

void orc_result_free(orc_result *r) { delete r; }

} // extern "C"
