// Host side of sjq_run: validation, the plan (evaluation order, which tables
// are staged in shared memory, which aggregation path), and the launches.
//
// The order rule follows the paper's observation that bytes moved, not
// arithmetic, decide the run time (Section 3.2): evaluate first what removes
// the most rows per byte read, so that later columns are loaded for few rows.
// The aggregation rule follows Section 3.3: privatise the group table in
// shared memory only when it fits and many survivors contend on it; keep the
// global table when few rows survive or the groups are many.  The rows-per-
// thread choice of Section 4.3.1 ("asymmetric batching") is the fixed four
// rows per 128-bit load here; occupancy supplies the memory-level parallelism.
#include <algorithm>
#include <cstring>
#include <vector>

#include "sjq_run.cuh"

// Block size the ahead-of-time kernels are built for (their launch bound); a build for experiments may set another.
#ifndef SJQ_LB_THREADS
#define SJQ_LB_THREADS 384
#endif
#define SJQ_LB_THREADS_MAX SJQ_LB_THREADS

namespace sjq {

sjq_status fused_occupancy(int agg, bool mul, bool hash, int block, size_t smem, int *ctas_per_sm);
sjq_status jit_occupancy(const RunParams &P, int agg, bool mul, bool hash, int block, int lb_blocks, size_t smem,
                         int *ctas_per_sm);
sjq_status jit_launch(const RunParams &P, int agg, bool mul, bool hash, int grid, int block, int lb_blocks,
                      size_t smem, cudaStream_t stream);
sjq_status fused_launch(int agg, bool mul, bool hash, int grid, int block, size_t smem, const RunParams &P,
                        cudaStream_t stream);
sjq_status clear_launch(int64_t *sums, int64_t *counts, int64_t cells, int64_t *gkeys, int64_t gslots,
                        int64_t *n_groups, int32_t *status, int sm_count, cudaStream_t stream);
sjq_status compact_launch(const int64_t *gkeys, const int64_t *gsums, const int64_t *gcounts, int64_t gslots,
                          bool indexed, int64_t dense_base, int64_t *keys, int64_t *sums, int64_t *counts,
                          int64_t capacity, int64_t *n_groups, int32_t *status, int sm_count, cudaStream_t stream);

size_t unfused_scratch_bytes(int64_t n, int gathering_joins);
sjq_status unfused_launch(const RunParams &P, int nfilter, int agg, bool mul, bool has_hash, void *scratch,
                          size_t scratch_bytes, int sm_count, cudaStream_t stream, int *launches);
sjq_status sample_launch(const sjq_col *fact, const DPred *preds, int npreds, int64_t n, unsigned long long *counts,
                         cudaStream_t stream);
sjq_status hot_launch(const void *col, bool is64, int64_t n, const sjq_table *T, void *scratch, cudaStream_t stream,
                      const void **hot_table, int *launches);
sjq_status merge_launch(const int64_t *keys, const int64_t *sums, const int64_t *counts, int64_t n, int64_t *gkeys,
                        int64_t *gsums, int64_t *gcounts, uint64_t gmask, int32_t *status, int sm_count,
                        cudaStream_t stream);

namespace {

struct StageSpec {
    int kind;     // ST_PRED / ST_PROBE / ST_LOAD
    int index;    // predicate or join index (-1 for loads)
    int col;      // fact column
    double sel;   // estimated fraction of rows passing
    double cost;  // relative cost per row evaluated
    int prefilter; // 1: only the presence bitmap of a hashed join; 2: the exact probe that follows one
};

// share of the rows surviving all filters from which a compiled kernel drops the survivor queues
constexpr double kDirectSurvival = 0.35;       // register accumulators
constexpr double kDirectSurvivalGrouped = 0.75; // group tables

double pred_selectivity(const sjq_pred &p)
{
    switch (p.op) {
    case SJQ_EQ: return 0.1;
    case SJQ_NE: return 0.9;
    case SJQ_IN: return std::min(0.5, 0.1 * std::max(1, p.nset));
    case SJQ_BETWEEN: return 0.25;
    default: return 0.4;
    }
}

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

uint64_t hashed_slots(int64_t capacity)
{
    uint64_t want = (uint64_t)std::max<int64_t>(capacity, 8) * 2;
    uint64_t slots = 16;
    while (slots < want) slots <<= 1;
    return slots;
}

bool valid_term(const sjq_term &t, int nfact, const sjq_join *joins, int njoins)
{
    if (t.src == SJQ_SRC_FACT) return t.a >= 0 && t.a < nfact;
    if (t.src == SJQ_SRC_PAYLOAD)
        return t.a >= 0 && t.a < njoins && t.b >= 0 && t.b < joins[t.a].table->layout.npayload;
    return false;
}

// The filter stages of a query (its predicates and joins; a hashed join with a presence bitmap is two
// stages) with estimated selectivities and relative costs, and the order they are evaluated in: the
// caller's, or by rank (1 - selectivity) / cost.
sjq_status order_stages(const sjq_col *fact, const sjq_pred *preds, int npreds, const sjq_join *joins, int njoins,
                        const sjq_run_opts &opts, std::vector<StageSpec> *specs_out, std::vector<int> *order_out)
{
    std::vector<StageSpec> &specs = *specs_out;
    std::vector<int> &order = *order_out;
    // a measured pass fraction (parts per million) replaces the estimate where the caller supplies one
    auto hinted = [&](int i, double estimate) {
        const int32_t ppm = opts.pass_ppm[i];
        return ppm > 0 ? std::min(1.0, ppm / 1e6) : estimate;
    };
    for (int p = 0; p < npreds; ++p) {
        const double bytes = fact[preds[p].col].dtype == SJQ_I64 ? 2.0 : 1.0;
        specs.push_back({ST_PRED, p, preds[p].col, hinted(p, pred_selectivity(preds[p])), bytes, 0});
    }
    for (int j = 0; j < njoins; ++j) {
        const sjq_table *T = joins[j].table;
        const sjq_dim_layout &L = T->layout;
        const double bytes = L.key_dtype == SJQ_I64 ? 2.0 : 1.0;
        const double sel = hinted(npreds + j, L.dim_rows > 0 ? (double)L.entries / (double)L.dim_rows : 0.0);
        // bytes a filter stage on this table touches: the presence bitmap when a direct table has one
        const size_t tb = (is_direct_kind(L.kind) && L.filter_bits > 0 && T->filter && !opts.no_filter_bitmap)
                              ? (size_t)(L.filter_bits / 8)
                              : L.table_bytes;
        // relative cost of one probe: a table the L1 mostly holds, one the L2 holds (measured on the four-join
        // workload: the 3 MB map before the 175 KB bitmap when it drops twice as many rows), one in HBM
        double probe = tb <= (size_t)200 << 10 ? 0.3 : tb <= (size_t)32 << 20 ? 0.6 : 4.0;
        if (is_hash_kind(L.kind) && T->filter && L.filter_bits > 0) {
            // a hashed join is two stages: its presence bitmap (cheap, passes the hits and ~1/16 of the
            // misses) early, the exact probe (expensive) on what is left
            const double fp = std::min(1.0, (double)L.entries / (double)L.filter_bits);
            const double pass = std::min(1.0, sel + (1.0 - sel) * fp);
            specs.push_back({ST_PROBE, j, joins[j].fk_col, pass, bytes + 0.7, 1});
            specs.push_back({ST_PROBE, j, joins[j].fk_col, pass > 0 ? std::min(1.0, sel / pass) : 1.0,
                             bytes + probe + 4.0, 2});
            continue;
        }
        specs.push_back({ST_PROBE, j, joins[j].fk_col, std::min(1.0, sel), bytes + probe, 0});
    }
    const int nfilter = (int)specs.size();
    if (opts.norder) {
        // the caller orders predicates and joins; a hashed join's bitmap and exact probe stay adjacent
        std::vector<char> seen(npreds + njoins, 0);
        for (int i = 0; i < npreds + njoins; ++i) {
            const int o = opts.order[i];
            if (o < 0 || o >= npreds + njoins || seen[o]) return SJQ_ERR_INVALID_ARG;
            seen[o] = 1;
            for (int k = 0; k < nfilter; ++k) {
                const bool match = o < npreds ? (specs[k].kind == ST_PRED && specs[k].index == o)
                                              : (specs[k].kind == ST_PROBE && specs[k].index == o - npreds);
                if (match) order.push_back(k);
            }
        }
    } else {
        order.resize(nfilter);
        for (int i = 0; i < nfilter; ++i) order[i] = i;
        std::stable_sort(order.begin(), order.end(), [&](int a, int b) {
            // exact probes of prefiltered hashed joins go last: they run at the final level
            if ((specs[a].prefilter == 2) != (specs[b].prefilter == 2)) return specs[b].prefilter == 2;
            return (1.0 - specs[a].sel) / specs[a].cost > (1.0 - specs[b].sel) / specs[b].cost;
        });
    }

    return SJQ_OK;
}

} // namespace
} // namespace sjq

using namespace sjq;

extern "C" sjq_status sjq_unfused_scratch_bytes(int64_t rows, int njoins, size_t *bytes)
{
    if (rows < 0 || njoins < 0 || njoins > SJQ_MAX_JOINS || !bytes) return SJQ_ERR_INVALID_ARG;
    *bytes = unfused_scratch_bytes(rows, njoins);
    return SJQ_OK;
}

extern "C" sjq_status sjq_run_workspace_bytes(const sjq_result_spec *spec, size_t *bytes)
{
    if (!spec || !bytes) return SJQ_ERR_INVALID_ARG;
    *bytes = 0;
    if (spec->mode == SJQ_HASHED) {
        if (spec->capacity <= 0) return SJQ_ERR_INVALID_ARG;
        *bytes = align_up((size_t)(hashed_slots(spec->capacity) + 1) * 8, 256) * 3;
    } else if (spec->mode != SJQ_SCALAR && spec->mode != SJQ_DENSE) {
        return SJQ_ERR_INVALID_ARG;
    }
    return SJQ_OK;
}

// ---------------------------------------------------------------------------
// Measured predicate selectivities.
namespace {

int32_t ppm_of(int64_t passed, int64_t sampled)
{
    if (sampled <= 0) return 0; // nothing sampled: no hint
    const int64_t ppm = (passed * 1000000 + sampled / 2) / sampled;
    return (int32_t)std::min<int64_t>(std::max<int64_t>(ppm, 1), 1000000);
}

} // namespace

extern "C" sjq_status sjq_pred_sample_begin(const sjq_col *fact, int nfact, const sjq_pred *preds, int npreds,
                                            void *scratch_dev, int64_t *host_counts, void *stream_)
{
    if (!fact || nfact <= 0 || nfact > 64 || npreds < 0 || npreds > SJQ_MAX_PREDS || (npreds && !preds) ||
        !scratch_dev || !host_counts)
        return SJQ_ERR_INVALID_ARG;
    if (!aligned16(scratch_dev)) return SJQ_ERR_ALIGN;
    const int64_t n = fact[0].n;
    DPred d[SJQ_MAX_PREDS];
    for (int c = 0; c < nfact; ++c) {
        if (fact[c].n != n || n < 0 || (fact[c].dtype != SJQ_I32 && fact[c].dtype != SJQ_I64) ||
            (n > 0 && !fact[c].data))
            return SJQ_ERR_INVALID_ARG;
        if (!aligned16(fact[c].data)) return SJQ_ERR_ALIGN;
    }
    for (int p = 0; p < npreds; ++p) {
        if (preds[p].col < 0 || preds[p].col >= nfact) return SJQ_ERR_INVALID_ARG;
        if (!canon_pred(preds[p], fact[preds[p].col].dtype, &d[p])) return SJQ_ERR_INVALID_ARG;
    }
    cudaStream_t stream = (cudaStream_t)stream_;
    unsigned long long *counts = static_cast<unsigned long long *>(scratch_dev);
    sjq_status st = sample_launch(fact, d, npreds, n, counts, stream);
    if (st != SJQ_OK) return st;
    if (cudaMemcpyAsync(host_counts, counts, (SJQ_MAX_PREDS + 1) * sizeof(int64_t), cudaMemcpyDeviceToHost, stream) !=
        cudaSuccess) {
        (void)cudaGetLastError();
        return SJQ_ERR_CUDA;
    }
    return SJQ_OK;
}

extern "C" sjq_status sjq_pred_sample_end(const int64_t *host_counts, int npreds, int32_t *pass_ppm)
{
    if (!host_counts || npreds < 0 || npreds > SJQ_MAX_PREDS || (npreds && !pass_ppm)) return SJQ_ERR_INVALID_ARG;
    for (int p = 0; p < npreds; ++p) pass_ppm[p] = ppm_of(host_counts[1 + p], host_counts[0]);
    return SJQ_OK;
}

extern "C" sjq_status sjq_pred_sample(const sjq_col *fact, int nfact, const sjq_pred *preds, int npreds,
                                      void *scratch_dev, void *stream_, int32_t *pass_ppm)
{
    int64_t h[SJQ_MAX_PREDS + 1];
    sjq_status st = sjq_pred_sample_begin(fact, nfact, preds, npreds, scratch_dev, h, stream_);
    if (st != SJQ_OK) return st;
    if (cudaStreamSynchronize((cudaStream_t)stream_) != cudaSuccess) {
        (void)cudaGetLastError();
        return SJQ_ERR_CUDA;
    }
    return sjq_pred_sample_end(h, npreds, pass_ppm);
}

extern "C" sjq_status sjq_run(const sjq_col *fact, int nfact, const sjq_pred *preds, int npreds,
                              const sjq_join *joins, int njoins, const sjq_key_expr *key, const sjq_agg_expr *agg,
                              const sjq_result_spec *spec, const sjq_result *out, const sjq_run_opts *opts_,
                              void *stream_, sjq_run_info *info)
{
    // ------------------------------------------------------------ validation
    if (!fact || nfact <= 0 || nfact > 64 || npreds < 0 || npreds > SJQ_MAX_PREDS || (npreds && !preds) ||
        njoins < 0 || njoins > SJQ_MAX_JOINS || (njoins && !joins) || !agg || !spec || !out || !out->status ||
        !out->sums)
        return SJQ_ERR_INVALID_ARG;
    sjq_run_opts opts{};
    if (opts_) opts = *opts_;
    const int64_t n = fact[0].n;
    if (n < 0) return SJQ_ERR_INVALID_ARG;
    for (int c = 0; c < nfact; ++c) {
        if (fact[c].n != n || (fact[c].dtype != SJQ_I32 && fact[c].dtype != SJQ_I64)) return SJQ_ERR_INVALID_ARG;
        if (n > 0 && !fact[c].data) return SJQ_ERR_INVALID_ARG;
        if (!aligned16(fact[c].data)) return SJQ_ERR_ALIGN;
    }
    if (spec->mode != SJQ_SCALAR && spec->mode != SJQ_DENSE && spec->mode != SJQ_HASHED) return SJQ_ERR_INVALID_ARG;
    if ((spec->mode == SJQ_SCALAR) != (key == nullptr)) return SJQ_ERR_INVALID_ARG;
    if (spec->mode == SJQ_DENSE && spec->num_groups <= 0) return SJQ_ERR_INVALID_ARG;
    if (spec->mode == SJQ_HASHED &&
        (spec->capacity <= 0 || !out->keys || !out->counts || !out->n_groups || !out->workspace))
        return SJQ_ERR_INVALID_ARG;
    if (agg->want_count && !out->counts) return SJQ_ERR_INVALID_ARG;
    if (agg->op < SJQ_AGG_COL || agg->op > SJQ_AGG_ADD) return SJQ_ERR_INVALID_ARG;
    if (!aligned16(out->sums) || !aligned16(out->counts) || !aligned16(out->keys) || !aligned16(out->workspace) ||
        (reinterpret_cast<uintptr_t>(out->status) & 3u) || (reinterpret_cast<uintptr_t>(out->n_groups) & 7u))
        return SJQ_ERR_ALIGN;
    for (int j = 0; j < njoins; ++j) {
        const sjq_table *T = joins[j].table;
        if (!T || T->magic != kTableMagic || joins[j].fk_col < 0 || joins[j].fk_col >= nfact)
            return SJQ_ERR_INVALID_ARG;
        if (fact[joins[j].fk_col].dtype != T->layout.key_dtype) return SJQ_ERR_UNSUPPORTED;
    }
    for (int p = 0; p < npreds; ++p)
        if (preds[p].col < 0 || preds[p].col >= nfact) return SJQ_ERR_INVALID_ARG;
    if (key) {
        if (key->nterms < 0 || key->nterms > SJQ_MAX_KEY_TERMS) return SJQ_ERR_INVALID_ARG;
        for (int t = 0; t < key->nterms; ++t)
            if (!valid_term(key->t[t], nfact, joins, njoins)) return SJQ_ERR_INVALID_ARG;
    }
    if (!valid_term(agg->x, nfact, joins, njoins)) return SJQ_ERR_INVALID_ARG;
    if (agg->op != SJQ_AGG_COL && !valid_term(agg->y, nfact, joins, njoins)) return SJQ_ERR_INVALID_ARG;
    // the ahead-of-time kernels are bounded at SJQ_LB_THREADS_MAX; a specialised kernel is compiled for its block size
    if (opts.block_threads && (opts.block_threads < 128 || opts.block_threads % 32 ||
                               opts.block_threads > (opts.specialise ? 1024 : SJQ_LB_THREADS_MAX)))
        return SJQ_ERR_INVALID_ARG;
    if (opts.rows_per_lane != 0 && opts.rows_per_lane != 4 && !(opts.rows_per_lane == 8 && opts.specialise))
        return SJQ_ERR_INVALID_ARG;
    if (opts.dense_slots != 0 && opts.dense_slots != 2 && !(opts.dense_slots == 4 && opts.specialise))
        return SJQ_ERR_INVALID_ARG;
    if (opts.norder && opts.norder != npreds + njoins) return SJQ_ERR_INVALID_ARG;
    if (opts.hot_keys < 0 || opts.hot_keys > 2) return SJQ_ERR_INVALID_ARG;
    if (opts.hot_scratch && !aligned16(opts.hot_scratch)) return SJQ_ERR_ALIGN;

    DeviceInfo dev;
    sjq_status st = device_info(&dev);
    if (st != SJQ_OK) return st;
    cudaStream_t stream = (cudaStream_t)stream_;

    // ------------------------------------------------------------ stage list
    std::vector<StageSpec> specs;
    std::vector<int> order;
    if ((st = order_stages(fact, preds, npreds, joins, njoins, opts, &specs, &order)) != SJQ_OK) return st;
    const int nfilter = (int)specs.size();

    // ------------------------------------------------------------ accumulators
    // Every term adds mult * value to one accumulator; fold the expressions
    // into per-source multipliers: src_mult[source][dest].
    struct Contribution { int src, a, b, dest; int64_t mult; };
    std::vector<Contribution> contrib;
    auto add_term = [&](const sjq_term &t, int dest, int64_t sign) {
        contrib.push_back({t.src, t.a, t.b, dest, (int64_t)((uint64_t)t.mult * (uint64_t)sign)});
    };
    // a key taken modulo 1 is 0 whatever its terms are: they are neither loaded nor gathered
    if (key && key->modulo != 1)
        for (int t = 0; t < key->nterms; ++t) add_term(key->t[t], kAccKey, 1);
    const bool mul = agg->op == SJQ_AGG_MUL;
    add_term(agg->x, kAccX, 1);
    if (agg->op == SJQ_AGG_MUL) add_term(agg->y, kAccY, 1);
    if (agg->op == SJQ_AGG_SUB) add_term(agg->y, kAccX, -1);
    if (agg->op == SJQ_AGG_ADD) add_term(agg->y, kAccX, 1);

    RunParams P;
    std::memset(&P, 0, sizeof(P));
    P.n = n;
    int ns = 0;
    int nsets = 0;
    std::vector<int> stage_of_join(njoins, -1);
    std::vector<int> stage_of_col(nfact, -1);
    std::vector<int> stage_label;
    auto fill_stage = [&](DStage &S, const StageSpec &sp) -> sjq_status {
        S.kind = (uint8_t)sp.kind;
        S.col = fact[sp.col].data;
        S.is64 = (uint8_t)(fact[sp.col].dtype == SJQ_I64);
        S.op = OP_LOAD;
        if (sp.kind == ST_PRED) {
            DPred d;
            if (!canon_pred(preds[sp.index], fact[sp.col].dtype, &d)) return SJQ_ERR_INVALID_ARG;
            if (d.nset) {
                S.op = OP_PRED_SET;
                S.nset = d.nset;
                S.set_idx = (uint8_t)nsets;
                for (int k = 0; k < d.nset; ++k) P.sets[nsets][k] = d.set[k];
                ++nsets;
            } else {
                S.op = OP_PRED_RANGE;
                S.lo = d.lo;
                S.hi = d.hi;
                S.neg = d.neg;
                S.never = d.never;
                S.lo32 = d.lo32;
                S.width32 = d.never ? 0u : (uint32_t)d.hi32 - (uint32_t)d.lo32;
            }
        } else if (sp.kind == ST_PROBE) {
            const sjq_table *T = joins[sp.index].table;
            const sjq_dim_layout &L = T->layout;
            if (L.slots > ((int64_t)1 << 31) && is_hash_kind(L.kind)) return SJQ_ERR_UNSUPPORTED;
            S.op = (uint8_t)(L.kind == SJQ_TABLE_DIRECT_BITMAP ? OP_DIRECT_BITMAP
                             : L.kind == SJQ_TABLE_DIRECT_U8   ? OP_DIRECT_U8
                             : L.kind == SJQ_TABLE_DIRECT_U16  ? OP_DIRECT_U16
                             : L.kind == SJQ_TABLE_DIRECT_U32  ? OP_DIRECT_U32
                             : L.kind == SJQ_TABLE_DIRECT_U64  ? OP_DIRECT_U64
                             : L.kind == SJQ_TABLE_DIRECT_U4   ? OP_DIRECT_U4
                             : L.kind == SJQ_TABLE_DIRECT_U2   ? OP_DIRECT_U2
                             : L.kind == SJQ_TABLE_HASH_I32    ? OP_HASH32
                                                               : OP_HASH64);
            S.tab = T->slots;
            S.kmin = L.kmin;
            S.last = (uint64_t)L.slots - 1;
            S.full = (uint8_t)(L.code_bits > 0 && L.code_bits < 8 && L.entries == L.slots);
            if (is_hash_kind(L.kind)) {
                S.last = (uint64_t)(T->slots_bytes / kBucketBytes); // bucket count
                S.wide = (uint8_t)((reinterpret_cast<uintptr_t>(T->slots) & 31u) == 0);
                if (sp.prefilter == 1) {
                    S.op = OP_HASHBITS;
                    S.tab = T->filter;
                }
            }
            S.kmin32 = (int32_t)L.kmin;
            S.last32 = (uint32_t)std::min<uint64_t>((uint64_t)L.slots - 1, 0xFFFFFFFFull);
            // with 2^32 slots or more every 32-bit index is in range and nothing is clamped
            S.clamp32 = (uint32_t)std::min<uint64_t>((uint64_t)L.slots, 0xFFFFFFFFull);
            S.hmask = sp.prefilter == 1 ? (uint64_t)L.filter_bits - 1 : 0;
            S.pmin0 = L.pay_min[0];
            S.pmin1 = L.pay_min[1];
            S.pbits0 = (uint8_t)L.pay_bits[0];
            S.pmask0 = L.pay_bits[0] >= 64 ? ~0ULL : ((1ULL << L.pay_bits[0]) - 1ULL);
            S.code_bits = (uint8_t)L.code_bits;
            S.tab_bytes = (uint32_t)std::min<size_t>(T->slots_bytes, 0xFFFFFFF0u);
        }
        return SJQ_OK;
    };
    for (int i = 0; i < nfilter; ++i) {
        const StageSpec &sp = specs[order[i]];
        if (ns >= kMaxStages) return SJQ_ERR_UNSUPPORTED;
        if ((st = fill_stage(P.st[ns], sp)) != SJQ_OK) return st;
        if (sp.kind == ST_PROBE && sp.prefilter != 1) stage_of_join[sp.index] = ns;
        if (stage_of_col[sp.col] < 0) stage_of_col[sp.col] = ns;
        stage_label.push_back(sp.kind == ST_PRED ? sp.index : npreds + sp.index);
        ++ns;
    }
    P.want_count = agg->want_count ? 1 : 0;
    P.status = out->status;
    if (key) {
        P.key_offset = key->offset;
        P.modulo = key->modulo;
        if (key->modulo > 0 && (key->modulo & (key->modulo - 1)) == 0) P.modmask = (uint64_t)key->modulo - 1;
        P.mod32 = key->modulo > 0 && key->modulo <= 0xFFFFFFFFLL;
    }

    // ------------------------------------------------------------ dense / sparse split
    // Fraction of rows reaching each filter stage, from the estimates.
    std::vector<double> reach(nfilter + 1, 1.0);
    for (int s = 0; s < nfilter; ++s) reach[s + 1] = reach[s] * specs[order[s]].sel;
    const double survivors = (double)n * reach[nfilter];
    // Level 0 runs, on thread-owned rows, the leading filter stages that still see a fair share of
    // the rows (a dense stage costs about the same per table row whatever survives, a queue-fed
    // level costs per surviving row, several times more: measured break-even between 20 % and 30 %).
    // Up to kMaxQueues - 1 later filter stages run as queue-fed levels; the rest at the final level.
    // Eager loading and compaction = never use no queue at all.
    int nd0 = 0, nfq = 0;
    // Most rows surviving every filter (by the measured fractions): each column is read for nearly every
    // 32-byte sector anyway, so queues would only add shared-memory traffic and turn 128-bit loads into 4-byte
    // ones.  A kernel compiled for the query then keeps thread-owned rows throughout and requests its columns
    // up front.
    // (A group-by terminal works on whatever lanes still hold a row, so with a shared-memory or global group
    // table compacted survivors keep paying until nearly all rows survive: measured on the selectivity sweep at
    // 50 %, one group 1.78 -> 1.44 ms without queues, a thousand groups 2.13 -> 2.32 ms.)
    const bool register_terminal = spec->mode == SJQ_SCALAR || (spec->mode == SJQ_DENSE && spec->num_groups == 1);
    const bool mostly_survive = opts.specialise && opts.compaction == 0 &&
                                reach[nfilter] >= (register_terminal ? kDirectSurvival : kDirectSurvivalGrouped);
    const bool direct = opts.eager_loads || opts.compaction == 1 || nfilter == 0 || opts.unfused || mostly_survive;
    if (!direct) {
        nd0 = 1;
        if (opts.compaction != 2) {
            const double dense_reach = 0.3;
            while (nd0 < nfilter && specs[order[nd0]].sel < 0.9 && reach[nd0] > dense_reach &&
                   specs[order[nd0]].prefilter != 2)
                ++nd0;
            while (nd0 + nfq < nfilter && nfq < kMaxQueues - 1 && specs[order[nd0 + nfq]].sel < 0.9 &&
                   reach[nd0 + nfq] > 0.002 && specs[order[nd0 + nfq]].prefilter != 2)
                ++nfq;
        }
    }
    const int ndense = nd0 + nfq; // stages that only filter (no accumulators)
    P.nd0 = nd0;
    P.nq = direct ? 0 : nfq + 1;
    P.rows = opts.rows_per_lane ? opts.rows_per_lane : 4;
    P.slots = (opts.specialise && opts.dense_slots == 4) ? 4 : 2;
    // a third or more of the rows reaching the first queue: pushes are dense enough for bank conflicts to matter
    P.qfold = (opts.specialise && P.nq && reach[nd0] >= 0.3) ? 7u : 0u;
    // fewer than about one row in seven surviving level 0: pushing by walking the set bits of a thread's mask beats
    // testing its eight rows one by one (city x brand 0.72 -> 0.68 ms, city x city 0.72 -> 0.71; at one in five,
    // the four-join workload, it loses: 1.19 -> 1.21 ms)
    P.sparse_push = (opts.specialise && P.nq && reach[nd0] < 0.15) ? 1 : 0;

    // Sources of the accumulators.  A dense stage cannot feed an accumulator
    // (it only keeps a bit per row), so a value it would supply is gathered
    // again for the survivors by a sparse copy of the stage.
    std::vector<int> gather_of_stage(ns, -1);
    for (const Contribution &c : contrib) {
        int s, src;
        if (c.src == SJQ_SRC_FACT) {
            if (stage_of_col[c.a] < 0) { // a column nobody filters on: plain load stage at the end
                if (ns >= kMaxStages) return SJQ_ERR_UNSUPPORTED;
                StageSpec sp{ST_LOAD, -1, c.a, 1.0, 1.0, 0};
                fill_stage(P.st[ns], sp);
                stage_of_col[c.a] = ns;
                stage_label.push_back(-1);
                gather_of_stage.push_back(-1);
                ++ns;
            }
            s = stage_of_col[c.a];
            src = 0;
        } else {
            s = stage_of_join[c.a];
            src = 1 + c.b;
        }
        if (s < ndense) {
            if (gather_of_stage[s] < 0) {
                if (ns >= kMaxStages) return SJQ_ERR_UNSUPPORTED;
                P.st[ns] = P.st[s];
                gather_of_stage[s] = ns;
                stage_label.push_back(stage_label[s]);
                gather_of_stage.push_back(-1);
                ++ns;
            }
            s = gather_of_stage[s];
        }
        DStage &S = P.st[s];
        const int slot = 3 * src + c.dest;
        S.mult[slot] = (int64_t)((uint64_t)S.mult[slot] + (uint64_t)c.mult);
        S.acc |= (uint16_t)(1u << slot);
    }
    // a gathered copy that only needs the raw value need not filter again
    for (int s = ndense; s < ns; ++s) {
        DStage &S = P.st[s];
        bool is_copy = false;
        for (int d = 0; d < ndense; ++d) is_copy |= gather_of_stage[d] == s;
        if (is_copy && (S.acc & ~0x7u) == 0) {
            S.kind = ST_LOAD;
            S.op = OP_LOAD;
        }
    }
    // A filter stage on a direct table with payloads probes the table's presence bitmap (an eighth to a
    // sixty-fourth of the code array, so far more of it stays in L1/L2); the payload is gathered from the
    // codes by the sparse copy, for the survivors only.
    std::vector<char> via_bitmap(ns, 0);
    if (!opts.no_filter_bitmap) {
        for (int s = 0; s < ndense; ++s) {
            DStage &S = P.st[s];
            if (S.kind != ST_PROBE || !is_code_op(S.op)) continue;
            const sjq_table *T = joins[specs[order[s]].index].table;
            if (!T->filter || T->layout.filter_bits <= 0) continue;
            S.op = OP_DIRECT_BITMAP;
            S.tab = T->filter;
            S.tab_bytes = (uint32_t)std::min<size_t>((size_t)(T->layout.filter_bits / 8), 0xFFFFFFF0u);
            via_bitmap[s] = 1;
        }
    }
    // 32-bit fast path of the accumulators: int32 column, multipliers and payload ranges within int32
    for (int s2 = 0; s2 < ns; ++s2) {
        DStage &S = P.st[s2];
        bool ok = !S.is64;
        for (int i = 0; i < 9; ++i) {
            ok = ok && S.mult[i] >= INT32_MIN && S.mult[i] <= INT32_MAX;
            S.mult32[i] = (int32_t)S.mult[i];
        }
        if (S.kind == ST_PROBE) {
            const int64_t hi0 = S.pmin0 + (int64_t)std::min<uint64_t>(S.pmask0, (uint64_t)INT32_MAX);
            ok = ok && S.code_bits <= 32 && S.pmin0 >= INT32_MIN && hi0 <= INT32_MAX && S.pmask0 <= 0x7FFFFFFFull;
            if (S.acc & 0x1C0u) {
                const int bits1 = (int)S.code_bits - (int)S.pbits0;
                ok = ok && bits1 < 31 && S.pmin1 >= INT32_MIN && S.pmin1 + ((int64_t)1 << std::max(bits1, 0)) <= INT32_MAX;
            }
        }
        S.acc32 = ok ? 1 : 0;
        S.simple = 0;
        if (ok && S.op == OP_LOAD && (S.acc == 1u || S.acc == 2u || S.acc == 4u))
            S.simple = (uint8_t)(1 + (S.acc == 1u ? 0 : S.acc == 2u ? 1 : 2));
    }
    P.nstages = ns;
    P.eager = opts.eager_loads ? 1 : 0;
    P.count32 = n < ((int64_t)1 << 32) ? 1 : 0;
    // Load schedule of the final level (used by kernels compiled for the query): a column is requested
    // once the last stage before it that is expected to drop rows has produced its mask, and at most
    // three columns ahead of the stage being processed.
    // Without queues a thread keeps its four consecutive rows and loads them with one 128-bit load, which is
    // skipped only when all four are dead: waiting for a mask pays only behind a stage that keeps less than
    // about one row in six; everything else is requested up front, four columns deep.
    {
        const int first = ndense, depth = P.nq ? 3 : 4;
        const double drop_below = P.nq ? 0.9 : 0.16;
        int last_barrier = first - 1;
        for (int t = first; t < ns; ++t) {
            P.st[t].issue_after = (int8_t)std::max(std::max(last_barrier, t - depth), first - 1);
            const bool drops = t < nfilter && specs[order[t]].sel < drop_below;
            if (drops) last_barrier = t;
        }
    }

    // A hashed result whose key is taken modulo M can only hold keys in (-M, M): when 2M - 1 cells fit the
    // workspace arrays the group table is indexed directly by key + M - 1 (no key array, no hashing, no claim:
    // two atomics per row instead of a look-up and two atomics; every dense aggregation path applies) and the
    // compaction recovers the keys from the cell numbers (config 4, G = 10^6 at 10 %: 3.2 -> 1.6 ms).
    // The same holds for a key without a modulo whose every term is a gathered payload: the tables know the
    // range of each payload among the rows they hold, so the key's range is known before the run (the
    // paper's city x city and city x brand keys, Section 3.3, are of this kind).  Whenever the range fits, the
    // indexed table is chosen: its clear and its compaction touch no more cells than the hash table's (whose
    // size follows the capacity, not the survivors), and a row costs less.
    const uint64_t gslots_all = spec->mode == SJQ_HASHED ? hashed_slots(spec->capacity) : 0;
    bool key_bounded = spec->mode == SJQ_HASHED && key != nullptr;
    __int128 key_lo = key ? key->offset : 0, key_hi = key_lo;
    for (int t = 0; key_bounded && t < key->nterms; ++t) {
        const sjq_term &T = key->t[t];
        if (T.src != SJQ_SRC_PAYLOAD) {
            key_bounded = false;
            break;
        }
        const sjq_dim_layout &L = joins[T.a].table->layout;
        const __int128 a = (__int128)T.mult * L.pay_min[T.b], b = (__int128)T.mult * L.pay_max[T.b];
        key_lo += a < b ? a : b;
        key_hi += a < b ? b : a;
    }
    if (key && key->modulo > 0) {
        // C remainder: the sign follows the dividend, the magnitude stays below the modulus
        const __int128 m1 = (__int128)key->modulo - 1;
        const bool nonneg = key_bounded && key_lo >= 0, nonpos = key_bounded && key_hi <= 0;
        key_lo = nonneg ? 0 : -m1;
        key_hi = nonpos ? 0 : m1;
        key_bounded = spec->mode == SJQ_HASHED;
    }
    const __int128 key_cells = key_hi - key_lo + 1;
    const bool direct_groups = key_bounded && !opts.group_hash_always && key_cells >= 1 &&
                               key_cells <= (__int128)gslots_all + 1 && key_lo > INT64_MIN && key_hi < INT64_MAX;
    const int64_t table_groups = direct_groups ? (int64_t)key_cells : spec->num_groups;
    if (direct_groups) {
        P.post_offset = (int64_t)-key_lo;
        P.want_count = 1; // the counts tell which cells hold a group
    }
    // ------------------------------------------------------------ aggregation path
    int aggp;
    size_t group_bytes = 0;
    const int approx_grid = dev.sm_count * 2;
    if (spec->mode == SJQ_SCALAR) {
        aggp = AGG_SCALAR;
    } else if (spec->mode == SJQ_HASHED && !direct_groups) {
        aggp = AGG_HASH;
    } else if (spec->mode == SJQ_DENSE && spec->num_groups == 1) {
        aggp = AGG_SCALAR; // a single group: register accumulation, key only range-checked
        P.has_key = 1;
    } else {
        const size_t gb = (size_t)table_groups * 8 * (P.want_count ? 2 : 1);
        const bool fits = gb <= (size_t)64 << 10;
        bool contended = survivors / approx_grid >= 8.0 * (double)table_groups;
        if (opts.unfused) {
            aggp = AGG_GLOBAL;
        } else if (opts.agg_path == 1) {
            if (!fits) return SJQ_ERR_UNSUPPORTED;
            aggp = AGG_SMEM;
        } else if (opts.agg_path == 2) {
            aggp = AGG_GLOBAL;
        } else {
            aggp = (fits && contended) ? AGG_SMEM : AGG_GLOBAL;
        }
        if (aggp == AGG_SMEM) group_bytes = gb;
    }
    P.num_groups = spec->mode == SJQ_DENSE ? spec->num_groups : direct_groups ? table_groups : 0;
    // Adding the values of equal keys inside the warp before the atomics is an option, never the default: per-lane
    // shared-memory atomics on a few counters were faster at every group count measured (selectivity sweep at
    // 100 %: 2 groups 4.1 vs 4.4 ms, 4 groups 3.3 vs 5.2, 16 groups 2.7 vs 15, 1000 groups 2.9 vs 34).
    if (opts.warp_agg < 0 || opts.warp_agg > 2) return SJQ_ERR_INVALID_ARG;
    P.warp_agg = (aggp == AGG_SMEM || aggp == AGG_GLOBAL) && !opts.unfused && opts.warp_agg == 1;

    // ------------------------------------------------------------ result buffers
    int64_t *gkeys = nullptr, *gsums = nullptr, *gcounts = nullptr;
    uint64_t gslots = 0;
    if (spec->mode == SJQ_HASHED) {
        size_t need = 0;
        sjq_run_workspace_bytes(spec, &need);
        if (out->workspace_bytes < need) return SJQ_ERR_BUFFER_SMALL;
        gslots = hashed_slots(spec->capacity);
        const size_t arr = align_up((size_t)(gslots + 1) * 8, 256);
        gkeys = reinterpret_cast<int64_t *>(static_cast<char *>(out->workspace));
        gsums = reinterpret_cast<int64_t *>(static_cast<char *>(out->workspace) + arr);
        gcounts = reinterpret_cast<int64_t *>(static_cast<char *>(out->workspace) + 2 * arr);
        P.gmask = gslots - 1;
        P.gkeys = direct_groups ? nullptr : gkeys;
        P.sums = gsums;
        P.counts = gcounts;
    } else {
        P.sums = out->sums;
        P.counts = agg->want_count ? out->counts : nullptr;
    }

    // ------------------------------------------------------------ hot-key table
    // The first open-addressing join that filters through its presence bitmap gets a table of its heaviest
    // foreign keys in shared memory (built by three small kernels right before the fused pass), consulted by the
    // bitmap stage and by the exact probe.  Whether the keys are skewed at all is decided on the device (an empty
    // table switches the look-ups off).  Measured on the Zipf-skewed 64-bit-key workload (300 M rows, 2 009 keys
    // held, covering 47 % of the sample): fused kernel 1.61 -> 1.53 ms, whole call 1.65 -> 1.61 ms (the three
    // kernels cost about 40 us), so by default only a kernel compiled for the query on at least 2^26 rows uses it;
    // the interpreted kernel loses with it (3.5 -> 4.9 ms: the look-up does not fit its register budget).
    int hot_stage = -1;
    if (opts.hot_keys != 2 && opts.hot_scratch && opts.hot_scratch_bytes >= SJQ_HOT_SCRATCH_BYTES && !opts.unfused &&
        n > 0 && (opts.hot_keys == 1 || (opts.specialise && n >= ((int64_t)1 << 26)))) {
        for (int s2 = 0; s2 < ns && hot_stage < 0; ++s2)
            if (P.st[s2].op == OP_HASHBITS && P.st[s2].code_bits <= 32) hot_stage = s2;
    }
    size_t hot_bytes = hot_stage >= 0 ? align_up((size_t)(kHotSlots + 1) * 16, 16) : 0;

    // ------------------------------------------------------------ shared memory layout
    // [stage descriptors][staged tables][hot-key table][group table][per-warp survivor queues]
    int block = opts.block_threads ? opts.block_threads : SJQ_LB_THREADS;
    // A compiled kernel without queues whose rows all meet in a shared group table runs as two blocks of 640
    // threads per SM: two copies of the table instead of three and 40 warps instead of 36 (selectivity sweep at
    // 100 %, a thousand groups: 2.73 -> 2.52 ms; 64 groups 2.57 -> 2.39; 4000 groups 3.25 -> 2.56).
    // With register accumulators two blocks of 768 threads (48 warps at 42 registers) help while some rows still
    // drop (the sweep at 50 %, one group: 1.48 -> 1.41 ms) and cost a little when none does (100 %: 2.18 -> 2.22).
    const bool two_wide_blocks = opts.specialise && !opts.unfused && !opts.block_threads && !opts.ctas_per_sm &&
                                 P.nq == 0 && (aggp == AGG_SMEM || (aggp == AGG_SCALAR && reach[nfilter] < 0.8));
    if (two_wide_blocks) block = aggp == AGG_SMEM ? 640 : 768;
    const size_t smem_cap = (size_t)dev.max_smem_optin - 1024; // static reduce scratch + slack
    const size_t stage_bytes = align_up((size_t)ns * sizeof(DStage), 16);
    if (hot_bytes && stage_bytes + hot_bytes + group_bytes +
                             (P.nq ? (size_t)(block / 32) * (size_t)(queue0_cap_for(P.slots) + (P.nq - 1) * queue_cap_for(P.rows)) * 4 : 0) >
                         smem_cap) {
        hot_stage = -1; // no room beside the group table and the queues
        hot_bytes = 0;
    }
    auto queue_bytes = [&](int threads) { return P.nq ? (size_t)(threads / 32) * (size_t)(queue0_cap_for(P.slots) + (P.nq - 1) * queue_cap_for(P.rows)) * 4 : (size_t)0; };
    // Direct tables (and presence bitmaps) worth a copy in shared memory, most probes per staged byte first.
    auto stage_tables = [&](int threads, size_t *tables_out) -> bool {
        for (int s2 = 0; s2 < ns; ++s2) P.st[s2].in_smem = 0, P.st[s2].smem_off = 0;
        const size_t fixed = stage_bytes + hot_bytes + group_bytes + queue_bytes(threads);
        if (fixed > smem_cap) return false;
        const size_t table_budget = smem_cap - fixed;
        size_t tables = 0;
        if (opts.smem_tables != 1 && !opts.unfused) {
            std::vector<int> cand;
            for (int s = 0; s < nfilter; ++s)
                if (is_direct_op(P.st[s].op)) cand.push_back(s);
            std::stable_sort(cand.begin(), cand.end(), [&](int a, int b) {
                return reach[a] / (double)P.st[a].tab_bytes > reach[b] / (double)P.st[b].tab_bytes;
            });
            for (int s : cand) {
                DStage &S = P.st[s];
                const size_t tb = align_up(S.tab_bytes, 16);
                if (tables + tb > table_budget) continue;
                // larger tables are left to L1/L2: shared memory taken here is L1 capacity lost to every other table
                if (opts.smem_tables == 0 && tb > (size_t)32 << 10) continue;
                if (opts.smem_tables >= 1024 && tb > (size_t)opts.smem_tables) continue; // experiment: size limit in bytes
                // worth it only if a block probes the table more often than it costs to copy
                const double probes_per_cta = (double)n * reach[s] / approx_grid;
                if (probes_per_cta * 4.0 < (double)tb) continue;
                S.in_smem = 1;
                S.smem_off = (uint32_t)(stage_bytes + tables);
                tables += tb;
                if (s < ndense && gather_of_stage[s] >= 0 && !via_bitmap[s]) { // the sparse copy reads the same staged table
                    P.st[gather_of_stage[s]].in_smem = 1;
                    P.st[gather_of_stage[s]].smem_off = S.smem_off;
                }
            }
        }
        *tables_out = tables;
        return true;
    };
    size_t tables = 0;
    if (!stage_tables(block, &tables)) return SJQ_ERR_UNSUPPORTED;
    // Two blocks per SM each carry their own copies of the staged tables and the group table, and their
    // queues.  A kernel compiled for the query can run as one block of 1024 threads per SM instead: one
    // copy, 32 warps instead of 24.  Measured better whenever the copies are sizeable or shared memory
    // would crowd out the L1 (config 3: 1.43 -> 1.32 ms, config 5: 2.8 -> 1.8 ms), given enough tiles per
    // block to even out the tail.
    bool single_block = false;
    // Between the two: a kernel with queues whose shared memory is moderate (more than three 384-thread blocks
    // could share, at most 100 KB as a 640-thread block) runs as two 640-thread blocks: 40 warps instead of 24 or
    // 32 and the L1 keeps half of the SM's memory (two-join workload 0.101 -> 0.094 ms, city x brand 0.681 ->
    // 0.667, city x city 0.700 -> 0.691).
    bool two_wide_queue_blocks = false;
    if (opts.specialise && !opts.block_threads && !opts.ctas_per_sm && P.nq && !opts.unfused &&
        stage_bytes + tables + hot_bytes + group_bytes + queue_bytes(block) > ((size_t)48 << 10)) {
        size_t tables640 = 0;
        if (stage_tables(640, &tables640) &&
            stage_bytes + tables640 + hot_bytes + group_bytes + queue_bytes(640) <= ((size_t)100 << 10)) {
            block = 640;
            tables = tables640;
            two_wide_queue_blocks = true;
        } else if (!stage_tables(block, &tables)) {
            return SJQ_ERR_UNSUPPORTED;
        }
    }
    if (opts.specialise && !opts.block_threads && !opts.ctas_per_sm && P.nq && !two_wide_queue_blocks) {
        const size_t copies = tables + hot_bytes + group_bytes;
        const int64_t tiles_per_block = n / ((int64_t)1024 * 4 * P.slots) / dev.sm_count;
        size_t tables1024 = 0;
        if ((copies >= ((size_t)16 << 10) || stage_bytes + copies + queue_bytes(block) > ((size_t)80 << 10)) &&
            tiles_per_block >= 128 && stage_tables(1024, &tables1024)) {
            block = 1024;
            single_block = true;
            tables = tables1024;
        } else if (!stage_tables(block, &tables)) {
            return SJQ_ERR_UNSUPPORTED;
        }
    }
    P.smem_stages = 0;
    P.smem_groups = (uint32_t)(stage_bytes + tables + hot_bytes);
    P.smem_queue = (uint32_t)(stage_bytes + tables + hot_bytes + group_bytes);
    size_t smem = stage_bytes + tables + hot_bytes + group_bytes + queue_bytes(block);
    if (hot_stage >= 0) {
        // the bitmap stage copies the table into shared memory; every stage of the same join reads that copy
        const void *bucket_array = joins[specs[order[hot_stage]].index].table->slots;
        for (int s2 = 0; s2 < ns; ++s2) {
            DStage &S = P.st[s2];
            const bool same_join = s2 == hot_stage || ((S.op == OP_HASH32 || S.op == OP_HASH64) && S.tab == bucket_array);
            if (!same_join) continue;
            S.hot = s2 == hot_stage ? 1 : 2;
            S.hot_off = (uint32_t)(stage_bytes + tables);
        }
    }

    // ------------------------------------------------------------ bulk-asynchronous staging of the first column
    // A kernel compiled for a query with survivor queues can have its first column copied into shared memory by
    // the copy engine, one tile (block size x 4 x slots values) per copy, three in flight per block.  Only when
    // asked for: measured on the selectivity sweep (600 M rows) the staged kernel is slower than 128-bit loads
    // with L2 prefetch at every point (0.01 %: 0.42 vs 0.37 ms; 1 %: 0.64 vs 0.53; 10 %, 1000 groups: 1.25 vs 1.21)
    // and much slower where its buffers crowd the shared memory (city x city: 1.09 vs 0.73 ms), although a bare
    // scan kernel built on the same copies moves 7.3 TB/s against 6.7 TB/s for loads: the warps of the fused
    // kernel consume a tile at their own pace, so the refill of a buffer waits for the slowest of them.
    const size_t smem_without_bulk = smem;
    if (opts.l0_bulk < 0 || opts.l0_bulk > 3) return SJQ_ERR_INVALID_ARG;
    if (opts.specialise && !opts.unfused && P.nq > 0 && n > 0 && (opts.l0_bulk == 1 || opts.l0_bulk == 3)) {
        const size_t tile_bytes = (size_t)block * 4 * P.slots * (P.st[0].is64 ? 8 : 4);
        const size_t at = align_up(smem, 128);
        const size_t total = at + 3 * tile_bytes + 3 * 8 + 3 * 4 + 4;
        if (total <= smem_cap) {
            P.l0_bulk = opts.l0_bulk == 3 ? 2 : 1; // 2: the kernel waits for copies nobody issues (failure-path test)
            P.smem_l0 = (uint32_t)at;
            smem = total;
        }
    }

    bool has_hash = false; // kernels without the hash probe are leaner; pick by what the stages need
    for (int s2 = 0; s2 < ns; ++s2)
        has_hash |= P.st[s2].op == OP_HASH32 || P.st[s2].op == OP_HASH64 || P.st[s2].op == OP_HASHBITS;

    // ------------------------------------------------------------ launch shape
    int per_sm = 0;
    const bool jit = opts.specialise != 0 && !opts.unfused;
    // register budget a specialised kernel is compiled for
    // (three blocks of 384 threads when their shared memory leaves the L1 alone: 56 registers are enough for the
    // short pipelines that have so little state, and 36 warps hide more latency than 24)
    const int lb_blocks = single_block ? 1
                          : (two_wide_blocks || two_wide_queue_blocks) ? 2
                          : opts.ctas_per_sm > 0 ? opts.ctas_per_sm
                          : block > 512 ? 1
                          : (block <= 384 && smem_without_bulk <= ((size_t)48 << 10)) ? 3
                                                                        : 2;
    st = jit ? jit_occupancy(P, aggp, mul, has_hash, block, lb_blocks, smem, &per_sm)
             : fused_occupancy(aggp, mul, has_hash, block, smem, &per_sm);
    if (st != SJQ_OK) return st;
    if (per_sm < 1) return SJQ_ERR_UNSUPPORTED;
    if (opts.ctas_per_sm > 0) per_sm = std::min(per_sm, opts.ctas_per_sm);
    const int64_t tile_rows = (int64_t)block * (P.nq ? 4 * P.slots : kDirectRows);
    const int64_t ntiles = (n + tile_rows - 1) / tile_rows;
    if (ntiles >= ((int64_t)1 << 31)) return SJQ_ERR_UNSUPPORTED;
    int grid = (int)std::min<int64_t>((int64_t)dev.sm_count * per_sm, std::max<int64_t>(ntiles, 1));

    // ------------------------------------------------------------ launches
    int launches = 0;
    if (!opts.accumulate) {
        int64_t cells = spec->mode == SJQ_SCALAR ? 1
                        : spec->mode == SJQ_DENSE ? spec->num_groups
                        : direct_groups           ? table_groups
                                                  : (int64_t)gslots + 1;
        st = clear_launch(P.sums, spec->mode == SJQ_HASHED ? gcounts : out->counts, cells, gkeys,
                          (spec->mode == SJQ_HASHED && !direct_groups) ? (int64_t)gslots + 1 : 0, out->n_groups,
                          out->status, dev.sm_count, stream);
        if (st != SJQ_OK) return st;
        ++launches;
    } else if (spec->mode == SJQ_HASHED) {
        if (cudaMemsetAsync(out->n_groups, 0, sizeof(int64_t), stream) != cudaSuccess) return SJQ_ERR_CUDA;
    }
    if (hot_stage >= 0) {
        const StageSpec &sp = specs[order[hot_stage]];
        const void *hot_table = nullptr;
        st = hot_launch(fact[sp.col].data, fact[sp.col].dtype == SJQ_I64, n, joins[sp.index].table, opts.hot_scratch,
                        stream, &hot_table, &launches);
        if (st != SJQ_OK) return st;
        for (int s2 = 0; s2 < ns; ++s2)
            if (P.st[s2].hot) P.st[s2].hot_tab = hot_table;
    }
    if ((opts.event_before != nullptr) != (opts.event_after != nullptr)) return SJQ_ERR_INVALID_ARG;
    if (opts.event_before && cudaEventRecord((cudaEvent_t)opts.event_before, stream) != cudaSuccess)
        return SJQ_ERR_CUDA;
    if (n > 0 && opts.unfused) {
        if (!aligned16(opts.unfused_scratch)) return SJQ_ERR_ALIGN;
        st = unfused_launch(P, nfilter, aggp, mul, has_hash, opts.unfused_scratch, opts.unfused_scratch_bytes,
                            dev.sm_count, stream, &launches);
        if (st != SJQ_OK) return st;
    } else if (n > 0) {
        st = jit ? jit_launch(P, aggp, mul, has_hash, grid, block, lb_blocks, smem, stream)
                 : fused_launch(aggp, mul, has_hash, grid, block, smem, P, stream);
        if (st != SJQ_OK) return st;
        ++launches;
    }
    if (opts.event_after && cudaEventRecord((cudaEvent_t)opts.event_after, stream) != cudaSuccess)
        return SJQ_ERR_CUDA;
    if (spec->mode == SJQ_HASHED) {
        st = compact_launch(gkeys, gsums, gcounts, direct_groups ? table_groups - 1 : (int64_t)gslots,
                            direct_groups, P.post_offset, out->keys, out->sums, out->counts, spec->capacity,
                            out->n_groups, out->status, dev.sm_count, stream);
        if (st != SJQ_OK) return st;
        ++launches;
    }
    if (info) {
        std::memset(info, 0, sizeof(*info));
        info->nstages = ns;
        const int shown = std::min<int>(ns, (int)(sizeof(info->order) / sizeof(info->order[0])));
        info->nstages = shown;
        for (int s = 0; s < shown; ++s) {
            info->order[s] = stage_label[s];
            info->stage_in_smem[s] = P.st[s].in_smem;
        }
        info->first_sparse_stage = P.nq ? P.nd0 : 0;
        info->reserved_levels = P.nq;
        info->agg_path = aggp;
        info->grid = grid;
        info->block = block;
        info->smem_bytes = (int32_t)smem;
        info->kernel_launches = launches;
    }
    return SJQ_OK;
}


// ---------------------------------------------------------------------------
// Merge of hashed results (the exchange step of a row-sharded run).
extern "C" sjq_status sjq_merge_groups(const int64_t *keys, const int64_t *sums, const int64_t *counts, int64_t n,
                                       int64_t capacity, const sjq_result *out, void *stream_)
{
    if (n < 0 || capacity <= 0 || !out || !out->keys || !out->sums || !out->counts || !out->n_groups ||
        !out->status || !out->workspace || (n > 0 && (!keys || !sums || !counts)))
        return SJQ_ERR_INVALID_ARG;
    if (!aligned16(out->sums) || !aligned16(out->counts) || !aligned16(out->keys) || !aligned16(out->workspace) ||
        (reinterpret_cast<uintptr_t>(keys) & 7u) || (reinterpret_cast<uintptr_t>(sums) & 7u) ||
        (reinterpret_cast<uintptr_t>(counts) & 7u) || (reinterpret_cast<uintptr_t>(out->status) & 3u) ||
        (reinterpret_cast<uintptr_t>(out->n_groups) & 7u))
        return SJQ_ERR_ALIGN;
    sjq_result_spec spec{SJQ_HASHED, 0, capacity};
    size_t need = 0;
    sjq_run_workspace_bytes(&spec, &need);
    if (out->workspace_bytes < need) return SJQ_ERR_BUFFER_SMALL;
    DeviceInfo dev;
    sjq_status st = device_info(&dev);
    if (st != SJQ_OK) return st;
    cudaStream_t stream = (cudaStream_t)stream_;
    const uint64_t gslots = hashed_slots(capacity);
    const size_t arr = align_up((size_t)(gslots + 1) * 8, 256);
    int64_t *gkeys = reinterpret_cast<int64_t *>(static_cast<char *>(out->workspace));
    int64_t *gsums = reinterpret_cast<int64_t *>(static_cast<char *>(out->workspace) + arr);
    int64_t *gcounts = reinterpret_cast<int64_t *>(static_cast<char *>(out->workspace) + 2 * arr);
    if ((st = clear_launch(gsums, gcounts, (int64_t)gslots + 1, gkeys, (int64_t)gslots + 1, out->n_groups, out->status,
                           dev.sm_count, stream)) != SJQ_OK)
        return st;
    if ((st = merge_launch(keys, sums, counts, n, gkeys, gsums, gcounts, gslots - 1, out->status, dev.sm_count,
                           stream)) != SJQ_OK)
        return st;
    return compact_launch(gkeys, gsums, gcounts, (int64_t)gslots, false, 0, out->keys, out->sums, out->counts, capacity,
                          out->n_groups, out->status, dev.sm_count, stream);
}

// ---------------------------------------------------------------------------
// Host-buffer entry point: chunked, double-buffered copy + run.
namespace {

struct HostPipe {
    cudaStream_t s[2] = {nullptr, nullptr};
    cudaEvent_t start = nullptr, done[2] = {nullptr, nullptr};
    bool ok = false;
};

thread_local HostPipe g_pipes[64];

HostPipe *host_pipe()
{
    HostPipe *pipes = g_pipes;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    HostPipe &p = pipes[dev];
    if (!p.ok) {
        if (cudaStreamCreateWithFlags(&p.s[0], cudaStreamNonBlocking) != cudaSuccess ||
            cudaStreamCreateWithFlags(&p.s[1], cudaStreamNonBlocking) != cudaSuccess ||
            cudaEventCreateWithFlags(&p.start, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&p.done[0], cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&p.done[1], cudaEventDisableTiming) != cudaSuccess) {
            (void)cudaGetLastError();
            return nullptr;
        }
        p.ok = true;
    }
    return &p;
}

} // namespace

namespace {

enum { HOST_COPY = 0, HOST_IN_PLACE = 1, HOST_SKIP = 2 };

// How each host-resident column reaches the kernel.  A column most rows still need is copied chunk by
// chunk; one that only a few per cent of the rows reach (lazy loading: it is read for survivors only) is
// read by the kernel straight from the page-locked host buffer, 32 bytes per touched sector, which moves
// far fewer bytes over the bus than the whole column (measured on the four-join workload, 600 M rows:
// revenue and supplycost 16 ms instead of 87 ms of copies; break-even near 5 % of the rows); a column the
// query never references is not transferred at all.  `need`: share of the rows each column is first read
// for (< 0: never).  Invalid queries get "copy everything" and are rejected later by sjq_run.
void host_transfer_plan(const sjq_col *fact_host, int nfact, const sjq_pred *preds, int npreds,
                        const sjq_join *joins, int njoins, const sjq_key_expr *key, const sjq_agg_expr *agg,
                        sjq_run_opts *opts_io, std::vector<int> *how_out, std::vector<const char *> *base_out,
                        std::vector<double> *need_out)
{
    sjq_run_opts &opts = *opts_io; // predicates measured here are written back as hints for the runs
    std::vector<int> &how = *how_out;
    std::vector<const char *> &direct_base = *base_out;
    how.assign(nfact, HOST_COPY);
    direct_base.assign(nfact, nullptr);
    need_out->assign(nfact, 1.0);
    const int64_t n = fact_host[0].n;
    bool ok = npreds >= 0 && npreds <= SJQ_MAX_PREDS && njoins >= 0 && njoins <= SJQ_MAX_JOINS &&
              (!npreds || preds) && (!njoins || joins) && n > 0 && agg;
    for (int p = 0; ok && p < npreds; ++p) ok = preds[p].col >= 0 && preds[p].col < nfact;
    for (int j = 0; ok && j < njoins; ++j)
        ok = joins[j].table && joins[j].table->magic == kTableMagic && joins[j].fk_col >= 0 && joins[j].fk_col < nfact;
    auto term_ok = [&](const sjq_term &t) { return t.src != SJQ_SRC_FACT || (t.a >= 0 && t.a < nfact); };
    if (ok && key) {
        ok = key->nterms >= 0 && key->nterms <= SJQ_MAX_KEY_TERMS;
        for (int t = 0; ok && t < key->nterms; ++t) ok = term_ok(key->t[t]);
    }
    ok = ok && term_ok(agg->x) && (agg->op == SJQ_AGG_COL || term_ok(agg->y));
    std::vector<StageSpec> specs;
    std::vector<int> order;
    // The columns are in host memory here, so predicates without a measured pass fraction are measured on
    // the spot: a few thousand evenly spaced rows read by the host.  (A guess that is far too low would send
    // a column most rows need over the bus sector by sector.)
    sjq_run_opts &measured = opts;
    for (int p = 0; ok && p < npreds; ++p) {
        if (measured.pass_ppm[p] > 0) continue;
        const sjq_col &c = fact_host[preds[p].col];
        DPred d;
        if (!c.data || !canon_pred(preds[p], c.dtype, &d)) continue;
        const int64_t samples = std::min<int64_t>(n, 8192), stride = n / samples;
        int64_t pass = 0;
        for (int64_t i = 0; i < samples; ++i) {
            const int64_t r = i * stride;
            const int64_t v = c.dtype == SJQ_I64 ? static_cast<const int64_t *>(c.data)[r]
                                                 : (int64_t) static_cast<const int32_t *>(c.data)[r];
            bool in;
            if (d.nset) {
                in = false;
                for (int k = 0; k < d.nset; ++k) in |= v == d.set[k];
            } else {
                in = (v >= d.lo && v <= d.hi) != (bool)d.neg;
            }
            pass += in;
        }
        measured.pass_ppm[p] = ppm_of(pass, samples);
    }
    if (!ok || order_stages(fact_host, preds, npreds, joins, njoins, measured, &specs, &order) != SJQ_OK) return;
    std::vector<double> &need = *need_out;
    need.assign(nfact, -1.0);
    double reach = 1.0;
    for (int i : order) {
        if (need[specs[i].col] < 0) need[specs[i].col] = reach;
        reach *= specs[i].sel;
    }
    auto use = [&](const sjq_term &t) {
        if (t.src == SJQ_SRC_FACT && need[t.a] < 0) need[t.a] = reach;
    };
    if (key && key->modulo != 1) // (modulo 1: the planner drops the key's terms)
        for (int t = 0; t < key->nterms; ++t) use(key->t[t]);
    use(agg->x);
    if (agg->op != SJQ_AGG_COL) use(agg->y);
    for (int c = 0; c < nfact; ++c) {
        if (need[c] < 0) {
            how[c] = HOST_SKIP;
        } else if (need[c] <= 0.04 && !opts.eager_loads && !opts.host_copy_all) {
            cudaPointerAttributes attr;
            if (cudaPointerGetAttributes(&attr, fact_host[c].data) == cudaSuccess && attr.type == cudaMemoryTypeHost &&
                attr.devicePointer && aligned16(attr.devicePointer)) {
                how[c] = HOST_IN_PLACE;
                direct_base[c] = static_cast<const char *>(attr.devicePointer);
            } else {
                (void)cudaGetLastError(); // pageable memory: copy it
            }
        }
    }
}

} // namespace

extern "C" sjq_status sjq_host_transfer_plan(const sjq_col *fact_host, int nfact, const sjq_pred *preds, int npreds,
                                             const sjq_join *joins, int njoins, const sjq_key_expr *key,
                                             const sjq_agg_expr *agg, const sjq_run_opts *opts_, int32_t *how,
                                             double *share)
{
    if (!fact_host || nfact <= 0 || nfact > 64 || !agg || !how) return SJQ_ERR_INVALID_ARG;
    sjq_run_opts opts{};
    if (opts_) opts = *opts_;
    std::vector<int> h;
    std::vector<const char *> base;
    std::vector<double> need;
    host_transfer_plan(fact_host, nfact, preds, npreds, joins, njoins, key, agg, &opts, &h, &base, &need);
    for (int c = 0; c < nfact; ++c) {
        how[c] = h[c];
        if (share) share[c] = need[c] < 0 ? 0.0 : need[c];
    }
    return SJQ_OK;
}

extern "C" sjq_status sjq_run_host(const sjq_col *fact_host, int nfact, const sjq_pred *preds, int npreds,
                                   const sjq_join *joins, int njoins, const sjq_key_expr *key,
                                   const sjq_agg_expr *agg, const sjq_result_spec *spec, const sjq_result *out,
                                   const sjq_run_opts *opts_, void *staging_dev, size_t staging_bytes,
                                   int64_t chunk_rows, int64_t *host_sums, int64_t *host_counts, int64_t *host_keys,
                                   int64_t *host_n_groups, int32_t *host_status, void *stream_)
{
    if (!fact_host || nfact <= 0 || nfact > 64 || !staging_dev || chunk_rows <= 0 || (chunk_rows & 3) || !spec ||
        !out || !agg)
        return SJQ_ERR_INVALID_ARG;
    if (!aligned16(staging_dev)) return SJQ_ERR_ALIGN;
    const int64_t n = fact_host[0].n;
    if (n < 0) return SJQ_ERR_INVALID_ARG;
    size_t half = 0;
    std::vector<size_t> col_off(nfact);
    for (int c = 0; c < nfact; ++c) {
        if (fact_host[c].n != n || (fact_host[c].dtype != SJQ_I32 && fact_host[c].dtype != SJQ_I64) ||
            (n > 0 && !fact_host[c].data))
            return SJQ_ERR_INVALID_ARG;
        col_off[c] = half;
        half += align_up((size_t)chunk_rows * (fact_host[c].dtype == SJQ_I64 ? 8 : 4), 256);
    }
    if (staging_bytes < 2 * half) return SJQ_ERR_BUFFER_SMALL;
    HostPipe *hp = host_pipe();
    if (!hp) return SJQ_ERR_CUDA;
    cudaStream_t stream = (cudaStream_t)stream_;
    sjq_run_opts opts{};
    if (opts_) opts = *opts_;
    opts.event_before = opts.event_after = nullptr;

    std::vector<int> how;
    std::vector<const char *> direct_base;
    std::vector<double> need_share;
    host_transfer_plan(fact_host, nfact, preds, npreds, joins, njoins, key, agg, &opts, &how, &direct_base, &need_share);

    // internal streams start after whatever is already queued on the caller's stream
    if (cudaEventRecord(hp->start, stream) != cudaSuccess) return SJQ_ERR_CUDA;
    for (int b = 0; b < 2; ++b)
        if (cudaStreamWaitEvent(hp->s[b], hp->start, 0) != cudaSuccess) return SJQ_ERR_CUDA;

    const int64_t nchunks = n == 0 ? 1 : (n + chunk_rows - 1) / chunk_rows;
    std::vector<sjq_col> dev_cols(nfact);
    for (int64_t k = 0; k < nchunks; ++k) {
        const int b = (int)(k & 1);
        const int64_t r0 = k * chunk_rows;
        const int64_t rows = std::min<int64_t>(chunk_rows, n - r0);
        char *base = static_cast<char *>(staging_dev) + (size_t)b * half;
        // copies into this half follow run k-2 by stream order and overlap run k-1 on the other stream
        for (int c = 0; c < nfact; ++c) {
            const size_t w = fact_host[c].dtype == SJQ_I64 ? 8 : 4;
            dev_cols[c] = sjq_col{base + col_off[c], fact_host[c].dtype, rows};
            if (how[c] == HOST_SKIP) continue; // never dereferenced
            if (how[c] == HOST_IN_PLACE) {
                dev_cols[c].data = direct_base[c] + (size_t)r0 * w;
                continue;
            }
            if (rows > 0 &&
                cudaMemcpyAsync(base + col_off[c], static_cast<const char *>(fact_host[c].data) + (size_t)r0 * w,
                                (size_t)rows * w, cudaMemcpyHostToDevice, hp->s[b]) != cudaSuccess)
                return SJQ_ERR_CUDA;
        }
        // runs accumulate into the same result and must not overlap: run k waits for run k-1
        if (k > 0 && cudaStreamWaitEvent(hp->s[b], hp->done[b ^ 1], 0) != cudaSuccess) return SJQ_ERR_CUDA;
        opts.accumulate = (k > 0 || (opts_ && opts_->accumulate)) ? 1 : 0;
        opts.hot_keys = 2; // a chunk's foreign keys may still be in host memory: no sampling pass over them
        sjq_status st = sjq_run(dev_cols.data(), nfact, preds, npreds, joins, njoins, key, agg, spec, out, &opts,
                                hp->s[b], nullptr);
        if (st != SJQ_OK) return st;
        if (cudaEventRecord(hp->done[b], hp->s[b]) != cudaSuccess) return SJQ_ERR_CUDA;
    }
    const int last = (int)((nchunks - 1) & 1);
    if (cudaStreamWaitEvent(stream, hp->done[last], 0) != cudaSuccess) return SJQ_ERR_CUDA;
    if (nchunks > 1 && cudaStreamWaitEvent(stream, hp->done[last ^ 1], 0) != cudaSuccess) return SJQ_ERR_CUDA;
    const int64_t cells = spec->mode == SJQ_SCALAR ? 1 : spec->mode == SJQ_DENSE ? spec->num_groups : spec->capacity;
    bool ok = true;
    if (host_sums) ok = ok && cudaMemcpyAsync(host_sums, out->sums, (size_t)cells * 8, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    if (host_counts && out->counts)
        ok = ok && cudaMemcpyAsync(host_counts, out->counts, (size_t)cells * 8, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    if (host_keys && out->keys)
        ok = ok && cudaMemcpyAsync(host_keys, out->keys, (size_t)cells * 8, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    if (host_n_groups && out->n_groups)
        ok = ok && cudaMemcpyAsync(host_n_groups, out->n_groups, 8, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    if (host_status) ok = ok && cudaMemcpyAsync(host_status, out->status, 4, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    return ok ? SJQ_OK : SJQ_ERR_CUDA;
}


namespace sjq {
int fused_cache_clear();
}

extern "C" int32_t sjq_release(void)
{
    int32_t released = 0;
    int current = 0;
    const bool have_device = cudaGetDevice(&current) == cudaSuccess;
    for (int d = 0; d < 64; ++d) {
        HostPipe &p = g_pipes[d];
        if (!p.ok) continue;
        if (have_device && cudaSetDevice(d) == cudaSuccess) {
            for (cudaStream_t &st : p.s)
                if (st && cudaStreamDestroy(st) == cudaSuccess) ++released;
            for (cudaEvent_t ev : {p.start, p.done[0], p.done[1]})
                if (ev && cudaEventDestroy(ev) == cudaSuccess) ++released;
        }
        p = HostPipe();
    }
    if (have_device) (void)cudaSetDevice(current);
    (void)cudaGetLastError();
    released += sjq_jit_cache_clear();
    released += sjq::fused_cache_clear();
    return released;
}

// ---------------------------------------------------------------------------
// Hashed group-by with the group table in the library's own device image, for
// callers that cannot allocate device memory.
namespace {

// 2 * SJQ_STATIC_MAX_GROUPS slots + the side slot, three int64 arrays, each padded to 256 bytes.
static __device__ __align__(256) unsigned char g_static_group_table[SJQ_STATIC_WORKSPACE_BYTES];

} // namespace

extern "C" sjq_status sjq_run_hashed_static(const sjq_col *fact, int nfact, const sjq_pred *preds, int npreds,
                                            const sjq_join *joins, int njoins, const sjq_key_expr *key,
                                            const sjq_agg_expr *agg, int64_t capacity, const sjq_result *out,
                                            const sjq_run_opts *opts_, void *stream, sjq_run_info *info)
{
    if (!out || capacity <= 0) return SJQ_ERR_INVALID_ARG;
    if (capacity > SJQ_STATIC_MAX_GROUPS) return SJQ_ERR_STATIC_LIMIT;
    sjq_result_spec spec{SJQ_HASHED, 0, capacity};
    size_t need = 0;
    if (sjq_run_workspace_bytes(&spec, &need) != SJQ_OK || need > SJQ_STATIC_WORKSPACE_BYTES)
        return SJQ_ERR_STATIC_LIMIT;

    // In host code the array's name is only a stand-in; the kernels need its device address,
    // looked up once per device with that device current.
    static thread_local void *table_addr[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
        (void)cudaGetLastError();
        return SJQ_ERR_CUDA;
    }
    if (!table_addr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_group_table) != cudaSuccess || !p) {
            (void)cudaGetLastError();
            return SJQ_ERR_CUDA;
        }
        table_addr[dev] = p;
    }
    sjq_result r = *out;
    r.workspace = table_addr[dev];
    r.workspace_bytes = SJQ_STATIC_WORKSPACE_BYTES;
    sjq_run_opts opts{};
    if (opts_) opts = *opts_;
    opts.accumulate = 0; // the shared table holds the last call's groups: always start from a cleared table
    opts.specialise = 0; // loading a compiled module allocates device memory: this entry point only interprets
    return sjq_run(fact, nfact, preds, npreds, joins, njoins, key, agg, &spec, &r, &opts, stream, info);
}
