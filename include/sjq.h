/*
 * sjq -- fused star-join query pipeline for NVIDIA B200 (sm_100a).
 *
 * C ABI of the library.  The operation is the fused per-row pipeline of the
 * paper (Section 3.1 "Kernel Composition", Section 3.2 Listing 2, Section 3.3
 * "Workload-Specific Optimizations", Section 4.2.2 "Fusion in SYCLDB"): one
 * pass over a columnar fact table that evaluates the fact predicates, probes
 * one dimension table per join (a miss drops the row, a hit gathers the
 * dimension's payload), and aggregates the survivors (scalar sum, dense
 * group array, or hashed groups); the dimension tables are produced
 * beforehand by a separate build kernel from the filtered dimension columns.
 *
 * Conventions
 *   - Every `data`, `*_dev`, `table_mem`, result and workspace pointer is a
 *     DEVICE pointer owned by the caller, 16-byte aligned, and must stay
 *     valid and unmodified until the work enqueued on `stream` has finished.
 *     Descriptor structs (columns, predicates, expressions, options) are HOST
 *     memory and are copied during the call.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *   - The library allocates no device memory for data.  (A run that asks for
 *     run-time specialisation loads a compiled module the first time it meets
 *     a query shape; the CUDA driver places the module's code on the device.)
 *     All kernels are enqueued on the given stream; calls return after
 *     enqueueing unless stated otherwise.
 *   - Functions return 0 (SJQ_OK) or a host-detected error code.  Errors only
 *     the device can see are written to the caller's int32 status word (first
 *     error wins); kernels never trap and never spin without a bound.  Results
 *     are undefined when the status word is non-zero after the stream syncs.
 *   - Columns are int32 or int64, contiguous, little-endian.  All arithmetic
 *     on values is done after sign-extension to 64 bits and wraps modulo 2^64
 *     (the 64-bit product of Listing 2); `%` truncates toward zero as in C.
 *   - No CPU fallback exists: without a CUDA device every compute call fails
 *     with SJQ_ERR_CUDA.
 */
#ifndef SJQ_H
#define SJQ_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t sjq_status;

enum {
    SJQ_OK = 0,
    /* host-detected (returned) */
    SJQ_ERR_INVALID_ARG = 1,
    SJQ_ERR_UNSUPPORTED = 2,
    SJQ_ERR_ALIGN = 3,        /* a device pointer is not 16-byte aligned */
    SJQ_ERR_CUDA = 4,         /* a CUDA runtime call failed (no device, launch error) */
    SJQ_ERR_BUFFER_SMALL = 5, /* caller-provided table / workspace memory too small */
    SJQ_ERR_STATIC_LIMIT = 6, /* request exceeds the built-in scratch of a no-allocation entry point */
    SJQ_ERR_JIT = 7,          /* run-time specialisation asked for but the compiler, the device sources or the
                                 compiled module are unavailable (sjq_jit_log has the details) */
    /* device-detected (written to the status word) */
    SJQ_ERR_DUP_KEY = 16,        /* two dimension rows passing the filter share a key */
    SJQ_ERR_TABLE_FULL = 17,     /* open-addressing insert found no free slot */
    SJQ_ERR_GROUP_RANGE = 18,    /* dense mode: a group key fell outside [0, num_groups) */
    SJQ_ERR_GROUP_OVERFLOW = 19, /* hashed mode: more distinct groups than the capacity */
    SJQ_ERR_RESERVED_KEY = 20,   /* a dimension key equals the reserved empty marker (minimum of its type) */
    SJQ_ERR_LAYOUT_MISMATCH = 21, /* build saw a key or payload outside the planned layout */
    SJQ_ERR_ASYNC_WAIT = 22       /* a bounded wait for a bulk-asynchronous copy ran out; the kernel went on with
                                     plain loads, so the result is still exact, but the device needs a look */
};

enum { SJQ_I32 = 0, SJQ_I64 = 1 };

/* One column: n values of `dtype` at device address `data`. */
typedef struct sjq_col {
    const void *data;
    int32_t dtype;
    int64_t n;
} sjq_col;

/* Predicate on one column; a query carries a conjunction of these
 * (Section 4.2.2: a BETWEEN is the AND of its two inclusive bounds; the
 * disjunction on one column in the Q4.1 text of Section 3.3 is an IN set). */
enum { SJQ_EQ = 0, SJQ_NE, SJQ_LT, SJQ_LE, SJQ_GT, SJQ_GE, SJQ_BETWEEN, SJQ_IN };
#define SJQ_MAX_IN_SET 16
typedef struct sjq_pred {
    int32_t col;        /* index into the column array it is applied to */
    int32_t op;         /* SJQ_EQ ... SJQ_IN; one-sided ops compare with `lo` */
    int64_t lo, hi;     /* BETWEEN: lo <= v <= hi */
    const int64_t *set; /* IN: host array of nset values (nset <= SJQ_MAX_IN_SET) */
    int32_t nset;
} sjq_pred;

/* A value available to the group key and the aggregate: a fact column
 * (a = fact column index) or a payload gathered by a join (a = join index,
 * b = payload index of that join's table), scaled by `mult`. */
enum { SJQ_SRC_FACT = 0, SJQ_SRC_PAYLOAD = 1 };
typedef struct sjq_term {
    int32_t src, a, b;
    int64_t mult;
} sjq_term;

/* key = (offset + sum_t mult_t * value_t) [% modulo]; modulo 0 = none. */
#define SJQ_MAX_KEY_TERMS 4
typedef struct sjq_key_expr {
    sjq_term t[SJQ_MAX_KEY_TERMS];
    int32_t nterms;
    int64_t offset, modulo;
} sjq_key_expr;

/* Aggregated value per surviving row: COL: x; MUL: x*y; SUB: x-y; ADD: x+y
 * (each of x, y already scaled by its `mult`); summed per group in int64. */
enum { SJQ_AGG_COL = 0, SJQ_AGG_MUL, SJQ_AGG_SUB, SJQ_AGG_ADD };
typedef struct sjq_agg_expr {
    int32_t op;
    sjq_term x, y;
    int32_t want_count; /* non-zero: also count the rows per group */
} sjq_agg_expr;

/* ------------------------------------------------------------------ */
/* Dimension tables (Section 3.3: direct-mapped and byte-packed maps for
 * dense keys, an open-addressing table otherwise; Section 4.3.1: the key
 * range is verified at run time and the packed or the unpacked form chosen). */

enum {
    SJQ_TABLE_AUTO = 0,
    SJQ_TABLE_DIRECT_BITMAP = 1, /* 1 bit per key in [kmin, kmax]: filter only, no payload */
    SJQ_TABLE_DIRECT_U8 = 2,     /* 1 byte per key: packed payload code, 0xFF = miss */
    SJQ_TABLE_DIRECT_U16 = 3,
    SJQ_TABLE_DIRECT_U32 = 4,
    SJQ_TABLE_DIRECT_U64 = 5,
    SJQ_TABLE_HASH_I32 = 6, /* open addressing over 32-byte buckets of keys and codes, linear probing, int32 keys */
    SJQ_TABLE_HASH_I64 = 7,
    SJQ_TABLE_DIRECT_U4 = 8, /* 4 bits per key, eight codes to a 32-bit word: 0xF = miss unless every key of the
                                range is present (entries == slots), in which case the range test alone decides */
    SJQ_TABLE_DIRECT_U2 = 9, /* 2 bits per key, sixteen to a word; same rule */
    SJQ_TABLE_FORCE_DIRECT = 100, /* build option only */
    SJQ_TABLE_FORCE_HASH = 101    /* build option only */
};

#define SJQ_MAX_PAYLOADS 2
#define SJQ_PLAN_SCRATCH_BYTES 256

typedef struct sjq_build_opts {
    int32_t force_kind;       /* SJQ_TABLE_AUTO, SJQ_TABLE_FORCE_DIRECT or SJQ_TABLE_FORCE_HASH */
    int32_t hash_load_pct;    /* 0 = default 40: slots >= entries * 100 / pct, in whole 32-byte buckets; <= 90 */
    int64_t max_direct_bytes; /* 0 = default 64 MiB: larger direct tables fall back to hashing */
    int32_t min_code_bits;    /* narrowest packed code of a direct table: 0 = default 2 (sub-byte codes where the
                                 payload range allows: a probed structure a quarter the size of Section 3.3's byte
                                 map stays closer to the SMs), 8 = one byte or wider, as in the paper */
    int32_t reserved;
} sjq_build_opts;

/* Shape of a table, decided from the data by sjq_dim_plan. Plain host data. */
typedef struct sjq_dim_layout {
    int32_t kind;      /* one of SJQ_TABLE_DIRECT_* / SJQ_TABLE_HASH_* */
    int32_t key_dtype; /* SJQ_I32 / SJQ_I64 */
    int32_t npayload;
    int32_t code_bits;                 /* width of the packed payload code stored per key (0, 2, 4, 8, 16, 32, 64) */
    int64_t dim_rows;                  /* rows of the dimension */
    int64_t entries;                   /* rows passing the filter */
    int64_t kmin, kmax;                /* key range among the passing rows (0,0 if none) */
    int64_t pay_min[SJQ_MAX_PAYLOADS]; /* payload i is stored as (value - pay_min[i]) in pay_bits[i] bits */
    int64_t pay_max[SJQ_MAX_PAYLOADS];
    int32_t pay_bits[SJQ_MAX_PAYLOADS];
    int64_t slots;      /* direct: kmax-kmin+1; hash: key slots = 32-byte buckets x keys per bucket (a bucket holds
                           K keys then their K codes: K = 8, 4 or 2 for 32-bit keys and 4, 2 or 2 for 64-bit keys
                           with no, 32-bit or 64-bit codes) */
    int64_t filter_bits; /* direct with payloads: bits of the presence bitmap over the slots (a multiple of 128);
                            hash: size (power of two, 0 = none) of the presence bitmap indexed by the key's hash,
                            probed before the table so that most absent keys never touch it */
    size_t table_bytes; /* device bytes sjq_build_dim needs at table_mem */
} sjq_dim_layout;

typedef struct sjq_table sjq_table; /* opaque host handle */

/*
 * Scan the filtered dimension once (key range, passing-row count, payload
 * ranges) and choose the table shape: Section 4.3.1 of the paper has the
 * engine verify the key range at run time and pick the packed direct map or
 * the unpacked table; Section 3.3 gives the forms.  The layout also carries
 * the device bytes the table needs, so this call stands where a separate
 * "how much memory" query would: the caller allocates `table_bytes` and hands
 * them to sjq_build_dim.  Enqueues one kernel on `stream`, copies
 * 64 bytes back and SYNCHRONISES the stream before returning.
 *   cols/ncols      dimension columns (device), all of equal length
 *   preds/npreds    conjunction over those columns (npreds <= 16)
 *   key_col         index of the key column
 *   payload_cols    indices of up to SJQ_MAX_PAYLOADS payload columns
 *   scratch_dev     device scratch of SJQ_PLAN_SCRATCH_BYTES bytes
 * Errors: INVALID_ARG, ALIGN, UNSUPPORTED (payload ranges too wide to pack
 * into 64 bits), CUDA.
 */
sjq_status sjq_dim_plan(const sjq_col *cols, int ncols, const sjq_pred *preds, int npreds, int key_col,
                        const int *payload_cols, int npayload, const sjq_build_opts *opts, void *scratch_dev,
                        void *stream, sjq_dim_layout *layout);

/*
 * The same in two halves, so that several dimensions can be planned with one
 * wait: `_begin` enqueues the scan on `stream` and an asynchronous copy of the
 * eight int64 statistics into `host_stats` (page-locked host memory, 64 bytes)
 * and returns at once; after the caller has synchronised that stream (or an
 * event recorded on it), `_end` turns the statistics into the layout on the
 * host.  `cols`/`ncols`/`key_col`/`npayload`/`opts` must describe the same
 * dimension in both calls.
 */
sjq_status sjq_dim_plan_begin(const sjq_col *cols, int ncols, const sjq_pred *preds, int npreds, int key_col,
                              const int *payload_cols, int npayload, void *scratch_dev, int64_t *host_stats,
                              void *stream);
sjq_status sjq_dim_plan_end(const sjq_col *cols, int ncols, int key_col, int npayload, const sjq_build_opts *opts,
                            const int64_t *host_stats, sjq_dim_layout *layout);

/*
 * Build the table described by `layout` into caller memory `table_mem`
 * (>= layout->table_bytes, else BUFFER_SMALL) and return a handle.  The
 * layout normally comes from sjq_dim_plan; whatever its origin, its sizes are
 * recomputed and a self-contradictory layout is INVALID_ARG.  A layout that
 * is consistent but too small for the data is caught on the device
 * (LAYOUT_MISMATCH: key or payload outside the planned ranges; TABLE_FULL:
 * the open-addressing table has no free slot left).  Enqueues
 * a fill, the build kernel and a verification kernel; does not synchronise.
 * Direct tables are written by race-free direct stores indexed by key
 * (Section 3.3); hash tables by atomicCAS on the key word with a bounded
 * linear probe.  Keys must be unique among the passing rows: a repeated key
 * sets SJQ_ERR_DUP_KEY in *status_dev.  Zero passing rows is valid (every
 * probe then misses).  *status_dev is NOT cleared by this call.
 */
sjq_status sjq_build_dim(const sjq_col *cols, int ncols, const sjq_pred *preds, int npreds, int key_col,
                         const int *payload_cols, int npayload, const sjq_dim_layout *layout, void *table_mem,
                         size_t table_bytes, int32_t *status_dev, void *stream, sjq_table **table);

/*
 * Device bytes a table of the given shape occupies, recomputed from `kind`,
 * `key_dtype`, `npayload`, `code_bits`, `slots` and `filter_bits` (the
 * layout's own `table_bytes` is not read).  A caller that edits a planned
 * layout (Section 4.3.1 lets the engine choose the table form at run time;
 * here the caller may override that choice, e.g. give an open-addressing
 * table more slots) must store the answer in `table_bytes` before handing the
 * layout to sjq_build_dim, which rejects a layout whose fields contradict one
 * another (INVALID_ARG) instead of writing past `table_mem`.  Host only.
 */
sjq_status sjq_dim_layout_bytes(const sjq_dim_layout *layout, size_t *bytes);

/* Copy of the layout the table was built with: kind, key range, entries, slots and bytes, i.e. what decides
 * whether the probed structure stays in L1 / L2 (Section 3.3: the packed map is sized to stay cache-resident). */
sjq_status sjq_table_info(const sjq_table *table, sjq_dim_layout *layout);

/* Kernels sjq_build_dim enqueued for this table: one that prepares the memory, the build unless the dimension
 * is empty, and for a direct table the occupancy count that ends with the duplicate check. */
int32_t sjq_table_kernel_launches(const sjq_table *table);

/* Frees the host handle only (the device memory belongs to the caller). */
void sjq_table_destroy(sjq_table *table);

/* ------------------------------------------------------------------ */
/* The fused run. */

typedef struct sjq_join {
    int32_t fk_col;         /* fact column holding the foreign key (same dtype as the table's key) */
    const sjq_table *table; /* table probed with it */
} sjq_join;

enum { SJQ_SCALAR = 0, SJQ_DENSE = 1, SJQ_HASHED = 2 };

typedef struct sjq_result_spec {
    int32_t mode;
    int64_t num_groups; /* DENSE: keys must lie in [0, num_groups) */
    int64_t capacity;   /* HASHED: maximum number of distinct groups */
} sjq_result_spec;

/* Device buffers receiving the result.
 *   SCALAR: sums[0], counts[0].
 *   DENSE : sums[num_groups], counts[num_groups] (absent groups are zero).
 *   HASHED: keys/sums/counts[capacity] hold *n_groups entries in no particular
 *           order; `workspace` is the group table (scratch): an
 *           open-addressing hash table, or, when the key is taken modulo M and
 *           2M - 1 cells fit, a table indexed by the key itself.
 * `counts` may be NULL when want_count is 0 (SCALAR and DENSE only).
 * `n_groups` is required for HASHED.  `status` is always required. */
typedef struct sjq_result {
    int64_t *sums;
    int64_t *counts;
    int64_t *keys;
    int64_t *n_groups;
    int32_t *status;
    void *workspace;
    size_t workspace_bytes;
} sjq_result;

#define SJQ_MAX_PREDS 16
#define SJQ_MAX_JOINS 8

/* Tuning and ablation switches; a zeroed struct (or NULL) means defaults. */
typedef struct sjq_run_opts {
    int32_t block_threads; /* 0 = library chooses (384; a kernel compiled for the query may run 640 or 1024); else a
                              multiple of 32 in 128..384, or up to 1024 together with `specialise` */
    int32_t ctas_per_sm;   /* 0 = as many as fit */
    int32_t eager_loads;   /* 1 = load every column for every row (ablation of lazy loading) */
    int32_t agg_path;      /* 0 auto, 1 shared-memory privatised table, 2 global atomics (DENSE) */
    int32_t smem_tables;   /* 0 auto (direct tables and presence bitmaps up to 32 KiB are copied into shared
                              memory), 1 never, 2 every one that fits, >= 1024: size limit in bytes */
    int32_t compaction;    /* 0 auto; 1 never queue survivors (every stage on thread-owned rows);
                              2 one queue only (first stage dense, everything else at the final level) */
    int32_t accumulate;    /* 1 = add into the result buffers instead of clearing them first */
    int32_t norder;        /* 0 = library chooses the evaluation order */
    int32_t order[SJQ_MAX_PREDS + SJQ_MAX_JOINS]; /* entry < npreds: predicate index; else npreds + join index */
    void *event_before; /* optional cudaEvent_t recorded on `stream` right before the fused kernel */
    void *event_after;  /* optional cudaEvent_t recorded right after it (both or neither) */
    int32_t specialise; /* 1 = compile the fused kernel for this query's shape at run time (NVRTC) and cache the
                           module for later runs of the same shape; 0 = interpret the descriptor (default).  Key
                           ranges, thresholds, table sizes and pointers stay run-time values, so a compiled module
                           is reused when only they change.  Same results either way. */
    int32_t rows_per_lane; /* rows a lane handles per batch at the queue-fed levels: 0 = library chooses, 4, or 8
                              (8 only with specialise: the ahead-of-time kernels are built for 4) */
    int32_t no_filter_bitmap; /* 1 = filter stages probe a direct table's code array even when the table has a
                                 presence bitmap (ablation) */
    int32_t host_copy_all; /* sjq_run_host: 1 = copy every referenced column to the device; 0 = columns that only a
                              few per cent of the rows reach are read by the kernel from the page-locked host
                              buffer instead */
    int32_t dense_slots; /* level 0: groups of four consecutive rows a thread owns per tile: 0 = library chooses, 2,
                            or 4 (4 only with specialise) */
    int32_t group_hash_always; /* HASHED results: 1 = always use the group hash table; 0 = a key taken modulo M whose
                                  2M - 1 possible values fit the workspace is aggregated in a table indexed by the
                                  key itself */
    int32_t warp_agg; /* group-by terminal (shared-memory table or global atomics): 1 = lanes of a warp holding the
                         same group key add their values inside the warp and one of them issues the atomics
                         (north-star "warp-level reductions"; the point of Section 3.3's privatisation is
                         contention on a few counters); 0 or 2 = off, the default: measured slower than per-lane
                         shared-memory atomics at every group count from 2 to 1000 */
    int32_t unfused; /* 1 = ablation: run the query operator at a time instead of fused (Section 4.1's engine before
                        fusion, Section 5.4's first step): one kernel per predicate and per join over the whole
                        table, a flag byte per row that every operator reads and rewrites, gathered payloads
                        written out as columns, then an aggregation kernel with global atomics.  Same result;
                        needs `unfused_scratch`.  Ignores specialise and the queue / shared-memory options. */
    void *unfused_scratch;       /* device scratch of at least sjq_unfused_scratch_bytes() bytes (16-byte aligned) */
    size_t unfused_scratch_bytes;
    int32_t pass_ppm[SJQ_MAX_PREDS + SJQ_MAX_JOINS]; /* measured pass fractions in parts per million, predicates
                                  first, then joins (index npreds + join): 0 = not known, the library estimates
                                  (a fact predicate from its operator alone, a join from the share of dimension
                                  rows its table holds); k > 0 = k / 1e6 of the rows pass that filter taken on its
                                  own (use 1 for "none seen").  sjq_pred_sample measures the predicates.  The
                                  estimates order the stages, split them into levels, pick the aggregation path
                                  and decide copy versus in-place reads in sjq_run_host: they change the run time,
                                  never the result. */
    int32_t hot_keys; /* open-addressing joins: 0 = library chooses (a hot-key table is used when `hot_scratch` is
                         given, the table sits behind its presence bitmap, its codes are at most 32 bits wide, the
                         kernel is compiled for the query (`specialise`) and the fact table has at least 2^26
                         rows), 1 = whenever the scratch is given, 2 = never.
                         Section 3.3 keeps the probed structure small enough to stay in cache; an open-addressing
                         table over millions of keys cannot, but with skewed foreign keys the answers for the few
                         keys that carry most rows can: before the fused pass three small kernels sample the
                         foreign-key column (2^18 evenly spaced rows), pick the keys seen most often and look each
                         up in the dimension table once; the fused kernel holds the 2048 answers (present with
                         this code / absent) in shared memory and consults them before the bitmap and before the
                         exact probe.  When the keys held cover less than a tenth of the sample the table is left
                         empty and the kernel skips the look-ups.  Same result either way; no host wait. */
    void *hot_scratch;        /* device scratch of at least SJQ_HOT_SCRATCH_BYTES bytes (16-byte aligned), used by */
    size_t hot_scratch_bytes; /* this run only; NULL = no hot-key table */
    int32_t l0_bulk; /* first column of a query with survivor queues, compiled kernels only: 1 = bring it into
                        shared memory with bulk-asynchronous copies (`cp.async.bulk` global -> shared completing on
                        an mbarrier; one copy per block tile of 12 to 64 KB, three in flight per block; no tensor
                        map, no cluster multicast, this GPU's memory only) whenever the shared memory is there;
                        0 or 2 = 128-bit loads with L2 prefetch, the default: Section 3.2's scan is bound by the
                        bytes in flight, and in this kernel, whose warps run independently, the loads keep more
                        of them in flight than the staged tiles do (measured slower at every point of the
                        selectivity sweep).  Every wait on a copy is bounded; one that runs out sets
                        SJQ_ERR_ASYNC_WAIT in *out->status and the kernel goes on with loads.  3 = as 1, but the
                        copies are never issued: every wait runs out (well under a second each), which is how the
                        tests reach that path without faulting anything; the result is still exact. */
} sjq_run_opts;

#define SJQ_HOT_SCRATCH_BYTES ((size_t)3 * 1048576 + 65536)

/* What the planner decided for a run (for reports and tests). */
typedef struct sjq_run_info {
    int32_t nstages;
    int32_t order[SJQ_MAX_PREDS + SJQ_MAX_JOINS + 8]; /* as in sjq_run_opts.order; -1 = plain column load */
    int32_t stage_in_smem[SJQ_MAX_PREDS + SJQ_MAX_JOINS + 8];
    int32_t first_sparse_stage; /* stages before this one filter thread-owned rows (level 0); later stages run
                                   on compacted survivors; 0 = no queues at all */
    int32_t reserved_levels;    /* number of queue-fed levels (the last one is the final level) */
    int32_t agg_path;           /* 0 scalar registers, 1 shared-memory table, 2 global atomics, 3 global hash */
    int32_t grid, block;
    int32_t smem_bytes;
    int32_t kernel_launches; /* kernels enqueued by the call */
} sjq_run_info;

/*
 * Measure the pass fraction of every fact predicate on an evenly spaced
 * sample of the table (65 536 groups of four rows), each predicate on its own.
 * Section 3.2 of the paper ties run time to the bytes the lazily loaded columns
 * move, which the selectivities decide, and Section 4.3.1 has the engine check
 * properties of the data at run time instead of assuming them; here the
 * planner's selectivity guesses are replaced by measured ones.
 *   scratch_dev  device scratch of SJQ_PLAN_SCRATCH_BYTES bytes
 *   pass_ppm     receives npreds entries, laid out like sjq_run_opts.pass_ppm
 *                (a predicate that passed no sampled row gets 1, not 0)
 * sjq_pred_sample enqueues one small kernel on `stream`, copies the counters
 * back and SYNCHRONISES the stream.  The two halves let the wait be shared
 * with other planning work: `_begin` enqueues the kernel and an asynchronous
 * copy of SJQ_MAX_PREDS + 1 counters into `host_counts` (page-locked host
 * memory) and returns; after the caller has synchronised that stream, `_end`
 * turns the counters into pass_ppm on the host.
 * Errors: INVALID_ARG, ALIGN, CUDA.
 */
sjq_status sjq_pred_sample(const sjq_col *fact, int nfact, const sjq_pred *preds, int npreds, void *scratch_dev,
                           void *stream, int32_t *pass_ppm);
sjq_status sjq_pred_sample_begin(const sjq_col *fact, int nfact, const sjq_pred *preds, int npreds,
                                 void *scratch_dev, int64_t *host_counts, void *stream);
sjq_status sjq_pred_sample_end(const int64_t *host_counts, int npreds, int32_t *pass_ppm);

/* Device bytes the operator-at-a-time ablation (sjq_run_opts.unfused) needs as scratch for a fact table of
 * `rows` rows and `njoins` joins: one flag byte per row and one 8-byte cell per row and join. */
sjq_status sjq_unfused_scratch_bytes(int64_t rows, int njoins, size_t *bytes);

/* Device bytes needed at sjq_result.workspace for `spec` (0 unless HASHED): room for the global group table
 * of Section 3.3 ("the global table" kept for queries with very many groups), three int64 arrays of twice the
 * capacity, rounded up to a power of two, plus one side slot. */
sjq_status sjq_run_workspace_bytes(const sjq_result_spec *spec, size_t *bytes);

/*
 * One fused pass over the fact table: Section 4.2.2's operator vocabulary
 * (a selection narrows the set of passing rows, a join probe drops the rows
 * without a match, a gather pulls one dimension attribute into the row, the
 * terminal consumes the survivors) run per row in one kernel, with Section
 * 3.2's lazy loading (a later column is read only for rows that are still
 * alive) and Section 3.3's terminals (register sum with one atomic per block,
 * shared-memory privatised group table, global table).
 *   fact/nfact   fact columns (device), equal length N >= 0 (N need not be a
 *                multiple of anything)
 *   preds        conjunction over fact columns (npreds <= SJQ_MAX_PREDS)
 *   joins        inner equi-joins (njoins <= SJQ_MAX_JOINS): a row survives
 *                iff every fk finds its key; a key outside a direct table's
 *                range is a miss, never an out-of-bounds access
 *   key          group key expression (NULL iff spec->mode == SJQ_SCALAR)
 *   agg          value summed per group
 *   out          result buffers; cleared by this call unless opts->accumulate
 *   info         optional: receives the plan that was used
 * Enqueues a clear kernel, the fused kernel and (HASHED) a compaction kernel
 * on `stream`; does not synchronise.  Host-detected errors are returned;
 * device-detected errors (GROUP_RANGE, GROUP_OVERFLOW) go to *out->status.
 */
sjq_status sjq_run(const sjq_col *fact, int nfact, const sjq_pred *preds, int npreds, const sjq_join *joins,
                   int njoins, const sjq_key_expr *key, const sjq_agg_expr *agg, const sjq_result_spec *spec,
                   const sjq_result *out, const sjq_run_opts *opts, void *stream, sjq_run_info *info);

/*
 * Put a HASHED result into its canonical order: ascending (signed) key.
 * Section 3.3's global table returns its groups in table order, which depends
 * on the hash function and the capacity; the paper compares results through an
 * order-free checksum (Section 2.2), this library gives the list itself an
 * order instead.  A radix sort of (key, position) pairs on the device, then
 * one gather of the three arrays.
 *   keys/sums/counts  device arrays of `capacity` entries (8-byte aligned), of
 *                     which the first *n_groups hold the result; sorted in place
 *   n_groups          device pointer, read by the kernels (no host wait)
 *   scratch           device scratch of sjq_result_sort_scratch_bytes(capacity)
 *                     bytes, 16-byte aligned (about 40 bytes per entry)
 * capacity <= 2^31.  Enqueues 27 small kernels on `stream`; does not
 * synchronise.  Errors: INVALID_ARG, ALIGN, BUFFER_SMALL, CUDA.
 */
sjq_status sjq_result_sort_scratch_bytes(int64_t capacity, size_t *bytes);
sjq_status sjq_result_sort(int64_t *keys, int64_t *sums, int64_t *counts, const int64_t *n_groups, int64_t capacity,
                           void *scratch, size_t scratch_bytes, void *stream);

/*
 * Merge lists of (key, sum, count) triples into one list with one entry per
 * distinct key, sums and counts added (int64, wrapping).  This is the exchange
 * step of a row-sharded run over several GPUs (the paper's second scale point,
 * Section 5.1, is a table twice the size of the first): every GPU runs sjq_run
 * on its row range, the per-GPU HASHED lists are gathered, and this call
 * folds them; integer sums make the result independent of the split.
 *   keys/sums/counts  device arrays of n entries (8-byte aligned; a key may
 *                     occur any number of times)
 *   capacity          maximum number of distinct keys
 *   out               keys/sums/counts[capacity], n_groups, status, and a
 *                     workspace of sjq_run_workspace_bytes({SJQ_HASHED, 0,
 *                     capacity}) bytes; all cleared by this call.  The output
 *                     arrays must not overlap the inputs.
 * Enqueues three kernels on `stream`; does not synchronise.  More distinct
 * keys than `capacity` sets SJQ_ERR_GROUP_OVERFLOW in *out->status.
 */
sjq_status sjq_merge_groups(const int64_t *keys, const int64_t *sums, const int64_t *counts, int64_t n,
                            int64_t capacity, const sjq_result *out, void *stream);

/*
 * The same query over fact columns that live in HOST memory (page-locked for
 * full copy speed): the table is cut into chunks of `chunk_rows` rows; each
 * chunk's columns are copied into one half of the device staging buffer while
 * the previous chunk is being processed from the other half (two internal
 * streams, ordered after and joined back into `stream`), every chunk runs
 * sjq_run with `accumulate` into `out`, and at the end the result arrays are
 * copied to the host.
 *   fact_host     columns whose `data` are HOST pointers (n = total rows)
 *   staging_dev   device buffer of at least 2 * chunk_rows * (sum of column
 *                 widths, each rounded up to 16 bytes per chunk) bytes
 *   chunk_rows    rows per chunk, a positive multiple of 4
 *   host_sums / host_counts / host_keys / host_n_groups / host_status
 *                 host destinations (page-locked for an asynchronous copy) of
 *                 the arrays of `out`; NULL = do not copy that one.  HASHED
 *                 results copy `capacity` entries.
 * A column that most rows still need when it is first read is copied whole.
 * A column that at most a few per cent of the rows reach (by the planner's
 * estimate) is not copied when its buffer is page-locked: the kernel reads it
 * in place over the bus, for the surviving rows only, which moves far fewer
 * bytes (opts->host_copy_all = 1 copies it all the same; a pageable buffer is
 * always copied).  A column the query does not reference is not transferred.
 * The host buffers must stay valid and unchanged until `stream` has finished.
 * Enqueues only; the caller synchronises `stream`.  Errors as sjq_run, plus
 * BUFFER_SMALL.
 */
sjq_status sjq_run_host(const sjq_col *fact_host, int nfact, const sjq_pred *preds, int npreds,
                        const sjq_join *joins, int njoins, const sjq_key_expr *key, const sjq_agg_expr *agg,
                        const sjq_result_spec *spec, const sjq_result *out, const sjq_run_opts *opts,
                        void *staging_dev, size_t staging_bytes, int64_t chunk_rows, int64_t *host_sums,
                        int64_t *host_counts, int64_t *host_keys, int64_t *host_n_groups, int32_t *host_status,
                        void *stream);

/*
 * What sjq_run_host would do with each column of `fact_host` for this query:
 * how[c] = 0 copied chunk by chunk, 1 read in place from the page-locked host
 * buffer by the kernel, 2 not transferred (the query does not reference it);
 * share[c] (optional) = estimated share of the rows the column is first read
 * for.  Enqueues nothing.
 */
sjq_status sjq_host_transfer_plan(const sjq_col *fact_host, int nfact, const sjq_pred *preds, int npreds,
                                  const sjq_join *joins, int njoins, const sjq_key_expr *key,
                                  const sjq_agg_expr *agg, const sjq_run_opts *opts, int32_t *how, double *share);

/*
 * Hashed group-by without any workspace from the caller.  (The paper has no
 * counterpart: this entry point exists for embedders, not for the method.)
 *
 * Who needs it: code that runs where device allocation is forbidden or
 * impossible -- a plug-in handed a fixed arena by its host process, a
 * real-time or safety-certified loop whose rules ban allocator calls after
 * start-up, a process whose memory pool is owned by another runtime.  Such a
 * caller can still own its input columns and result arrays (they were given
 * to it), but it has nowhere to get the group hash table that sjq_run takes
 * as `workspace` in HASHED mode.
 *
 * What it does: exactly sjq_run with spec->mode == SJQ_HASHED, except that the
 * group table lives in a fixed array inside the library's device image
 * (SJQ_STATIC_WORKSPACE_BYTES, about 3 MiB, held by every GPU that loads the
 * library until the process exits).  `out->workspace` and
 * `out->workspace_bytes` are ignored; `out->keys/sums/counts` need `capacity`
 * entries, `out->n_groups` and `out->status` as for sjq_run.
 *
 * Limits and rules:
 *   - capacity must be 1 .. SJQ_STATIC_MAX_GROUPS; a larger request returns
 *     SJQ_ERR_STATIC_LIMIT and enqueues nothing.
 *   - `opts->accumulate` is ignored: the table is cleared at the start of
 *     every call, because it is shared by all calls and still holds the
 *     previous call's groups.
 *   - `opts->specialise` is ignored: a module compiled at run time is loaded
 *     when its query shape is first met, which places code on the device at an
 *     arbitrary moment, so this entry point always runs the interpreted kernel.
 *   - Calls whose kernels could overlap on the GPU (different streams, several
 *     host threads) race on the one table; run them one after another.
 *   - The first call on a device looks the array's device address up once, and
 *     the CUDA driver loads each ahead-of-time kernel the first time it is
 *     launched (that loading is the driver's own and may reserve device memory
 *     for code).  Make one call per query shape you will use during start-up,
 *     outside any stream capture; later calls take nothing from the device.
 *   - What is promised: the library itself calls no cudaMalloc,
 *     cudaMallocAsync, cudaFree or allocating library routine on this path,
 *     and needs no workspace from the caller.
 */
#define SJQ_STATIC_MAX_GROUPS 65536
#define SJQ_STATIC_WORKSPACE_BYTES ((size_t)3 * 1024 * 1024 + 768 + 3 * 256)
sjq_status sjq_run_hashed_static(const sjq_col *fact, int nfact, const sjq_pred *preds, int npreds,
                                 const sjq_join *joins, int njoins, const sjq_key_expr *key,
                                 const sjq_agg_expr *agg, int64_t capacity, const sjq_result *out,
                                 const sjq_run_opts *opts, void *stream, sjq_run_info *info);

const char *sjq_strerror(sjq_status status);
const char *sjq_version(void);

/*
 * Give back what the library holds on behalf of the calling thread and the
 * process: the two internal streams and three events sjq_run_host creates per
 * device and thread on first use, the modules compiled at run time, and the
 * remembered occupancy answers.  Nothing the library enqueued may still be
 * running.  Later calls create what they need again.  Returns the number of
 * objects released.  (Host-side bookkeeping only; the paper has no counterpart.)
 */
int32_t sjq_release(void);

/*
 * Run-time specialisation (Section 4.2 of the paper fuses a query's operators before it runs; here the fused
 * kernel is compiled for the query's shape with NVRTC when sjq_run_opts.specialise is set).
 * Compiled modules are cached per process, keyed by the query's shape.  The compiler needs the device sources:
 * they are looked for in csrc/ beside the library and ../include (the environment variables SJQ_SOURCE_DIR and
 * SJQ_INCLUDE_DIR name other places); SJQ_JIT_VERBOSE=1 prints the compiler's output to stderr.  SJQ_JIT_EXTRA
 * (extra compiler options, part of the cache key) is a development hook, not a supported interface.
 * sjq_jit_log copies the compiler output of the most recent compilation into `buf` (NUL-terminated, truncated
 * to `bytes`) and returns its full length.  sjq_jit_selftest compiles one of a few built-in query shapes
 * (shape_id 0 .. sjq_jit_selftest(-1, ...) - 1) without touching a device: SJQ_OK if the device code
 * compiles for sm_100a, SJQ_ERR_JIT otherwise, with the compiler output in `log`; shape_id -1 returns the number
 * of built-in shapes instead of a status.
 */
size_t sjq_jit_log(char *buf, size_t bytes);
/* Unload every module compiled at run time in this process and forget them (the next specialised run of a shape
 * compiles or loads it again); returns how many were unloaded.  No kernel of such a module may still be running. */
int32_t sjq_jit_cache_clear(void);
int32_t sjq_jit_selftest(int32_t shape_id, char *log, size_t log_bytes);

#ifdef __cplusplus
}
#endif
#endif /* SJQ_H */
