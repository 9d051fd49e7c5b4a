// Device-side description of one fused run: a chain of stages over the fact
// table followed by a terminal.  The chain plays the role of the paper's slot
// sequence (Section 4.2.2: select-literal, probe, gather, then the terminal);
// the query's identity is data in this struct, not generated code.
#ifndef SJQ_RUN_CUH
#define SJQ_RUN_CUH

#include "sjq_internal.h"

namespace sjq {

enum : uint8_t { ST_PRED = 0, ST_PROBE = 1, ST_LOAD = 2 };
enum : int32_t { AGG_SCALAR = 0, AGG_SMEM = 1, AGG_GLOBAL = 2, AGG_HASH = 3 };

// Stage bodies (uniform switch per stage, straight-line code inside).
enum : uint8_t {
    OP_LOAD = 0,
    OP_PRED_RANGE = 1,
    OP_PRED_SET = 2,
    OP_DIRECT_BITMAP = 3,
    OP_DIRECT_U8 = 4,
    OP_DIRECT_U16 = 5,
    OP_DIRECT_U32 = 6,
    OP_DIRECT_U64 = 7,
    OP_HASH32 = 8,
    OP_HASH64 = 9,
    OP_HASHBITS = 10, // presence bitmap in front of an open-addressing table, indexed by a hash of the key
    OP_DIRECT_U4 = 11, // sub-byte codes, eight / sixteen to a 32-bit word
    OP_DIRECT_U2 = 12
};
__host__ __device__ constexpr bool is_code_op(int op)
{
    return (op >= OP_DIRECT_U8 && op <= OP_DIRECT_U64) || op == OP_DIRECT_U4 || op == OP_DIRECT_U2;
}
__host__ __device__ constexpr bool is_direct_op(int op) { return op == OP_DIRECT_BITMAP || is_code_op(op); }

// which accumulators a stage's values feed: bit = 3 * source + destination,
// source 0 = the fact value itself, 1 = payload 0, 2 = payload 1;
// destination 0 = group key, 1 = X, 2 = Y.  value = X (or X*Y for a product).
constexpr int kAccKey = 0, kAccX = 1, kAccY = 2;

// predicates + joins (two stages when hashed) + plain loads + gather copies.  A kernel compiled for one query
// carries exactly that query's stages: its parameter block is a tenth of the general one, which takes about
// 4 us off every launch (launch latency by parameter size, measured: 64 B 4.5 us, 2 KB 4.7, 8 KB 5.7, 21 KB 8.7).
#if defined(SJQ_JIT)
constexpr int kMaxStages = SJQ_JIT_nstages > 0 ? SJQ_JIT_nstages : 1;
#else
constexpr int kMaxStages = 72;
#endif

// Geometry of the fused kernel.
#ifndef SJQ_SLOTS
#define SJQ_SLOTS 2
#endif
constexpr int kSlots = SJQ_SLOTS;        // level 0: 128-bit loads per thread per tile
constexpr int kDenseRows = 4 * kSlots;   // rows a thread owns at level 0
#ifndef SJQ_ROWS
#define SJQ_ROWS 4 // the ahead-of-time kernels; a kernel compiled for one query may use 8
#endif
constexpr int kRows = SJQ_ROWS;          // rows a lane handles per batch at the queue-fed levels
constexpr int kDirectRows = 4;           // rows a thread owns when there are no queues at all (one 128-bit load)
constexpr int kBatch = 32 * kRows;       // rows a warp processes at once at those levels
constexpr int queue0_cap_for(int slots) { return slots <= 2 ? 512 : 1024; }
constexpr int kQueue0Cap = queue0_cap_for(kSlots); // first queue of a warp: a batch minus one plus a whole tile fit
constexpr int queue_cap_for(int rows) { return 64 * rows; }
constexpr int kQueueCap = queue_cap_for(kRows); // its later queues: a batch minus one plus a batch fit
constexpr int kMaxQueues = 3;            // queue-fed levels per warp (the last one is the final level)

struct DStage {
    const void *col;   // fact column read by this stage
    const void *tab;   // direct: code array / bitmap words; hash: bucket array; presence bitmap: its words
    int64_t kmin;      // direct: slot index = key - kmin
    uint64_t last;     // direct: last valid slot index (slots - 1); hash (and its bitmap stage): bucket count
    int64_t lo, hi;    // 64-bit predicate range
    uint64_t hmask;    // presence bitmap of a hash table: bits - 1
    int64_t pmin0, pmin1;
    uint64_t pmask0;
    int64_t mult[9];
    int32_t mult32[9]; // the same multipliers when acc32
    int32_t acc32;     // every multiplier, raw value and payload of this stage fits in 32 bits
    int32_t lo32;      // 32-bit predicate: pass iff (uint32)(v - lo32) <= width32
    uint32_t width32;
    int32_t kmin32;    // 32-bit direct probe: idx = min((uint32)v - (uint32)kmin32, clamp32)
    uint32_t last32;
    uint32_t clamp32;  // index of the spare, never set entry after the last slot (every key outside the range lands there)
    uint32_t smem_off;  // byte offset of the staged copy in dynamic shared memory
    uint32_t tab_bytes; // bytes to stage
    uint16_t acc;
    uint8_t op, is64, neg, never, nset, set_idx, pbits0, code_bits, in_smem, kind;
    uint8_t simple; // 1 + destination (0 key, 1 X, 2 Y): plain int32 load feeding one accumulator through mult32
    int8_t issue_after; // final level of a compiled kernel: the column is requested once this stage's mask is known
                        // (a stage before the level's first one = on entry)
    uint8_t full;   // sub-byte direct table holding every key of its range: a probe hits iff its key is in range
    uint8_t hot;    // open-addressing join (its bitmap stage and its exact probe): consult the hot-key table first
    uint8_t wide;   // open-addressing probe: the bucket array starts on a 32-byte boundary, so a bucket is one 256-bit load
    const void *hot_tab; // hot-key table in global memory (kHotSlots + 1 entries), copied to shared memory per block
    uint32_t hot_off;    // byte offset of that copy in dynamic shared memory
    uint32_t hot_pad;
};
static_assert(sizeof(DStage) % 8 == 0, "stage descriptors are copied as 64-bit words");

struct RunParams {
    DStage st[kMaxStages];
    int64_t sets[SJQ_MAX_PREDS][SJQ_MAX_IN_SET];
    int64_t n;
    int64_t key_offset;
    int64_t modulo;   // 0 = none
    int64_t post_offset; // added to the key after the modulo (a hashed result kept as a direct-indexed table)
    uint64_t modmask; // modulo - 1 when modulo is a power of two, else 0
    int64_t num_groups;
    uint64_t gmask; // hashed: group-table slots - 1
    int64_t *sums;  // scalar/dense: result; hashed: table sums
    int64_t *counts; // may be NULL
    int64_t *gkeys;  // hashed: table keys
    int32_t *status;
    int32_t nstages;
    int32_t nq;     // queue-fed levels: 0 = none (every stage on thread-owned rows); else stages 0 .. nd0-1
                    // filter thread-owned rows at level 0, stages nd0 .. nd0+nq-2 are queue-fed filters and
                    // stages from nd0+nq-1 on run at the final level
    int32_t nd0;
    int32_t rows;   // rows per lane and batch at the queue-fed levels: 4, or 8 in a kernel compiled for it
    int32_t slots;  // level 0: groups of four rows a thread owns per tile: 2, or 4 in a kernel compiled for it
    uint32_t qfold; // 7: queue slots are swizzled (dense survivors), 0: ring positions are used as they are
    int32_t want_count;
    int32_t eager;   // load every column for every row
    int32_t has_key; // scalar path of a one-group dense result: key is computed and range-checked
    int32_t mod32;   // modulo fits in 32 bits
    int32_t warp_agg; // group-by terminal: equal keys of a warp are added inside the warp before the atomics
    uint32_t smem_stages; // byte offset of the stage descriptors copied to shared memory
    uint32_t smem_groups; // byte offset of the shared group table
    uint32_t smem_queue;  // byte offset of the per-warp survivor queues
    uint32_t smem_l0;     // byte offset of the per-warp staging buffers of the first column (then their mbarriers)
    int32_t sparse_push;  // few rows survive level 0: the push into the first queue walks the set bits of the mask
    int32_t count32;      // fewer than 2^32 fact rows: a block's count of a group fits 32 bits (no carry into the high word)
    int32_t l0_bulk;      // compiled kernels: the first column arrives by bulk-asynchronous copies into shared memory
};

#if !defined(SJQ_JIT)
// The sixteen ahead-of-time variants of the fused kernel (aggregation path x product aggregate x "some table is
// open-addressing"), instantiated in one translation unit per aggregation path.
typedef void (*fused_fn)(const RunParams);
fused_fn fused_variant_scalar(bool mul, bool hash);
fused_fn fused_variant_smem(bool mul, bool hash);
fused_fn fused_variant_global(bool mul, bool hash);
fused_fn fused_variant_hash(bool mul, bool hash);
#endif

} // namespace sjq

#endif
