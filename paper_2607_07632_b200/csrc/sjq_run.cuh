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

// which accumulators a stage's values feed: bit = 3 * source + destination,
// source 0 = the fact value itself, 1 = payload 0, 2 = payload 1;
// destination 0 = group key, 1 = X, 2 = Y.  value = X (or X*Y for a product).
constexpr int kAccKey = 0, kAccX = 1, kAccY = 2;

constexpr int kMaxStages = SJQ_MAX_PREDS + SJQ_MAX_JOINS + 8;

struct DStage {
    const void *col;   // fact column read by this stage
    const void *tab;   // direct: code array / bitmap words; hash: key array
    const void *codes; // hash: payload codes
    int64_t kmin;      // direct: slot index = key - kmin
    uint64_t span;     // direct: number of slots
    uint64_t hmask;    // hash: slots - 1
    int64_t pmin0, pmin1;
    uint64_t pmask0;
    int64_t mult[9];
    DPred pred;
    uint32_t smem_off;  // byte offset of the staged copy in dynamic shared memory
    uint32_t tab_bytes; // bytes to stage
    uint16_t acc;
    uint8_t kind, is64, tkind, in_smem, pbits0, code_bits;
};

struct RunParams {
    DStage st[kMaxStages];
    int64_t n;
    int64_t key_offset;
    int64_t modulo;   // 0 = none
    uint64_t modmask; // modulo - 1 when modulo is a power of two, else 0
    int64_t num_groups;
    uint64_t gmask;    // hashed: group-table slots - 1
    int64_t *sums;     // scalar/dense: result; hashed: table sums
    int64_t *counts;   // may be NULL
    int64_t *gkeys;    // hashed: table keys
    int32_t *status;
    int32_t nstages;
    int32_t first_sparse; // stages >= this run on compacted survivors
    int32_t want_count;
    int32_t eager;
    int32_t has_key;      // compute and range-check the key (dense with one group in scalar path)
    int32_t mod32;        // modulo fits in 32 bits
    uint32_t smem_groups; // byte offset of the shared group table
    uint32_t smem_queue;  // byte offset of the per-warp survivor queues
    uint32_t carry;       // bit 0 key, 1 X, 2 Y: accumulators live at the dense->sparse switch
};

} // namespace sjq
#endif
