// Internal structures shared by the translation units of libsjq.
#ifndef SJQ_INTERNAL_H
#define SJQ_INTERNAL_H

#include <cuda_runtime.h>
#include <stdint.h>

#include "sjq.h"

namespace sjq {

// ---------------------------------------------------------------- predicates
// Canonical form of one predicate: an inclusive range [lo, hi], optionally
// negated, or a small set.  An empty range is encoded as lo > hi.
struct DPred {
    int64_t lo, hi;
    int64_t set[SJQ_MAX_IN_SET];
    int32_t lo32, hi32; // the same range clamped to int32 (for int32 columns)
    int32_t col;
    uint8_t neg;   // pass iff NOT in range
    uint8_t nset;  // > 0: pass iff value in set[0..nset)
    uint8_t is64;  // dtype of the column
    uint8_t never; // range empty for this dtype: nothing passes (before negation)
};

bool canon_pred(const sjq_pred &p, int dtype, DPred *out);

// ---------------------------------------------------------------- tables
constexpr int64_t kEmptyKey64 = INT64_MIN;
constexpr int32_t kEmptyKey32 = INT32_MIN;
// An open-addressing table is an array of 32-byte buckets (one memory sector), each holding K keys followed
// by their K payload codes, so that a probe step is one sector and a hit finds its code in the sector it
// already has (Section 3.3's point about the unpacked table: what a probe touches decides its cost).  A key's
// linear probe starts at its home bucket (multiply-high range reduction of its hash, so the bucket count need
// not be a power of two), a lookup loads whole buckets and stops at the first one with a free slot; inserts
// fill a bucket's slots in order.  Measured on the skewed 64-bit-key workload (300 M probes, 2 M keys, load
// 0.5): keys and codes in separate arrays with 32-byte key buckets 1.76 ms, 64-byte buckets of keys and codes
// 2.19 ms (two sectors per step), 32-byte buckets of keys and codes 1.71 ms.
constexpr int kBucketBytes = 32;
// keys per bucket for a key of kb bytes with a code of cb bytes (0, 4 or 8): the largest K with
// K * kb rounded up to the code's alignment + K * cb <= the bucket size
__host__ __device__ constexpr int bucket_code_offset(int kb, int cb, int k)
{
    return cb == 0 ? k * kb : (k * kb + cb - 1) / cb * cb;
}
__host__ __device__ constexpr int bucket_keys(int kb, int cb)
{
    int k = kBucketBytes / (kb + cb);
    while (k > 1 && bucket_code_offset(kb, cb, k) + k * cb > kBucketBytes) --k;
    return k;
}
static_assert(bucket_keys(8, 4) == 2 && bucket_keys(8, 8) == 2 && bucket_keys(8, 0) == 4, "64-bit keys");
static_assert(bucket_keys(4, 4) == 4 && bucket_keys(4, 8) == 2 && bucket_keys(4, 0) == 8, "32-bit keys");
constexpr size_t kTableHeaderBytes = 256; // device-side counters at the start of table_mem

} // namespace sjq

struct sjq_table {
    sjq_dim_layout layout;
    char *base;          // table_mem
    char *slots;         // direct: code array / bitmap words; hash: bucket array
    char *filter;        // presence bitmap (NULL when none)
    size_t slots_bytes;  // bytes of the direct array (for shared-memory staging) or of the bucket array
    int32_t launches;    // kernels sjq_build_dim enqueued
    uint32_t magic;
};

namespace sjq {

constexpr uint32_t kTableMagic = 0x534a5154u; // "SJQT"

inline bool is_hash_kind(int kind) { return kind == SJQ_TABLE_HASH_I32 || kind == SJQ_TABLE_HASH_I64; }
inline bool is_direct_kind(int kind)
{
    return (kind >= SJQ_TABLE_DIRECT_BITMAP && kind <= SJQ_TABLE_DIRECT_U64) || kind == SJQ_TABLE_DIRECT_U4 ||
           kind == SJQ_TABLE_DIRECT_U2;
}
// width of the code a direct kind stores per key (0: bitmap)
inline int direct_kind_bits(int kind)
{
    switch (kind) {
    case SJQ_TABLE_DIRECT_U2: return 2;
    case SJQ_TABLE_DIRECT_U4: return 4;
    case SJQ_TABLE_DIRECT_U8: return 8;
    case SJQ_TABLE_DIRECT_U16: return 16;
    case SJQ_TABLE_DIRECT_U32: return 32;
    case SJQ_TABLE_DIRECT_U64: return 64;
    default: return 0;
    }
}

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Hash of a 64-bit key for the dimension hash tables and the group hash table: fold the high half
// into the low one, one odd 64-bit multiply, take the upper word.  Every bit of the key reaches the
// low bits of the result (the slot index) at the price of about six instructions.
__host__ __device__ inline uint64_t hash64(uint64_t k)
{
    k ^= k >> 32;
    k *= 0x9E3779B97F4A7C15ULL;
    return k >> 32;
}

// Home bucket of a key in a table of `buckets` buckets (any count below 2^32).
__host__ __device__ inline uint32_t home_bucket(uint64_t k, uint32_t buckets)
{
    return (uint32_t)((hash64(k) * (uint64_t)buckets) >> 32);
}

// A second, independent hash for the presence bitmap in front of an open-addressing table.
__host__ __device__ inline uint32_t filter_hash(uint64_t k)
{
    k ^= k >> 29;
    k *= 0xD6E8FEB86659FD93ULL;
    return (uint32_t)(k >> 32);
}

// Hot-key table of an open-addressing join (built per run from a sample of the foreign keys, held in shared
// memory by the fused kernel): direct-mapped, 16-byte entries {key low word, key high word, payload code,
// state}; state 0 = free, 1 = the key is in the dimension table (code valid), 2 = the key is absent.  Entry
// kHotSlots is a header whose first word counts the keys stored.
constexpr int kHotSlots = 2048;            // 32 KB of shared memory
constexpr int kHotCountSlots = 1 << 18;    // sample count table (global scratch)
constexpr int kHotSamples = 1 << 18;       // foreign keys sampled per run
__host__ __device__ inline uint32_t hot_hash(uint64_t k)
{
    k ^= k >> 31;
    k *= 0xBF58476D1CE4E5B9ULL;
    return (uint32_t)(k >> 37);
}

// first-error-wins store into the status word
__device__ inline void set_status(int32_t *status, int32_t code) { atomicCAS(status, 0, code); }

template <typename T>
__device__ inline bool pred_eval(const DPred &d, T v)
{
    if (d.nset) {
        bool f = false;
        for (int k = 0; k < d.nset; ++k) f |= ((int64_t)v == d.set[k]);
        return f;
    }
    bool in;
    if (sizeof(T) == 4) in = ((int32_t)v >= d.lo32) & ((int32_t)v <= d.hi32) & !d.never;
    else in = ((int64_t)v >= d.lo) & ((int64_t)v <= d.hi);
    return in != (bool)d.neg;
}

__device__ inline int64_t load_cell(const void *col, int is64, int64_t i)
{
    return is64 ? static_cast<const int64_t *>(col)[i] : (int64_t) static_cast<const int32_t *>(col)[i];
}

struct DeviceInfo {
    int device;
    int sm_count;
    int max_smem_optin;
    int l2_bytes;
};
sjq_status device_info(DeviceInfo *out);

} // namespace sjq

#endif
