// The fused probe kernel: one pass over the fact table.
//
// Execution model.  A machine-sized grid of persistent blocks strides over
// tiles of the fact table (Section 3.2 of the paper, "grid-stride persistent
// threads").  Every warp runs a small push pipeline of its own:
//
//  level 0   (dense) every thread owns kSlots groups of four consecutive
//            rows, so one 128-bit load brings four values of the first
//            column and a warp reads 512 contiguous bytes; the first stage
//            keeps one bit per row.  The sixteen loads and probes of a thread
//            are independent, which keeps enough bytes in flight to cover
//            HBM latency.
//  level l   the survivors of level l-1 are compacted (popcount + warp scan)
//            into queue l of the warp in shared memory; whenever a queue
//            holds a full batch (kRows per lane) the warp runs the next filter
//            stage on it, loading that stage's column with one 4-byte load per
//            surviving row only (lazy loading, Section 3.2: a later column is
//            never read for an eliminated row), and pushes the survivors on.
//  last      the final level gathers the group-key payloads and the measure
//            columns of the survivors into register accumulators and runs the
//            terminal.
//
// A probe is a range-checked single load from a direct-mapped table (global or
// staged in shared memory) or a bounded lock-step linear probe of an
// open-addressing table (Section 3.3).  The terminal is a register accumulator
// with one atomic per block, a shared-memory privatised group table flushed
// with one atomic per touched group per block, global atomics, or a global
// group hash table (Section 3.3 "Shared-memory privatized group-by").
#include <type_traits>

#include "sjq_run.cuh"

#ifndef SJQ_LB_THREADS
#define SJQ_LB_THREADS 384
#define SJQ_LB_BLOCKS 2
#endif
#ifndef SJQ_HASH_INLINE
#define SJQ_HASH_INLINE __forceinline__
#endif
#ifndef SJQ_PREFETCH_DIST
#define SJQ_PREFETCH_DIST 2
#endif

namespace sjq {

namespace {

template <typename T>
struct Vec4;
template <>
struct Vec4<int32_t> {
    static __device__ __forceinline__ void load(const int32_t *p, int32_t *v)
    {
        const int4 a = __ldcs(reinterpret_cast<const int4 *>(p));
        v[0] = a.x, v[1] = a.y, v[2] = a.z, v[3] = a.w;
    }
};
template <>
struct Vec4<int64_t> {
    static __device__ __forceinline__ void load(const int64_t *p, int64_t *v)
    {
        const longlong2 a = __ldcs(reinterpret_cast<const longlong2 *>(p));
        const longlong2 b = __ldcs(reinterpret_cast<const longlong2 *>(p) + 1);
        v[0] = a.x, v[1] = a.y, v[2] = b.x, v[3] = b.y;
    }
};

// One value of a later column for one surviving row.
#if defined(SJQ_SPARSE_PLAIN)
__device__ __forceinline__ int32_t ld_sparse(const int32_t *p)
{
    int32_t v;
    asm volatile("ld.global.b32 %0, [%1];" : "=r"(v) : "l"(p));
    return v;
}
__device__ __forceinline__ int64_t ld_sparse(const int64_t *p)
{
    int64_t v;
    asm volatile("ld.global.b64 %0, [%1];" : "=l"(v) : "l"(p));
    return v;
}
#else
__device__ __forceinline__ int32_t ld_sparse(const int32_t *p) { return __ldg(p); }
__device__ __forceinline__ int64_t ld_sparse(const int64_t *p) { return __ldg(p); }
#endif

template <typename T>
struct Index {
    typedef uint64_t type;
};
template <>
struct Index<int32_t> {
    typedef uint32_t type;
};

// ------------------------------------------------------------------ stage bodies
// Each body takes the values v[0..NR) of the rows whose bit is set in m and
// returns the mask of rows that pass.  Values of rows outside m are ignored.

template <typename T, int NR>
__device__ __forceinline__ uint32_t body_pred_range(const DStage &S, const T (&v)[NR], uint32_t m)
{
    uint32_t pass = 0;
    if (sizeof(T) == 4) {
        if (!S.never) {
#pragma unroll
            for (int i = 0; i < NR; ++i)
                pass |= (uint32_t)(((uint32_t)v[i] - (uint32_t)S.lo32) <= S.width32) << i;
        }
    } else {
#pragma unroll
        for (int i = 0; i < NR; ++i) pass |= (uint32_t)(((int64_t)v[i] >= S.lo) & ((int64_t)v[i] <= S.hi)) << i;
    }
    if (S.neg) pass = ~pass;
    return m & pass;
}

template <typename T, int NR>
__device__ __forceinline__ uint32_t body_pred_set(const RunParams &P, const DStage &S, const T (&v)[NR], uint32_t m)
{
    uint32_t pass = 0;
    for (int k = 0; k < S.nset; ++k) {
        const int64_t lit = P.sets[S.set_idx][k];
#pragma unroll
        for (int i = 0; i < NR; ++i) pass |= (uint32_t)((int64_t)v[i] == lit) << i;
    }
    return m & pass;
}

template <typename T, int OP, bool SMEM, int NR, bool WANT>
__device__ __forceinline__ uint32_t body_direct(const DStage &S, const unsigned char *smem, const T (&v)[NR],
                                                uint32_t m, uint64_t (&code)[NR])
{
    const unsigned char *base = SMEM ? smem + S.smem_off : static_cast<const unsigned char *>(S.tab);
    typename Index<T>::type idx[NR];
    uint32_t in = 0;
#pragma unroll
    for (int i = 0; i < NR; ++i) {
        if (sizeof(T) == 4) {
            const uint32_t d = (uint32_t)v[i] - (uint32_t)S.kmin32;
            idx[i] = d;
            in |= (uint32_t)(d <= S.last32) << i;
        } else {
            const uint64_t d = (uint64_t)v[i] - (uint64_t)S.kmin;
            idx[i] = d;
            in |= (uint32_t)(d <= S.last) << i;
        }
    }
    in &= m; // a key outside the table's range is a miss, never an access
    uint32_t hit = 0;
    if (OP == OP_DIRECT_BITMAP) {
        uint32_t w[NR];
#pragma unroll
        for (int i = 0; i < NR; ++i) {
            w[i] = 0;
            if ((in >> i) & 1u) {
                const uint32_t *p = reinterpret_cast<const uint32_t *>(base) + (idx[i] >> 5);
                w[i] = SMEM ? *p : __ldg(p);
            }
        }
#pragma unroll
        for (int i = 0; i < NR; ++i) hit |= ((w[i] >> (idx[i] & 31)) & 1u) << i;
        return in & hit;
    }
    uint64_t c[NR];
#pragma unroll
    for (int i = 0; i < NR; ++i) {
        c[i] = ~0ULL;
        if ((in >> i) & 1u) {
            if (OP == OP_DIRECT_U8) {
                const uint8_t *p = base + idx[i];
                c[i] = SMEM ? *p : __ldg(p);
            } else if (OP == OP_DIRECT_U16) {
                const uint16_t *p = reinterpret_cast<const uint16_t *>(base) + idx[i];
                c[i] = SMEM ? *p : __ldg(p);
            } else if (OP == OP_DIRECT_U32) {
                const uint32_t *p = reinterpret_cast<const uint32_t *>(base) + idx[i];
                c[i] = SMEM ? *p : __ldg(p);
            } else {
                const uint64_t *p = reinterpret_cast<const uint64_t *>(base) + idx[i];
                c[i] = SMEM ? *p : __ldg(p);
            }
        }
    }
    const uint64_t miss = OP == OP_DIRECT_U8 ? 0xFFull : OP == OP_DIRECT_U16 ? 0xFFFFull
                          : OP == OP_DIRECT_U32 ? 0xFFFFFFFFull : ~0ULL;
#pragma unroll
    for (int i = 0; i < NR; ++i) {
        hit |= (uint32_t)(c[i] != miss) << i;
        if (WANT) code[i] = c[i];
    }
    return in & hit;
}

// Open addressing with 32-byte buckets (4 int64 or 8 int32 keys): a key's linear probe starts at the
// first slot of its home bucket, so a lookup loads one whole bucket per step (two 128-bit loads),
// compares every key in it, and stops at a match or at the first bucket with a free slot.  The rows of
// a chunk advance in lock step so that their loads overlap; bounded by the bucket count.
__device__ __forceinline__ void load_bucket(const int64_t *p, int64_t (&k)[kBucketKeys64])
{
    const longlong2 a = __ldg(reinterpret_cast<const longlong2 *>(p));
    const longlong2 b = __ldg(reinterpret_cast<const longlong2 *>(p) + 1);
    k[0] = a.x, k[1] = a.y, k[2] = b.x, k[3] = b.y;
}
__device__ __forceinline__ void load_bucket(const int32_t *p, int32_t (&k)[kBucketKeys32])
{
    const int4 a = __ldg(reinterpret_cast<const int4 *>(p));
    const int4 b = __ldg(reinterpret_cast<const int4 *>(p) + 1);
    k[0] = a.x, k[1] = a.y, k[2] = a.z, k[3] = a.w, k[4] = b.x, k[5] = b.y, k[6] = b.z, k[7] = b.w;
}

template <typename T, int NR, bool WANT>
__device__ SJQ_HASH_INLINE uint32_t body_hash(const DStage &S, const T (&v)[NR], uint32_t m, uint64_t (&code)[NR])
{
    constexpr int KPB = sizeof(T) == 4 ? kBucketKeys32 : kBucketKeys64;
#ifndef SJQ_HASH_CH
#define SJQ_HASH_CH 2
#endif
    constexpr int CH = NR < SJQ_HASH_CH ? NR : SJQ_HASH_CH; // rows advancing together
    const T empty = sizeof(T) == 4 ? (T)kEmptyKey32 : (T)kEmptyKey64;
    const T *keys = static_cast<const T *>(S.tab);
    const uint32_t bmask = (uint32_t)(S.hmask / KPB); // buckets - 1
    uint32_t hit = 0;
    uint32_t slot[NR];
#pragma unroll
    for (int base = 0; base < NR; base += CH) {
        uint32_t bucket[CH];
        uint32_t pending = 0;
#pragma unroll
        for (int i = 0; i < CH; ++i) {
            bucket[i] = (uint32_t)hash64((uint64_t)(int64_t)v[base + i]) & bmask;
            slot[base + i] = 0;
            pending |= (uint32_t)(((m >> (base + i)) & 1u) && v[base + i] != empty) << i; // the marker is never a key
        }
        for (uint32_t it = 0; pending != 0 && it <= bmask; ++it) {
            T bk[CH][KPB];
#pragma unroll
            for (int i = 0; i < CH; ++i) {
#pragma unroll
                for (int j = 0; j < KPB; ++j) bk[i][j] = empty;
                if ((pending >> i) & 1u) load_bucket(keys + (size_t)bucket[i] * KPB, bk[i]);
            }
#pragma unroll
            for (int i = 0; i < CH; ++i) {
                if ((pending >> i) & 1u) {
                    bool found = false, has_free = false;
                    uint32_t at = 0;
#pragma unroll
                    for (int j = 0; j < KPB; ++j) {
                        if (bk[i][j] == v[base + i]) {
                            found = true;
                            at = j;
                        }
                        has_free |= bk[i][j] == empty;
                    }
                    if (found) {
                        hit |= 1u << (base + i);
                        slot[base + i] = bucket[i] * KPB + at;
                        pending &= ~(1u << i);
                    } else if (has_free) {
                        pending &= ~(1u << i);
                    } else {
                        bucket[i] = (bucket[i] + 1) & bmask;
                    }
                }
            }
        }
    }
    if (WANT && S.codes) {
#pragma unroll
        for (int i = 0; i < NR; ++i) {
            code[i] = 0;
            if ((hit >> i) & 1u)
                code[i] = S.code_bits == 64 ? __ldg(static_cast<const uint64_t *>(S.codes) + slot[i])
                                            : (uint64_t)__ldg(static_cast<const uint32_t *>(S.codes) + slot[i]);
        }
    }
    return hit;
}

// Presence bitmap of an open-addressing table: one bit per hash value; a clear bit proves the key
// absent, a set bit sends the row on to the exact probe.
template <typename T, int NR>
__device__ __forceinline__ uint32_t body_hashbits(const DStage &S, const T (&v)[NR], uint32_t m)
{
    const uint32_t *bits = static_cast<const uint32_t *>(S.tab);
    const uint32_t fmask = (uint32_t)S.hmask;
    uint32_t w[NR], idx[NR];
#pragma unroll
    for (int i = 0; i < NR; ++i) {
        idx[i] = filter_hash((uint64_t)(int64_t)v[i]) & fmask;
        w[i] = 0;
        if ((m >> i) & 1u) w[i] = __ldg(bits + (idx[i] >> 5));
    }
    uint32_t hit = 0;
#pragma unroll
    for (int i = 0; i < NR; ++i) hit |= ((w[i] >> (idx[i] & 31)) & 1u) << i;
    return m & hit;
}

template <typename T, int NR, bool WANT, bool HASH>
__device__ __forceinline__ uint32_t run_stage(const RunParams &P, const DStage &S, const unsigned char *smem,
                                              const T (&v)[NR], uint32_t m, uint64_t (&code)[NR])
{
    switch (S.op * 2 + S.in_smem) {
    case OP_PRED_RANGE * 2: return body_pred_range<T, NR>(S, v, m);
    case OP_PRED_SET * 2: return body_pred_set<T, NR>(P, S, v, m);
    case OP_DIRECT_BITMAP * 2: return body_direct<T, OP_DIRECT_BITMAP, false, NR, WANT>(S, smem, v, m, code);
    case OP_DIRECT_BITMAP * 2 + 1: return body_direct<T, OP_DIRECT_BITMAP, true, NR, WANT>(S, smem, v, m, code);
    case OP_DIRECT_U8 * 2: return body_direct<T, OP_DIRECT_U8, false, NR, WANT>(S, smem, v, m, code);
    case OP_DIRECT_U8 * 2 + 1: return body_direct<T, OP_DIRECT_U8, true, NR, WANT>(S, smem, v, m, code);
    case OP_DIRECT_U16 * 2: return body_direct<T, OP_DIRECT_U16, false, NR, WANT>(S, smem, v, m, code);
    case OP_DIRECT_U16 * 2 + 1: return body_direct<T, OP_DIRECT_U16, true, NR, WANT>(S, smem, v, m, code);
    case OP_DIRECT_U32 * 2: return body_direct<T, OP_DIRECT_U32, false, NR, WANT>(S, smem, v, m, code);
    case OP_DIRECT_U32 * 2 + 1: return body_direct<T, OP_DIRECT_U32, true, NR, WANT>(S, smem, v, m, code);
    case OP_DIRECT_U64 * 2: return body_direct<T, OP_DIRECT_U64, false, NR, WANT>(S, smem, v, m, code);
    case OP_DIRECT_U64 * 2 + 1: return body_direct<T, OP_DIRECT_U64, true, NR, WANT>(S, smem, v, m, code);
    case OP_HASHBITS * 2: return body_hashbits<T, NR>(S, v, m);
    case OP_HASH32 * 2:
    case OP_HASH64 * 2:
        if (HASH) return body_hash<T, NR, WANT>(S, v, m, code);
        return 0; // kernels built without the hash probe are never given such a stage
    default: return m; // OP_LOAD
    }
}

// ------------------------------------------------------------------ accumulators

// Feed a batch's values into the accumulators.  Every test on the stage's
// recipe is uniform and sits outside the row loop; a row contributes iff its
// bit is set in m.  acc32: every multiplier of the stage and every value it
// can see fits in 32 bits, so a contribution is one widening multiply-add.
template <int NR, typename V>
__device__ __forceinline__ void add_scaled(int64_t (&dst)[NR], int64_t mult, const V (&val)[NR], uint32_t m)
{
#pragma unroll
    for (int k = 0; k < NR; ++k)
        if ((m >> k) & 1u) dst[k] += mult * (int64_t)val[k];
}
template <int NR>
__device__ __forceinline__ void add_scaled32(int64_t (&dst)[NR], int32_t mult, const int32_t (&val)[NR], uint32_t m)
{
#pragma unroll
    for (int k = 0; k < NR; ++k)
        if ((m >> k) & 1u) dst[k] += (int64_t)mult * val[k]; // one widening multiply-add
}

template <bool MUL, typename T, int NR>
__device__ __forceinline__ void accumulate(const DStage &S, const T (&v)[NR], const uint64_t (&code)[NR], uint32_t m,
                                           int64_t (&key)[NR], int64_t (&X)[NR], int64_t (&Y)[NR])
{
    const uint32_t acc = S.acc;
    if (S.acc32 && sizeof(T) == 4) {
        if (acc & 0x7u) {
            int32_t r[NR];
#pragma unroll
            for (int k = 0; k < NR; ++k) r[k] = (int32_t)v[k];
            if (acc & 1u) add_scaled32<NR>(key, S.mult32[0], r, m);
            if (acc & 2u) add_scaled32<NR>(X, S.mult32[1], r, m);
            if (MUL && (acc & 4u)) add_scaled32<NR>(Y, S.mult32[2], r, m);
        }
        if (acc & 0x38u) {
            const uint32_t mask0 = (uint32_t)S.pmask0;
            const int32_t min0 = (int32_t)S.pmin0;
            int32_t p0[NR];
#pragma unroll
            for (int k = 0; k < NR; ++k) p0[k] = (int32_t)((uint32_t)code[k] & mask0) + min0;
            if (acc & 8u) add_scaled32<NR>(key, S.mult32[3], p0, m);
            if (acc & 16u) add_scaled32<NR>(X, S.mult32[4], p0, m);
            if (MUL && (acc & 32u)) add_scaled32<NR>(Y, S.mult32[5], p0, m);
        }
        if (acc & 0x1C0u) {
            const uint32_t sh = S.pbits0;
            const int32_t min1 = (int32_t)S.pmin1;
            int32_t p1[NR];
#pragma unroll
            for (int k = 0; k < NR; ++k) p1[k] = (int32_t)((uint32_t)code[k] >> sh) + min1;
            if (acc & 64u) add_scaled32<NR>(key, S.mult32[6], p1, m);
            if (acc & 128u) add_scaled32<NR>(X, S.mult32[7], p1, m);
            if (MUL && (acc & 256u)) add_scaled32<NR>(Y, S.mult32[8], p1, m);
        }
        return;
    }
    if (acc & 0x7u) {
        if (acc & 1u) add_scaled<NR>(key, S.mult[0], v, m);
        if (acc & 2u) add_scaled<NR>(X, S.mult[1], v, m);
        if (MUL && (acc & 4u)) add_scaled<NR>(Y, S.mult[2], v, m);
    }
    if (acc & 0x38u) {
        const uint64_t mask0 = S.pmask0;
        const int64_t min0 = S.pmin0;
        int64_t p0[NR];
#pragma unroll
        for (int k = 0; k < NR; ++k) p0[k] = (int64_t)(code[k] & mask0) + min0;
        if (acc & 8u) add_scaled<NR>(key, S.mult[3], p0, m);
        if (acc & 16u) add_scaled<NR>(X, S.mult[4], p0, m);
        if (MUL && (acc & 32u)) add_scaled<NR>(Y, S.mult[5], p0, m);
    }
    if (acc & 0x1C0u) {
        const uint32_t sh = S.pbits0;
        const int64_t min1 = S.pmin1;
        int64_t p1[NR];
#pragma unroll
        for (int k = 0; k < NR; ++k) p1[k] = (int64_t)(code[k] >> sh) + min1;
        if (acc & 64u) add_scaled<NR>(key, S.mult[6], p1, m);
        if (acc & 128u) add_scaled<NR>(X, S.mult[7], p1, m);
        if (MUL && (acc & 256u)) add_scaled<NR>(Y, S.mult[8], p1, m);
    }
}

__device__ __forceinline__ int64_t reduce_key(const RunParams &P, int64_t g)
{
    if (P.modulo != 0) {
        if (g >= 0 && P.modmask) g &= (int64_t)P.modmask;
        else if (P.mod32 && (uint64_t)g <= 0xFFFFFFFFull) g = (int64_t)((uint32_t)g % (uint32_t)P.modulo);
        else g = g % P.modulo;
    }
    return g;
}

// Insert-or-find in the global group table (open addressing, linear probe,
// bounded), then add.  The reserved empty marker as a key uses the side slot
// after the last regular slot.
__device__ __forceinline__ void hash_aggregate(const RunParams &P, int64_t g, int64_t val)
{
    uint64_t slot;
    if (g == kEmptyKey64) {
        slot = P.gmask + 1;
    } else {
        unsigned long long *keys = reinterpret_cast<unsigned long long *>(P.gkeys);
        slot = hash64((uint64_t)g) & P.gmask;
        bool found = false;
        for (uint64_t it = 0; it <= P.gmask; ++it) {
            unsigned long long cur = *reinterpret_cast<volatile unsigned long long *>(&keys[slot]);
            if (cur == (unsigned long long)g) {
                found = true;
                break;
            }
            if (cur == (unsigned long long)kEmptyKey64) {
                cur = atomicCAS(&keys[slot], (unsigned long long)kEmptyKey64, (unsigned long long)g);
                if (cur == (unsigned long long)kEmptyKey64 || cur == (unsigned long long)g) {
                    found = true;
                    break;
                }
            }
            slot = (slot + 1) & P.gmask;
        }
        if (!found) {
            set_status(P.status, SJQ_ERR_GROUP_OVERFLOW);
            return;
        }
    }
    atomicAdd(reinterpret_cast<unsigned long long *>(P.sums) + slot, (unsigned long long)val);
    atomicAdd(reinterpret_cast<unsigned long long *>(P.counts) + slot, 1ull);
}

// 64-bit add into shared memory as two native 32-bit atomics: the low word's
// returned old value tells this thread whether its own add carried, so every
// carry is propagated exactly once and the 64-bit total is exact.
__device__ __forceinline__ void smem_add64(unsigned long long *cell, uint64_t val)
{
    unsigned int *w = reinterpret_cast<unsigned int *>(cell);
    const unsigned int lo = (unsigned int)val;
    unsigned int hi = (unsigned int)(val >> 32);
    const unsigned int old = atomicAdd(w, lo);
    hi += (unsigned int)((old + lo) < old);
    if (hi) atomicAdd(w + 1, hi);
}

// The terminal on a batch: group keys of all rows first (their divisions overlap), then the
// aggregation; every test on the query shape is uniform and outside the row loops.
template <int AGG, bool MUL, int NR>
__device__ __forceinline__ void terminal(const RunParams &P, unsigned char *smem, const int64_t (&key)[NR],
                                         const int64_t (&X)[NR], const int64_t (&Y)[NR], uint32_t m, int64_t &lsum,
                                         int64_t &lcnt)
{
    if (!m) return;
    int64_t val[NR];
#pragma unroll
    for (int k = 0; k < NR; ++k) val[k] = MUL ? X[k] * Y[k] : X[k];
    int64_t g[NR];
    if (AGG != AGG_SCALAR || P.has_key) {
        const int64_t modulo = P.modulo;
        if (modulo == 0) {
#pragma unroll
            for (int k = 0; k < NR; ++k) g[k] = key[k];
        } else if (P.modmask) {
            const int64_t mask = (int64_t)P.modmask;
#pragma unroll
            for (int k = 0; k < NR; ++k) g[k] = key[k] >= 0 ? (key[k] & mask) : (key[k] % modulo);
        } else if (P.mod32) {
            const uint32_t d = (uint32_t)modulo;
#pragma unroll
            for (int k = 0; k < NR; ++k)
                g[k] = (uint64_t)key[k] <= 0xFFFFFFFFull ? (int64_t)((uint32_t)key[k] % d) : (key[k] % modulo);
        } else {
#pragma unroll
            for (int k = 0; k < NR; ++k) g[k] = key[k] % modulo;
        }
    }
    if (AGG == AGG_SCALAR) {
        if (P.has_key) {
#pragma unroll
            for (int k = 0; k < NR; ++k)
                if (((m >> k) & 1u) && g[k] != 0) {
                    set_status(P.status, SJQ_ERR_GROUP_RANGE);
                    m &= ~(1u << k);
                }
        }
#pragma unroll
        for (int k = 0; k < NR; ++k)
            if ((m >> k) & 1u) lsum += val[k];
        lcnt += __popc(m);
        return;
    }
    if (AGG == AGG_HASH) {
#pragma unroll
        for (int k = 0; k < NR; ++k)
            if ((m >> k) & 1u) hash_aggregate(P, g[k], val[k]);
        return;
    }
    const uint64_t ng = (uint64_t)P.num_groups;
#pragma unroll
    for (int k = 0; k < NR; ++k)
        if (((m >> k) & 1u) && (uint64_t)g[k] >= ng) {
            set_status(P.status, SJQ_ERR_GROUP_RANGE);
            m &= ~(1u << k);
        }
    const bool want_count = P.want_count != 0;
    if (AGG == AGG_SMEM) {
        unsigned long long *ss = reinterpret_cast<unsigned long long *>(smem + P.smem_groups);
#pragma unroll
        for (int k = 0; k < NR; ++k)
            if ((m >> k) & 1u) smem_add64(ss + g[k], (uint64_t)val[k]);
        if (want_count) {
#pragma unroll
            for (int k = 0; k < NR; ++k)
                if ((m >> k) & 1u) smem_add64(ss + ng + g[k], 1ull);
        }
    } else {
        unsigned long long *gs = reinterpret_cast<unsigned long long *>(P.sums);
#pragma unroll
        for (int k = 0; k < NR; ++k)
            if ((m >> k) & 1u) atomicAdd(gs + g[k], (unsigned long long)val[k]);
        if (want_count) {
            unsigned long long *gc = reinterpret_cast<unsigned long long *>(P.counts);
#pragma unroll
            for (int k = 0; k < NR; ++k)
                if ((m >> k) & 1u) atomicAdd(gc + g[k], 1ull);
        }
    }
}

// ------------------------------------------------------------------ row batches
// A batch is up to kRows rows per lane, named by 32-bit offsets from a base
// row that is uniform over the warp (so a column address costs one multiply-
// add per row).  CONTIG: the lane owns four consecutive rows (one 128-bit
// load); otherwise the rows are survivors popped from a queue (one 4- or
// 8-byte load each).

template <typename T, bool CONTIG>
__device__ __forceinline__ void load_rows(const DStage &S, int64_t base, const uint32_t (&off)[kRows], uint32_t valid,
                                          uint32_t need, T (&v)[kRows])
{
    const T *c = static_cast<const T *>(S.col) + base;
    if (CONTIG && valid == 0xFu) {
        Vec4<T>::load(c + off[0], v);
        return;
    }
#pragma unroll
    for (int k = 0; k < kRows; ++k) {
        v[k] = 0;
        if ((need >> k) & 1u) v[k] = ld_sparse(c + off[k]);
    }
}

// One pure filter stage on a batch: returns the mask of rows that pass.
template <bool HASH>
__device__ __forceinline__ uint32_t filter_rows(const RunParams &P, const DStage &S, const unsigned char *smem,
                                                int64_t base, const uint32_t (&off)[kRows], uint32_t valid)
{
    uint64_t unused[kRows];
    if (S.is64) {
        int64_t v[kRows];
        load_rows<int64_t, false>(S, base, off, valid, valid, v);
        return run_stage<int64_t, kRows, false, HASH>(P, S, smem, v, valid, unused);
    }
    int32_t v[kRows];
    load_rows<int32_t, false>(S, base, off, valid, valid, v);
    return run_stage<int32_t, kRows, false, HASH>(P, S, smem, v, valid, unused);
}

// Stages [first, nstages) with accumulators, then the terminal.  The column of
// the next stage is requested before the current stage's probe is resolved, so
// a stage costs one memory latency, not two.
template <int AGG, bool MUL, bool CONTIG, bool HASH>
__device__ __forceinline__ void final_rows(const RunParams &P, const DStage *st, unsigned char *smem, int first,
                                           int64_t base, const uint32_t (&off)[kRows], uint32_t valid, int64_t &lsum,
                                           int64_t &lcnt)
{
    uint32_t m = valid;
    int64_t key[kRows], X[kRows], Y[kRows];
#pragma unroll
    for (int k = 0; k < kRows; ++k) {
        key[k] = P.key_offset;
        X[k] = 0;
        Y[k] = 0;
    }
    int32_t vnext[kRows];
    bool have_next = false;
    for (int s = first; s < P.nstages; ++s) {
        const DStage &S = st[s];
        const uint32_t need = P.eager ? valid : m;
        if (!need) break;
        const uint32_t simple = S.simple;
        if (simple) { // a plain int32 column feeding one accumulator: no probe, no recipe to interpret
            int32_t v[kRows];
            if (have_next) {
#pragma unroll
                for (int k = 0; k < kRows; ++k) v[k] = vnext[k];
            } else {
                load_rows<int32_t, CONTIG>(S, base, off, valid, need, v);
            }
            have_next = (s + 1 < P.nstages) && !st[s + 1].is64;
            if (have_next) load_rows<int32_t, CONTIG>(st[s + 1], base, off, valid, need, vnext);
            const int32_t mult = S.mult32[simple - 1];
            if (simple == 2) add_scaled32<kRows>(X, mult, v, m);
            else if (simple == 1) add_scaled32<kRows>(key, mult, v, m);
            else if (MUL) add_scaled32<kRows>(Y, mult, v, m);
            continue;
        }
        uint64_t code[kRows];
#pragma unroll
        for (int k = 0; k < kRows; ++k) code[k] = 0;
        if (S.is64) {
            int64_t v[kRows];
            load_rows<int64_t, CONTIG>(S, base, off, valid, need, v);
            have_next = false;
            m = run_stage<int64_t, kRows, true, HASH>(P, S, smem, v, m, code);
            if (S.acc) accumulate<MUL, int64_t, kRows>(S, v, code, m, key, X, Y);
        } else {
            int32_t v[kRows];
            if (have_next) {
#pragma unroll
                for (int k = 0; k < kRows; ++k) v[k] = vnext[k];
            } else {
                load_rows<int32_t, CONTIG>(S, base, off, valid, need, v);
            }
            have_next = (s + 1 < P.nstages) && !st[s + 1].is64;
            if (have_next) load_rows<int32_t, CONTIG>(st[s + 1], base, off, valid, need, vnext);
            m = run_stage<int32_t, kRows, true, HASH>(P, S, smem, v, m, code);
            if (S.acc) accumulate<MUL, int32_t, kRows>(S, v, code, m, key, X, Y);
        }
    }
    terminal<AGG, MUL, kRows>(P, smem, key, X, Y, m, lsum, lcnt);
}

// ------------------------------------------------------------------ level 0
// One filter stage on the thread's own kSlots groups of four consecutive rows
// of a tile: the column is loaded for a group only while one of its rows is
// alive.  FULL: the whole tile lies inside the table (no bounds masks).
template <typename T, bool FULL, bool HASH>
__device__ __forceinline__ uint32_t dense_stage(const RunParams &P, const DStage &S, const unsigned char *smem,
                                                int64_t row0, int32_t slot_stride, uint32_t valid, uint32_t alive)
{
    T v[kDenseRows];
    const T *c = static_cast<const T *>(S.col) + row0;
#pragma unroll
    for (int u = 0; u < kSlots; ++u) {
#pragma unroll
        for (int r = 0; r < 4; ++r) v[4 * u + r] = 0;
        if ((alive >> (4 * u)) & 0xFu) {
            if (FULL) {
                Vec4<T>::load(c + u * slot_stride, &v[4 * u]);
            } else {
                const uint32_t nv = (valid >> (4 * u)) & 0xFu;
#pragma unroll
                for (int r = 0; r < 4; ++r)
                    if ((nv >> r) & 1u) v[4 * u + r] = __ldcs(c + u * slot_stride + r);
            }
        }
    }
    uint64_t unused[kDenseRows];
    return run_stage<T, kDenseRows, false, HASH>(P, S, smem, v, alive, unused);
}

template <bool FULL, bool HASH>
__device__ __forceinline__ uint32_t level0(const RunParams &P, const DStage *st, const unsigned char *smem,
                                           int64_t row0, int32_t slot_stride, uint32_t valid)
{
    uint32_t alive = valid;
    for (int s = 0; s < P.nd0; ++s) {
        if (!alive) break;
        const DStage &S = st[s];
        alive = S.is64 ? dense_stage<int64_t, FULL, HASH>(P, S, smem, row0, slot_stride, valid, alive)
                       : dense_stage<int32_t, FULL, HASH>(P, S, smem, row0, slot_stride, valid, alive);
    }
    return alive;
}

// ------------------------------------------------------------------ per-warp queues
// Queue l of a warp (a ring of 32-bit row offsets in shared memory) holds the
// rows that passed stages 0 .. nd0+l-1.  The level fed by queue l runs filter
// stage nd0+l and pushes to queue l+1, or, for the last queue, runs the
// remaining stages and the terminal.  Heads and counts live in registers and are
// selected without indexing so that they never spill to local memory.
struct QueueState {
    uint32_t h0, h1, h2, c0, c1, c2;
    __device__ __forceinline__ uint32_t head(int l) const { return l == 0 ? h0 : (l == 1 ? h1 : h2); }
    __device__ __forceinline__ uint32_t count(int l) const { return l == 0 ? c0 : (l == 1 ? c1 : c2); }
    __device__ __forceinline__ void set_head(int l, uint32_t v)
    {
        h0 = l == 0 ? v : h0;
        h1 = l == 1 ? v : h1;
        h2 = l == 2 ? v : h2;
    }
    __device__ __forceinline__ void set_count(int l, uint32_t v)
    {
        c0 = l == 0 ? v : c0;
        c1 = l == 1 ? v : c1;
        c2 = l == 2 ? v : c2;
    }
};

__device__ __forceinline__ uint32_t queue_cap(int l) { return l == 0 ? (uint32_t)kQueue0Cap : (uint32_t)kQueueCap; }
__device__ __forceinline__ uint32_t queue_base(int l)
{
    return l == 0 ? 0u : (uint32_t)(kQueue0Cap + (l - 1) * kQueueCap);
}

template <int AGG, bool MUL, bool HASH>
__global__ void __launch_bounds__(SJQ_LB_THREADS, SJQ_LB_BLOCKS) fused_kernel(const __grid_constant__ RunParams P)
{
    extern __shared__ __align__(16) unsigned char smem[];
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int warp = tid >> 5;

    // Stage descriptors and small direct tables -> shared memory (once per block).
    DStage *st = reinterpret_cast<DStage *>(smem + P.smem_stages);
    {
        const uint32_t words = (uint32_t)(P.nstages * sizeof(DStage) / 8);
        const uint64_t *src = reinterpret_cast<const uint64_t *>(&P.st[0]);
        uint64_t *dst = reinterpret_cast<uint64_t *>(st);
        for (uint32_t i = tid; i < words; i += blockDim.x) dst[i] = src[i];
    }
    for (int s = 0; s < P.nstages; ++s) {
        const DStage &S = P.st[s];
        if (S.in_smem) {
            const uint4 *src = static_cast<const uint4 *>(S.tab);
            uint4 *dst = reinterpret_cast<uint4 *>(smem + S.smem_off);
            for (uint32_t i = tid; i < S.tab_bytes / 16; i += blockDim.x) dst[i] = __ldg(src + i);
        }
    }
    if (AGG == AGG_SMEM) {
        unsigned long long *ss = reinterpret_cast<unsigned long long *>(smem + P.smem_groups);
        const int64_t cells = P.num_groups * (P.want_count ? 2 : 1);
        for (int64_t i = tid; i < cells; i += blockDim.x) ss[i] = 0ull;
    }
    __syncthreads();

    int64_t lsum = 0, lcnt = 0;

    if (P.nq == 0) {
        // No queue: every stage runs on the thread's own four consecutive rows.
        const int64_t tile_rows = (int64_t)blockDim.x * kRows;
        const int64_t ntiles = (P.n + tile_rows - 1) / tile_rows;
        uint32_t off[kRows];
#pragma unroll
        for (int k = 0; k < kRows; ++k) off[k] = (uint32_t)(4 * tid + k);
        for (int64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
            const int64_t base = tile * tile_rows;
            const int64_t rem = P.n - base - 4 * (int64_t)tid;
            const uint32_t valid = rem >= 4 ? 0xFu : (rem > 0 ? ((1u << (int)rem) - 1u) : 0u);
            final_rows<AGG, MUL, true, HASH>(P, st, smem, 0, base, off, valid, lsum, lcnt);
        }
    } else {
        const int nq = P.nq;
        uint32_t *const qmem = reinterpret_cast<uint32_t *>(smem + P.smem_queue) +
                               warp * (kQueue0Cap + (nq - 1) * kQueueCap);
        QueueState Q{0, 0, 0, 0, 0, 0};
        const bool wide = P.n > 0xFFFFFFFFll; // offsets are tile-relative and the queues are flushed per tile
        const int32_t slot_stride = (int32_t)blockDim.x * 4;
        const int32_t tile_rows = slot_stride * kSlots;
        const uint32_t ntiles = (uint32_t)((P.n + tile_rows - 1) / tile_rows); // host checks n / tile_rows < 2^31
        int64_t qbase = 0;
        uint32_t tile = blockIdx.x;
        bool flushing = false;

        // One loop, one call site per piece of work: pick the deepest queue holding a full
        // batch (so that a push never meets a full queue); else filter the next tile and push
        // its survivors; at the end drain what is left.
        for (;;) {
            int l = (nq >= 3 && Q.c2 >= (uint32_t)kBatch) ? 2
                    : (nq >= 2 && Q.c1 >= (uint32_t)kBatch) ? 1
                    : (Q.c0 >= (uint32_t)kBatch)            ? 0
                                                            : -1;
            uint32_t nb = kBatch;
            if (l < 0) {
                if (flushing) {
                    l = Q.c0 ? 0 : (Q.c1 ? 1 : (Q.c2 ? 2 : -1));
                    if (l < 0) {
                        flushing = false;
                        if (tile >= ntiles) break;
                        continue;
                    }
                    nb = Q.count(l) < (uint32_t)kBatch ? Q.count(l) : (uint32_t)kBatch;
                } else if (tile < ntiles) {
                    // level 0: the first stage on the thread's own rows of the next tile
                    const int64_t tile_base = (int64_t)tile * tile_rows;
                    const int64_t row0 = tile_base + 4 * tid;
                    if (wide) qbase = tile_base;
#if !defined(SJQ_NO_PREFETCH)
                    {   // ask L2 for the first column of the tile this block filters next
                        const int64_t nrow = row0 + (int64_t)gridDim.x * tile_rows * SJQ_PREFETCH_DIST;
                        if (nrow + tile_rows <= P.n) {
                            const DStage &S0 = st[0];
                            const char *pc = static_cast<const char *>(S0.col) + nrow * (S0.is64 ? 8 : 4);
#pragma unroll
                            for (int k = 0; k < kSlots; ++k)
                                asm volatile("prefetch.global.L2 [%0];" ::"l"(pc + (int64_t)k * slot_stride * (S0.is64 ? 8 : 4)));
                        }
                    }
#endif
                    uint32_t alive;
                    if (tile_base + tile_rows <= P.n) {
                        alive = level0<true, HASH>(P, st, smem, row0, slot_stride, kDenseRows >= 32 ? 0xFFFFFFFFu : ((1u << kDenseRows) - 1u));
                    } else {
                        uint32_t valid = 0;
#pragma unroll
                        for (int k = 0; k < kSlots; ++k) {
                            const int64_t rem = P.n - (row0 + k * slot_stride);
                            const uint32_t nv = rem >= 4 ? 0xFu : (rem > 0 ? ((1u << (int)rem) - 1u) : 0u);
                            valid |= nv << (4 * k);
                        }
                        alive = level0<false, HASH>(P, st, smem, row0, slot_stride, valid);
                    }
#if defined(SJQ_EXP_NO_QUEUE)
                    lcnt += __popc(alive);
                    tile += gridDim.x;
                    continue;
#endif
                    if (!__any_sync(0xffffffffu, alive != 0)) { // a very selective first stage: nothing to push
                        tile += gridDim.x;
                        if (wide) flushing = true;
                        continue;
                    }
                    // compact the warp's survivors into queue 0
                    const uint32_t mine = (uint32_t)__popc(alive);
                    uint32_t incl = mine;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
                        if (lane >= o) incl += t;
                    }
                    const uint32_t tot = __shfl_sync(0xffffffffu, incl, 31);
                    if (tot) {
                        uint32_t pos = Q.h0 + Q.c0 + incl - mine;
                        const uint32_t off0 = (uint32_t)(row0 - qbase);
#pragma unroll
                        for (int k = 0; k < kDenseRows; ++k) {
                            if ((alive >> k) & 1u) {
                                qmem[pos & (kQueue0Cap - 1)] = off0 + (uint32_t)((k >> 2) * slot_stride + (k & 3));
                                ++pos;
                            }
                        }
                        Q.c0 += tot;
                        __syncwarp();
                    }
                    tile += gridDim.x;
                    if (wide) flushing = true;
                    continue;
                } else {
                    if ((Q.c0 | Q.c1 | Q.c2) == 0) break;
                    flushing = true;
                    continue;
                }
            }

            // Run one batch of nb rows at the level fed by queue l.
            uint32_t off[kRows];
            uint32_t valid = 0;
            {
                const uint32_t *q = qmem + queue_base(l);
                const uint32_t h = Q.head(l), cap = queue_cap(l);
#pragma unroll
                for (int k = 0; k < kRows; ++k) {
                    const uint32_t e = (uint32_t)(k * 32 + lane);
                    off[k] = 0;
                    if (e < nb) {
                        off[k] = q[(h + e) & (cap - 1)];
                        valid |= 1u << k;
                    }
                }
                __syncwarp();
                Q.set_head(l, (h + nb) & (cap - 1));
                Q.set_count(l, Q.count(l) - nb);
            }
            if (l + 1 == nq) {
                final_rows<AGG, MUL, false, HASH>(P, st, smem, P.nd0 + l, qbase, off, valid, lsum, lcnt);
            } else {
                const uint32_t m = filter_rows<HASH>(P, st[P.nd0 + l], smem, qbase, off, valid);
                const uint32_t mine = (uint32_t)__popc(m);
                uint32_t incl = mine;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
                    if (lane >= o) incl += t;
                }
                const uint32_t tot = __shfl_sync(0xffffffffu, incl, 31);
                if (tot) {
                    uint32_t *q = qmem + queue_base(l + 1);
                    uint32_t pos = Q.head(l + 1) + Q.count(l + 1) + incl - mine;
#pragma unroll
                    for (int k = 0; k < kRows; ++k) {
                        if ((m >> k) & 1u) {
                            q[pos & (kQueueCap - 1)] = off[k];
                            ++pos;
                        }
                    }
                    Q.set_count(l + 1, Q.count(l + 1) + tot);
                    __syncwarp();
                }
            }
        }
    }

    if (AGG == AGG_SCALAR) {
        // block reduce, then one global atomic per block
        for (int o = 16; o > 0; o >>= 1) {
            lsum += __shfl_xor_sync(0xffffffffu, lsum, o);
            lcnt += __shfl_xor_sync(0xffffffffu, lcnt, o);
        }
        __shared__ int64_t part[64];
        if (lane == 0) {
            part[warp] = lsum;
            part[32 + warp] = lcnt;
        }
        __syncthreads();
        if (warp == 0) {
            const int nw = (blockDim.x + 31) >> 5;
            lsum = lane < nw ? part[lane] : 0;
            lcnt = lane < nw ? part[32 + lane] : 0;
            for (int o = 16; o > 0; o >>= 1) {
                lsum += __shfl_xor_sync(0xffffffffu, lsum, o);
                lcnt += __shfl_xor_sync(0xffffffffu, lcnt, o);
            }
            if (lane == 0 && lcnt != 0) {
                atomicAdd(reinterpret_cast<unsigned long long *>(P.sums), (unsigned long long)lsum);
                if (P.counts) atomicAdd(reinterpret_cast<unsigned long long *>(P.counts), (unsigned long long)lcnt);
            }
        }
    } else if (AGG == AGG_SMEM) {
        // one global atomic per touched group per block
        __syncthreads();
        const unsigned long long *ss = reinterpret_cast<const unsigned long long *>(smem + P.smem_groups);
        for (int64_t g = tid; g < P.num_groups; g += blockDim.x) {
            const unsigned long long s = ss[g];
            const unsigned long long c = P.want_count ? ss[P.num_groups + g] : 0ull;
            if (s != 0ull) atomicAdd(reinterpret_cast<unsigned long long *>(P.sums) + g, s);
            if (c != 0ull) atomicAdd(reinterpret_cast<unsigned long long *>(P.counts) + g, c);
        }
    }
}

struct ClearParams {
    int64_t *sums;
    int64_t *counts;
    int64_t cells; // entries of sums / counts to zero
    int64_t *gkeys;
    int64_t gslots; // entries of gkeys to set to the empty marker
    int64_t *n_groups;
    int32_t *status;
};

__global__ void __launch_bounds__(256) clear_kernel(const ClearParams C)
{
    const int64_t stride = (int64_t)blockDim.x * gridDim.x;
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (int64_t i = t; i < C.cells; i += stride) {
        C.sums[i] = 0;
        if (C.counts) C.counts[i] = 0;
    }
    for (int64_t i = t; i < C.gslots; i += stride) C.gkeys[i] = kEmptyKey64;
    if (t == 0) {
        if (C.status) *C.status = 0;
        if (C.n_groups) *C.n_groups = 0;
    }
}

struct CompactParams {
    const int64_t *gkeys, *gsums, *gcounts;
    int64_t gslots; // regular slots; the side slot follows
    int64_t *keys, *sums, *counts;
    int64_t capacity;
    int64_t *n_groups;
    int32_t *status;
};

// Group table -> list of (key, sum, count).
__global__ void __launch_bounds__(256) compact_kernel(const CompactParams C)
{
    const int64_t stride = (int64_t)blockDim.x * gridDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i <= C.gslots; i += stride) {
        const bool side = i == C.gslots;
        const int64_t k = side ? kEmptyKey64 : C.gkeys[i];
        const bool used = side ? (C.gcounts[i] != 0) : (k != kEmptyKey64);
        if (!used) continue;
        const int64_t pos = (int64_t)atomicAdd(reinterpret_cast<unsigned long long *>(C.n_groups), 1ull);
        if (pos < C.capacity) {
            C.keys[pos] = k;
            C.sums[pos] = C.gsums[i];
            C.counts[pos] = C.gcounts[i];
        } else {
            set_status(C.status, SJQ_ERR_GROUP_OVERFLOW);
        }
    }
}

typedef void (*fused_fn)(const RunParams);

fused_fn pick_kernel(int agg, bool mul, bool hash)
{
    switch (agg * 4 + (mul ? 2 : 0) + (hash ? 1 : 0)) {
    case 0: return fused_kernel<AGG_SCALAR, false, false>;
    case 1: return fused_kernel<AGG_SCALAR, false, true>;
    case 2: return fused_kernel<AGG_SCALAR, true, false>;
    case 3: return fused_kernel<AGG_SCALAR, true, true>;
    case 4: return fused_kernel<AGG_SMEM, false, false>;
    case 5: return fused_kernel<AGG_SMEM, false, true>;
    case 6: return fused_kernel<AGG_SMEM, true, false>;
    case 7: return fused_kernel<AGG_SMEM, true, true>;
    case 8: return fused_kernel<AGG_GLOBAL, false, false>;
    case 9: return fused_kernel<AGG_GLOBAL, false, true>;
    case 10: return fused_kernel<AGG_GLOBAL, true, false>;
    case 11: return fused_kernel<AGG_GLOBAL, true, true>;
    case 12: return fused_kernel<AGG_HASH, false, false>;
    case 13: return fused_kernel<AGG_HASH, false, true>;
    case 14: return fused_kernel<AGG_HASH, true, false>;
    default: return fused_kernel<AGG_HASH, true, true>;
    }
}

} // namespace

// ---- launch helpers used by the planner (sjq_run.cu) ----------------------

sjq_status fused_occupancy(int agg, bool mul, bool hash, int block, size_t smem, int *ctas_per_sm)
{
    fused_fn fn = pick_kernel(agg, mul, hash);
    if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess ||
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(ctas_per_sm, fn, block, smem) != cudaSuccess) {
        (void)cudaGetLastError();
        return SJQ_ERR_CUDA;
    }
    return SJQ_OK;
}

sjq_status fused_launch(int agg, bool mul, bool hash, int grid, int block, size_t smem, const RunParams &P,
                        cudaStream_t stream)
{
    fused_fn fn = pick_kernel(agg, mul, hash);
    fn<<<grid, block, smem, stream>>>(P);
    if (cudaGetLastError() != cudaSuccess) return SJQ_ERR_CUDA;
    return SJQ_OK;
}

sjq_status clear_launch(int64_t *sums, int64_t *counts, int64_t cells, int64_t *gkeys, int64_t gslots,
                        int64_t *n_groups, int32_t *status, int sm_count, cudaStream_t stream)
{
    ClearParams C{sums, counts, cells, gkeys, gslots, n_groups, status};
    int64_t work = cells > gslots ? cells : gslots;
    int64_t blocks = (work + 255) / 256;
    if (blocks > (int64_t)sm_count * 8) blocks = (int64_t)sm_count * 8;
    if (blocks < 1) blocks = 1;
    clear_kernel<<<(int)blocks, 256, 0, stream>>>(C);
    return cudaGetLastError() == cudaSuccess ? SJQ_OK : SJQ_ERR_CUDA;
}

sjq_status compact_launch(const int64_t *gkeys, const int64_t *gsums, const int64_t *gcounts, int64_t gslots,
                          int64_t *keys, int64_t *sums, int64_t *counts, int64_t capacity, int64_t *n_groups,
                          int32_t *status, int sm_count, cudaStream_t stream)
{
    CompactParams C{gkeys, gsums, gcounts, gslots, keys, sums, counts, capacity, n_groups, status};
    int64_t blocks = (gslots + 256) / 256;
    if (blocks > (int64_t)sm_count * 8) blocks = (int64_t)sm_count * 8;
    compact_kernel<<<(int)blocks, 256, 0, stream>>>(C);
    return cudaGetLastError() == cudaSuccess ? SJQ_OK : SJQ_ERR_CUDA;
}

} // namespace sjq
