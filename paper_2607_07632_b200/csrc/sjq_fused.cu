// The fused probe kernel: one pass over the fact table.
//
// Execution model (Section 3.2 of the paper, "grid-stride persistent
// threads"): a machine-sized grid; each thread owns four consecutive rows of a
// tile and strides over tiles, so one 128-bit load brings the four values of a
// column; later columns are loaded only while at least one of the thread's
// rows is still alive (lazy loading, Section 3.2 "Latency-hidden join"), a
// probe is a range-checked single load from a direct-mapped table or a bounded
// linear probe of an open-addressing table (Section 3.3), and the terminal is
// a register accumulator, a shared-memory privatised group table or global
// atomics (Section 3.3 "Shared-memory privatized group-by").
#include "sjq_run.cuh"

namespace sjq {

namespace {

__device__ __forceinline__ int4 ld_stream16(const void *p)
{
    return __ldcs(static_cast<const int4 *>(p));
}
__device__ __forceinline__ longlong2 ld_stream16ll(const void *p)
{
    return __ldcs(static_cast<const longlong2 *>(p));
}

// Probe of one table with key v.  Returns hit; on a hit `code` holds the
// packed payload code.  SMEM: the direct table was staged into shared memory.
template <typename T>
__device__ __forceinline__ bool probe(const DStage &S, const unsigned char *smem, T v, uint64_t &code)
{
    if (S.tkind <= SJQ_TABLE_DIRECT_U64) {
        const uint64_t idx = (uint64_t)(int64_t)v - (uint64_t)S.kmin;
        if (idx >= S.span) return false; // outside the key range: a miss, never an access
        if (S.in_smem) {
            const unsigned char *t = smem + S.smem_off;
            switch (S.tkind) {
            case SJQ_TABLE_DIRECT_BITMAP:
                return (reinterpret_cast<const uint32_t *>(t)[idx >> 5] >> (idx & 31)) & 1u;
            case SJQ_TABLE_DIRECT_U8: code = t[idx]; return code != 0xFFu;
            case SJQ_TABLE_DIRECT_U16: code = reinterpret_cast<const uint16_t *>(t)[idx]; return code != 0xFFFFu;
            case SJQ_TABLE_DIRECT_U32: code = reinterpret_cast<const uint32_t *>(t)[idx]; return code != 0xFFFFFFFFu;
            default: code = reinterpret_cast<const uint64_t *>(t)[idx]; return code != ~0ULL;
            }
        }
        switch (S.tkind) {
        case SJQ_TABLE_DIRECT_BITMAP:
            return (__ldg(static_cast<const uint32_t *>(S.tab) + (idx >> 5)) >> (idx & 31)) & 1u;
        case SJQ_TABLE_DIRECT_U8: code = __ldg(static_cast<const uint8_t *>(S.tab) + idx); return code != 0xFFu;
        case SJQ_TABLE_DIRECT_U16: code = __ldg(static_cast<const uint16_t *>(S.tab) + idx); return code != 0xFFFFu;
        case SJQ_TABLE_DIRECT_U32:
            code = __ldg(static_cast<const uint32_t *>(S.tab) + idx);
            return code != 0xFFFFFFFFu;
        default: code = __ldg(static_cast<const uint64_t *>(S.tab) + idx); return code != ~0ULL;
        }
    }
    if (S.tkind == SJQ_TABLE_HASH_I64) {
        const int64_t k = (int64_t)v;
        if (k == kEmptyKey64) return false;
        const int64_t *keys = static_cast<const int64_t *>(S.tab);
        uint64_t slot = hash64((uint64_t)k) & S.hmask;
        for (uint64_t it = 0; it <= S.hmask; ++it) {
            const int64_t cur = __ldg(keys + slot);
            if (cur == k) {
                if (S.codes)
                    code = (S.code_bits == 64) ? __ldg(static_cast<const uint64_t *>(S.codes) + slot)
                                         : (uint64_t)__ldg(static_cast<const uint32_t *>(S.codes) + slot);
                return true;
            }
            if (cur == kEmptyKey64) return false;
            slot = (slot + 1) & S.hmask;
        }
        return false;
    }
    { // HASH_I32
        const int32_t k = (int32_t)v;
        if ((int64_t)v != (int64_t)k || k == kEmptyKey32) return false;
        const int32_t *keys = static_cast<const int32_t *>(S.tab);
        uint64_t slot = hash64((uint64_t)(int64_t)k) & S.hmask;
        for (uint64_t it = 0; it <= S.hmask; ++it) {
            const int32_t cur = __ldg(keys + slot);
            if (cur == k) {
                if (S.codes)
                    code = (S.code_bits == 64) ? __ldg(static_cast<const uint64_t *>(S.codes) + slot)
                                         : (uint64_t)__ldg(static_cast<const uint32_t *>(S.codes) + slot);
                return true;
            }
            if (cur == kEmptyKey32) return false;
            slot = (slot + 1) & S.hmask;
        }
        return false;
    }
}

// One stage applied to one row: filter, then feed the accumulators.
template <typename T, bool MUL>
__device__ __forceinline__ bool apply(const DStage &S, const unsigned char *smem, T v, int64_t &key, int64_t &X,
                                      int64_t &Y)
{
    uint64_t code = 0;
    bool pass = true;
    if (S.kind == ST_PRED) pass = pred_eval<T>(S.pred, v);
    else if (S.kind == ST_PROBE) pass = probe<T>(S, smem, v, code);
    if (pass && S.acc) {
        const uint32_t acc = S.acc;
        if (acc & 0x7u) {
            const int64_t raw = (int64_t)v;
            if (acc & 1u) key += S.mult[0] * raw;
            if (acc & 2u) X += S.mult[1] * raw;
            if (MUL && (acc & 4u)) Y += S.mult[2] * raw;
        }
        if (acc & 0x38u) {
            const int64_t p0 = (int64_t)(code & S.pmask0) + S.pmin0;
            if (acc & 8u) key += S.mult[3] * p0;
            if (acc & 16u) X += S.mult[4] * p0;
            if (MUL && (acc & 32u)) Y += S.mult[5] * p0;
        }
        if (acc & 0x1C0u) {
            const int64_t p1 = (int64_t)(code >> S.pbits0) + S.pmin1;
            if (acc & 64u) key += S.mult[6] * p1;
            if (acc & 128u) X += S.mult[7] * p1;
            if (MUL && (acc & 256u)) Y += S.mult[8] * p1;
        }
    }
    return pass;
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

template <int AGG, bool MUL>
__device__ __forceinline__ void terminal(const RunParams &P, unsigned char *smem, int64_t key, int64_t X, int64_t Y,
                                         int64_t &lsum, int64_t &lcnt)
{
    const int64_t val = MUL ? X * Y : X;
    if (AGG == AGG_SCALAR) {
        if (P.has_key) {
            const int64_t g = reduce_key(P, key);
            if (g != 0) {
                set_status(P.status, SJQ_ERR_GROUP_RANGE);
                return;
            }
        }
        lsum += val;
        lcnt += 1;
        return;
    }
    const int64_t g = reduce_key(P, key);
    if (AGG == AGG_HASH) {
        hash_aggregate(P, g, val);
        return;
    }
    if ((uint64_t)g >= (uint64_t)P.num_groups) {
        set_status(P.status, SJQ_ERR_GROUP_RANGE);
        return;
    }
    if (AGG == AGG_SMEM) {
        unsigned long long *ss = reinterpret_cast<unsigned long long *>(smem + P.smem_groups);
        atomicAdd(ss + g, (unsigned long long)val);
        if (P.want_count) atomicAdd(ss + P.num_groups + g, 1ull);
    } else {
        atomicAdd(reinterpret_cast<unsigned long long *>(P.sums) + g, (unsigned long long)val);
        if (P.want_count) atomicAdd(reinterpret_cast<unsigned long long *>(P.counts) + g, 1ull);
    }
}

template <int AGG, bool MUL>
__global__ void __launch_bounds__(1024) fused_kernel(const __grid_constant__ RunParams P)
{
    extern __shared__ __align__(16) unsigned char smem[];
    const int tid = threadIdx.x;

    // Stage small direct tables into shared memory (one copy per CTA).
    for (int s = 0; s < P.nstages; ++s) {
        const DStage &S = P.st[s];
        if (S.kind == ST_PROBE && S.in_smem) {
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
    const int64_t tile_rows = (int64_t)blockDim.x * 4;
    const int64_t ntiles = (P.n + tile_rows - 1) / tile_rows;
    for (int64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
        const int64_t row0 = tile * tile_rows + 4 * (int64_t)tid;
        const int64_t rem = P.n - row0;
        const uint32_t valid = rem >= 4 ? 0xFu : (rem > 0 ? ((1u << (int)rem) - 1u) : 0u);
        uint32_t alive = valid;
        int64_t key[4], X[4], Y[4];
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            key[r] = P.key_offset;
            X[r] = 0;
            Y[r] = 0;
        }
        for (int s = 0; s < P.nstages; ++s) {
            const DStage &S = P.st[s];
            const uint32_t need = P.eager ? valid : alive;
            if (!need) continue;
            if (S.is64) {
                int64_t v[4] = {0, 0, 0, 0};
                const int64_t *c = static_cast<const int64_t *>(S.col) + row0;
                if (valid == 0xFu) {
                    const longlong2 a = ld_stream16ll(c), b = ld_stream16ll(c + 2);
                    v[0] = a.x, v[1] = a.y, v[2] = b.x, v[3] = b.y;
                } else {
#pragma unroll
                    for (int r = 0; r < 4; ++r)
                        if ((valid >> r) & 1u) v[r] = __ldcs(c + r);
                }
#pragma unroll
                for (int r = 0; r < 4; ++r)
                    if ((alive >> r) & 1u)
                        if (!apply<int64_t, MUL>(S, smem, v[r], key[r], X[r], Y[r])) alive &= ~(1u << r);
            } else {
                int32_t v[4] = {0, 0, 0, 0};
                const int32_t *c = static_cast<const int32_t *>(S.col) + row0;
                if (valid == 0xFu) {
                    const int4 a = ld_stream16(c);
                    v[0] = a.x, v[1] = a.y, v[2] = a.z, v[3] = a.w;
                } else {
#pragma unroll
                    for (int r = 0; r < 4; ++r)
                        if ((valid >> r) & 1u) v[r] = __ldcs(c + r);
                }
#pragma unroll
                for (int r = 0; r < 4; ++r)
                    if ((alive >> r) & 1u)
                        if (!apply<int32_t, MUL>(S, smem, v[r], key[r], X[r], Y[r])) alive &= ~(1u << r);
            }
        }
#pragma unroll
        for (int r = 0; r < 4; ++r)
            if ((alive >> r) & 1u) terminal<AGG, MUL>(P, smem, key[r], X[r], Y[r], lsum, lcnt);
    }

    if (AGG == AGG_SCALAR) {
        // block reduce, then one global atomic per block
        for (int o = 16; o > 0; o >>= 1) {
            lsum += __shfl_xor_sync(0xffffffffu, lsum, o);
            lcnt += __shfl_xor_sync(0xffffffffu, lcnt, o);
        }
        __shared__ int64_t part[64];
        const int warp = tid >> 5, lane = tid & 31;
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

fused_fn pick_kernel(int agg, bool mul)
{
    switch (agg * 2 + (mul ? 1 : 0)) {
    case 0: return fused_kernel<AGG_SCALAR, false>;
    case 1: return fused_kernel<AGG_SCALAR, true>;
    case 2: return fused_kernel<AGG_SMEM, false>;
    case 3: return fused_kernel<AGG_SMEM, true>;
    case 4: return fused_kernel<AGG_GLOBAL, false>;
    case 5: return fused_kernel<AGG_GLOBAL, true>;
    case 6: return fused_kernel<AGG_HASH, false>;
    default: return fused_kernel<AGG_HASH, true>;
    }
}

} // namespace

// ---- launch helpers used by the planner (sjq_run.cu) ----------------------

sjq_status fused_occupancy(int agg, bool mul, int block, size_t smem, int *ctas_per_sm)
{
    fused_fn fn = pick_kernel(agg, mul);
    if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess ||
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(ctas_per_sm, fn, block, smem) != cudaSuccess) {
        (void)cudaGetLastError();
        return SJQ_ERR_CUDA;
    }
    return SJQ_OK;
}

sjq_status fused_launch(int agg, bool mul, int grid, int block, size_t smem, const RunParams &P, cudaStream_t stream)
{
    fused_fn fn = pick_kernel(agg, mul);
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
