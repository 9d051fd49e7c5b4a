// Dimension-table planning and build kernels.
//
// Section 3.3 of the paper: dense primary keys allow a directly indexed map
// whose build is a race-free direct store and whose probe is one load; the
// filter and the gathered attribute are fused into one narrow code per key
// with a reserved all-ones sentinel for "filtered out".  Sparse keys fall back
// to an open-addressing table populated with atomicCAS.  Section 4.3.1: the
// key range is verified at run time and the packed or unpacked form chosen.
#include <algorithm>
#include <new>

#include "sjq_internal.h"

namespace sjq {

namespace {

constexpr int kMaxDimCols = 32;

struct DimParams {
    const void *col[kMaxDimCols];
    uint8_t is64[kMaxDimCols];
    DPred preds[SJQ_MAX_PREDS];
    int32_t npreds;
    int32_t key_col;
    int32_t pay_col[SJQ_MAX_PAYLOADS];
    int32_t npayload;
    int64_t n;
};

__device__ inline bool dim_row_passes(const DimParams &P, int64_t r)
{
    bool ok = true;
    for (int k = 0; k < P.npreds && ok; ++k) {
        const DPred &d = P.preds[k];
        if (d.is64) ok = pred_eval<int64_t>(d, static_cast<const int64_t *>(P.col[d.col])[r]);
        else ok = pred_eval<int32_t>(d, static_cast<const int32_t *>(P.col[d.col])[r]);
    }
    return ok;
}

__device__ inline int64_t warp_min(int64_t v)
{
    for (int o = 16; o > 0; o >>= 1) {
        int64_t t = __shfl_xor_sync(0xffffffffu, v, o);
        v = t < v ? t : v;
    }
    return v;
}
__device__ inline int64_t warp_max(int64_t v)
{
    for (int o = 16; o > 0; o >>= 1) {
        int64_t t = __shfl_xor_sync(0xffffffffu, v, o);
        v = t > v ? t : v;
    }
    return v;
}
__device__ inline int64_t warp_sum(int64_t v)
{
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Sum over a block of at most 256 threads; the total is valid in thread 0.
__device__ inline unsigned long long block_sum(unsigned long long v)
{
    __shared__ unsigned long long part[8];
    v = (unsigned long long)warp_sum((int64_t)v);
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = v;
    __syncthreads();
    unsigned long long t = 0;
    if (threadIdx.x == 0)
        for (int w = 0; w < (int)((blockDim.x + 31) >> 5); ++w) t += part[w];
    return t;
}

// scratch: [0] kmin [1] kmax [2] count [3] p0min [4] p0max [5] p1min [6] p1max
__global__ void plan_init_kernel(int64_t *s)
{
    if (threadIdx.x < 8) {
        int64_t v = 0;
        if (threadIdx.x == 0 || threadIdx.x == 3 || threadIdx.x == 5) v = INT64_MAX;
        if (threadIdx.x == 1 || threadIdx.x == 4 || threadIdx.x == 6) v = INT64_MIN;
        s[threadIdx.x] = v;
    }
}

__global__ void __launch_bounds__(256) plan_scan_kernel(const __grid_constant__ DimParams P, int64_t *scratch)
{
    int64_t kmin = INT64_MAX, kmax = INT64_MIN, cnt = 0;
    int64_t pmin[SJQ_MAX_PAYLOADS] = {INT64_MAX, INT64_MAX}, pmax[SJQ_MAX_PAYLOADS] = {INT64_MIN, INT64_MIN};
    const int64_t stride = (int64_t)blockDim.x * gridDim.x;
    for (int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; r < P.n; r += stride) {
        if (!dim_row_passes(P, r)) continue;
        int64_t k = load_cell(P.col[P.key_col], P.is64[P.key_col], r);
        kmin = k < kmin ? k : kmin;
        kmax = k > kmax ? k : kmax;
        ++cnt;
        for (int i = 0; i < P.npayload; ++i) {
            int64_t v = load_cell(P.col[P.pay_col[i]], P.is64[P.pay_col[i]], r);
            pmin[i] = v < pmin[i] ? v : pmin[i];
            pmax[i] = v > pmax[i] ? v : pmax[i];
        }
    }
    kmin = warp_min(kmin);
    kmax = warp_max(kmax);
    cnt = warp_sum(cnt);
    for (int i = 0; i < SJQ_MAX_PAYLOADS; ++i) {
        pmin[i] = warp_min(pmin[i]);
        pmax[i] = warp_max(pmax[i]);
    }
    // one set of atomics per block, not per warp: they all land on the same seven words
    __shared__ int64_t part[8][3 + 2 * SJQ_MAX_PAYLOADS];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) {
        part[warp][0] = kmin;
        part[warp][1] = kmax;
        part[warp][2] = cnt;
        for (int i = 0; i < SJQ_MAX_PAYLOADS; ++i) {
            part[warp][3 + 2 * i] = pmin[i];
            part[warp][4 + 2 * i] = pmax[i];
        }
    }
    __syncthreads();
    if (threadIdx.x < 3 + 2 * SJQ_MAX_PAYLOADS) {
        const int f = threadIdx.x; // 0 kmin, 1 kmax, 2 count, then (min, max) per payload
        const bool is_min = f == 0 || (f >= 3 && ((f - 3) & 1) == 0), is_sum = f == 2;
        int64_t v = part[0][f];
        for (int w = 1; w < (int)(blockDim.x >> 5); ++w) {
            const int64_t t = part[w][f];
            v = is_sum ? v + t : is_min ? (t < v ? t : v) : (t > v ? t : v);
        }
        int64_t block_cnt = 0;
        for (int w = 0; w < (int)(blockDim.x >> 5); ++w) block_cnt += part[w][2];
        if (block_cnt > 0 && f < 3 + 2 * P.npayload) {
            if (is_sum) atomicAdd((unsigned long long *)&scratch[f], (unsigned long long)v);
            else if (is_min) atomicMin((long long *)&scratch[f], (long long)v);
            else atomicMax((long long *)&scratch[f], (long long)v);
        }
    }
}

struct BuildParams {
    DimParams dim;
    int32_t kind;
    int32_t code_bits;
    int64_t kmin;
    uint64_t span;  // direct
    uint32_t buckets; // hash: number of buckets
    int32_t bucket_k; // hash: keys per bucket
    int32_t code_off; // hash: byte offset of the codes inside a bucket
    int64_t pay_min[SJQ_MAX_PAYLOADS], pay_max[SJQ_MAX_PAYLOADS];
    int32_t pay_bits[SJQ_MAX_PAYLOADS];
    void *slots;
    unsigned int *filter; // presence bitmap words (hash: indexed by a hash of the key; direct with payloads: by slot)
    uint32_t fmask;       // hash: filter bits - 1
    unsigned long long *header; // [0] rows inserted, [1] slots occupied
    int32_t *status;
};

// One launch prepares a table's memory: the header counters and the presence bitmap to zero, the slot array to
// its empty pattern (bitmap: zeros; packed codes: all ones; open addressing: the empty key in every word).
// All three regions start on 16-byte boundaries and are padded to a multiple of 16 bytes by the layout.
struct InitParams {
    uint4 *header, *slots, *filter;
    size_t header16, slots16, filter16; // sizes in 16-byte units
    uint4 pattern;
};

__global__ void __launch_bounds__(256) table_init_kernel(const __grid_constant__ InitParams I)
{
    const size_t stride = (size_t)blockDim.x * gridDim.x;
    const size_t total = I.header16 + I.slots16 + I.filter16;
    const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
        if (i < I.header16) I.header[i] = zero;
        else if (i < I.header16 + I.slots16) I.slots[i - I.header16] = I.pattern;
        else I.filter[i - I.header16 - I.slots16] = zero;
    }
}

__device__ inline bool pack_code(const BuildParams &B, int64_t r, uint64_t *code)
{
    uint64_t c = 0;
    int shift = 0;
    for (int i = 0; i < B.dim.npayload; ++i) {
        int64_t v = load_cell(B.dim.col[B.dim.pay_col[i]], B.dim.is64[B.dim.pay_col[i]], r);
        if (v < B.pay_min[i] || v > B.pay_max[i]) return false;
        c |= ((uint64_t)v - (uint64_t)B.pay_min[i]) << shift;
        shift += B.pay_bits[i];
    }
    *code = c;
    return true;
}

__device__ inline void store_code(void *codes, int bits, uint64_t idx, uint64_t c)
{
    if (bits < 8) {
        // several codes share a word that starts as all ones: clear this code's zero bits (the keys are
        // unique, so no two rows touch the same bits)
        const int per = 32 / bits;
        const unsigned int sh = (unsigned int)(idx % (uint64_t)per) * (unsigned int)bits;
        const unsigned int mask = ((1u << bits) - 1u) << sh;
        atomicAnd(static_cast<unsigned int *>(codes) + idx / (uint64_t)per, ~mask | ((unsigned int)c << sh));
        return;
    }
    switch (bits) {
    case 8: static_cast<uint8_t *>(codes)[idx] = (uint8_t)c; break;
    case 16: static_cast<uint16_t *>(codes)[idx] = (uint16_t)c; break;
    case 32: static_cast<uint32_t *>(codes)[idx] = (uint32_t)c; break;
    case 64: static_cast<uint64_t *>(codes)[idx] = c; break;
    default: break;
    }
}

// Claim the first free slot on the key's probe path (bucket after bucket from its home bucket, the slots of
// a bucket in order) with atomicCAS on the key word, then store the code beside it.  Bounded by the number
// of buckets; a key met on the way is a duplicate.
template <typename W>
__device__ inline void hash_insert(const BuildParams &B, W key, W empty, uint64_t hashed, uint64_t code)
{
    char *base = static_cast<char *>(B.slots);
    uint32_t b = home_bucket(hashed, B.buckets);
    for (uint32_t it = 0; it < B.buckets; ++it) {
        char *bucket = base + (size_t)b * kBucketBytes;
        W *keys = reinterpret_cast<W *>(bucket);
        for (int j = 0; j < B.bucket_k; ++j) {
            W old = *reinterpret_cast<volatile W *>(&keys[j]);
            if (old == empty) old = atomicCAS(&keys[j], empty, key);
            if (old == empty) {
                if (B.code_bits == 32) reinterpret_cast<uint32_t *>(bucket + B.code_off)[j] = (uint32_t)code;
                else if (B.code_bits == 64) reinterpret_cast<uint64_t *>(bucket + B.code_off)[j] = code;
                return;
            }
            if (old == key) {
                set_status(B.status, SJQ_ERR_DUP_KEY);
                return;
            }
        }
        b = b + 1 == B.buckets ? 0 : b + 1;
    }
    set_status(B.status, SJQ_ERR_TABLE_FULL);
}

__global__ void __launch_bounds__(256) build_kernel(const __grid_constant__ BuildParams B)
{
    const DimParams &P = B.dim;
    const int64_t stride = (int64_t)blockDim.x * gridDim.x;
    unsigned long long inserted = 0;
    for (int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; r < P.n; r += stride) {
        if (!dim_row_passes(P, r)) continue;
        const int64_t k = load_cell(P.col[P.key_col], P.is64[P.key_col], r);
        uint64_t code = 0;
        if (!pack_code(B, r, &code)) {
            set_status(B.status, SJQ_ERR_LAYOUT_MISMATCH);
            continue;
        }
        ++inserted;
        if (B.kind != SJQ_TABLE_HASH_I32 && B.kind != SJQ_TABLE_HASH_I64) {
            const uint64_t idx = (uint64_t)k - (uint64_t)B.kmin;
            if (idx >= B.span) {
                set_status(B.status, SJQ_ERR_LAYOUT_MISMATCH);
                continue;
            }
            if (B.kind == SJQ_TABLE_DIRECT_BITMAP)
                atomicOr(static_cast<unsigned int *>(B.slots) + (idx >> 5), 1u << (idx & 31));
            else {
                store_code(B.slots, B.code_bits, idx, code); // race-free: keys are unique
                if (B.filter) atomicOr(B.filter + (idx >> 5), 1u << (idx & 31));
            }
        } else if (B.kind == SJQ_TABLE_HASH_I64) {
            if (k == kEmptyKey64) {
                set_status(B.status, SJQ_ERR_RESERVED_KEY);
                continue;
            }
            if (B.filter) {
                const uint32_t fb = filter_hash((uint64_t)k) & B.fmask;
                atomicOr(B.filter + (fb >> 5), 1u << (fb & 31));
            }
            hash_insert<unsigned long long>(B, (unsigned long long)k, (unsigned long long)kEmptyKey64, (uint64_t)k, code);
        } else { // HASH_I32
            const int32_t k32 = (int32_t)k;
            if (k32 == kEmptyKey32) {
                set_status(B.status, SJQ_ERR_RESERVED_KEY);
                continue;
            }
            if (B.filter) {
                const uint32_t fb = filter_hash((uint64_t)(int64_t)k32) & B.fmask;
                atomicOr(B.filter + (fb >> 5), 1u << (fb & 31));
            }
            hash_insert<unsigned int>(B, (unsigned int)k32, (unsigned int)kEmptyKey32, (uint64_t)(int64_t)k32, code);
        }
    }
    inserted = block_sum(inserted);
    if (threadIdx.x == 0 && inserted) atomicAdd(&B.header[0], inserted);
}

// Count occupied slots of a direct table; a repeated key leaves fewer occupied slots than inserted rows.  The
// block that finishes last (a ticket in header[2]) compares the two counters.  `expect_full` >= 0: the layout
// promises that every key of the range is present (a probe then trusts the range test alone), so exactly that
// many rows must have been stored.
__global__ void __launch_bounds__(256) direct_count_kernel(const __grid_constant__ BuildParams B, long long expect_full)
{
    const uint64_t stride = (uint64_t)blockDim.x * gridDim.x;
    unsigned long long occ = 0;
    if (B.kind == SJQ_TABLE_DIRECT_BITMAP || B.filter) {
        // one bit per occupied slot: the table itself, or the presence bitmap beside the codes
        const uint64_t words = (B.span + 31) >> 5;
        const unsigned int *w = B.kind == SJQ_TABLE_DIRECT_BITMAP ? static_cast<const unsigned int *>(B.slots) : B.filter;
        for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < words; i += stride) occ += __popc(w[i]);
    } else {
        for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < B.span; i += stride) {
            bool set;
            switch (B.code_bits) {
            case 8: set = static_cast<const uint8_t *>(B.slots)[i] != 0xFFu; break;
            case 16: set = static_cast<const uint16_t *>(B.slots)[i] != 0xFFFFu; break;
            case 32: set = static_cast<const uint32_t *>(B.slots)[i] != 0xFFFFFFFFu; break;
            default: set = static_cast<const uint64_t *>(B.slots)[i] != ~0ULL; break;
            }
            occ += set;
        }
    }
    occ = block_sum(occ);
    if (threadIdx.x == 0) {
        if (occ) atomicAdd(&B.header[1], occ);
        __threadfence();
        if (atomicAdd(&B.header[2], 1ULL) == (unsigned long long)gridDim.x - 1) {
            __threadfence();
            const unsigned long long inserted = atomicAdd(&B.header[0], 0ULL), occupied = atomicAdd(&B.header[1], 0ULL);
            if (inserted != occupied) set_status(B.status, SJQ_ERR_DUP_KEY);
            else if (expect_full >= 0 && occupied != (unsigned long long)expect_full)
                set_status(B.status, SJQ_ERR_LAYOUT_MISMATCH);
        }
    }
}

int bits_for(uint64_t range)
{
    int b = 0;
    while (b < 64 && (range >> b) != 0) ++b;
    return b;
}

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Bytes of a direct table's slot array (bitmap words or packed codes), spare entry included.
size_t direct_array_bytes(const sjq_dim_layout &L)
{
    const uint64_t span = (uint64_t)L.slots;
    const uint64_t bits = L.kind == SJQ_TABLE_DIRECT_BITMAP ? 1 : (uint64_t)L.code_bits;
    return align_up((size_t)(((span + 1) * bits + 31) / 32 * 4), 16); // whole 32-bit words
}

// Device bytes a table of this shape occupies, recomputed from kind, slots, code_bits and filter_bits (never
// taken from the struct); false when the fields contradict one another.  sjq_dim_plan_end sizes tables with
// it and sjq_build_dim checks a caller-supplied layout against it, so that a stale or hand-edited layout is
// rejected on the host instead of making the fills and the build kernel write past table_mem.
bool layout_table_bytes(const sjq_dim_layout &L, size_t *bytes)
{
    if (L.slots <= 0 || L.npayload < 0 || L.npayload > SJQ_MAX_PAYLOADS || L.filter_bits < 0) return false;
    if (is_direct_kind(L.kind)) {
        if ((uint64_t)L.slots > ((uint64_t)1 << 40)) return false;
        if (L.code_bits != direct_kind_bits(L.kind) || (L.kind == SJQ_TABLE_DIRECT_BITMAP) != (L.npayload == 0))
            return false;
        // a sub-byte table without its presence bitmap could not tell a repeated key from a missing one
        if (L.code_bits > 0 && L.code_bits < 8 && L.filter_bits == 0) return false;
        if (L.filter_bits != 0 &&
            (L.kind == SJQ_TABLE_DIRECT_BITMAP || L.filter_bits <= L.slots || L.filter_bits % 128 != 0))
            return false;
        *bytes = kTableHeaderBytes + align_up(direct_array_bytes(L), 256) + align_up((size_t)(L.filter_bits / 8), 256);
        return true;
    }
    if (L.kind == SJQ_TABLE_HASH_I32 || L.kind == SJQ_TABLE_HASH_I64) {
        if ((L.kind == SJQ_TABLE_HASH_I64) != (L.key_dtype == SJQ_I64)) return false;
        if (L.npayload == 0 ? L.code_bits != 0 : (L.code_bits != 32 && L.code_bits != 64)) return false;
        const int k = bucket_keys(L.key_dtype == SJQ_I64 ? 8 : 4, L.code_bits / 8);
        if (L.slots % k != 0 || L.slots > ((int64_t)1 << 31)) return false; // whole buckets
        if ((L.filter_bits & (L.filter_bits - 1)) || L.filter_bits > ((int64_t)1 << 32)) return false;
        *bytes = kTableHeaderBytes + align_up((size_t)(L.slots / k) * kBucketBytes, 256) +
                 align_up((size_t)(L.filter_bits / 8), 256);
        return true;
    }
    return false;
}

sjq_status fill_dim_params(const sjq_col *cols, int ncols, const sjq_pred *preds, int npreds, int key_col,
                           const int *payload_cols, int npayload, DimParams *P)
{
    if (!cols || ncols <= 0 || ncols > kMaxDimCols || npreds < 0 || npreds > SJQ_MAX_PREDS || (npreds && !preds) ||
        key_col < 0 || key_col >= ncols || npayload < 0 || npayload > SJQ_MAX_PAYLOADS || (npayload && !payload_cols))
        return SJQ_ERR_INVALID_ARG;
    const int64_t n = cols[key_col].n;
    if (n < 0) return SJQ_ERR_INVALID_ARG;
    for (int c = 0; c < ncols; ++c) {
        if (cols[c].n != n || (cols[c].dtype != SJQ_I32 && cols[c].dtype != SJQ_I64)) return SJQ_ERR_INVALID_ARG;
        if (n > 0 && !cols[c].data) return SJQ_ERR_INVALID_ARG;
        if (!aligned16(cols[c].data)) return SJQ_ERR_ALIGN;
        P->col[c] = cols[c].data;
        P->is64[c] = (uint8_t)cols[c].dtype;
    }
    for (int k = 0; k < npreds; ++k) {
        if (preds[k].col < 0 || preds[k].col >= ncols) return SJQ_ERR_INVALID_ARG;
        if (!canon_pred(preds[k], cols[preds[k].col].dtype, &P->preds[k])) return SJQ_ERR_INVALID_ARG;
    }
    for (int i = 0; i < npayload; ++i) {
        if (payload_cols[i] < 0 || payload_cols[i] >= ncols) return SJQ_ERR_INVALID_ARG;
        P->pay_col[i] = payload_cols[i];
    }
    P->npreds = npreds;
    P->key_col = key_col;
    P->npayload = npayload;
    P->n = n;
    return SJQ_OK;
}

int grid_for(int64_t n, int sm_count)
{
    int64_t blocks = (n + 255) / 256;
    int64_t cap = (int64_t)sm_count * 8;
    if (blocks > cap) blocks = cap;
    return blocks < 1 ? 1 : (int)blocks;
}

} // namespace

bool canon_pred(const sjq_pred &p, int dtype, DPred *d)
{
    *d = DPred{};
    d->col = p.col;
    d->is64 = (uint8_t)(dtype == SJQ_I64);
    bool empty = false;
    switch (p.op) {
    case SJQ_EQ: d->lo = d->hi = p.lo; break;
    case SJQ_NE: d->lo = d->hi = p.lo; d->neg = 1; break;
    case SJQ_LT:
        if (p.lo == INT64_MIN) empty = true;
        else { d->lo = INT64_MIN; d->hi = p.lo - 1; }
        break;
    case SJQ_LE: d->lo = INT64_MIN; d->hi = p.lo; break;
    case SJQ_GT:
        if (p.lo == INT64_MAX) empty = true;
        else { d->lo = p.lo + 1; d->hi = INT64_MAX; }
        break;
    case SJQ_GE: d->lo = p.lo; d->hi = INT64_MAX; break;
    case SJQ_BETWEEN: d->lo = p.lo; d->hi = p.hi; break;
    case SJQ_IN:
        if (p.nset < 0 || p.nset > SJQ_MAX_IN_SET || (p.nset && !p.set)) return false;
        if (p.nset == 0) empty = true;
        for (int k = 0; k < p.nset; ++k) d->set[k] = p.set[k];
        d->nset = (uint8_t)p.nset;
        break;
    default: return false;
    }
    if (empty || d->lo > d->hi) {
        d->lo = 1;
        d->hi = 0;
    }
    // int32 view of the range
    if (d->lo > d->hi || d->lo > INT32_MAX || d->hi < INT32_MIN) {
        d->never = 1;
        d->lo32 = 1;
        d->hi32 = 0;
    } else {
        d->lo32 = d->lo < INT32_MIN ? INT32_MIN : (int32_t)d->lo;
        d->hi32 = d->hi > INT32_MAX ? INT32_MAX : (int32_t)d->hi;
    }
    return true;
}

sjq_status device_info(DeviceInfo *out)
{
    static thread_local DeviceInfo cache[64];
    static thread_local bool have[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        (void)cudaGetLastError();
        return SJQ_ERR_CUDA;
    }
    if (dev >= 0 && dev < 64 && have[dev]) {
        *out = cache[dev];
        return SJQ_OK;
    }
    DeviceInfo d{};
    d.device = dev;
    if (cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&d.max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&d.l2_bytes, cudaDevAttrL2CacheSize, dev) != cudaSuccess) {
        (void)cudaGetLastError();
        return SJQ_ERR_CUDA;
    }
    if (dev >= 0 && dev < 64) {
        cache[dev] = d;
        have[dev] = true;
    }
    *out = d;
    return SJQ_OK;
}

} // namespace sjq

using namespace sjq;

extern "C" sjq_status sjq_dim_plan_begin(const sjq_col *cols, int ncols, const sjq_pred *preds, int npreds,
                                         int key_col, const int *payload_cols, int npayload, void *scratch_dev,
                                         int64_t *host_stats, void *stream_)
{
    if (!scratch_dev || !host_stats) return SJQ_ERR_INVALID_ARG;
    if (!aligned16(scratch_dev)) return SJQ_ERR_ALIGN;
    DimParams P{};
    sjq_status st = fill_dim_params(cols, ncols, preds, npreds, key_col, payload_cols, npayload, &P);
    if (st != SJQ_OK) return st;
    DeviceInfo dev;
    if ((st = device_info(&dev)) != SJQ_OK) return st;
    cudaStream_t stream = (cudaStream_t)stream_;
    int64_t *scratch = static_cast<int64_t *>(scratch_dev);
    plan_init_kernel<<<1, 32, 0, stream>>>(scratch);
    if (P.n > 0) plan_scan_kernel<<<grid_for(P.n, dev.sm_count), 256, 0, stream>>>(P, scratch);
    if (cudaGetLastError() != cudaSuccess ||
        cudaMemcpyAsync(host_stats, scratch, 8 * sizeof(int64_t), cudaMemcpyDeviceToHost, stream) != cudaSuccess) {
        (void)cudaGetLastError();
        return SJQ_ERR_CUDA;
    }
    return SJQ_OK;
}

extern "C" sjq_status sjq_dim_plan(const sjq_col *cols, int ncols, const sjq_pred *preds, int npreds, int key_col,
                                   const int *payload_cols, int npayload, const sjq_build_opts *opts,
                                   void *scratch_dev, void *stream_, sjq_dim_layout *layout)
{
    int64_t h[8];
    sjq_status st = sjq_dim_plan_begin(cols, ncols, preds, npreds, key_col, payload_cols, npayload, scratch_dev, h,
                                       stream_);
    if (st != SJQ_OK) return st;
    if (cudaStreamSynchronize((cudaStream_t)stream_) != cudaSuccess) {
        (void)cudaGetLastError();
        return SJQ_ERR_CUDA;
    }
    return sjq_dim_plan_end(cols, ncols, key_col, npayload, opts, h, layout);
}

extern "C" sjq_status sjq_dim_plan_end(const sjq_col *cols, int ncols, int key_col, int npayload,
                                       const sjq_build_opts *opts, const int64_t *h, sjq_dim_layout *layout)
{
    if (!layout || !h || !cols || ncols <= 0 || key_col < 0 || key_col >= ncols || npayload < 0 ||
        npayload > SJQ_MAX_PAYLOADS)
        return SJQ_ERR_INVALID_ARG;
    struct { int64_t n; } P{cols[key_col].n};

    sjq_dim_layout L{};
    L.key_dtype = cols[key_col].dtype;
    L.npayload = npayload;
    L.dim_rows = P.n;
    L.entries = h[2];
    if (L.entries > 0) {
        L.kmin = h[0];
        L.kmax = h[1];
    }
    uint64_t maxcode = 0;
    int total_bits = 0;
    for (int i = 0; i < npayload; ++i) {
        L.pay_min[i] = L.entries > 0 ? h[3 + 2 * i] : 0;
        L.pay_max[i] = L.entries > 0 ? h[4 + 2 * i] : 0;
        const uint64_t range = (uint64_t)L.pay_max[i] - (uint64_t)L.pay_min[i];
        L.pay_bits[i] = bits_for(range);
        if (total_bits + L.pay_bits[i] > 63) return SJQ_ERR_UNSUPPORTED;
        maxcode |= range << total_bits;
        total_bits += L.pay_bits[i];
    }
    // Narrowest code that leaves all-ones free as the miss marker; a table that holds every key of its range
    // (entries == slots) needs no marker below one byte, because there the range test alone decides a hit.
    const uint64_t span_if_any = (uint64_t)L.kmax - (uint64_t)L.kmin; // span - 1
    const bool every_key = L.entries > 0 && span_if_any + 1 == (uint64_t)L.entries;
    const int min_bits = (opts && opts->min_code_bits > 0) ? opts->min_code_bits : 2;
    if (min_bits != 2 && min_bits != 4 && min_bits != 8) return SJQ_ERR_INVALID_ARG;
    int code_bits = 0;
    if (npayload > 0) {
        if (min_bits <= 2 && (every_key ? maxcode <= 0x3u : maxcode < 0x3u)) code_bits = 2;
        else if (min_bits <= 4 && (every_key ? maxcode <= 0xFu : maxcode < 0xFu)) code_bits = 4;
        else if (maxcode < 0xFFu) code_bits = 8;
        else if (maxcode < 0xFFFFu) code_bits = 16;
        else if (maxcode < 0xFFFFFFFFu) code_bits = 32;
        else code_bits = 64;
    }
    const int force = opts ? opts->force_kind : SJQ_TABLE_AUTO;
    if (force != SJQ_TABLE_AUTO && force != SJQ_TABLE_FORCE_DIRECT && force != SJQ_TABLE_FORCE_HASH)
        return SJQ_ERR_INVALID_ARG;
    const int64_t max_direct = (opts && opts->max_direct_bytes > 0) ? opts->max_direct_bytes : (int64_t)64 << 20;
    // (the skewed 64-bit-key workload: 1.61 / 1.65 / 1.71 / 1.91 ms at load 33 / 40 / 50 / 60 %)
    const int load_pct = (opts && opts->hash_load_pct > 0) ? opts->hash_load_pct : 40;
    if (load_pct > 90) return SJQ_ERR_INVALID_ARG;

    const uint64_t span_m1 = (uint64_t)L.kmax - (uint64_t)L.kmin; // span - 1, no overflow
    bool direct_ok = span_m1 < ((uint64_t)1 << 40);
    size_t direct_bytes = 0;
    if (direct_ok) {
        const uint64_t span = span_m1 + 1;
        // one spare entry after the last slot, never set: a probe clamps its index there instead of testing the range
        direct_bytes = align_up((size_t)(((span + 1) * (uint64_t)(npayload == 0 ? 1 : code_bits) + 31) / 32 * 4), 16);
    }
    bool use_direct;
    if (force == SJQ_TABLE_FORCE_DIRECT) {
        if (!direct_ok || direct_bytes > ((size_t)1 << 36)) return SJQ_ERR_UNSUPPORTED;
        use_direct = true;
    } else if (force == SJQ_TABLE_FORCE_HASH) {
        use_direct = false;
    } else {
        use_direct = direct_ok && (int64_t)direct_bytes <= max_direct;
    }
    if (use_direct) {
        L.slots = (int64_t)(span_m1 + 1);
        L.code_bits = code_bits;
        L.kind = npayload == 0 ? SJQ_TABLE_DIRECT_BITMAP
                 : code_bits == 2 ? SJQ_TABLE_DIRECT_U2
                 : code_bits == 4 ? SJQ_TABLE_DIRECT_U4
                 : code_bits == 8 ? SJQ_TABLE_DIRECT_U8
                 : code_bits == 16 ? SJQ_TABLE_DIRECT_U16
                 : code_bits == 32 ? SJQ_TABLE_DIRECT_U32
                                   : SJQ_TABLE_DIRECT_U64;
        // a code array is 8 to 64 times the size of a bitmap over the same slots: keep both, so that a
        // filter stage probes the bitmap and only the survivors gather their payload from the codes
        if (npayload > 0) L.filter_bits = (int64_t)((span_m1 + 129) / 128 * 128); // at least one spare bit after the last slot
    } else {
        L.kind = L.key_dtype == SJQ_I64 ? SJQ_TABLE_HASH_I64 : SJQ_TABLE_HASH_I32;
        L.code_bits = npayload == 0 ? 0 : (code_bits <= 32 ? 32 : 64);
        const uint64_t k = (uint64_t)bucket_keys(L.key_dtype == SJQ_I64 ? 8 : 4, L.code_bits / 8);
        const uint64_t want = ((uint64_t)L.entries * 100u + (uint64_t)load_pct - 1) / (uint64_t)load_pct;
        const uint64_t buckets = std::max<uint64_t>((want + k - 1) / k, 2);
        L.slots = (int64_t)(buckets * k);
        // presence bitmap: 16 bits per entry (about 6 % false positives), at least 1024 bits, at most 2^32
        uint64_t fbits = 1024;
        while (fbits < (uint64_t)L.entries * 16 && fbits < ((uint64_t)1 << 32)) fbits <<= 1;
        L.filter_bits = (int64_t)fbits;
    }
    if (!layout_table_bytes(L, &L.table_bytes)) return SJQ_ERR_UNSUPPORTED;
    *layout = L;
    return SJQ_OK;
}

extern "C" sjq_status sjq_build_dim(const sjq_col *cols, int ncols, const sjq_pred *preds, int npreds, int key_col,
                                    const int *payload_cols, int npayload, const sjq_dim_layout *layout,
                                    void *table_mem, size_t table_bytes, int32_t *status_dev, void *stream_,
                                    sjq_table **table)
{
    if (!layout || !table_mem || !status_dev || !table) return SJQ_ERR_INVALID_ARG;
    if (!aligned16(table_mem)) return SJQ_ERR_ALIGN;
    BuildParams B{};
    sjq_status st = fill_dim_params(cols, ncols, preds, npreds, key_col, payload_cols, npayload, &B.dim);
    if (st != SJQ_OK) return st;
    const sjq_dim_layout &L = *layout;
    // The layout is the caller's: every size used below is recomputed from its shape fields, never taken
    // from its table_bytes, and a layout whose fields contradict one another is rejected here.
    size_t need_bytes = 0;
    if (L.npayload != npayload || L.key_dtype != cols[key_col].dtype || L.dim_rows != B.dim.n ||
        !layout_table_bytes(L, &need_bytes) || need_bytes != L.table_bytes)
        return SJQ_ERR_INVALID_ARG;
    for (int i = 0; i < npayload; ++i)
        if (L.pay_bits[i] < 0 || L.pay_bits[i] > 63) return SJQ_ERR_INVALID_ARG;
    if (table_bytes < need_bytes) return SJQ_ERR_BUFFER_SMALL;
    DeviceInfo dev;
    if ((st = device_info(&dev)) != SJQ_OK) return st;
    cudaStream_t stream = (cudaStream_t)stream_;

    sjq_table *T = new (std::nothrow) sjq_table();
    if (!T) return SJQ_ERR_INVALID_ARG;
    T->layout = L;
    T->base = static_cast<char *>(table_mem);
    T->slots = T->base + kTableHeaderBytes;
    T->filter = nullptr;
    T->magic = kTableMagic;

    B.kind = L.kind;
    B.code_bits = L.code_bits;
    B.kmin = L.kmin;
    B.span = (uint64_t)L.slots;
    for (int i = 0; i < SJQ_MAX_PAYLOADS; ++i) {
        B.pay_min[i] = L.pay_min[i];
        B.pay_max[i] = L.pay_max[i];
        B.pay_bits[i] = L.pay_bits[i];
    }
    B.header = reinterpret_cast<unsigned long long *>(T->base);
    B.status = status_dev;
    B.slots = T->slots;

    InitParams I{};
    I.header = reinterpret_cast<uint4 *>(T->base);
    I.header16 = kTableHeaderBytes / 16;
    I.slots = reinterpret_cast<uint4 *>(T->slots);
    const bool direct = is_direct_kind(L.kind);
    size_t filter_bytes = 0;
    if (direct) {
        const size_t bytes = direct_array_bytes(L);
        T->slots_bytes = bytes;
        const unsigned int fill = L.kind == SJQ_TABLE_DIRECT_BITMAP ? 0u : 0xFFFFFFFFu;
        I.pattern = make_uint4(fill, fill, fill, fill);
        if (L.filter_bits) {
            T->filter = T->slots + align_up(bytes, 256);
            B.filter = reinterpret_cast<unsigned int *>(T->filter);
            filter_bytes = (size_t)(L.filter_bits / 8);
        }
    } else {
        const int kb = L.key_dtype == SJQ_I64 ? 8 : 4, cb = L.code_bits / 8;
        B.bucket_k = bucket_keys(kb, cb);
        B.code_off = bucket_code_offset(kb, cb, B.bucket_k);
        B.buckets = (uint32_t)(L.slots / B.bucket_k);
        const size_t bytes = (size_t)B.buckets * kBucketBytes;
        T->slots_bytes = bytes;
        if (L.filter_bits) {
            T->filter = T->slots + align_up(bytes, 256);
            B.filter = reinterpret_cast<unsigned int *>(T->filter);
            B.fmask = (uint32_t)(L.filter_bits - 1);
            filter_bytes = (size_t)(L.filter_bits / 8);
        }
        // Every word of a bucket starts as the empty marker's pattern: both markers (the minimum of the key
        // type) are a repeated 0x80 00 .. 00 word, so the codes start as that pattern too and are overwritten
        // when their slot is claimed.
        I.pattern = L.key_dtype == SJQ_I64 ? make_uint4(0u, 0x80000000u, 0u, 0x80000000u)
                                           : make_uint4(0x80000000u, 0x80000000u, 0x80000000u, 0x80000000u);
    }
    I.slots16 = (T->slots_bytes + 15) / 16;
    I.filter = reinterpret_cast<uint4 *>(T->filter);
    I.filter16 = (filter_bytes + 15) / 16; // the layout pads the bitmap's region to 256 bytes
    table_init_kernel<<<grid_for((int64_t)(I.header16 + I.slots16 + I.filter16), dev.sm_count), 256, 0, stream>>>(I);
    ++T->launches;
    if (B.dim.n > 0) {
        build_kernel<<<grid_for(B.dim.n, dev.sm_count), 256, 0, stream>>>(B);
        ++T->launches;
    }
    if (direct) {
        const bool promises_every_key = L.code_bits > 0 && L.code_bits < 8 && L.entries == L.slots;
        direct_count_kernel<<<grid_for(L.slots, dev.sm_count), 256, 0, stream>>>(
            B, promises_every_key ? (long long)L.entries : -1);
        ++T->launches;
    }
    if (cudaGetLastError() != cudaSuccess) {
        (void)cudaGetLastError();
        delete T;
        return SJQ_ERR_CUDA;
    }
    *table = T;
    return SJQ_OK;
}

extern "C" sjq_status sjq_dim_layout_bytes(const sjq_dim_layout *layout, size_t *bytes)
{
    if (!layout || !bytes) return SJQ_ERR_INVALID_ARG;
    return layout_table_bytes(*layout, bytes) ? SJQ_OK : SJQ_ERR_INVALID_ARG;
}

extern "C" sjq_status sjq_table_info(const sjq_table *table, sjq_dim_layout *layout)
{
    if (!table || table->magic != kTableMagic || !layout) return SJQ_ERR_INVALID_ARG;
    *layout = table->layout;
    return SJQ_OK;
}

extern "C" int32_t sjq_table_kernel_launches(const sjq_table *table)
{
    return (table && table->magic == kTableMagic) ? table->launches : 0;
}

extern "C" void sjq_table_destroy(sjq_table *table)
{
    if (table && table->magic == kTableMagic) {
        table->magic = 0;
        delete table;
    }
}

extern "C" const char *sjq_strerror(sjq_status s)
{
    switch (s) {
    case SJQ_OK: return "ok";
    case SJQ_ERR_INVALID_ARG: return "invalid argument";
    case SJQ_ERR_UNSUPPORTED: return "unsupported query or table shape";
    case SJQ_ERR_ALIGN: return "device pointer not 16-byte aligned";
    case SJQ_ERR_CUDA: return "CUDA runtime error (no device or launch failure)";
    case SJQ_ERR_BUFFER_SMALL: return "caller-provided buffer too small";
    case SJQ_ERR_STATIC_LIMIT: return "request exceeds the built-in scratch of the no-allocation entry point";
    case SJQ_ERR_JIT: return "run-time specialisation unavailable (compiler, device sources or module load)";
    case SJQ_ERR_DUP_KEY: return "duplicate dimension key among rows passing the filter";
    case SJQ_ERR_TABLE_FULL: return "hash table full";
    case SJQ_ERR_GROUP_RANGE: return "group key outside [0, num_groups)";
    case SJQ_ERR_GROUP_OVERFLOW: return "more distinct groups than the hashed capacity";
    case SJQ_ERR_RESERVED_KEY: return "dimension key equals the reserved empty marker";
    case SJQ_ERR_LAYOUT_MISMATCH: return "dimension data does not match the planned layout";
    case SJQ_ERR_ASYNC_WAIT: return "a bounded wait for a bulk-asynchronous copy ran out (result still exact)";
    default: return "unknown status";
    }
}

extern "C" const char *sjq_version(void) { return "sjq 0.1 (sm_100a)"; }
