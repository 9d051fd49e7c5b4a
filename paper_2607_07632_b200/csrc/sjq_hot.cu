// Hot-key table of an open-addressing join.
//
// Section 3.3 of the paper sizes the probed structure so that it stays in cache; an open-addressing table over
// millions of 64-bit keys cannot, and every probe of it (and of the presence bitmap in front of it) is a random
// global load.  When the foreign keys are skewed, a few keys carry a large share of the fact rows: the answers
// for those keys (present with this payload code / absent) fit in shared memory, where a warp's 32 look-ups
// cost a few cycles instead of one L1 tag cycle each.  Three small kernels, enqueued before the fused pass and
// never waited for on the host, find the heavy keys from an evenly spaced sample of the foreign-key column and
// resolve each of them against the dimension table once.  The fused kernel copies the resulting table into
// shared memory and consults it before the bitmap and before the exact probe; a key it does not hold takes the
// usual path, so the table changes the run time, never the result.
#include <algorithm>

#include "sjq_run.cuh"

namespace sjq {

namespace {

static_assert((size_t)kHotCountSlots * 12 + (size_t)kHotSlots * 4 + (size_t)(kHotSlots + 1) * 16 <= SJQ_HOT_SCRATCH_BYTES,
              "hot scratch");
static_assert(kHotCountSlots == (1 << 18) && kHotSlots % 1024 == 0, "claims pack a count-table slot into 18 bits");
constexpr unsigned long long kUnused = ~0ULL; // count-table key word of a free slot (set by a 0xFF memset)

struct HotParams {
    const void *col; // foreign-key column
    int64_t n;
    int32_t is64;
    int64_t stride;   // sample row i * stride
    int32_t nsamples;
    const char *buckets; // the dimension's open-addressing table
    uint32_t nb;
    int32_t bucket_k, code_off, code_bytes;
    unsigned long long *ckeys; // count table: keys and counts (count word starts at 0xFFFFFFFF = zero occurrences)
    unsigned int *ccounts;
    unsigned int *claims;      // per hot slot: the heaviest claim so far
    uint4 *hot;                // kHotSlots entries, then one header entry whose first word is the number of keys held
};

__device__ __forceinline__ int64_t sample_key(const HotParams &H, int64_t row)
{
    return H.is64 ? static_cast<const int64_t *>(H.col)[row] : (int64_t) static_cast<const int32_t *>(H.col)[row];
}

// Add `occ` occurrences of `key` to the global count table (bounded linear probe; a sample that finds no slot
// is dropped: the counts only rank candidates).
__device__ __forceinline__ void count_global(const HotParams &H, unsigned long long key, unsigned int occ)
{
    uint32_t h = (uint32_t)hash64(key) & (kHotCountSlots - 1);
    for (int it = 0; it < 16; ++it) {
        unsigned long long old = H.ckeys[h];
        if (old == kUnused) old = atomicCAS(&H.ckeys[h], kUnused, key);
        if (old == kUnused || old == key) {
            atomicAdd(&H.ccounts[h], occ);
            return;
        }
        h = (h + 1) & (kHotCountSlots - 1);
    }
}

// One sample per thread, counted in a shared-memory table of the block first so that a key holding several per
// cent of the rows costs one global atomic per block instead of one per occurrence.
__global__ void __launch_bounds__(1024) hot_sample_kernel(const __grid_constant__ HotParams H)
{
    constexpr int kLocal = 2048;
    __shared__ unsigned long long lkeys[kLocal];
    __shared__ unsigned int lcounts[kLocal];
    for (int i = threadIdx.x; i < kLocal; i += blockDim.x) {
        lkeys[i] = kUnused;
        lcounts[i] = 0;
    }
    __syncthreads();
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < H.nsamples) {
        const int64_t row = i * H.stride;
        if (row < H.n) {
            const int64_t v = sample_key(H, row);
            const unsigned long long key = (unsigned long long)v;
            // the free-slot pattern and the tables' empty markers are never cached
            if (key != kUnused && v != (H.is64 ? kEmptyKey64 : (int64_t)kEmptyKey32)) {
                uint32_t h = (uint32_t)(hash64(key) >> 7) & (kLocal - 1);
                bool placed = false;
                for (int it = 0; it < 8 && !placed; ++it) {
                    unsigned long long old = lkeys[h];
                    if (old == kUnused) old = atomicCAS(&lkeys[h], kUnused, key);
                    if (old == kUnused || old == key) {
                        atomicAdd(&lcounts[h], 1u);
                        placed = true;
                    }
                    h = (h + 1) & (kLocal - 1);
                }
                if (!placed) count_global(H, key, 1u);
            }
        }
    }
    __syncthreads();
    for (int s = threadIdx.x; s < kLocal; s += blockDim.x)
        if (lkeys[s] != kUnused) count_global(H, lkeys[s], lcounts[s]);
}

// Exact look-up of one key in the dimension's open-addressing table (the fused kernel's probe, one row at a time).
__device__ bool dim_lookup(const HotParams &H, int64_t v, uint32_t *code)
{
    uint32_t b = home_bucket((uint64_t)v, H.nb);
    for (uint32_t it = 0; it < H.nb; ++it) {
        const char *bucket = H.buckets + (size_t)b * kBucketBytes;
        bool has_free = false;
        for (int j = 0; j < H.bucket_k; ++j) {
            int64_t kj;
            bool free_slot;
            if (H.is64) {
                kj = reinterpret_cast<const int64_t *>(bucket)[j];
                free_slot = kj == kEmptyKey64;
            } else {
                const int32_t k32 = reinterpret_cast<const int32_t *>(bucket)[j];
                kj = (int64_t)k32;
                free_slot = k32 == kEmptyKey32;
            }
            if (!free_slot && kj == v) {
                *code = H.code_bytes == 4 ? reinterpret_cast<const uint32_t *>(bucket + H.code_off)[j] : 0u;
                return true;
            }
            has_free |= free_slot;
        }
        if (has_free) return false;
        b = b + 1 == H.nb ? 0 : b + 1;
    }
    return false;
}

// Every sampled key seen at least three times claims the slot its hash names in the hot table; the heaviest
// claim wins (atomicMax on occurrences << 18 | count-table slot).
__global__ void __launch_bounds__(1024) hot_claim_kernel(const __grid_constant__ HotParams H)
{
    const int s = blockIdx.x * blockDim.x + threadIdx.x;
    if (s >= kHotCountSlots) return;
    const unsigned long long key = H.ckeys[s];
    if (key == kUnused) return;
    const unsigned int occ = H.ccounts[s] + 1u; // the count word started at all ones
    if (occ < 3u) return;
    atomicMax(&H.claims[hot_hash(key) & (kHotSlots - 1)], ((occ < 16383u ? occ : 16383u) << 18) | (unsigned int)s);
}

// One thread per hot slot: the winning key is looked up in the dimension table once and stored with the
// answer.  The block that finishes last writes the header: the number of keys held, or zero when the keys held
// cover less than a tenth of the sample (no skew worth a look-up per row).
__global__ void __launch_bounds__(1024) hot_resolve_kernel(const __grid_constant__ HotParams H)
{
    const int slot = blockIdx.x * blockDim.x + threadIdx.x;
    unsigned int held = 0, covered = 0;
    if (slot < kHotSlots) {
        const unsigned int claim = H.claims[slot];
        uint4 e = make_uint4(0u, 0u, 0u, 0u);
        if (claim != 0u) {
            const unsigned long long key = H.ckeys[claim & (kHotCountSlots - 1)];
            uint32_t code = 0;
            const bool present = dim_lookup(H, (int64_t)key, &code);
            e = make_uint4((uint32_t)key, (uint32_t)(key >> 32), code, present ? 1u : 2u);
            held = 1;
            covered = claim >> 18;
        }
        H.hot[slot] = e;
    }
    __shared__ unsigned int sh[2];
    if (threadIdx.x < 2) sh[threadIdx.x] = 0;
    __syncthreads();
    if (held) {
        atomicAdd(&sh[0], 1u);
        atomicAdd(&sh[1], covered);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned int *hdr = reinterpret_cast<unsigned int *>(&H.hot[kHotSlots]); // {n_hot, held, covered, ticket}
        atomicAdd(&hdr[1], sh[0]);
        atomicAdd(&hdr[2], sh[1]);
        __threadfence();
        if (atomicAdd(&hdr[3], 1u) == gridDim.x - 1) {
            __threadfence();
            const unsigned int all = atomicAdd(&hdr[1], 0u), cov = atomicAdd(&hdr[2], 0u);
            hdr[0] = (uint64_t)cov * 10u >= (uint64_t)H.nsamples ? all : 0u;
        }
    }
}

} // namespace

// Enqueue the kernels.  `scratch` holds the count table (keys, then counts), the claims and the hot table;
// returns the device address of the hot table (kHotSlots + 1 entries of 16 bytes).
sjq_status hot_launch(const void *col, bool is64, int64_t n, const sjq_table *T, void *scratch, cudaStream_t stream,
                      const void **hot_table, int *launches)
{
    char *base = static_cast<char *>(scratch);
    HotParams H{};
    H.col = col;
    H.n = n;
    H.is64 = is64 ? 1 : 0;
    H.nsamples = (int32_t)std::min<int64_t>(n, kHotSamples);
    H.stride = std::max<int64_t>(1, n / std::max<int32_t>(H.nsamples, 1));
    const int kb = is64 ? 8 : 4, cb = T->layout.code_bits / 8;
    H.buckets = T->slots;
    H.nb = (uint32_t)(T->slots_bytes / kBucketBytes);
    H.bucket_k = bucket_keys(kb, cb);
    H.code_off = bucket_code_offset(kb, cb, H.bucket_k);
    H.code_bytes = cb;
    const size_t count_bytes = (size_t)kHotCountSlots * 12, claim_bytes = (size_t)kHotSlots * 4;
    H.ckeys = reinterpret_cast<unsigned long long *>(base);
    H.ccounts = reinterpret_cast<unsigned int *>(base + (size_t)kHotCountSlots * 8);
    H.claims = reinterpret_cast<unsigned int *>(base + count_bytes);
    H.hot = reinterpret_cast<uint4 *>(base + count_bytes + claim_bytes);
    if (cudaMemsetAsync(base, 0xFF, count_bytes, stream) != cudaSuccess ||
        cudaMemsetAsync(base + count_bytes, 0, claim_bytes + (size_t)(kHotSlots + 1) * 16, stream) != cudaSuccess) {
        (void)cudaGetLastError();
        return SJQ_ERR_CUDA;
    }
    if (H.nsamples > 0) hot_sample_kernel<<<(H.nsamples + 1023) / 1024, 1024, 0, stream>>>(H);
    hot_claim_kernel<<<kHotCountSlots / 1024, 1024, 0, stream>>>(H);
    hot_resolve_kernel<<<kHotSlots / 1024, 1024, 0, stream>>>(H);
    if (cudaGetLastError() != cudaSuccess) return SJQ_ERR_CUDA;
    *hot_table = H.hot;
    *launches += 3;
    return SJQ_OK;
}

} // namespace sjq
