// Canonical order of a hashed result: ascending key.
//
// The global group table of Section 3.3 hands its groups back in table order, which depends on the hash function
// and on the capacity; two runs of the same query agree only as sets.  sjq_result_sort puts the list of
// (key, sum, count) triples into ascending signed key order on the device: a least-significant-digit radix sort
// of (key, position) pairs, eight passes of eight bits (histogram per tile, one scan, stable scatter), then one
// gather of the three arrays.  The number of groups is read from device memory by every kernel, so the call
// needs no host wait; grids are sized for the capacity.
#include <algorithm>

#include "sjq_internal.h"

namespace sjq {
namespace {

constexpr int kSortThreads = 256;
constexpr int kSortRounds = 4;
constexpr int kSortTile = kSortThreads * kSortRounds; // elements per block

struct SortParams {
    const int64_t *n_groups; // device: number of entries
    int64_t capacity;
    const unsigned long long *keys_in; // keys of this pass (sign bit already flipped)
    const unsigned int *pos_in;
    unsigned long long *keys_out;
    unsigned int *pos_out;
    unsigned int *hist; // [256][nblocks] counts, scanned in place to offsets
    int32_t nblocks;
    int32_t shift;
};

__device__ __forceinline__ int64_t sort_count(const SortParams &S)
{
    const int64_t n = *S.n_groups;
    return n < 0 ? 0 : (n > S.capacity ? S.capacity : n);
}

// Pass 0 input: keys with the sign bit flipped (unsigned order = signed order) and the identity permutation.
__global__ void __launch_bounds__(kSortThreads) sort_init_kernel(const int64_t *keys, const int64_t *n_groups,
                                                                 int64_t capacity, unsigned long long *k0,
                                                                 unsigned int *p0)
{
    int64_t n = *n_groups;
    n = n < 0 ? 0 : (n > capacity ? capacity : n);
    const int64_t stride = (int64_t)blockDim.x * gridDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
        k0[i] = (unsigned long long)keys[i] ^ 0x8000000000000000ull;
        p0[i] = (unsigned int)i;
    }
}

__global__ void __launch_bounds__(kSortThreads) sort_hist_kernel(const __grid_constant__ SortParams S)
{
    __shared__ unsigned int h[256];
    h[threadIdx.x] = 0;
    __syncthreads();
    const int64_t n = sort_count(S);
    const int64_t base = (int64_t)blockIdx.x * kSortTile;
    for (int r = 0; r < kSortRounds; ++r) {
        const int64_t i = base + r * kSortThreads + threadIdx.x;
        if (i < n) atomicAdd(&h[(unsigned int)(S.keys_in[i] >> S.shift) & 255u], 1u);
    }
    __syncthreads();
    S.hist[(size_t)threadIdx.x * S.nblocks + blockIdx.x] = h[threadIdx.x];
}

// Exclusive scan of the 256 x nblocks counts in digit-major order: entry (d, b) becomes the output position of the
// first element of tile b whose digit is d.  One block; every thread scans a contiguous run.
__global__ void __launch_bounds__(1024) sort_scan_kernel(unsigned int *hist, int64_t total)
{
    __shared__ unsigned int part[1024];
    const int64_t per = (total + 1023) / 1024;
    int64_t lo = (int64_t)threadIdx.x * per, hi;
    lo = lo < total ? lo : total;
    hi = lo + per < total ? lo + per : total;
    unsigned int sum = 0;
    for (int64_t i = lo; i < hi; ++i) sum += hist[i];
    part[threadIdx.x] = sum;
    __syncthreads();
    // inclusive scan of the 1024 partial sums
    for (int off = 1; off < 1024; off <<= 1) {
        const unsigned int v = threadIdx.x >= off ? part[threadIdx.x - off] : 0u;
        __syncthreads();
        part[threadIdx.x] += v;
        __syncthreads();
    }
    unsigned int run = part[threadIdx.x] - sum;
    for (int64_t i = lo; i < hi; ++i) {
        const unsigned int c = hist[i];
        hist[i] = run;
        run += c;
    }
}

// Stable scatter of one tile: elements are taken in index order (round by round, thread by thread); an element's
// position is the tile's offset for its digit plus the number of earlier elements of the tile with that digit.
__global__ void __launch_bounds__(kSortThreads) sort_scatter_kernel(const __grid_constant__ SortParams S)
{
    __shared__ unsigned int offset[256];                      // next output position per digit
    __shared__ unsigned int wcount[kSortThreads / 32][256];   // this round: elements per warp and digit
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    offset[threadIdx.x] = S.hist[(size_t)threadIdx.x * S.nblocks + blockIdx.x];
    const int64_t n = sort_count(S);
    const int64_t base = (int64_t)blockIdx.x * kSortTile;
    for (int r = 0; r < kSortRounds; ++r) {
        for (int w = 0; w < kSortThreads / 32; ++w) wcount[w][threadIdx.x] = 0;
        __syncthreads();
        const int64_t i = base + r * kSortThreads + threadIdx.x;
        const bool valid = i < n;
        unsigned long long key = 0;
        unsigned int pos = 0, digit = 0;
        if (valid) {
            key = S.keys_in[i];
            pos = S.pos_in[i];
            digit = (unsigned int)(key >> S.shift) & 255u;
        }
        // lanes of the warp with the same digit; a lane without an element matches nobody
        const unsigned int peers = __match_any_sync(0xffffffffu, valid ? digit : 256u + (unsigned int)lane);
        const unsigned int before = __popc(peers & ((1u << lane) - 1u));
        if (valid && before == 0) wcount[warp][digit] = __popc(peers);
        __syncthreads();
        if (valid) {
            unsigned int at = offset[digit] + before;
            for (int w = 0; w < warp; ++w) at += wcount[w][digit];
            S.keys_out[at] = key;
            S.pos_out[at] = pos;
        }
        __syncthreads();
        unsigned int add = 0;
        for (int w = 0; w < kSortThreads / 32; ++w) add += wcount[w][threadIdx.x];
        offset[threadIdx.x] += add;
        __syncthreads();
    }
}

// Apply the permutation: out[i] = in[pos[i]] for the three arrays (sorted keys come from the last pass).
__global__ void __launch_bounds__(kSortThreads) sort_gather_kernel(const unsigned long long *skeys, const unsigned int *pos,
                                                                   const int64_t *n_groups, int64_t capacity,
                                                                   const int64_t *sums, const int64_t *counts,
                                                                   int64_t *tmp_sums, int64_t *tmp_counts, int64_t *keys)
{
    int64_t n = *n_groups;
    n = n < 0 ? 0 : (n > capacity ? capacity : n);
    const int64_t stride = (int64_t)blockDim.x * gridDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
        const unsigned int p = pos[i];
        keys[i] = (int64_t)(skeys[i] ^ 0x8000000000000000ull);
        tmp_sums[i] = sums[p];
        tmp_counts[i] = counts[p];
    }
}

__global__ void __launch_bounds__(kSortThreads) sort_copy_back_kernel(const int64_t *n_groups, int64_t capacity,
                                                                      const int64_t *tmp_sums, const int64_t *tmp_counts,
                                                                      int64_t *sums, int64_t *counts)
{
    int64_t n = *n_groups;
    n = n < 0 ? 0 : (n > capacity ? capacity : n);
    const int64_t stride = (int64_t)blockDim.x * gridDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
        sums[i] = tmp_sums[i];
        counts[i] = tmp_counts[i];
    }
}

size_t up256(size_t v) { return (v + 255) / 256 * 256; }

struct SortLayout {
    size_t k0, k1, p0, p1, hist, tsums, tcounts, total;
    int nblocks;
};

SortLayout sort_layout(int64_t capacity)
{
    SortLayout L{};
    const size_t c = (size_t)std::max<int64_t>(capacity, 1);
    L.nblocks = (int)((c + kSortTile - 1) / kSortTile);
    size_t at = 0;
    L.k0 = at, at += up256(c * 8);
    L.k1 = at, at += up256(c * 8);
    L.p0 = at, at += up256(c * 4);
    L.p1 = at, at += up256(c * 4);
    L.hist = at, at += up256((size_t)256 * L.nblocks * 4);
    L.tsums = at, at += up256(c * 8);
    L.tcounts = at, at += up256(c * 8);
    L.total = at;
    return L;
}

} // namespace
} // namespace sjq

using namespace sjq;

extern "C" sjq_status sjq_result_sort_scratch_bytes(int64_t capacity, size_t *bytes)
{
    if (capacity <= 0 || capacity > ((int64_t)1 << 31) || !bytes) return SJQ_ERR_INVALID_ARG;
    *bytes = sort_layout(capacity).total;
    return SJQ_OK;
}

extern "C" sjq_status sjq_result_sort(int64_t *keys, int64_t *sums, int64_t *counts, const int64_t *n_groups,
                                      int64_t capacity, void *scratch, size_t scratch_bytes, void *stream_)
{
    if (!keys || !sums || !counts || !n_groups || !scratch || capacity <= 0 || capacity > ((int64_t)1 << 31))
        return SJQ_ERR_INVALID_ARG;
    if (!aligned16(scratch) || (reinterpret_cast<uintptr_t>(keys) & 7u) || (reinterpret_cast<uintptr_t>(sums) & 7u) ||
        (reinterpret_cast<uintptr_t>(counts) & 7u) || (reinterpret_cast<uintptr_t>(n_groups) & 7u))
        return SJQ_ERR_ALIGN;
    const SortLayout L = sort_layout(capacity);
    if (scratch_bytes < L.total) return SJQ_ERR_BUFFER_SMALL;
    DeviceInfo dev;
    sjq_status st = device_info(&dev);
    if (st != SJQ_OK) return st;
    cudaStream_t stream = (cudaStream_t)stream_;
    char *base = static_cast<char *>(scratch);
    unsigned long long *k[2] = {reinterpret_cast<unsigned long long *>(base + L.k0),
                                reinterpret_cast<unsigned long long *>(base + L.k1)};
    unsigned int *p[2] = {reinterpret_cast<unsigned int *>(base + L.p0), reinterpret_cast<unsigned int *>(base + L.p1)};
    int64_t *tsums = reinterpret_cast<int64_t *>(base + L.tsums), *tcounts = reinterpret_cast<int64_t *>(base + L.tcounts);
    const int stream_grid = (int)std::min<int64_t>((capacity + kSortThreads - 1) / kSortThreads, (int64_t)dev.sm_count * 8);
    sort_init_kernel<<<stream_grid, kSortThreads, 0, stream>>>(keys, n_groups, capacity, k[0], p[0]);
    for (int pass = 0; pass < 8; ++pass) {
        SortParams S{};
        S.n_groups = n_groups;
        S.capacity = capacity;
        S.keys_in = k[pass & 1];
        S.pos_in = p[pass & 1];
        S.keys_out = k[(pass & 1) ^ 1];
        S.pos_out = p[(pass & 1) ^ 1];
        S.hist = reinterpret_cast<unsigned int *>(base + L.hist);
        S.nblocks = L.nblocks;
        S.shift = 8 * pass;
        sort_hist_kernel<<<L.nblocks, kSortThreads, 0, stream>>>(S);
        sort_scan_kernel<<<1, 1024, 0, stream>>>(S.hist, (int64_t)256 * L.nblocks);
        sort_scatter_kernel<<<L.nblocks, kSortThreads, 0, stream>>>(S);
    }
    // eight passes: the sorted pairs are back in buffer 0
    sort_gather_kernel<<<stream_grid, kSortThreads, 0, stream>>>(k[0], p[0], n_groups, capacity, sums, counts, tsums,
                                                              tcounts, keys);
    sort_copy_back_kernel<<<stream_grid, kSortThreads, 0, stream>>>(n_groups, capacity, tsums, tcounts, sums, counts);
    if (cudaGetLastError() != cudaSuccess) return SJQ_ERR_CUDA;
    return SJQ_OK;
}
