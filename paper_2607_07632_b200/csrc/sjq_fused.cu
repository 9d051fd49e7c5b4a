// Ahead-of-time instantiations of the fused probe kernel (the query is a descriptor interpreted at
// run time), result housekeeping kernels and the launch helpers used by the planner.
#include <mutex>
#include <unordered_map>

#include "sjq_fused_device.cuh"

namespace sjq {
namespace {

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
    int64_t dense_base; // indexed: cell number = key + dense_base
    int32_t indexed;    // the table is indexed by the key itself and has no key array
    int64_t gslots; // regular slots; the side slot follows (direct-indexed: cells - 1)
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
        const bool direct = C.indexed != 0;
        const bool side = !direct && i == C.gslots;
        const int64_t k = direct ? i - C.dense_base : side ? kEmptyKey64 : C.gkeys[i];
        const bool used = (direct || side) ? (C.gcounts[i] != 0) : (k != kEmptyKey64);
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

struct MergeParams {
    const int64_t *keys, *sums, *counts; // the lists to merge, n entries
    int64_t n;
    int64_t *gkeys, *gsums, *gcounts; // group table
    uint64_t gmask;
    int32_t *status;
};

// Lists of (key, sum, count) -> group table: one insert-or-find and two adds per entry.
__global__ void __launch_bounds__(256) merge_kernel(const MergeParams M)
{
    const int64_t stride = (int64_t)blockDim.x * gridDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < M.n; i += stride)
        group_table_add(M.gkeys, M.gsums, M.gcounts, M.gmask, M.status, M.keys[i], M.sums[i], M.counts[i]);
}

struct SampleParams {
    const void *col[SJQ_MAX_PREDS];
    DPred preds[SJQ_MAX_PREDS];
    int32_t npreds;
    int64_t n;       // rows of the table
    int64_t groups;  // sampled groups of four consecutive rows
    int64_t stride;  // rows between the starts of two sampled groups (a multiple of 4)
    unsigned long long *counts; // [0] rows sampled, [1 + p] rows among them passing predicate p
};

// Every predicate evaluated on its own over an evenly spaced sample of the table: the marginal pass
// fractions the planner orders the stages by.  One 16- or 32-byte load per predicate and group.
__global__ void __launch_bounds__(256) sample_kernel(const __grid_constant__ SampleParams S)
{
    __shared__ unsigned int block_counts[SJQ_MAX_PREDS + 1];
    if (threadIdx.x <= SJQ_MAX_PREDS) block_counts[threadIdx.x] = 0;
    __syncthreads();
    const int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (g < S.groups) {
        const int64_t r0 = g * S.stride;
        const int rows = (int)(S.n - r0 < 4 ? S.n - r0 : 4);
        atomicAdd(&block_counts[0], (unsigned int)rows);
        for (int p = 0; p < S.npreds; ++p) {
            const DPred &d = S.preds[p];
            unsigned int pass = 0;
            for (int r = 0; r < rows; ++r)
                pass += d.is64 ? pred_eval<int64_t>(d, static_cast<const int64_t *>(S.col[p])[r0 + r])
                               : pred_eval<int32_t>(d, static_cast<const int32_t *>(S.col[p])[r0 + r]);
            if (pass) atomicAdd(&block_counts[1 + p], pass);
        }
    }
    __syncthreads();
    if (threadIdx.x <= S.npreds && block_counts[threadIdx.x])
        atomicAdd(&S.counts[threadIdx.x], (unsigned long long)block_counts[threadIdx.x]);
}

fused_fn pick_kernel(int agg, bool mul, bool hash)
{
    switch (agg) {
    case AGG_SCALAR: return fused_variant_scalar(mul, hash);
    case AGG_SMEM: return fused_variant_smem(mul, hash);
    case AGG_GLOBAL: return fused_variant_global(mul, hash);
    default: return fused_variant_hash(mul, hash);
    }
}

} // namespace

// ---- launch helpers used by the planner (sjq_run.cu) ----------------------

// Shared-memory opt-in and occupancy of a kernel variant; both answers are remembered per device, so a
// repeated query costs two map look-ups instead of two runtime calls.
namespace {
std::mutex g_occ_mutex;
std::unordered_map<uint64_t, int> g_occupancy; // (device, variant, block, smem) -> blocks per SM
std::unordered_map<uint32_t, int> g_opted;     // (device, variant) -> largest smem opted in for
} // namespace

int fused_cache_clear()
{
    std::lock_guard<std::mutex> lock(g_occ_mutex);
    const int n = (int)g_occupancy.size();
    g_occupancy.clear(); // the shared-memory opt-in of a kernel is a property of the function: kept
    return n;
}

sjq_status fused_occupancy(int agg, bool mul, bool hash, int block, size_t smem, int *ctas_per_sm)
{
    std::mutex &mutex = g_occ_mutex;
    std::unordered_map<uint64_t, int> &occupancy = g_occupancy;
    std::unordered_map<uint32_t, int> &opted = g_opted;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return SJQ_ERR_CUDA;
    const uint32_t variant = (uint32_t)(agg * 4 + (mul ? 2 : 0) + (hash ? 1 : 0));
    const uint32_t fkey = (uint32_t)dev * 64u + variant;
    const uint64_t okey = ((uint64_t)fkey << 40) | ((uint64_t)block << 24) | (uint64_t)(smem & 0xFFFFFF);
    std::lock_guard<std::mutex> lock(mutex);
    fused_fn fn = pick_kernel(agg, mul, hash);
    auto o = opted.find(fkey);
    if (o == opted.end() || o->second < (int)smem) {
        if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
            (void)cudaGetLastError();
            return SJQ_ERR_CUDA;
        }
        opted[fkey] = (int)smem;
    }
    auto it = occupancy.find(okey);
    if (it == occupancy.end()) {
        int n = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, fn, block, smem) != cudaSuccess) {
            (void)cudaGetLastError();
            return SJQ_ERR_CUDA;
        }
        it = occupancy.emplace(okey, n).first;
    }
    *ctas_per_sm = it->second;
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

// Enqueue the sampling kernel: `counts` (device, SJQ_MAX_PREDS + 1 words) is cleared first.
sjq_status sample_launch(const sjq_col *fact, const DPred *preds, int npreds, int64_t n, unsigned long long *counts,
                         cudaStream_t stream)
{
    if (cudaMemsetAsync(counts, 0, (SJQ_MAX_PREDS + 1) * sizeof(unsigned long long), stream) != cudaSuccess)
        return SJQ_ERR_CUDA;
    if (n <= 0 || npreds <= 0) return SJQ_OK;
    SampleParams S{};
    for (int p = 0; p < npreds; ++p) {
        S.col[p] = fact[preds[p].col].data;
        S.preds[p] = preds[p];
    }
    S.npreds = npreds;
    S.n = n;
    S.counts = counts;
    const int64_t quads = (n + 3) / 4;
    const int64_t want = (int64_t)1 << 16; // 65 536 groups of four rows
    S.groups = quads < want ? quads : want;
    S.stride = 4 * (quads / S.groups);
    sample_kernel<<<(int)((S.groups + 255) / 256), 256, 0, stream>>>(S);
    return cudaGetLastError() == cudaSuccess ? SJQ_OK : SJQ_ERR_CUDA;
}

sjq_status merge_launch(const int64_t *keys, const int64_t *sums, const int64_t *counts, int64_t n, int64_t *gkeys,
                        int64_t *gsums, int64_t *gcounts, uint64_t gmask, int32_t *status, int sm_count,
                        cudaStream_t stream)
{
    if (n <= 0) return SJQ_OK;
    MergeParams M{keys, sums, counts, n, gkeys, gsums, gcounts, gmask, status};
    int64_t blocks = (n + 255) / 256;
    if (blocks > (int64_t)sm_count * 8) blocks = (int64_t)sm_count * 8;
    merge_kernel<<<(int)blocks, 256, 0, stream>>>(M);
    return cudaGetLastError() == cudaSuccess ? SJQ_OK : SJQ_ERR_CUDA;
}

sjq_status compact_launch(const int64_t *gkeys, const int64_t *gsums, const int64_t *gcounts, int64_t gslots,
                          bool indexed, int64_t dense_base, int64_t *keys, int64_t *sums, int64_t *counts,
                          int64_t capacity, int64_t *n_groups, int32_t *status, int sm_count, cudaStream_t stream)
{
    CompactParams C{gkeys, gsums, gcounts, dense_base, indexed ? 1 : 0, gslots, keys, sums, counts, capacity, n_groups,
                    status};
    int64_t blocks = (gslots + 256) / 256;
    if (blocks > (int64_t)sm_count * 8) blocks = (int64_t)sm_count * 8;
    compact_kernel<<<(int)blocks, 256, 0, stream>>>(C);
    return cudaGetLastError() == cudaSuccess ? SJQ_OK : SJQ_ERR_CUDA;
}

} // namespace sjq
