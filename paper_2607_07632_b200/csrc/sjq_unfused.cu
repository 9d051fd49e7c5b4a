// Operator-at-a-time execution of the same query, for the ablation only.
//
// Section 4.1 of the paper describes the engine before fusion: one kernel per
// operator, a global flag array that every selection and every join ANDs its
// verdict into, and the gathered dimension attributes written out as whole
// columns for the operator that follows; Section 5.4 measures what fusing
// those passes into one kernel saves.  This file restates that baseline on the
// same stage descriptors the fused kernel interprets, so the two can be timed
// on the same plan:
//
//   filter pass (one per predicate or join)   reads its fact column for every
//       row, reads the flags (except the first pass), evaluates the rows still
//       flagged, writes the flags back; a join that gathers a payload also
//       writes the packed payload code of every surviving row to a column of
//       its own;
//   aggregate pass                             reads the flags, and for flagged
//       rows the measure columns and the materialised payload columns, forms
//       group key and value, and adds them with global atomics (a scalar sum
//       is reduced per block first).
//
// Every row pays for every column, for the flag traffic and for one launch per
// operator: exactly what fusion removes.
#include "sjq_fused_device.cuh"

namespace sjq {
namespace {

struct MatColumns {
    void *col[kMaxStages]; // per stage: the materialised payload codes (NULL: the stage gathers nothing)
};

// rows [r, r + 4) of a flag array as a mask (flags are bytes holding 0 or 1)
__device__ __forceinline__ uint32_t load_flags4(const uint8_t *flags, int64_t r)
{
    const uint32_t w = *reinterpret_cast<const uint32_t *>(flags + r);
    return (w & 1u) | ((w >> 7) & 2u) | ((w >> 14) & 4u) | ((w >> 21) & 8u);
}

template <typename T, bool HASH>
__device__ __forceinline__ void filter_group(const RunParams &P, const DStage &S, int64_t r, uint32_t valid,
                                             uint8_t *flags, bool first, void *mat, bool mat64)
{
    T v[4];
    const T *c = static_cast<const T *>(S.col) + r;
    if (valid == 0xFu) {
        Vec4<T>::load(c, v);
    } else {
#pragma unroll
        for (int k = 0; k < 4; ++k) v[k] = ((valid >> k) & 1u) ? c[k] : (T)0;
    }
    const uint32_t m = first ? valid : (load_flags4(flags, r) & valid);
    uint64_t code[4] = {0, 0, 0, 0};
    const uint32_t pass = run_stage<T, 4, true, HASH>(P, S, nullptr, v, m, code);
    *reinterpret_cast<uint32_t *>(flags + r) =
        (pass & 1u) | ((pass & 2u) << 7) | ((pass & 4u) << 14) | ((pass & 8u) << 21);
    if (mat) {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            if ((pass >> k) & 1u) {
                if (mat64) static_cast<uint64_t *>(mat)[r + k] = code[k];
                else static_cast<uint32_t *>(mat)[r + k] = (uint32_t)code[k];
            }
        }
    }
}

// One selection or one join probe over the whole table.
template <bool HASH>
__global__ void __launch_bounds__(256) unfused_filter_kernel(const __grid_constant__ RunParams P, int s, uint8_t *flags,
                                                             int first, void *mat, int mat64)
{
    const DStage &S = P.st[s];
    const int64_t groups = (P.n + 3) / 4;
    const int64_t stride = (int64_t)blockDim.x * gridDim.x;
    for (int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; g < groups; g += stride) {
        const int64_t r = 4 * g;
        const int64_t rem = P.n - r;
        const uint32_t valid = rem >= 4 ? 0xFu : ((1u << (int)rem) - 1u);
        if (S.is64) filter_group<int64_t, HASH>(P, S, r, valid, flags, first != 0, mat, mat64 != 0);
        else filter_group<int32_t, HASH>(P, S, r, valid, flags, first != 0, mat, mat64 != 0);
    }
}

// The terminal over the flagged rows: measure columns and materialised payloads in, atomics out.
template <int AGG, bool MUL>
__global__ void __launch_bounds__(256) unfused_aggregate_kernel(const __grid_constant__ RunParams P,
                                                                const uint8_t *flags,
                                                                const __grid_constant__ MatColumns M)
{
    const int64_t groups = (P.n + 3) / 4;
    const int64_t stride = (int64_t)blockDim.x * gridDim.x;
    int64_t lsum = 0, lcnt = 0;
    for (int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; g < groups; g += stride) {
        const int64_t r = 4 * g;
        const int64_t rem = P.n - r;
        const uint32_t valid = rem >= 4 ? 0xFu : ((1u << (int)rem) - 1u);
        const uint32_t m = flags ? (load_flags4(flags, r) & valid) : valid;
        if (!m) continue;
        int64_t key[4], X[4], Y[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) key[k] = P.key_offset, X[k] = 0, Y[k] = 0;
        for (int s = 0; s < P.nstages; ++s) {
            const DStage &S = P.st[s];
            if (!S.acc) continue;
            uint64_t code[4] = {0, 0, 0, 0};
            if (M.col[s]) {
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    if ((m >> k) & 1u)
                        code[k] = S.code_bits > 32 ? static_cast<const uint64_t *>(M.col[s])[r + k]
                                                   : (uint64_t) static_cast<const uint32_t *>(M.col[s])[r + k];
            }
            if (S.is64) {
                int64_t v[4] = {0, 0, 0, 0};
                if (S.acc & 0x7u) {
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        if ((m >> k) & 1u) v[k] = static_cast<const int64_t *>(S.col)[r + k];
                }
                accumulate<MUL, int64_t, 4>(S, v, code, m, key, X, Y);
            } else {
                int32_t v[4] = {0, 0, 0, 0};
                if (S.acc & 0x7u) {
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        if ((m >> k) & 1u) v[k] = static_cast<const int32_t *>(S.col)[r + k];
                }
                accumulate<MUL, int32_t, 4>(S, v, code, m, key, X, Y);
            }
        }
        terminal<AGG, MUL, 4>(P, nullptr, key, X, Y, m, lsum, lcnt);
    }
    if (AGG == AGG_SCALAR) scalar_block_reduce(P, lsum, lcnt);
}

} // namespace

size_t unfused_scratch_bytes(int64_t n, int gathering_joins)
{
    const size_t rows = (size_t)((n + 255) / 256 * 256);
    return rows + (size_t)gathering_joins * rows * 8;
}

// Enqueue the operator-at-a-time pipeline for a plan without queues, staged tables or gather copies:
// stages [0, nfilter) are the selections and joins, later stages plain column loads.
sjq_status unfused_launch(const RunParams &P, int nfilter, int agg, bool mul, bool has_hash, void *scratch,
                          size_t scratch_bytes, int sm_count, cudaStream_t stream, int *launches)
{
    const size_t rows = (size_t)((P.n + 255) / 256 * 256);
    int gathering = 0;
    for (int s = 0; s < nfilter; ++s) gathering += (P.st[s].kind == ST_PROBE && (P.st[s].acc & ~0x7u)) ? 1 : 0;
    if (!scratch || scratch_bytes < unfused_scratch_bytes(P.n, gathering)) return SJQ_ERR_BUFFER_SMALL;
    uint8_t *flags = static_cast<uint8_t *>(scratch);
    MatColumns M{};
    char *next = static_cast<char *>(scratch) + rows;
    const int64_t groups = (P.n + 3) / 4;
    int64_t blocks = (groups + 255) / 256;
    if (blocks > (int64_t)sm_count * 8) blocks = (int64_t)sm_count * 8;
    if (blocks < 1) blocks = 1;
    for (int s = 0; s < nfilter; ++s) {
        const DStage &S = P.st[s];
        void *mat = nullptr;
        if (S.kind == ST_PROBE && (S.acc & ~0x7u)) {
            mat = next;
            next += rows * 8;
            M.col[s] = mat;
        }
        if (has_hash) unfused_filter_kernel<true><<<(int)blocks, 256, 0, stream>>>(P, s, flags, s == 0, mat, S.code_bits > 32);
        else unfused_filter_kernel<false><<<(int)blocks, 256, 0, stream>>>(P, s, flags, s == 0, mat, S.code_bits > 32);
        ++*launches;
    }
    const uint8_t *f = nfilter ? flags : nullptr;
    switch (agg * 2 + (mul ? 1 : 0)) {
    case AGG_SCALAR * 2: unfused_aggregate_kernel<AGG_SCALAR, false><<<(int)blocks, 256, 0, stream>>>(P, f, M); break;
    case AGG_SCALAR * 2 + 1: unfused_aggregate_kernel<AGG_SCALAR, true><<<(int)blocks, 256, 0, stream>>>(P, f, M); break;
    case AGG_GLOBAL * 2: unfused_aggregate_kernel<AGG_GLOBAL, false><<<(int)blocks, 256, 0, stream>>>(P, f, M); break;
    case AGG_GLOBAL * 2 + 1: unfused_aggregate_kernel<AGG_GLOBAL, true><<<(int)blocks, 256, 0, stream>>>(P, f, M); break;
    case AGG_HASH * 2: unfused_aggregate_kernel<AGG_HASH, false><<<(int)blocks, 256, 0, stream>>>(P, f, M); break;
    case AGG_HASH * 2 + 1: unfused_aggregate_kernel<AGG_HASH, true><<<(int)blocks, 256, 0, stream>>>(P, f, M); break;
    default: return SJQ_ERR_UNSUPPORTED;
    }
    ++*launches;
    return cudaGetLastError() == cudaSuccess ? SJQ_OK : SJQ_ERR_CUDA;
}

} // namespace sjq
