/*
 * Device-side generator of the seeded synthetic columns: evaluates the input
 * definition of sjq_gen_core.h directly into device memory so that the large
 * fact tables never cross PCIe.  No query arithmetic lives here.
 */
#include "sjq_gen_core.h"
#include "sjq_gen.h"

#include <cuda_runtime.h>

namespace {

// One instantiation per column kind; every thread writes only rows i < n.
template <int KIND>
__global__ void __launch_bounds__(256)
gen_fill_kernel(uint64_t seed, uint64_t column, int64_t row0, int64_t n, int64_t a, int64_t b, int64_t divisor,
                uint64_t key_seed, const uint64_t *zipf_cum, int64_t zipf_k, void *out)
{
    int32_t *o32 = static_cast<int32_t *>(out);
    int64_t *o64 = static_cast<int64_t *>(out);
    const int64_t stride = (int64_t)blockDim.x * (int64_t)gridDim.x;
    for (int64_t i = (int64_t)blockIdx.x * (int64_t)blockDim.x + (int64_t)threadIdx.x; i < n; i += stride) {
        const uint64_t row = (uint64_t)(row0 + i);
        if (KIND == SJQ_GEN_UNIFORM_I32) {
            o32[i] = (int32_t)sjq_gen_uniform(sjq_gen_bits(seed, column, row), a, b);
        } else if (KIND == SJQ_GEN_UNIFORM_DIV_I32) {
            o32[i] = (int32_t)(sjq_gen_uniform(sjq_gen_bits(seed, column, row), a, b) / divisor);
        } else if (KIND == SJQ_GEN_DATE_FK_I32) {
            const int32_t day = (int32_t)sjq_gen_uniform(sjq_gen_bits(seed, column, row), 0, SJQ_GEN_DATE_ROWS - 1);
            o32[i] = sjq_gen_datekey(day);
        } else if (KIND == SJQ_GEN_SEQ_I32) {
            o32[i] = (int32_t)(row + 1);
        } else if (KIND == SJQ_GEN_DATE_KEY_I32) {
            o32[i] = sjq_gen_datekey((int32_t)row);
        } else if (KIND == SJQ_GEN_DATE_YEAR_I32) {
            o32[i] = sjq_gen_datekey((int32_t)row) / 10000;
        } else if (KIND == SJQ_GEN_MIXKEY_I64) {
            o64[i] = (int64_t)sjq_gen_mix(key_seed + row);
        } else {
            const int64_t rank = sjq_gen_zipf_rank(sjq_gen_bits(seed, column, row), zipf_cum, zipf_k);
            o64[i] = (int64_t)sjq_gen_mix(key_seed + (uint64_t)(rank - 1));
        }
    }
}

} // namespace

extern "C" int sjq_gen_fill_device(int kind, uint64_t seed, uint64_t column, int64_t row0, int64_t n, int64_t a,
                                   int64_t b, int64_t div, uint64_t key_seed, const uint64_t *zipf_cum,
                                   int64_t zipf_k, void *out, void *stream)
{
    if (n < 0 || out == nullptr || kind < 0 || kind > SJQ_GEN_ZIPF_FK_I64) return 1;
    if (kind == SJQ_GEN_UNIFORM_DIV_I32 && div == 0) return 1;
    if (kind == SJQ_GEN_ZIPF_FK_I64 && (zipf_cum == nullptr || zipf_k <= 0)) return 1;
    if (n == 0) return 0;
    int64_t blocks = (n + 255) / 256;
    if (blocks > 148 * 32) blocks = 148 * 32;
    const unsigned g = (unsigned)blocks;
    cudaStream_t st = (cudaStream_t)stream;
#define SJQ_GEN_LAUNCH(K) \
    gen_fill_kernel<K><<<g, 256, 0, st>>>(seed, column, row0, n, a, b, div, key_seed, zipf_cum, zipf_k, out)
    switch (kind) {
    case SJQ_GEN_UNIFORM_I32: SJQ_GEN_LAUNCH(SJQ_GEN_UNIFORM_I32); break;
    case SJQ_GEN_UNIFORM_DIV_I32: SJQ_GEN_LAUNCH(SJQ_GEN_UNIFORM_DIV_I32); break;
    case SJQ_GEN_DATE_FK_I32: SJQ_GEN_LAUNCH(SJQ_GEN_DATE_FK_I32); break;
    case SJQ_GEN_SEQ_I32: SJQ_GEN_LAUNCH(SJQ_GEN_SEQ_I32); break;
    case SJQ_GEN_DATE_KEY_I32: SJQ_GEN_LAUNCH(SJQ_GEN_DATE_KEY_I32); break;
    case SJQ_GEN_DATE_YEAR_I32: SJQ_GEN_LAUNCH(SJQ_GEN_DATE_YEAR_I32); break;
    case SJQ_GEN_MIXKEY_I64: SJQ_GEN_LAUNCH(SJQ_GEN_MIXKEY_I64); break;
    default: SJQ_GEN_LAUNCH(SJQ_GEN_ZIPF_FK_I64); break;
    }
#undef SJQ_GEN_LAUNCH
    return cudaGetLastError() == cudaSuccess ? 0 : 2;
}
