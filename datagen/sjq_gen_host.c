/*
 * Host-side generator of the seeded synthetic columns (multi-threaded with
 * OpenMP).  It only evaluates the input definition in sjq_gen_core.h; no
 * query arithmetic lives here.  The device generator produces the same bytes.
 */
#include "sjq_gen_core.h"
#include "sjq_gen.h"

#include <stddef.h>

int sjq_gen_fill_host(int kind, uint64_t seed, uint64_t column, int64_t row0, int64_t n,
                      int64_t a, int64_t b, int64_t div, uint64_t key_seed,
                      const uint64_t *zipf_cum, int64_t zipf_k, void *out)
{
    int32_t *o32 = (int32_t *)out;
    int64_t *o64 = (int64_t *)out;
    int32_t datekeys[SJQ_GEN_DATE_ROWS];
    int64_t i;

    if (n < 0 || out == NULL) return 1;
    if (kind == SJQ_GEN_DATE_FK_I32)
        for (i = 0; i < SJQ_GEN_DATE_ROWS; ++i) datekeys[i] = sjq_gen_datekey((int32_t)i);

    switch (kind) {
    case SJQ_GEN_UNIFORM_I32:
#pragma omp parallel for schedule(static)
        for (i = 0; i < n; ++i)
            o32[i] = (int32_t)sjq_gen_uniform(sjq_gen_bits(seed, column, (uint64_t)(row0 + i)), a, b);
        break;
    case SJQ_GEN_UNIFORM_DIV_I32:
        if (div == 0) return 1;
#pragma omp parallel for schedule(static)
        for (i = 0; i < n; ++i)
            o32[i] = (int32_t)(sjq_gen_uniform(sjq_gen_bits(seed, column, (uint64_t)(row0 + i)), a, b) / div);
        break;
    case SJQ_GEN_DATE_FK_I32:
#pragma omp parallel for schedule(static)
        for (i = 0; i < n; ++i)
            o32[i] = datekeys[sjq_gen_uniform(sjq_gen_bits(seed, column, (uint64_t)(row0 + i)), 0,
                                              SJQ_GEN_DATE_ROWS - 1)];
        break;
    case SJQ_GEN_SEQ_I32:
#pragma omp parallel for schedule(static)
        for (i = 0; i < n; ++i) o32[i] = (int32_t)(row0 + i + 1);
        break;
    case SJQ_GEN_DATE_KEY_I32:
        for (i = 0; i < n; ++i) o32[i] = sjq_gen_datekey((int32_t)(row0 + i));
        break;
    case SJQ_GEN_DATE_YEAR_I32:
        for (i = 0; i < n; ++i) o32[i] = sjq_gen_datekey((int32_t)(row0 + i)) / 10000;
        break;
    case SJQ_GEN_MIXKEY_I64:
#pragma omp parallel for schedule(static)
        for (i = 0; i < n; ++i) o64[i] = (int64_t)sjq_gen_mix(key_seed + (uint64_t)(row0 + i));
        break;
    case SJQ_GEN_ZIPF_FK_I64:
        if (zipf_cum == NULL || zipf_k <= 0) return 1;
#pragma omp parallel for schedule(static)
        for (i = 0; i < n; ++i) {
            int64_t rank = sjq_gen_zipf_rank(sjq_gen_bits(seed, column, (uint64_t)(row0 + i)), zipf_cum, zipf_k);
            o64[i] = (int64_t)sjq_gen_mix(key_seed + (uint64_t)(rank - 1));
        }
        break;
    default:
        return 1;
    }
    return 0;
}

/* cum[k] = sum_{j=1..k+1} floor(2^40 / j); serial prefix sum. */
int sjq_gen_zipf_table(int64_t k, uint64_t *cum)
{
    uint64_t acc = 0;
    int64_t j;
    if (k <= 0 || cum == NULL) return 1;
    for (j = 1; j <= k; ++j) {
        acc += SJQ_GEN_ZIPF_ONE / (uint64_t)j;
        cum[j - 1] = acc;
    }
    return 0;
}

uint64_t sjq_gen_mix_host(uint64_t z) { return sjq_gen_mix(z); }
