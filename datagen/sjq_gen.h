/*
 * C interface of the synthetic-input generators (host and device flavours).
 * Column kinds; every value is a pure function of (seed, column id, row).
 */
#ifndef SJQ_GEN_H
#define SJQ_GEN_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    SJQ_GEN_UNIFORM_I32 = 0,     /* int32 U[a,b] */
    SJQ_GEN_UNIFORM_DIV_I32 = 1, /* int32 U[a,b] / div (same bits as the UNIFORM column of that id) */
    SJQ_GEN_DATE_FK_I32 = 2,     /* int32 yyyymmdd of a uniformly drawn calendar day in [0, 2555] */
    SJQ_GEN_SEQ_I32 = 3,         /* int32 row + 1 (dense dimension key) */
    SJQ_GEN_DATE_KEY_I32 = 4,    /* int32 yyyymmdd of calendar day = row */
    SJQ_GEN_DATE_YEAR_I32 = 5,   /* int32 year of calendar day = row */
    SJQ_GEN_MIXKEY_I64 = 6,      /* int64 mix(key_seed + row): distinct sparse 64-bit keys */
    SJQ_GEN_ZIPF_FK_I64 = 7      /* int64 mix(key_seed + rank - 1), rank ~ Zipf(1.0) on [1, zipf_k] */
};

/* Fill out[0..n) with rows row0..row0+n of one column.  `out` is host memory.
 * Returns 0 on success, 1 on a bad argument. */
int sjq_gen_fill_host(int kind, uint64_t seed, uint64_t column, int64_t row0, int64_t n,
                      int64_t a, int64_t b, int64_t div, uint64_t key_seed,
                      const uint64_t *zipf_cum, int64_t zipf_k, void *out);

/* Same, `out` and `zipf_cum` are device memory; enqueued on `stream`
 * (a cudaStream_t passed as void*).  Returns 0, 1 (bad argument) or
 * 2 (CUDA launch error). */
int sjq_gen_fill_device(int kind, uint64_t seed, uint64_t column, int64_t row0, int64_t n,
                        int64_t a, int64_t b, int64_t div, uint64_t key_seed,
                        const uint64_t *zipf_cum, int64_t zipf_k, void *out, void *stream);

/* Cumulative Zipf(1.0) weight table (host memory, k entries). */
int sjq_gen_zipf_table(int64_t k, uint64_t *cum);

uint64_t sjq_gen_mix_host(uint64_t z);

#ifdef __cplusplus
}
#endif
#endif
