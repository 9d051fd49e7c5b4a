/*
 * Seeded synthetic input definition for the star-join workloads.
 *
 * This header IS the definition of the input data: every column value is a
 * pure function of (seed, column id, row).  It holds no query arithmetic
 * (no predicates, joins or aggregation) and is shared only by the host
 * generator (sjq_gen_host.c) and the device generator (sjq_gen_cuda.cu),
 * which must produce identical bytes.
 *
 * All arithmetic is unsigned 64-bit integer, so host and device agree
 * bit for bit on every platform.
 */
#ifndef SJQ_GEN_CORE_H
#define SJQ_GEN_CORE_H

#include <stdint.h>

#if defined(__CUDACC__)
#define SJQ_GEN_HD __host__ __device__ static inline
#else
#define SJQ_GEN_HD static inline
#endif

/* 64-bit finaliser: three xor-shifts interleaved with two odd multipliers.
 * Every step is invertible, so the whole map is a bijection on 64 bits. */
#define SJQ_GEN_M1 0xbf58476d1ce4e5b9ULL
#define SJQ_GEN_M2 0x94d049bb133111ebULL

SJQ_GEN_HD uint64_t sjq_gen_mix(uint64_t z)
{
    z ^= z >> 30;
    z *= SJQ_GEN_M1;
    z ^= z >> 27;
    z *= SJQ_GEN_M2;
    z ^= z >> 31;
    return z;
}

/* The 64 random bits of cell (column, row) under a master seed. */
SJQ_GEN_HD uint64_t sjq_gen_bits(uint64_t seed, uint64_t column, uint64_t row)
{
    return sjq_gen_mix(sjq_gen_mix(seed + column) + row);
}

/* Integer in [a, b], both ends included: a + floor(hi32(h) * span / 2^32). */
SJQ_GEN_HD int64_t sjq_gen_uniform(uint64_t h, int64_t a, int64_t b)
{
    uint64_t span = (uint64_t)(b - a) + 1ULL;
    return a + (int64_t)(((h >> 32) * span) >> 32);
}

/* Calendar: day index d (0 = 1992-01-01) -> yyyymmdd.  Gregorian rules. */
SJQ_GEN_HD int32_t sjq_gen_datekey(int32_t d)
{
    int32_t y = 1992;
    for (;;) {
        int32_t leap = ((y % 4 == 0) && (y % 100 != 0)) || (y % 400 == 0);
        int32_t len = 365 + leap;
        if (d < len) break;
        d -= len;
        ++y;
    }
    {
        int32_t leap = ((y % 4 == 0) && (y % 100 != 0)) || (y % 400 == 0);
        int32_t m = 1;
        for (;;) {
            int32_t ml = 31;
            if (m == 4 || m == 6 || m == 9 || m == 11) ml = 30;
            else if (m == 2) ml = 28 + leap;
            if (d < ml) break;
            d -= ml;
            ++m;
        }
        return y * 10000 + m * 100 + (d + 1);
    }
}

#define SJQ_GEN_DATE_ROWS 2556

/* Zipf(1.0) over ranks 1..K by integer weights w_j = floor(2^40 / j).
 * cum[k] = w_1 + ... + w_(k+1) for k = 0..K-1 (so cum[K-1] is the total).
 * A draw u in [0, total) maps to the smallest rank r with u < cum[r-1]. */
#define SJQ_GEN_ZIPF_ONE (1ULL << 40)

SJQ_GEN_HD uint64_t sjq_gen_mulhi64(uint64_t a, uint64_t b)
{
#if defined(__CUDA_ARCH__)
    return __umul64hi(a, b);
#else
    return (uint64_t)(((unsigned __int128)a * (unsigned __int128)b) >> 64);
#endif
}

/* rank in [1, K] for random bits h, given the cumulative table. */
SJQ_GEN_HD int64_t sjq_gen_zipf_rank(uint64_t h, const uint64_t *cum, int64_t K)
{
    uint64_t u = sjq_gen_mulhi64(h, cum[K - 1]); /* uniform in [0, total) */
    int64_t lo = 0, hi = K - 1;                  /* first index with u < cum[idx] */
    while (lo < hi) {
        int64_t mid = lo + ((hi - lo) >> 1);
        if (u < cum[mid]) hi = mid;
        else lo = mid + 1;
    }
    return lo + 1;
}

#endif /* SJQ_GEN_CORE_H */
