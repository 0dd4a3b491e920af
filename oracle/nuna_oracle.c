/*
 * CPU oracle for the emulated collectives.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the slow, plain definition that the CUDA library is checked
 * against.  It shares no code, header, table or helper with the CUDA path and
 * is called only by the tests, by the smoke check and by the benchmark's CPU
 * baseline leg.  Nothing on the product path may call it.
 *
 * What it computes.  The paper describes the collectives only at the level of
 * their meaning (Section 2.1: allreduce aggregates the partial activations of
 * all ranks, allgather assembles every rank's chunk in every rank's output;
 * Figure "Allocation_Diagram": allgather as local load + remote store of each
 * rank's chunk into every rank's buffer; Section 5.1: the direct / all-pairs
 * algorithm).  The numerics are fixed by this build's problem statement:
 * bf16 storage, binary32 accumulation in fixed rank order 0..N-1, one final
 * round-to-nearest-even to bf16, the same value in every destination.
 *
 *   f(h)   : bf16 pattern h  ->  binary32 whose bits are h << 16        (exact)
 *   rne(x) : binary32 -> bf16, round to nearest, ties to even; NaN -> 0x7FFF
 *   allreduce      dst[d][i]       = rne((((f(src[0][i]) + f(src[1][i])) + ...) + f(src[N-1][i])))
 *   reduce_scatter dst[r][j]       = the same fold over src[0..N-1][r*S + j]
 *   allgather      dst[d][r*S + j] = src[r][j]                          (16-bit copy)
 *   alltoall       dst[d][r*S + j] = src[r][d*S + j]                    (16-bit copy)
 *
 * The accumulator starts from f(src[0][i]), not from +0, so N values take N-1
 * additions and an all-(-0) column stays -0.  Every partial sum is a binary32
 * (SSE scalar add on x86-64: no extended precision, default rounding, no
 * flush-to-zero).  Compile without -ffast-math.
 *
 * Parity pins: see tests/test_oracle_pins.py (closed forms on exactly
 * representable integers, order / rounding / signed-zero / subnormal /
 * overflow pins, an exact-rational second model, brute force on tiny inputs).
 */
#include <stddef.h>
#include <stdint.h>
#include <string.h>

static float bf16_to_f32(uint16_t h)
{
    uint32_t u = (uint32_t)h << 16;
    float x;
    memcpy(&x, &u, sizeof x);
    return x;
}

static uint16_t f32_to_bf16_rne(float x)
{
    uint32_t u;
    memcpy(&u, &x, sizeof u);
    if ((u & 0x7F800000u) == 0x7F800000u && (u & 0x007FFFFFu) != 0u)
        return 0x7FFFu;                              /* NaN: canonical quiet NaN */
    /* Add half of the dropped field, minus one when the kept LSB is even, so a
       tie moves to the even neighbour.  A carry may run into the exponent,
       which is how the largest finite values round up to infinity. */
    u += 0x7FFFu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

/* Fold one column: the n values of one element index, in rank order. */
uint16_t nuna_oracle_fold_bf16(const uint16_t *vals, int n)
{
    volatile float acc = bf16_to_f32(vals[0]);       /* volatile: each partial sum is stored as binary32 */
    for (int r = 1; r < n; ++r)
        acc = acc + bf16_to_f32(vals[r]);
    return f32_to_bf16_rne(acc);
}

static uint16_t fold_column(const uint16_t *const *src, int nranks, size_t i)
{
    float acc = bf16_to_f32(src[0][i]);
    for (int r = 1; r < nranks; ++r)
        acc = acc + bf16_to_f32(src[r][i]);
    return f32_to_bf16_rne(acc);
}

/* allreduce: every dst[d] (count elements) receives the rank-ordered sum. */
void nuna_oracle_allreduce_bf16(const uint16_t *const *src, uint16_t *const *dst,
                                int nranks, size_t count, int nthreads)
{
    (void)nthreads;
#pragma omp parallel for schedule(static) num_threads(nthreads) if (nthreads > 1)
    for (size_t i = 0; i < count; ++i) {
        uint16_t out = fold_column(src, nranks, i);
        for (int d = 0; d < nranks; ++d)
            dst[d][i] = out;
    }
}

/* reduce_scatter: src[k] has nranks*shard elements, dst[r] has shard elements. */
void nuna_oracle_reduce_scatter_bf16(const uint16_t *const *src, uint16_t *const *dst,
                                     int nranks, size_t shard, int nthreads)
{
    (void)nthreads;
    for (int r = 0; r < nranks; ++r) {
#pragma omp parallel for schedule(static) num_threads(nthreads) if (nthreads > 1)
        for (size_t j = 0; j < shard; ++j)
            dst[r][j] = fold_column(src, nranks, (size_t)r * shard + j);
    }
}

/* allgather: src[r] has shard elements, every dst[d] has nranks*shard elements. */
void nuna_oracle_allgather_bf16(const uint16_t *const *src, uint16_t *const *dst,
                                int nranks, size_t shard, int nthreads)
{
    (void)nthreads;
    for (int d = 0; d < nranks; ++d)
        for (int r = 0; r < nranks; ++r) {
#pragma omp parallel for schedule(static) num_threads(nthreads) if (nthreads > 1)
            for (size_t j = 0; j < shard; ++j)
                dst[d][(size_t)r * shard + j] = src[r][j];
        }
}

/* alltoall (Section 2.1: token routing between experts, the paper's third collective): src[r] holds
 * nranks blocks of `block` elements, block d being what rank r sends to rank d; dst[d] holds nranks
 * blocks, block r being what it received from rank r.  dst[d][r*block + i] = src[r][d*block + i],
 * a 16-bit copy. */
void nuna_oracle_alltoall_bf16(const uint16_t *const *src, uint16_t *const *dst,
                               int nranks, size_t block, int nthreads)
{
    (void)nthreads;
    for (int d = 0; d < nranks; ++d)
        for (int r = 0; r < nranks; ++r) {
#pragma omp parallel for schedule(static) num_threads(nthreads) if (nthreads > 1)
            for (size_t i = 0; i < block; ++i)
                dst[d][(size_t)r * block + i] = src[r][(size_t)d * block + i];
        }
}

/* ---- other element types -----------------------------------------------------------------------------
 * The same fold with binary16 (IEEE half) or binary32 storage: widen exactly to binary32, add in rank
 * order in binary32, and round once to the storage type (binary32 storage needs no final rounding).
 * Half conversions are written out bit by bit: 1 sign, 5 exponent (bias 15), 10 fraction bits;
 * subnormals are kept in both directions; NaN becomes the canonical 0x7FFF; values that round to
 * 2^16 or more become infinity. */
static float f16_to_f32(uint16_t h)
{
    const uint32_t sign = (uint32_t)(h >> 15) << 31;
    const uint32_t expo = (h >> 10) & 0x1Fu, frac = h & 0x3FFu;
    uint32_t u;
    if (expo == 0x1Fu) {
        u = sign | 0x7F800000u | (frac << 13);                 /* Inf / NaN */
    } else if (expo != 0u) {
        u = sign | ((expo + 112u) << 23) | (frac << 13);       /* normal: rebias 15 -> 127 */
    } else if (frac == 0u) {
        u = sign;                                              /* +-0 */
    } else {
        /* subnormal: frac * 2^-24; normalise by hand */
        uint32_t f = frac;
        int e = -14;
        while ((f & 0x400u) == 0u) { f <<= 1; --e; }
        u = sign | ((uint32_t)(e + 127) << 23) | ((f & 0x3FFu) << 13);
    }
    float x;
    memcpy(&x, &u, sizeof x);
    return x;
}

static uint16_t f32_to_f16_rne(float x)
{
    uint32_t u;
    memcpy(&u, &x, sizeof u);
    const uint16_t sign = (uint16_t)((u >> 16) & 0x8000u);
    const uint32_t mag = u & 0x7FFFFFFFu;
    if (mag > 0x7F800000u) return 0x7FFFu;                     /* NaN */
    if (mag >= 0x477FF000u) return (uint16_t)(sign | 0x7C00u); /* >= 65520 rounds to infinity (Inf included) */
    if (mag >= 0x38800000u) {
        /* normal half range [2^-14, 65520): drop 13 fraction bits with round to nearest even */
        uint32_t v = mag - 0x38000000u;                        /* rebias 127 -> 15 */
        v += 0xFFFu + ((v >> 13) & 1u);
        return (uint16_t)(sign | (v >> 13));                   /* a carry may reach 0x7C00 only above the test */
    }
    if (mag < 0x33000000u) return sign;                        /* below 2^-25: rounds to zero (2^-25 itself ties to 0) */
    /* subnormal half: value = m * 2^-24 with m in [0, 1024]; shift the 24-bit significand right */
    const int e = (int)(mag >> 23) - 127;                      /* -25 .. -15 */
    const uint32_t sig = (mag & 0x7FFFFFu) | 0x800000u;        /* 1.f as a 24-bit integer, weight 2^(e-23) */
    const int shift = -e - 1;                                  /* sig * 2^(e-23) / 2^-24 = sig >> (-e-1) */
    uint32_t m = sig >> shift;
    const uint32_t rem = sig & ((1u << shift) - 1u), half = 1u << (shift - 1);
    if (rem > half || (rem == half && (m & 1u))) ++m;
    return (uint16_t)(sign | m);                               /* m == 1024 is the smallest normal: bits line up */
}

static uint16_t fold_column_f16(const uint16_t *const *src, int nranks, size_t i)
{
    float acc = f16_to_f32(src[0][i]);
    for (int r = 1; r < nranks; ++r)
        acc = acc + f16_to_f32(src[r][i]);
    return f32_to_f16_rne(acc);
}

static float fold_column_f32(const float *const *src, int nranks, size_t i)
{
    float acc = src[0][i];
    for (int r = 1; r < nranks; ++r)
        acc = acc + src[r][i];
    return acc;
}

void nuna_oracle_allreduce_f16(const uint16_t *const *src, uint16_t *const *dst,
                               int nranks, size_t count, int nthreads)
{
    (void)nthreads;
#pragma omp parallel for schedule(static) num_threads(nthreads) if (nthreads > 1)
    for (size_t i = 0; i < count; ++i) {
        uint16_t out = fold_column_f16(src, nranks, i);
        for (int d = 0; d < nranks; ++d)
            dst[d][i] = out;
    }
}

void nuna_oracle_allreduce_f32(const float *const *src, float *const *dst,
                               int nranks, size_t count, int nthreads)
{
    (void)nthreads;
#pragma omp parallel for schedule(static) num_threads(nthreads) if (nthreads > 1)
    for (size_t i = 0; i < count; ++i) {
        float out = fold_column_f32(src, nranks, i);
        for (int d = 0; d < nranks; ++d)
            dst[d][i] = out;
    }
}

void nuna_oracle_reduce_scatter_f16(const uint16_t *const *src, uint16_t *const *dst,
                                    int nranks, size_t shard, int nthreads)
{
    (void)nthreads;
    for (int r = 0; r < nranks; ++r) {
#pragma omp parallel for schedule(static) num_threads(nthreads) if (nthreads > 1)
        for (size_t j = 0; j < shard; ++j)
            dst[r][j] = fold_column_f16(src, nranks, (size_t)r * shard + j);
    }
}

void nuna_oracle_reduce_scatter_f32(const float *const *src, float *const *dst,
                                    int nranks, size_t shard, int nthreads)
{
    (void)nthreads;
    for (int r = 0; r < nranks; ++r) {
#pragma omp parallel for schedule(static) num_threads(nthreads) if (nthreads > 1)
        for (size_t j = 0; j < shard; ++j)
            dst[r][j] = fold_column_f32(src, nranks, (size_t)r * shard + j);
    }
}

uint16_t nuna_oracle_rne_f16(float x) { return f32_to_f16_rne(x); }
float nuna_oracle_widen_f16(uint16_t h) { return f16_to_f32(h); }

/* The two conversions on their own, so the tests can pin them separately. */
uint16_t nuna_oracle_rne_bf16(float x) { return f32_to_bf16_rne(x); }
float nuna_oracle_widen_bf16(uint16_t h) { return bf16_to_f32(h); }
