/*
 * CPU oracle for the symmetric-memory AllReduce(sum).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, obviously-correct statement
 * of what every AllReduce algorithm of the paper must produce.  Only the tests,
 * the smoke check and the benchmark's cpu_baseline / reference arm may call it;
 * the product (the CUDA library) shares no code with it and never links it.
 *
 * What it computes (paper Sec. III-A "One-shot AllReduce": every rank obtains
 * all contributions, reduces locally and writes the output; Sec. V "recvReduce":
 * contributions are converted to an accumulator type before the reduction
 * operator is applied; Table I: one-shot and two-shot are deterministic; Sec. IV
 * "Algorithm Comparison": all ranks must observe the same result):
 *
 *     for every element i:
 *         acc = widen(in[0][i])
 *         for q = 1 .. P-1:  acc = acc + widen(in[q][i])      (IEEE binary32, RNE)
 *         v = narrow(acc)
 *         for r = 0 .. P-1:  out[r][i] = v
 *
 * Readings where the paper is silent: the order is rank 0..P-1 on every rank;
 * the accumulator is binary32 for both element types; the accumulator starts
 * as the rank-0 value (not as +0.0); bf16 narrowing is round-to-nearest-even,
 * subnormals are kept, a NaN narrows to a quiet NaN of the same sign.
 *
 * Build:  gcc -O2 -fno-fast-math -ffp-contract=off -fexcess-precision=standard
 *             -fopenmp -shared -fPIC
 * (the flags keep every add a single correctly rounded binary32 operation).
 *
 * Parity pins live in tests/test_oracle_pins.py; none of the functions below is
 * "parity unpinned".
 */
#include <stddef.h>
#include <stdint.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

/* bf16 -> binary32: the 16 stored bits are the top half of the binary32 word. */
static float widen_bf16(uint16_t h)
{
    uint32_t w = (uint32_t)h << 16;
    float f;
    memcpy(&f, &w, sizeof f);
    return f;
}

/* binary32 -> bf16, round to nearest, ties to even. */
static uint16_t narrow_bf16(float f)
{
    uint32_t w;
    memcpy(&w, &f, sizeof w);
    if ((w & 0x7fffffffu) > 0x7f800000u) {
        /* NaN: keep the sign, force a quiet NaN so that the cut cannot yield Inf */
        return (uint16_t)((w >> 16) | 0x0040u);
    }
    uint32_t lsb = (w >> 16) & 1u;
    w += 0x7fffu + lsb;
    return (uint16_t)(w >> 16);
}

/* One element, fp32: the rank-ordered binary32 sum. */
static float reduce_f32(const float *in, int P, size_t count, size_t i)
{
    float acc = in[i];
    for (int q = 1; q < P; ++q)
        acc = acc + in[(size_t)q * count + i];
    return acc;
}

/* One element, bf16: widen, rank-ordered binary32 sum, one final narrowing. */
static uint16_t reduce_bf16(const uint16_t *in, int P, size_t count, size_t i)
{
    float acc = widen_bf16(in[i]);
    for (int q = 1; q < P; ++q)
        acc = acc + widen_bf16(in[(size_t)q * count + i]);
    return narrow_bf16(acc);
}

/*
 * in : P rows of `count` elements, row q = rank q's input   (row-major, host)
 * out: P rows of `count` elements, row r = rank r's output  (row-major, host)
 * Returns 0, or -1 on a bad argument.
 */
int oracle_allreduce_f32(const float *in, float *out, int P, size_t count)
{
    if (!in || !out || P < 1) return -1;
    for (size_t i = 0; i < count; ++i) {
        float v = reduce_f32(in, P, count, i);
        for (int r = 0; r < P; ++r)
            out[(size_t)r * count + i] = v;
    }
    return 0;
}

int oracle_allreduce_bf16(const uint16_t *in, uint16_t *out, int P, size_t count)
{
    if (!in || !out || P < 1) return -1;
    for (size_t i = 0; i < count; ++i) {
        uint16_t v = reduce_bf16(in, P, count, i);
        for (int r = 0; r < P; ++r)
            out[(size_t)r * count + i] = v;
    }
    return 0;
}

/*
 * The same loops with the element index split over host threads (OpenMP
 * parallel-for over i; elements are independent, so the arithmetic and its
 * order per element are unchanged).  Used only to time the oracle on all host
 * cores.  *threads_used receives the team size.
 */
int oracle_allreduce_f32_mt(const float *in, float *out, int P, size_t count,
                            int *threads_used)
{
    if (!in || !out || P < 1) return -1;
    int team = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp single
        team = omp_get_num_threads();
#pragma omp for schedule(static)
        for (long long i = 0; i < (long long)count; ++i) {
            float v = reduce_f32(in, P, count, (size_t)i);
            for (int r = 0; r < P; ++r)
                out[(size_t)r * count + (size_t)i] = v;
        }
    }
#else
    oracle_allreduce_f32(in, out, P, count);
#endif
    if (threads_used) *threads_used = team;
    return 0;
}

int oracle_allreduce_bf16_mt(const uint16_t *in, uint16_t *out, int P, size_t count,
                             int *threads_used)
{
    if (!in || !out || P < 1) return -1;
    int team = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp single
        team = omp_get_num_threads();
#pragma omp for schedule(static)
        for (long long i = 0; i < (long long)count; ++i) {
            uint16_t v = reduce_bf16(in, P, count, (size_t)i);
            for (int r = 0; r < P; ++r)
                out[(size_t)r * count + (size_t)i] = v;
        }
    }
#else
    oracle_allreduce_bf16(in, out, P, count);
#endif
    if (threads_used) *threads_used = team;
    return 0;
}

/*
 * Sibling collectives built from the same primitives (paper Sec. V, "NCCL Collective
 * Integration": low-latency Broadcast, Reduce, ReduceScatter and AllGather; Sec. III:
 * AllReduce decomposes into ReduceScatter + AllGather or Reduce + Broadcast).
 * es = element size in bytes (4: fp32, 2: bf16).  Reductions use the same
 * rank-ordered binary32 sum and single narrowing as the AllReduce above.
 *
 * reduce_scatter: in[P][P*n] -> out[P][n],   out[r][i] = sum_q in[q][r*n + i]
 * all_gather    : in[P][n]   -> out[P][P*n], out[r][q*n + i] = in[q][i]
 * broadcast     : in[P][n]   -> out[P][n],   out[r][i] = in[root][i]
 * reduce        : in[P][n]   -> out[n] (the root's result), sum over ranks
 */
int oracle_reduce_scatter(const void *in, void *out, int P, size_t n, int es)
{
    if (!in || !out || P < 1 || (es != 4 && es != 2)) return -1;
    const size_t row = (size_t)P * n;
    for (int r = 0; r < P; ++r)
        for (size_t i = 0; i < n; ++i) {
            if (es == 4)
                ((float *)out)[(size_t)r * n + i] = reduce_f32((const float *)in, P, row, (size_t)r * n + i);
            else
                ((uint16_t *)out)[(size_t)r * n + i] = reduce_bf16((const uint16_t *)in, P, row, (size_t)r * n + i);
        }
    return 0;
}

int oracle_all_gather(const void *in, void *out, int P, size_t n, int es)
{
    if (!in || !out || P < 1 || (es != 4 && es != 2)) return -1;
    const unsigned char *src = (const unsigned char *)in;
    unsigned char *dst = (unsigned char *)out;
    for (int r = 0; r < P; ++r)
        for (int q = 0; q < P; ++q)
            memcpy(dst + ((size_t)r * P + q) * n * es, src + (size_t)q * n * es, n * es);
    return 0;
}

int oracle_broadcast(const void *in, void *out, int P, size_t n, int es, int root)
{
    if (!in || !out || P < 1 || root < 0 || root >= P || (es != 4 && es != 2)) return -1;
    for (int r = 0; r < P; ++r)
        memcpy((unsigned char *)out + (size_t)r * n * es, (const unsigned char *)in + (size_t)root * n * es, n * es);
    return 0;
}

int oracle_reduce(const void *in, void *out, int P, size_t n, int es)
{
    if (!in || !out || P < 1 || (es != 4 && es != 2)) return -1;
    for (size_t i = 0; i < n; ++i) {
        if (es == 4) ((float *)out)[i] = reduce_f32((const float *)in, P, n, i);
        else ((uint16_t *)out)[i] = reduce_bf16((const uint16_t *)in, P, n, i);
    }
    return 0;
}

/* Team size of the *_mt entry points (0 or less: leave the runtime's default). */
void oracle_set_threads(int n)
{
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* Exposed so that the pins can test the two conversions on their own. */
uint16_t oracle_narrow_bf16(float f) { return narrow_bf16(f); }
float    oracle_widen_bf16(uint16_t h) { return widen_bf16(h); }
