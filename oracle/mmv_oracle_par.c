/*
 * CPU oracle, all-cores form of the fp16 segmented scan.
 *
 * TEST INFRASTRUCTURE ONLY (see mmv_oracle.c).  The same definition, Problem 2.1 / Eq. (1), run
 * chunk-parallel: the vector is cut into one contiguous chunk per thread, every thread applies the
 * sequential recurrence of mmv_oracle_seg_scan_f16 to its chunk (a later chunk honours its flag
 * byte 0 and otherwise continues with a running value of zero), and a sequential pass then hands
 * the running value at the end of each chunk to the elements of the next chunk that lie in front
 * of its first start (Section 4.2, steps 3-6, with one level and a chunk as the block).  It exists
 * to time the oracle on all host cores beside the one-core figure; results equal the sequential
 * function's up to the rounding of one extra fp64 addition per element, which its test checks.
 */
#include <math.h>
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>

void mmv_oracle_seg_scan_f16(const uint16_t *x, const uint8_t *f, int64_t n,
                             double *z, double *a, int has_prev, double *state);

typedef struct {
    const uint16_t *x;
    const uint8_t *f;
    double *z, *a;
    int64_t lo, hi;        /* the chunk [lo, hi) */
    int64_t first;         /* index of its first start, hi if none */
    int first_chunk;
} chunk_job;

static void *scan_chunk(void *arg)
{
    chunk_job *j = (chunk_job *)arg;
    double st[2] = {0.0, 0.0};
    mmv_oracle_seg_scan_f16(j->x + j->lo, j->f + j->lo, j->hi - j->lo, j->z + j->lo, j->a + j->lo,
                            j->first_chunk ? 0 : 1, st);
    j->first = j->hi;
    for (int64_t i = j->lo; i < j->hi; ++i)
        if ((j->first_chunk && i == j->lo) || j->f[i] != 0) { j->first = i; break; }
    return NULL;
}

typedef struct {
    double *z, *a;
    int64_t lo, hi;
    double cz, ca;
} fix_job;

static void *add_carry(void *arg)
{
    fix_job *j = (fix_job *)arg;
    for (int64_t i = j->lo; i < j->hi; ++i) { j->z[i] += j->cz; j->a[i] += j->ca; }
    return NULL;
}

/* Returns the number of threads used (<= nthreads), 0 on failure. */
int mmv_oracle_seg_scan_f16_chunks(const uint16_t *x, const uint8_t *f, int64_t n,
                                   double *z, double *a, int nthreads)
{
    if (nthreads < 1) nthreads = 1;
    if ((int64_t)nthreads > n) nthreads = n > 0 ? (int)n : 1;
    chunk_job *jobs = (chunk_job *)calloc((size_t)nthreads, sizeof(chunk_job));
    fix_job *fix = (fix_job *)calloc((size_t)nthreads, sizeof(fix_job));
    pthread_t *th = (pthread_t *)calloc((size_t)nthreads, sizeof(pthread_t));
    if (!jobs || !fix || !th) { free(jobs); free(fix); free(th); return 0; }
    for (int t = 0; t < nthreads; ++t) {
        jobs[t].x = x; jobs[t].f = f; jobs[t].z = z; jobs[t].a = a;
        jobs[t].lo = n * t / nthreads;
        jobs[t].hi = n * (t + 1) / nthreads;
        jobs[t].first_chunk = (t == 0);
    }
    for (int t = 1; t < nthreads; ++t) pthread_create(&th[t], NULL, scan_chunk, &jobs[t]);
    scan_chunk(&jobs[0]);
    for (int t = 1; t < nthreads; ++t) pthread_join(th[t], NULL);
    /* carries, chunk after chunk: what is open at the end of chunk t-1 (its own carry included when
       it has no start) reaches the elements of chunk t in front of its first start */
    double cz = 0.0, ca = 0.0;
    for (int t = 1; t < nthreads; ++t) {
        const chunk_job *p = &jobs[t - 1];
        if (p->hi > p->lo) {
            const int prev_has_start = p->first < p->hi;
            const double lz = z[p->hi - 1], la = a[p->hi - 1];     /* not yet fixed up */
            cz = prev_has_start ? lz : cz + lz;
            ca = prev_has_start ? la : ca + la;
        }
        fix[t].z = z; fix[t].a = a; fix[t].lo = jobs[t].lo; fix[t].hi = jobs[t].first;
        fix[t].cz = cz; fix[t].ca = ca;
    }
    for (int t = 1; t < nthreads; ++t) pthread_create(&th[t], NULL, add_carry, &fix[t]);
    for (int t = 1; t < nthreads; ++t) pthread_join(th[t], NULL);
    free(jobs); free(fix); free(th);
    return nthreads;
}
