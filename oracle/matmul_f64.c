/* Value oracle kernel: C = A * B in double precision.  TEST INFRASTRUCTURE ONLY.
 *
 * The plain definition of a matrix product, C[i][j] = sum_l A[i][l] * B[l][j], written as an
 * i-l-j triple loop over dense row-major buffers.  It ignores matrix properties on purpose: the
 * paper's own lowering multiplies dense buffers whose off-structure entries are stored zeros
 * (Section 2, "Matrix Attribute"; Listing 3 multiplies two lowerTri tensors with a plain matmul),
 * so a stored zero is multiplied like any other number.
 *
 * Rows of C are divided among POSIX threads; every row is computed by exactly one thread in the
 * same l-ascending order, so the result does not depend on the thread count.
 *
 * Nothing here is shared with, or called by, the CUDA library.
 */
#include <pthread.h>
#include <stdint.h>
#include <string.h>

typedef struct {
    const double *a, *b;
    double *c;
    int64_t row_begin, row_end, k, n;
} job_t;

static void *run_rows(void *arg) {
    job_t *j = (job_t *)arg;
    for (int64_t i = j->row_begin; i < j->row_end; ++i) {
        double *ci = j->c + i * j->n;
        memset(ci, 0, (size_t)j->n * sizeof(double));
        const double *ai = j->a + i * j->k;
        for (int64_t l = 0; l < j->k; ++l) {
            const double ail = ai[l];
            const double *bl = j->b + l * j->n;
            for (int64_t col = 0; col < j->n; ++col) ci[col] += ail * bl[col];
        }
    }
    return 0;
}

/* a: m x k, b: k x n, c: m x n (overwritten); all dense row-major.  threads >= 1.
 * Returns the number of threads actually used. */
int mom_oracle_matmul_f64(const double *a, const double *b, double *c,
                          int64_t m, int64_t k, int64_t n, int threads) {
    if (threads < 1) threads = 1;
    if (threads > 256) threads = 256;
    if ((int64_t)threads > m) threads = (int)(m > 0 ? m : 1);
    pthread_t tid[256];
    job_t jobs[256];
    int64_t per = (m + threads - 1) / threads;
    int started = 0;
    for (int t = 0; t < threads; ++t) {
        int64_t lo = t * per, hi = lo + per;
        if (hi > m) hi = m;
        if (lo >= hi) break;
        jobs[t] = (job_t){a, b, c, lo, hi, k, n};
        if (t == threads - 1 || (t + 1) * per >= m) {   /* last slice runs on the calling thread */
            run_rows(&jobs[t]);
            break;
        }
        pthread_create(&tid[t], 0, run_rows, &jobs[t]);
        ++started;
    }
    for (int t = 0; t < started; ++t) pthread_join(tid[t], 0);
    return started + 1;
}
