/*
 * TEST INFRASTRUCTURE ONLY - part of the CPU parity oracle.  Nothing on the
 * product path may call or link this file.
 *
 * LM-head logits of the draft model, written out from the definition
 * (paper Section 1: the draft model reuses the target's LM head; Algorithm 1
 * "Run draft model on beam"):
 *
 *     z[r][v] = s * sum_j W[v][j] * h[r][j] + bias[v]
 *
 * Every dot product is one plain left-to-right fp64 sum over j.  W stays in
 * its storage type (fp32 or bf16) and is widened element by element; widening
 * either type to fp64 is exact.  The only liberty taken is loop order: for one
 * vocab row v the R row accumulators advance together over j (h is passed
 * transposed, hT[j][r]), which does not change any individual sum.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define DDD_REF_MAX_ROWS 1024

static inline double widen_bf16(uint16_t bits) {
    uint32_t u = ((uint32_t)bits) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

__attribute__((target_clones("arch=haswell", "default")))
static void row_dots(const double *wrow, const double *hT, int64_t hidden, int rows, double *acc) {
    for (int r = 0; r < rows; ++r) acc[r] = 0.0;
    for (int64_t j = 0; j < hidden; ++j) {
        const double w = wrow[j];
        const double *hj = hT + j * rows;
        for (int r = 0; r < rows; ++r) acc[r] += w * hj[r];
    }
}

/* Returns 0 on success, -1 on bad arguments, -2 if memory ran out. */
int ddd_ref_logits(const void *W, int w_is_bf16, int64_t vocab, int64_t hidden,
                   const double *hT, int rows, double scale, const double *bias /* nullable */,
                   double *z /* [rows][vocab] */) {
    if (!W || !hT || !z || vocab <= 0 || hidden <= 0 || rows <= 0 || rows > DDD_REF_MAX_ROWS) return -1;
    int failed = 0;
#pragma omp parallel
    {
        double *wrow = (double *)malloc(sizeof(double) * (size_t)hidden);
        double *acc = (double *)malloc(sizeof(double) * (size_t)rows);
        if (!wrow || !acc) {
#pragma omp atomic write
            failed = 1;
        }
#pragma omp barrier
        if (!failed) {
#pragma omp for schedule(static)
            for (int64_t v = 0; v < vocab; ++v) {
                if (w_is_bf16) {
                    const uint16_t *src = (const uint16_t *)W + v * hidden;
                    for (int64_t j = 0; j < hidden; ++j) wrow[j] = widen_bf16(src[j]);
                } else {
                    const float *src = (const float *)W + v * hidden;
                    for (int64_t j = 0; j < hidden; ++j) wrow[j] = (double)src[j];
                }
                row_dots(wrow, hT, hidden, rows, acc);
                const double b = bias ? bias[v] : 0.0;
                for (int r = 0; r < rows; ++r) z[(int64_t)r * vocab + v] = scale * acc[r] + b;
            }
        }
        free(wrow);
        free(acc);
    }
    return failed ? -2 : 0;
}

int ddd_ref_num_threads(void) {
    int n = 1;
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    n = omp_get_max_threads();
#endif
    return n;
}
