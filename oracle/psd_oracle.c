/*
 * TEST INFRASTRUCTURE — the CPU oracle of the PSD confidence computation.
 *
 * Only tests, the smoke check and the benchmark's cpu_baseline leg may call this.
 * It shares no code with the CUDA path and is never a fallback for it.
 *
 * What it computes (paper Sec. 3.1, "Preliminaries"): for every row r of the final
 * hidden states, the model distribution over the vocabulary is the softmax of the
 * LM-head logits l_v = sum_j hidden[r, j] * W[v, j]; the prediction is
 * x^ = argmax_v p(v) and its confidence is c = max_v p(v).  The same quantities are
 * used again for every draft of the batched verification pass (Sec. 3.2, Stage 3;
 * Algorithm 1, the two model calls).
 *
 * Everything is the definition written out: inputs are bf16 bit patterns widened
 * exactly to fp64, every logit is one dot product summed in index order in fp64,
 * and max / argmax / sum of exponentials are plain loops over the vocabulary in
 * index order.  Threads split the vocabulary for the dot products only; no
 * summation is reordered by that.
 *
 * Readings where the paper is silent: softmax temperature 1; equal maxima resolve to
 * the lowest vocabulary index.
 *
 * Build: gcc -O2 -fopenmp -shared -fPIC psd_oracle.c -lm
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static inline double bf16_to_f64(uint16_t h)
{
    union { float f; uint32_t u; } c;
    c.u = (uint32_t)h << 16;
    return (double)c.f;
}

int psd_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* logits[r, v] = sum_j hidden[r, j] * W[v, j], fp64, j ascending. */
int psd_oracle_logits(const uint16_t *hidden, const uint16_t *W,
                      int64_t n_rows, int64_t H, int64_t V, double *logits)
{
    double *h = (double *)malloc(sizeof(double) * (size_t)(n_rows * H));
    if (!h) return -1;
    for (int64_t e = 0; e < n_rows * H; ++e) h[e] = bf16_to_f64(hidden[e]);
    int fail = 0;
#pragma omp parallel
    {
        double *w = (double *)malloc(sizeof(double) * (size_t)H);
        if (!w) {
#pragma omp atomic write
            fail = 1;
        }
#pragma omp barrier
        if (!fail) {
#pragma omp for schedule(static)
            for (int64_t v = 0; v < V; ++v) {
                for (int64_t j = 0; j < H; ++j) w[j] = bf16_to_f64(W[v * H + j]);
                for (int64_t r = 0; r < n_rows; ++r) {
                    const double *hr = h + r * H;
                    double acc = 0.0;
                    for (int64_t j = 0; j < H; ++j) acc += hr[j] * w[j];
                    logits[r * V + v] = acc;
                }
            }
        }
        free(w);
    }
    free(h);
    return fail ? -1 : 0;
}

/*
 * From one row of logits: m = max_v l_v; token = the lowest v with l_v = m;
 * S = sum_v exp(l_v - m) (v ascending); conf = 1/S = max_v softmax(l)_v;
 * lse = m + ln S; gap = m - (largest logit at any other index).
 */
void psd_oracle_row_stats(const double *l, int64_t V,
                          int32_t *token, double *conf, double *lse, double *gap)
{
    double m = l[0];
    int64_t a = 0;
    for (int64_t v = 1; v < V; ++v)
        if (l[v] > m) { m = l[v]; a = v; }
    double second = -INFINITY;
    for (int64_t v = 0; v < V; ++v)
        if (v != a && l[v] > second) second = l[v];
    double S = 0.0;
    for (int64_t v = 0; v < V; ++v) S += exp(l[v] - m);
    *token = (int32_t)a;
    *conf = 1.0 / S;
    *lse = m + log(S);
    *gap = m - second;
}

/* Confidence of every row; rows are processed in batches so the logits of a batch fit in memory. */
int psd_oracle_confidence(const uint16_t *hidden, const uint16_t *W,
                          int64_t n_rows, int64_t H, int64_t V,
                          int32_t *token, double *conf, double *lse, double *gap)
{
    int64_t batch = 64;
    double *logits = (double *)malloc(sizeof(double) * (size_t)(batch * V));
    if (!logits) return -1;
    for (int64_t r0 = 0; r0 < n_rows; r0 += batch) {
        int64_t nb = n_rows - r0 < batch ? n_rows - r0 : batch;
        if (psd_oracle_logits(hidden + r0 * H, W, nb, H, V, logits)) { free(logits); return -1; }
        for (int64_t r = 0; r < nb; ++r)
            psd_oracle_row_stats(logits + r * V, V, token + r0 + r, conf + r0 + r, lse + r0 + r, gap + r0 + r);
    }
    free(logits);
    return 0;
}
