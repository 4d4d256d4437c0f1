/*
 * Seeded synthetic inputs for the PSD hot path: an LM-head weight matrix and
 * final hidden states with planted confidence peaks.
 *
 * This file is input generation only.  It holds none of the method's
 * arithmetic (no softmax, no policy, no acceptance) and is the one piece of
 * code that both the CPU oracle's tests and the CUDA path's tests feed from,
 * so that both sides read the same bf16 bytes.
 *
 * Random numbers are counter based: value(seed, stream, index) is a pure
 * function, so any element can be generated in any order, on any thread.
 *
 * Build: gcc -O2 -fopenmp -shared -fPIC gen.c -lm
 */
#include <math.h>
#include <stdint.h>
#include <stddef.h>

enum {
    STREAM_W = 1,       /* LM-head weights                                */
    STREAM_Z = 2,       /* background noise of a hidden row               */
    STREAM_PRESENT = 3, /* does the row carry a planted peak              */
    STREAM_TOKEN = 4,   /* which vocabulary entry the peak points at      */
    STREAM_SCALE = 5,   /* peak scale s                                   */
    STREAM_REUSE = 6,   /* does level l keep level l-1's peak             */
    STREAM_MISC = 7     /* caller-defined extras (initial masks, ...)     */
};

#define GOLDEN 0x9E3779B97F4A7C15ull
#define MAX_LEVELS 64 /* levels -1..62 of one (block, slot) chain */

static inline uint64_t mix64(uint64_t z)
{
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

/* The idx-th output of a splitmix64 sequence whose start is fixed by (seed, stream). */
static inline uint64_t rng_u64(uint64_t seed, uint64_t stream, uint64_t idx)
{
    uint64_t key = mix64(mix64(seed + GOLDEN) ^ (stream * 0xD1342543DE82EF95ull));
    return mix64(key + (idx + 1) * GOLDEN);
}

/* Uniform in (0, 1]. */
static inline double rng_uniform(uint64_t seed, uint64_t stream, uint64_t idx)
{
    return (double)((rng_u64(seed, stream, idx) >> 11) + 1) * (1.0 / 9007199254740992.0);
}

/* Standard normal number k of a stream: Box-Muller on the pair (2p, 2p+1), p = k/2. */
static inline double rng_normal(uint64_t seed, uint64_t stream, uint64_t k)
{
    uint64_t p = k >> 1;
    double u1 = rng_uniform(seed, stream, 2 * p);
    double u2 = rng_uniform(seed, stream, 2 * p + 1);
    double r = sqrt(-2.0 * log(u1));
    double a = 6.283185307179586476925286766559 * u2;
    return (k & 1) ? r * sin(a) : r * cos(a);
}

/* fp32 -> bf16, round to nearest even. Inputs here are always finite. */
static inline uint16_t f32_to_bf16(float f)
{
    union { float f; uint32_t u; } c;
    c.f = f;
    uint32_t u = c.u;
    u += 0x7FFFu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

static inline float bf16_to_f32(uint16_t h)
{
    union { float f; uint32_t u; } c;
    c.u = (uint32_t)h << 16;
    return c.f;
}

/* Exported for tests of the generator itself. */
uint64_t psd_gen_u64(uint64_t seed, uint64_t stream, uint64_t idx) { return rng_u64(seed, stream, idx); }
double psd_gen_uniform(uint64_t seed, uint64_t stream, uint64_t idx) { return rng_uniform(seed, stream, idx); }
double psd_gen_normal(uint64_t seed, uint64_t stream, uint64_t k) { return rng_normal(seed, stream, k); }
uint16_t psd_gen_bf16(float f) { return f32_to_bf16(f); }

/* W[v, j] = bf16(std * n(seed, STREAM_W, v*H + j)), rows v0 .. v0+nv-1 into out[nv, H]. */
void psd_gen_weights(uint64_t seed, int64_t V, int64_t H, double std,
                     int64_t v0, int64_t nv, uint16_t *out)
{
    (void)V;
    int64_t total = nv * H;
    int64_t base = v0 * H;
    /* pairs of consecutive elements share one Box-Muller draw; H is even in every workload */
#pragma omp parallel for schedule(static)
    for (int64_t e = 0; e < total; ++e)
        out[e] = f32_to_bf16((float)(std * rng_normal(seed, STREAM_W, (uint64_t)(base + e))));
}

/*
 * Peak chain of one (block b, slot i): levels l = -1, 0, .., n_levels-2 stored at
 * index l+1.  Level -1 draws (present, token, scale) afresh; level l >= 0 keeps
 * level l-1's triple with probability rho, else draws afresh.
 */
void psd_gen_peaks(uint64_t seed, int64_t B, int64_t M, int64_t n_levels, int64_t V,
                   double frac, double rho, double s_lo, double s_hi,
                   int32_t *present, int32_t *token, double *scale /* each [B, M, n_levels] */)
{
    for (int64_t bm = 0; bm < B * M; ++bm) {
        int32_t cp = 0, ct = 0;
        double cs = 0.0;
        for (int64_t l = 0; l < n_levels; ++l) {
            uint64_t c = (uint64_t)bm * MAX_LEVELS + (uint64_t)l;
            int keep = (l > 0) && (rng_uniform(seed, STREAM_REUSE, c) <= rho);
            if (!keep) {
                cp = rng_uniform(seed, STREAM_PRESENT, c) <= frac;
                ct = (int32_t)(((rng_u64(seed, STREAM_TOKEN, c) >> 32) * (uint64_t)V) >> 32);
                cs = s_lo + (s_hi - s_lo) * rng_uniform(seed, STREAM_SCALE, c);
            }
            present[bm * n_levels + l] = cp;
            token[bm * n_levels + l] = ct;
            scale[bm * n_levels + l] = cs;
        }
    }
}

/*
 * hidden[row, j] = bf16( z[j] + gain * W[t, j] ) for the rows of levels
 * lvl0 .. lvl0+n_lvl-1 (level index as stored by psd_gen_peaks, i.e. l+1),
 * laid out [B, n_lvl, M, H]: row = (b*n_lvl + (lvl-lvl0))*M + i.
 *
 * gain_mode 0: gain = s (the scale used literally as a multiple of W[t]).
 * gain_mode 1: gain = (ln V + q/2 + 4*(s-3)) / |W[t]|^2 with q = H*std^2, so that
 *              s is in logit units: the planted logit sits 4*(s-3) nats above the
 *              log-partition of the background.
 * w_rows holds the bf16 rows W[token] for every (b, i, level) entry, gathered by
 * the caller: [B, M, n_levels, H].
 */
void psd_gen_hidden(uint64_t seed, int64_t B, int64_t M, int64_t n_levels, int64_t H, int64_t V,
                    double std, int32_t gain_mode, int64_t lvl0, int64_t n_lvl,
                    const int32_t *present, const double *scale, const uint16_t *w_rows,
                    uint16_t *hidden, double *gain_out /* nullable [B, n_lvl, M] */)
{
    double q = (double)H * std * std;
    int64_t rows = B * n_lvl * M;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        int64_t i = r % M;
        int64_t dl = (r / M) % n_lvl;
        int64_t b = r / (M * n_lvl);
        int64_t lvl = lvl0 + dl;
        int64_t e = (b * M + i) * n_levels + lvl;
        uint64_t c = (uint64_t)(b * M + i) * MAX_LEVELS + (uint64_t)lvl;
        const uint16_t *wr = w_rows + e * H;
        double gain = 0.0;
        if (present[e]) {
            if (gain_mode == 0) {
                gain = scale[e];
            } else {
                double n2 = 0.0;
                for (int64_t j = 0; j < H; ++j) {
                    double w = (double)bf16_to_f32(wr[j]);
                    n2 += w * w;
                }
                gain = (log((double)V) + 0.5 * q + 4.0 * (scale[e] - 3.0)) / n2;
            }
        }
        if (gain_out) gain_out[r] = gain;
        for (int64_t j = 0; j < H; ++j) {
            double z = rng_normal(seed, STREAM_Z, c * (uint64_t)H + (uint64_t)j);
            double x = z + gain * (double)bf16_to_f32(wr[j]);
            hidden[r * H + j] = f32_to_bf16((float)x);
        }
    }
}
