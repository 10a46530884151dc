/*
 * Seeded synthetic workloads for the ZipLine barrier-selection search.
 *
 * This file only produces inputs: per-worker predicted iteration end
 * timestamps (int64 microseconds), shaped [B][n][R].  It contains none of
 * the search arithmetic; both the CPU checker and the CUDA library read the
 * buffers it fills.
 *
 * Randomness is counter based: every draw is splitmix64 of a key built from
 * (seed, instance, worker, iteration, stream), so a buffer can be filled in
 * any order and by any number of threads with identical contents.
 * Normal deviates use Box-Muller on two such draws.
 *
 * Recipe per worker p of instance b (instance seed = base_seed + b):
 *   mean m_p (us)           : lognormal, fixed, or bimodal (see zl_workload)
 *   iteration length        : m_p * (1 + jitter * z), z ~ N(0,1)
 *                             optionally x5 with probability spike_prob
 *                             rounded to int64, clamped to >= 1 us
 *   end timestamp e^p_i     : off_p + running int64 sum of the lengths
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>

typedef struct {
    int32_t n, R, B;
    int32_t mean_kind;       /* 0 lognormal(ln mean_us, sigma); 1 bimodal halves mean_us / mean2_us */
    double  mean_us, sigma, mean2_us;
    double  jitter;          /* relative std of one iteration               */
    double  straggler_frac;  /* share of workers (ceil) whose mean is x straggler_mult */
    double  straggler_mult;
    double  spike_prob, spike_mult;
    double  offset_max_us;   /* start offset ~ U[0, offset_max_us)          */
    int64_t base_seed;
    int64_t epoch_us;        /* added to every timestamp                    */
} zl_workload;

static inline uint64_t splitmix64(uint64_t x) {
    x += 0x9E3779B97F4A7C15ull;
    x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
    x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
    return x ^ (x >> 31);
}

static inline uint64_t draw(uint64_t seed, uint64_t worker, uint64_t iter, uint64_t stream) {
    uint64_t h = splitmix64(seed);
    h = splitmix64(h ^ (worker * 0xD6E8FEB86659FD93ull));
    h = splitmix64(h ^ (iter * 0xA24BAED4963EE407ull));
    return splitmix64(h ^ (stream * 0x9FB21C651E98DF25ull));
}

static inline double unif01(uint64_t h) {            /* (0,1) open on both sides */
    return ((double)(h >> 11) + 0.5) * (1.0 / 9007199254740992.0);
}

static inline double normal(uint64_t seed, uint64_t worker, uint64_t iter, uint64_t stream) {
    double u1 = unif01(draw(seed, worker, iter, stream));
    double u2 = unif01(draw(seed, worker, iter, stream + 1));
    return sqrt(-2.0 * log(u1)) * cos(6.283185307179586476925 * u2);
}

enum { ST_MEAN = 1, ST_JIT = 3, ST_SPIKE = 5, ST_OFF = 6, ST_STRAG = 7 };

/* Fill out[B][n][R].  Returns 0, or -1 on bad arguments. */
int zl_generate(const zl_workload *w, int64_t *out) {
    if (!w || !out || w->n < 1 || w->R < 1 || w->B < 1) return -1;
    const int n = w->n, R = w->R;
    int n_strag = 0;
    if (w->straggler_frac > 0.0) n_strag = (int)ceil(w->straggler_frac * n - 1e-9);

#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t bp = 0; bp < (int64_t)w->B * n; ++bp) {
        const int b = (int)(bp / n), p = (int)(bp % n);
        const uint64_t seed = (uint64_t)(w->base_seed + b);
        double m;
        if (w->mean_kind == 1) m = (p < n / 2) ? w->mean_us : w->mean2_us;
        else m = exp(log(w->mean_us) + w->sigma * normal(seed, (uint64_t)p, 0, ST_MEAN));
        if (n_strag > 0) {
            /* worker p is a straggler when its hash ranks among the n_strag smallest */
            uint64_t mine = draw(seed, (uint64_t)p, 0, ST_STRAG);
            int rank = 0;
            for (int q = 0; q < n; ++q) {
                uint64_t other = draw(seed, (uint64_t)q, 0, ST_STRAG);
                if (other < mine || (other == mine && q < p)) ++rank;
            }
            if (rank < n_strag) m *= w->straggler_mult;
        }
        int64_t t = w->epoch_us;
        if (w->offset_max_us > 0.0)
            t += (int64_t)floor(unif01(draw(seed, (uint64_t)p, 0, ST_OFF)) * w->offset_max_us);
        int64_t *row = out + bp * R;
        for (int i = 0; i < R; ++i) {
            double dur = m * (1.0 + w->jitter * normal(seed, (uint64_t)p, (uint64_t)i + 1, ST_JIT));
            if (w->spike_prob > 0.0 &&
                unif01(draw(seed, (uint64_t)p, (uint64_t)i + 1, ST_SPIKE)) < w->spike_prob)
                dur *= w->spike_mult;
            long long d = llround(dur);
            if (d < 1) d = 1;
            t += (int64_t)d;
            row[i] = t;
        }
    }
    return 0;
}
