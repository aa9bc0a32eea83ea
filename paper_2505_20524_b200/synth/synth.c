/*
 * Seeded synthetic input generator (serves the tests, the benchmark and the oracle alike).
 * Holds none of the method's arithmetic: it only draws N(0, std) values from a counter-based
 * generator, applies the outlier edits the workload recipes ask for, and rounds to BF16 bits.
 *
 * elements 2j and 2j+1 of tensor `tid` under `seed` share one Box-Muller pair:
 *   u1, u2 = uniform(splitmix64(key + 2j)), uniform(splitmix64(key + 2j + 1)),
 *   key    = splitmix64(seed * 0x9E3779B97F4A7C15 + tid)
 *   z      = sqrt(-2 ln u1) * cos(2 pi u2)  for element 2j,  ... * sin(2 pi u2)  for element 2j+1   (double)
 *   v      = z * std, times col_factor if the column is an outlier column,
 *            or replaced by +-elem_value with probability elem_prob (third draw)
 *   out    = BF16(round-to-nearest-even(float(v)))
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

static inline uint64_t splitmix64(uint64_t x)
{
    x += 0x9E3779B97F4A7C15ull;
    x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
    x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
    return x ^ (x >> 31);
}

static inline double u01(uint64_t r) { return ((double)(r >> 11) + 0.5) * (1.0 / 9007199254740992.0); }

static inline uint16_t f32_to_bf16_rne(float f)
{
    uint32_t u;
    memcpy(&u, &f, 4);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7FFFu + lsb;
    return (uint16_t)(u >> 16);
}

uint64_t synth_hash(uint64_t x) { return splitmix64(x); }

void synth_fill_bf16(uint16_t *out, int64_t rows, int64_t cols, uint64_t seed, uint64_t tid, double std,
                     const uint8_t *col_is_outlier /* nullable, [cols] */, double col_factor,
                     double elem_prob, double elem_value)
{
    const uint64_t key = splitmix64(seed * 0x9E3779B97F4A7C15ull + tid);
    const uint64_t key2 = splitmix64(key ^ 0xD1B54A32D192ED03ull);
    const int64_t n = rows * cols;
#pragma omp parallel for schedule(static)
    for (int64_t ii = 0; ii < n; ++ii) {
        {
            const uint64_t i = (uint64_t)ii;
            const int64_t c = ii % cols;
            const uint64_t j = i >> 1;
            const double u1 = u01(splitmix64(key + 2 * j));
            const double u2 = u01(splitmix64(key + 2 * j + 1));
            const double ang = 6.283185307179586476925 * u2;
            double v = sqrt(-2.0 * log(u1)) * ((i & 1) ? sin(ang) : cos(ang)) * std;
            if (col_is_outlier && col_is_outlier[c]) v *= col_factor;
            if (elem_prob > 0.0) {
                const uint64_t r3 = splitmix64(key2 + i);
                if (u01(r3) < elem_prob) v = (r3 & 1u) ? elem_value : -elem_value;
            }
            out[i] = f32_to_bf16_rne((float)v);
        }
    }
}

/* Plain BF16 rounding of float32 values (used to hand identical bytes of a derived tensor to both sides). */
void synth_f32_to_bf16(const float *in, int64_t n, uint16_t *out)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) out[i] = f32_to_bf16_rne(in[i]);
}
