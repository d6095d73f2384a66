/*
 * Seeded synthetic value generator shared by the CPU oracle's tests and the GPU
 * tests/bench.  It holds none of the averaging method's arithmetic: it only
 * fills host fp32 buffers with reproducible random values.
 *
 * Generator: Philox4x32-10 (Salmon, Moraes, Dror, Shaw, "Parallel random numbers:
 * as easy as 1, 2, 3", SC'11), written from the published round function:
 *     (c0,c1,c2,c3) -> (hi(M1*c2)^c1^k0, lo(M1*c2), hi(M0*c0)^c3^k1, lo(M0*c0))
 * with key schedule k0 += W0, k1 += W1 each round.  It is counter based, so the
 * value at (seed, purpose, worker, layer, index) does not depend on the order or
 * the number of threads used to fill a buffer.
 *
 * Counter layout:  c0,c1 = 64-bit block index inside the (worker, layer) stream,
 *                  c2 = worker, c3 = layer.      Key: k0 = seed, k1 = purpose.
 * One block gives four 32-bit words -> two Box-Muller pairs -> four N(0,1) draws.
 */
#include <math.h>
#include <stdint.h>

#define PHILOX_M0 0xD2511F53u
#define PHILOX_M1 0xCD9E8D57u
#define PHILOX_W0 0x9E3779B9u
#define PHILOX_W1 0xBB67AE85u

static inline void philox4x32_10(uint32_t c[4], uint32_t k0, uint32_t k1)
{
    for (int r = 0; r < 10; ++r) {
        uint64_t p0 = (uint64_t)PHILOX_M0 * c[0];
        uint64_t p1 = (uint64_t)PHILOX_M1 * c[2];
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c[1] ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c[3] ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c[0] = n0; c[1] = n1; c[2] = n2; c[3] = n3;
        k0 += PHILOX_W0;
        k1 += PHILOX_W1;
    }
}

/* Raw block, exported so that the tests can check the published known answers. */
void synth_philox_block(const uint32_t counter[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c[4] = {counter[0], counter[1], counter[2], counter[3]};
    philox4x32_10(c, key[0], key[1]);
    out[0] = c[0]; out[1] = c[1]; out[2] = c[2]; out[3] = c[3];
}

/* u in (0,1): the 32-bit word's bucket midpoint, never 0 or 1. */
static inline double u01(uint32_t w) { return ((double)w + 0.5) * (1.0 / 4294967296.0); }

static inline void normal4(uint64_t block, uint32_t seed, uint32_t purpose,
                           uint32_t worker, uint32_t layer, double z[4])
{
    uint32_t c[4] = {(uint32_t)block, (uint32_t)(block >> 32), worker, layer};
    philox4x32_10(c, seed, purpose);
    const double two_pi = 6.283185307179586476925286766559;
    double r0 = sqrt(-2.0 * log(u01(c[0])));
    double r1 = sqrt(-2.0 * log(u01(c[2])));
    double a0 = two_pi * u01(c[1]);
    double a1 = two_pi * u01(c[3]);
    z[0] = r0 * cos(a0); z[1] = r0 * sin(a0);
    z[2] = r1 * cos(a1); z[3] = r1 * sin(a1);
}

/* out[i] = (base ? base[i] : 0) + mean + std * z_i,  z_i ~ N(0,1), i in [0,n). */
void synth_fill_normal(float *out, const float *base, int64_t n, double mean, double std,
                       uint32_t seed, uint32_t purpose, uint32_t worker, uint32_t layer)
{
    int64_t nblocks = (n + 3) / 4;
#pragma omp parallel for schedule(static)
    for (int64_t b = 0; b < nblocks; ++b) {
        double z[4];
        normal4((uint64_t)b, seed, purpose, worker, layer, z);
        int64_t i0 = 4 * b;
        int lim = (n - i0 < 4) ? (int)(n - i0) : 4;
        for (int t = 0; t < lim; ++t) {
            double v = mean + std * z[t];
            if (base) v += (double)base[i0 + t];
            out[i0 + t] = (float)v;
        }
    }
}

/* out[i] = scale * Z / sqrt(V/3), Z ~ N(0,1), V = sum of three squared N(0,1): Student-t, nu = 3.
 * One Philox block per element (z[0] is Z; z[1..3] make V). */
void synth_fill_student_t3(float *out, int64_t n, double scale,
                           uint32_t seed, uint32_t purpose, uint32_t worker, uint32_t layer)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        double z[4];
        normal4((uint64_t)i, seed, purpose, worker, layer, z);
        double v = z[1] * z[1] + z[2] * z[2] + z[3] * z[3];
        out[i] = (float)(scale * z[0] / sqrt(v / 3.0));
    }
}

/* out[i] in (0,1), i in [0,n): uniform scalars (used for the per-(worker, layer) log-uniform sigmas). */
void synth_fill_uniform(double *out, int64_t n, uint32_t seed, uint32_t purpose,
                        uint32_t worker, uint32_t layer)
{
    for (int64_t b = 0; b < (n + 3) / 4; ++b) {
        uint32_t c[4] = {(uint32_t)b, (uint32_t)((uint64_t)b >> 32), worker, layer};
        philox4x32_10(c, seed, purpose);
        for (int t = 0; t < 4 && 4 * b + t < n; ++t) out[4 * b + t] = u01(c[t]);
    }
}

/* out[i] *= factor */
void synth_scale(float *out, int64_t n, double factor)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) out[i] = (float)((double)out[i] * factor);
}
