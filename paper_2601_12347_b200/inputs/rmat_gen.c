/* Seeded R-MAT candidate-pair generator (input harness only).
 *
 * Holds none of the method's arithmetic: it only draws vertex pairs.  Each pair i is a pure
 * function of (seed, i), through a counter-based 64-bit mixer, so the output does not depend
 * on the thread count or on how the index range is split into calls.
 */
#include <stdint.h>

static inline uint64_t mix64(uint64_t z) {
    z += 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

/* Draw `count` pairs with indices first..first+count-1 on a 2^scale x 2^scale grid.
 * At each of the `scale` levels a quadrant is picked with probabilities a, b, c, 1-a-b-c
 * (top-left, top-right, bottom-left, bottom-right); top/bottom sets the next bit of u,
 * left/right the next bit of v. */
void rmat_pairs(uint64_t seed, uint64_t first, int64_t count, int scale,
                double a, double b, double c, int32_t* u_out, int32_t* v_out) {
    const double ab = a + b, abc = a + b + c;
    const uint64_t s0 = mix64(seed ^ 0xA5A5A5A5DEADBEEFull);
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < count; ++i) {
        uint64_t idx = first + (uint64_t)i;
        uint32_t u = 0, v = 0;
        for (int k = 0; k < scale; ++k) {
            uint64_t r = mix64(s0 ^ mix64(idx * 64ull + (uint64_t)k));
            double x = (double)(r >> 11) * (1.0 / 9007199254740992.0);
            int q = (x >= a) + (x >= ab) + (x >= abc);
            u = (u << 1) | (uint32_t)(q >> 1);
            v = (v << 1) | (uint32_t)(q & 1);
        }
        u_out[i] = (int32_t)u;
        v_out[i] = (int32_t)v;
    }
}
