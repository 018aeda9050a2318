/* Native helper of datagen.py: fills large ternary tensors with the module's counter-based
 * generator, many times faster than the numpy formulation and bit for bit the same values.
 * It draws inputs only; it holds none of the method's arithmetic.
 *
 *   z = mix64((seed XOR stream * 0xD1B54A32D192ED03) + (i + 1) * 0x9E3779B97F4A7C15)  (mod 2^64)
 *   u = (z >> 11) * 2^-53;   trit = 0 if u < zero_density, +1 if u < zero_density + (1 - zero_density) / 2, else -1
 */
#include <stdint.h>

static uint64_t mix64(uint64_t z) {
    z ^= z >> 30;
    z *= 0xBF58476D1CE4E5B9ull;
    z ^= z >> 27;
    z *= 0x94D049BB133111EBull;
    z ^= z >> 31;
    return z;
}

void datagen_fill_trits(uint64_t seed, uint64_t stream, uint64_t start, uint64_t count, double zero_density, int8_t *out) {
    const uint64_t base = seed ^ (stream * 0xD1B54A32D192ED03ull);
    const double half = zero_density + (1.0 - zero_density) / 2.0;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < (int64_t)count; ++i) {
        const uint64_t z = mix64(base + (start + (uint64_t)i + 1) * 0x9E3779B97F4A7C15ull);
        const double u = (double)(z >> 11) * (1.0 / 9007199254740992.0);
        out[i] = (int8_t)(u < zero_density ? 0 : (u < half ? 1 : -1));
    }
}
