/*
 * Counter-based synthetic tensor generator (inputs only; none of the
 * convolution's arithmetic lives here).  Element i of tensor `tid` under
 * `seed` is a pure function of (seed, tid, i): two 64-bit mixing hashes give
 * two uniforms in (0,1); a normal draw is Box-Muller on them.  Values are
 * produced in double, rounded to float, and stored as float or as bf16 bit
 * patterns (round to nearest even).
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

static inline uint64_t mix64(uint64_t z) {
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

static inline uint64_t stream_key(uint64_t seed, uint64_t tid, uint64_t lane) {
    return seed * 0x632BE59BD9B4E019ull + tid * 0xD1B54A32D192ED03ull + lane * 0x8CB92BA72F3D8DD7ull + 0x1234567ull;
}

static inline double u01(uint64_t key, uint64_t i) {
    const uint64_t z = mix64(mix64(i * 0x9E3779B97F4A7C15ull + key));
    return ((double)(z >> 11) + 0.5) * (1.0 / 9007199254740992.0);
}

static inline uint16_t f32_to_bf16_rne(float f) {
    uint32_t b;
    memcpy(&b, &f, 4);
    b += 0x7FFFu + ((b >> 16) & 1u);
    return (uint16_t)(b >> 16);
}

/* kind: 0 = uniform in [a, b), 1 = normal with mean 0 and standard deviation a.
 * dtype: 0 = float32 output, 1 = bf16 bit patterns (uint16) output. */
void synth_fill(void* out, int64_t start, int64_t count, int kind, double a, double b, int dtype, uint64_t seed,
                uint64_t tid) {
    const uint64_t k0 = stream_key(seed, tid, 0), k1 = stream_key(seed, tid, 1);
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < count; ++j) {
        const uint64_t i = (uint64_t)(start + j);
        double v;
        if (kind == 0) {
            v = a + (b - a) * u01(k0, i);
        } else {
            const double u1 = u01(k0, i), u2 = u01(k1, i);
            v = a * sqrt(-2.0 * log(u1)) * cos(6.283185307179586476925286766559 * u2);
        }
        const float f = (float)v;
        if (dtype == 1) ((uint16_t*)out)[j] = f32_to_bf16_rne(f);
        else ((float*)out)[j] = f;
    }
}
