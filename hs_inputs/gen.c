/*
 * Seeded synthetic-input generator (counter based, stateless).
 *
 * This file only produces random bytes: uniform words, normal bf16 weights and
 * exactly representable uniform bf16 fill.  It contains none of the decoding
 * method's arithmetic.  The same bytes are handed to the CUDA library and to
 * the CPU oracle, which otherwise share nothing.
 *
 * Element idx of tensor tid under seed is a pure function of (seed, tid, idx):
 *   word(seed, tid, idx) = fin(base(seed, tid) + (idx + 1) * GAMMA)
 * with fin() the 64-bit splitmix finaliser, so any slice can be generated
 * independently and in parallel.
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

#define GAMMA 0x9E3779B97F4A7C15ull

static inline uint64_t fin64(uint64_t z) {
    z ^= z >> 30; z *= 0xBF58476D1CE4E5B9ull;
    z ^= z >> 27; z *= 0x94D049BB133111EBull;
    z ^= z >> 31;
    return z;
}

uint64_t hsin_base(uint64_t seed, uint64_t tid) {
    uint64_t s = fin64(seed + GAMMA);
    return fin64((s ^ (tid * 0xD1B54A32D192ED03ull)) + GAMMA);
}

static inline uint64_t word_at(uint64_t base, uint64_t idx) {
    return fin64(base + (idx + 1) * GAMMA);
}

/* raw 64-bit words, idx = first .. first+n-1 */
void hsin_words(uint64_t *out, int64_t n, uint64_t seed, uint64_t tid, int64_t first) {
    uint64_t base = hsin_base(seed, tid);
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) out[i] = word_at(base, (uint64_t)(first + i));
}

/* uniform in (0,1): ((w >> 11) + 0.5) / 2^53 */
static inline double u01(uint64_t w) { return ((double)(w >> 11) + 0.5) * (1.0 / 9007199254740992.0); }

static inline uint16_t f32_to_bf16_rne(float f) {
    uint32_t u; memcpy(&u, &f, 4);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7FFFu + lsb;
    return (uint16_t)(u >> 16);
}

/* N(0, std^2) rounded to bf16.  Elements 2j and 2j+1 form one Box-Muller pair
 * driven by words 2j (radius) and 2j+1 (angle).  first must be even. */
void hsin_normal_bf16(uint16_t *out, int64_t n, uint64_t seed, uint64_t tid, double std, int64_t first) {
    uint64_t base = hsin_base(seed, tid);
    int64_t npair = (n + 1) / 2;
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < npair; ++j) {
        uint64_t i0 = (uint64_t)first + 2 * (uint64_t)j;
        double u1 = u01(word_at(base, i0));
        double u2 = u01(word_at(base, i0 + 1));
        double r = sqrt(-2.0 * log(u1)) * std;
        double a = 6.283185307179586476925286766559 * u2;
        out[2 * j] = f32_to_bf16_rne((float)(r * cos(a)));
        if (2 * j + 1 < n) out[2 * j + 1] = f32_to_bf16_rne((float)(r * sin(a)));
    }
}

/* Uniform on a 2^16-point grid in [-scale, scale): value = (int16)(w >> 48) / 2^15 * scale,
 * then RNE to bf16.  Integer arithmetic up to the final exact scaling, so any
 * platform reproduces it bit for bit.  Used for injected contexts (KV rows, states). */
void hsin_grid_bf16(uint16_t *out, int64_t n, uint64_t seed, uint64_t tid, float scale, int64_t first) {
    uint64_t base = hsin_base(seed, tid);
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        int16_t v = (int16_t)(word_at(base, (uint64_t)(first + i)) >> 48);
        out[i] = f32_to_bf16_rne((float)v * (1.0f / 32768.0f) * scale);
    }
}

void hsin_grid_f32(float *out, int64_t n, uint64_t seed, uint64_t tid, float scale, int64_t first) {
    uint64_t base = hsin_base(seed, tid);
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        int16_t v = (int16_t)(word_at(base, (uint64_t)(first + i)) >> 48);
        out[i] = (float)v * (1.0f / 32768.0f) * scale;
    }
}
