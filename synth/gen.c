/*
 * Seeded synthetic-input generator (CPU side).
 *
 * This module makes INPUTS only: pseudo-random tensors that stand in for model
 * weights, context KV, drafter logits and token ids.  It holds none of the
 * verification method's arithmetic.  Everything is integer arithmetic followed
 * by at most one IEEE fp32 multiply, so any other implementation of the same
 * recipe (for instance a device fill kernel) yields the same bits.
 *
 * Recipe
 *   key(seed, tensor)   = mix(mix(seed) + tensor)
 *   word(key, c)        = mix(key + c * GAMMA)                 (64 random bits)
 *   normal(key, i)      = ((sum of the twelve 16-bit lanes of words 3i, 3i+1,
 *                          3i+2) - 6*65535) * (sigma / 65536)   (Irwin-Hall(12):
 *                          unit variance up to 1 - 2^-32, clipped at +-6 sigma)
 *   index(key, i, n)    = word(key, i) mod n
 *   unit(key, i)        = ((word(key, i) >> 40) + 0.5) * 2^-24  in (0, 1)
 * where mix is the splitmix64 finaliser.
 */
#include <stdint.h>
#include <stddef.h>
#include <string.h>

#define SYNTH_GAMMA 0x9E3779B97F4A7C15ull

static inline uint64_t synth_mix(uint64_t z)
{
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

static inline uint64_t synth_word(uint64_t key, uint64_t c)
{
    return synth_mix(key + c * SYNTH_GAMMA);
}

uint64_t synth_key(uint64_t seed, uint64_t tensor)
{
    return synth_mix(synth_mix(seed + SYNTH_GAMMA) + tensor * SYNTH_GAMMA + 1);
}

static inline int32_t synth_ih12(uint64_t key, uint64_t i)
{
    uint32_t s = 0;
    for (int j = 0; j < 3; ++j) {
        uint64_t w = synth_word(key, 3 * i + (uint64_t)j);
        s += (uint32_t)(w & 0xFFFF) + (uint32_t)((w >> 16) & 0xFFFF) +
             (uint32_t)((w >> 32) & 0xFFFF) + (uint32_t)(w >> 48);
    }
    return (int32_t)s - 6 * 65535;
}

static inline uint16_t synth_bf16_rne(float f)
{
    uint32_t u;
    memcpy(&u, &f, 4);
    u += 0x7FFFu + ((u >> 16) & 1u);   /* values are finite and far from overflow */
    return (uint16_t)(u >> 16);
}

/* out[i] = normal(key, first + i) * scale, fp32.  scale = sigma / 65536 as fp32. */
void synth_normal_f32(uint64_t key, uint64_t first, size_t n, float scale, float *out)
{
#pragma omp parallel for schedule(static)
    for (ptrdiff_t i = 0; i < (ptrdiff_t)n; ++i)
        out[i] = (float)synth_ih12(key, first + (uint64_t)i) * scale;
}

/* Same values rounded to bf16 (round to nearest even), stored as raw 16-bit words. */
void synth_normal_bf16(uint64_t key, uint64_t first, size_t n, float scale, uint16_t *out)
{
#pragma omp parallel for schedule(static)
    for (ptrdiff_t i = 0; i < (ptrdiff_t)n; ++i)
        out[i] = synth_bf16_rne((float)synth_ih12(key, first + (uint64_t)i) * scale);
}

/* out[i] = word(key, first + i) mod modulus, as int32. */
void synth_index_i32(uint64_t key, uint64_t first, size_t n, uint64_t modulus, int32_t *out)
{
#pragma omp parallel for schedule(static)
    for (ptrdiff_t i = 0; i < (ptrdiff_t)n; ++i)
        out[i] = (int32_t)(synth_word(key, first + (uint64_t)i) % modulus);
}

/* out[i] = unit(key, first + i): a uniform on (0,1), exact in fp32. */
void synth_unit_f32(uint64_t key, uint64_t first, size_t n, float *out)
{
#pragma omp parallel for schedule(static)
    for (ptrdiff_t i = 0; i < (ptrdiff_t)n; ++i)
        out[i] = ((float)(synth_word(key, first + (uint64_t)i) >> 40) + 0.5f) * 5.9604644775390625e-8f;
}
