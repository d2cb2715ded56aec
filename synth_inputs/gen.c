/*
 * Seeded synthetic inputs shared by the tests, the benchmark and the oracle
 * checks.  Holds none of the attention arithmetic: it only fills buffers with
 * reproducible bf16 bit patterns.
 *
 * Counter-based: element e of tensor (seed, tensor_id) depends on nothing but
 * (seed, tensor_id, e), so any slice of any tensor can be produced by any
 * number of threads with identical bits.
 *
 *   key   = mix(mix(seed) ^ (tensor_id * odd constant))
 *   bits  = mix(key ^ mix(pair index))           pair index = e / 2
 *   u1    = (bits 40..63 + 0.5) / 2^24  in (0,1],   u2 = bits 8..31 / 2^24   (single precision)
 *   z0,z1 = sqrt(-2 ln u1) * (cos, sin)(2 pi u2)   (Box-Muller), element e takes z_(e & 1)
 *   value = round-to-nearest-even bf16 of mult * z
 *
 * mix() is the SplitMix64 finaliser (Steele, Lea, Flood 2014).
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

static uint64_t mix(uint64_t x)
{
    x += 0x9E3779B97F4A7C15ull;
    x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
    x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
    return x ^ (x >> 31);
}

static uint64_t tensor_key(uint64_t seed, uint64_t tensor_id)
{
    return mix(mix(seed) ^ (tensor_id * 0xD1342543DE82EF95ull + 1ull));
}

static uint16_t f32_to_bf16_rne(float f)
{
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    u += 0x7FFFu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

/* 64 raw bits for counter c of a tensor; also used for integer draws (lengths). */
uint64_t synth_raw_bits(uint64_t seed, uint64_t tensor_id, uint64_t c)
{
    return mix(tensor_key(seed, tensor_id) ^ mix(c));
}

/* Fill out[0..count) with elements first .. first+count-1 of the tensor. */
void synth_normal_bf16(uint64_t seed, uint64_t tensor_id, double mult,
                       uint64_t first, uint64_t count, uint16_t *out)
{
    const uint64_t key = tensor_key(seed, tensor_id);
    const uint64_t p0 = first / 2, p1 = (first + count + 1) / 2;
    const float two_pi = 6.2831853071795864769f;
#pragma omp parallel for schedule(static)
    for (uint64_t p = p0; p < p1; ++p) {
        uint64_t bits = mix(key ^ mix(p));
        float u1 = ((float)(bits >> 40) + 0.5f) * (1.0f / 16777216.0f);
        float u2 = (float)((bits >> 8) & 0xFFFFFFull) * (1.0f / 16777216.0f);
        float r = sqrtf(-2.0f * logf(u1)) * (float)mult;
        float z0 = r * cosf(two_pi * u2), z1 = r * sinf(two_pi * u2);
        uint64_t e0 = 2 * p, e1 = 2 * p + 1;
        if (e0 >= first && e0 < first + count) out[e0 - first] = f32_to_bf16_rne(z0);
        if (e1 >= first && e1 < first + count) out[e1 - first] = f32_to_bf16_rne(z1);
    }
}
