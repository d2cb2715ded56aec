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
 *   u1    = (high 32 bits + 0.5) / 2^32  in (0,1),   u2 = low 32 bits / 2^32
 *   z0,z1 = sqrt(-2 ln u1) * (cos, sin)(2 pi u2)   (Box-Muller), element e takes z_(e & 1)
 *   value = round-to-nearest-even bf16 of (float)(mult * z)
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
    const double two_pi = 6.283185307179586476925286766559;
#pragma omp parallel for schedule(static)
    for (uint64_t p = p0; p < p1; ++p) {
        uint64_t bits = mix(key ^ mix(p));
        double u1 = ((double)(bits >> 32) + 0.5) * (1.0 / 4294967296.0);
        double u2 = (double)(bits & 0xFFFFFFFFull) * (1.0 / 4294967296.0);
        double r = sqrt(-2.0 * log(u1));
        double z0 = r * cos(two_pi * u2), z1 = r * sin(two_pi * u2);
        uint64_t e0 = 2 * p, e1 = 2 * p + 1;
        if (e0 >= first && e0 < first + count) out[e0 - first] = f32_to_bf16_rne((float)(mult * z0));
        if (e1 >= first && e1 < first + count) out[e1 - first] = f32_to_bf16_rne((float)(mult * z1));
    }
}
