/*
 * Seeded synthetic-input generator (data only; holds none of the method's arithmetic).
 *
 * Every value depends only on (seed, tensor_id, element index): a counter-based generator,
 * so a tensor can be produced in any chunking, on any number of threads, and always comes
 * out bit-identical.  No transcendental function is used:
 *   - a normal deviate is an Irwin-Hall sum of twelve 16-bit uniforms taken from three
 *     splitmix64-style hashes, centred and scaled with exact integer / power-of-two
 *     arithmetic, then multiplied once by the requested standard deviation in fp32 and
 *     rounded once (nearest-even) to bf16;
 *   - token ids are a hash reduced modulo the vocabulary, re-drawn while they hit one of
 *     two excluded ids.
 *
 * Build: gcc -O3 -fopenmp -shared -fPIC gen.c -o libodb_synth.so
 */
#include <stdint.h>
#include <string.h>

static inline uint64_t mix64(uint64_t z) {
    z += 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

static inline uint64_t key_of(uint64_t seed, uint64_t tensor_id) {
    return mix64(mix64(seed) ^ (tensor_id * 0xD6E8FEB86659FD93ull));
}

static inline uint16_t f32_to_bf16_rne(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    u += 0x7FFFu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

static inline int32_t sum4x16(uint64_t h) {
    return (int32_t)(h & 0xFFFF) + (int32_t)((h >> 16) & 0xFFFF) +
           (int32_t)((h >> 32) & 0xFFFF) + (int32_t)(h >> 48);
}

/* out[i] = bf16( std * z(seed, tensor_id, offset + i) ),  i in [0, n) */
void synth_normal_bf16(uint64_t seed, uint64_t tensor_id, uint64_t offset, uint64_t n,
                       float std, uint16_t* out) {
    const uint64_t key = key_of(seed, tensor_id);
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < (int64_t)n; ++i) {
        const uint64_t c = (offset + (uint64_t)i) * 3ull;
        const int32_t s = sum4x16(mix64(key ^ mix64(c))) + sum4x16(mix64(key ^ mix64(c + 1))) +
                          sum4x16(mix64(key ^ mix64(c + 2)));
        /* twelve uniforms on {0..65535}: mean 12*32767.5 = 393210, variance 12*(65536^2-1)/12 */
        const float z = (float)(s - 393210) * (1.0f / 65536.0f);
        out[i] = f32_to_bf16_rne(z * std);
    }
}

/* out[i] = id in [0, vocab) different from excl_a and excl_b */
void synth_tokens(uint64_t seed, uint64_t stream_id, uint64_t n, int32_t vocab, int32_t excl_a,
                  int32_t excl_b, int32_t* out) {
    const uint64_t key = key_of(seed, stream_id ^ 0x746F6B656E73ull);
    for (uint64_t i = 0; i < n; ++i) {
        uint64_t c = i << 8;
        int32_t t;
        do {
            t = (int32_t)(mix64(key ^ mix64(c)) % (uint64_t)vocab);
            ++c;
        } while (t == excl_a || t == excl_b);
        out[i] = t;
    }
}

/* out[i] = uniform in [0,1) with 24 bits, for seeded schedules (lengths, test logits) */
void synth_uniform_f32(uint64_t seed, uint64_t stream_id, uint64_t n, float* out) {
    const uint64_t key = key_of(seed, stream_id ^ 0x756E69666F726Dull);
    for (uint64_t i = 0; i < n; ++i)
        out[i] = (float)(mix64(key ^ mix64(i)) >> 40) * (1.0f / 16777216.0f);
}
