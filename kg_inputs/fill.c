/* Bulk host fill for the counter-based synthetic tensor generator (see synth.py for the
 * definition).  Input-generation only: nothing of the decode method lives here.
 * Build: gcc -O3 -fopenmp -shared -fPIC fill.c -o libkg_inputs_fill.so
 */
#include <stdint.h>
#include <string.h>

static inline uint64_t mix64(uint64_t z) {
    z += 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

static inline int32_t byte_sum(uint64_t u) {
    int32_t s = 0;
    for (int b = 0; b < 8; ++b) s += (int32_t)((u >> (8 * b)) & 0xFFu);
    return s - 1020;
}

static inline float bf16_rne(float x) {
    uint32_t bits;
    memcpy(&bits, &x, 4);
    uint32_t lsb = (bits >> 16) & 1u;
    bits = (bits + 0x7FFFu + lsb) & 0xFFFF0000u;
    memcpy(&x, &bits, 4);
    return x;
}

/* out[i] = value of element (start + i) of the stream whose base is `base`. */
void kgi_fill_f32(float* out, uint64_t base, uint64_t start, uint64_t count, float scale, int bf16) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < (int64_t)count; ++i) {
        uint64_t u = mix64(base + start + (uint64_t)i);
        float x = (float)byte_sum(u) * scale;
        out[i] = bf16 ? bf16_rne(x) : x;
    }
}
