/* Plain C twin of the synthetic input generator (harness only), for CPU runs over many millions of
 * elements where the numpy version is too slow.  Same definition as inputs/gen.py, bit for bit:
 * out[j] = cast( base + sigma_k * z(key, lo + j) ), z = float(sum of eight 16-bit lanes - 262140) * INV_STD,
 * every floating-point step rounded on its own (compile with -ffp-contract=off). */
#include <stdint.h>
#include <string.h>

static inline uint64_t mix64(uint64_t z) {
    z ^= z >> 30;
    z *= 0xBF58476D1CE4E5B9ull;
    z ^= z >> 27;
    z *= 0x94D049BB133111EBull;
    z ^= z >> 31;
    return z;
}

static inline int lane_sum(uint64_t h) {
    return (int)(h & 0xFFFF) + (int)((h >> 16) & 0xFFFF) + (int)((h >> 32) & 0xFFFF) + (int)(h >> 48);
}

static inline float unit_noise(uint64_t key, uint64_t idx) {
    const uint64_t x = key + idx * 0x9E3779B97F4A7C15ull;
    const int s = lane_sum(mix64(x)) + lane_sum(mix64(x ^ 0xD1B54A32D192ED03ull));
    return (float)(s - 262140) * 0x1.3988e2p-16f;
}

static inline float bf16_widen(uint16_t h) {
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

static inline uint16_t bf16_narrow(float f) { /* round to nearest even, finite inputs */
    uint32_t u;
    memcpy(&u, &f, 4);
    u += 0x7FFFu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

/* dtype 0 = fp32, 1 = bf16 patterns.  in may be NULL (then base_tbl[k] is the base).  tensor_off has
 * n_tensors + 1 entries; out/in cover the global indices [lo, lo + n).  The range is walked tensor by tensor so
 * that the inner loops have constant per-tensor factors and no control flow (they vectorise). */
void halos_synth_fill_cpu(void* out, const void* in, int dtype, const float* base_tbl, const float* sigma_tbl,
                          const uint64_t* tensor_off, uint32_t n_tensors, uint64_t key, uint64_t lo, uint64_t n) {
    uint32_t k = 0;
    while (k + 1 < n_tensors && tensor_off[k + 1] <= lo) ++k; /* last tensor that starts at or before lo */
    uint64_t j = 0;
    while (j < n) {
        const uint64_t g0 = lo + j;
        while (k + 1 < n_tensors && tensor_off[k + 1] <= g0) ++k;
        uint64_t seg = n - j; /* elements of [lo + j, lo + n) that belong to tensor k */
        if (k + 1 < n_tensors && tensor_off[k + 1] - g0 < seg) seg = tensor_off[k + 1] - g0;
        const float sigma = sigma_tbl[k], base_k = base_tbl[k];
        if (dtype == 0) {
            float* o = (float*)out + j;
            const float* src = in ? (const float*)in + j : 0;
            if (src) {
                for (uint64_t i = 0; i < seg; ++i) {
                    const float prod = sigma * unit_noise(key, g0 + i);
                    o[i] = src[i] + prod;
                }
            } else {
                for (uint64_t i = 0; i < seg; ++i) {
                    const float prod = sigma * unit_noise(key, g0 + i);
                    o[i] = base_k + prod;
                }
            }
        } else {
            uint16_t* o = (uint16_t*)out + j;
            const uint16_t* src = in ? (const uint16_t*)in + j : 0;
            for (uint64_t i = 0; i < seg; ++i) {
                const float prod = sigma * unit_noise(key, g0 + i);
                const float base = src ? bf16_widen(src[i]) : base_k;
                o[i] = bf16_narrow(base + prod);
            }
        }
        j += seg;
    }
}
