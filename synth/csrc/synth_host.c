/* Host twin (plain C, OpenMP) of the embedding generator in synth/graphs.py: the same integer recipe,
 * the same bits, only faster than numpy.  Inputs only: no arithmetic of the factorisation method. */
#include <stdint.h>
#include <string.h>

static inline uint64_t mix64(uint64_t z)
{
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}
static inline uint64_t hash2(uint64_t key, uint64_t a, uint64_t b) { return mix64(mix64(key ^ a) + b * 0x9E3779B97F4A7C15ull); }

#define NT_BITS 12
#define NT_FRAC_BITS 20

static inline float draw(uint64_t key, const int64_t *table, int64_t elem, double scale)
{
    const uint64_t h = hash2(key, (uint64_t)elem, 0);
    const int64_t cell = (int64_t)(h >> (64 - NT_BITS));
    const int64_t frac = (int64_t)((h >> (64 - NT_BITS - NT_FRAC_BITS)) & ((1ull << NT_FRAC_BITS) - 1));
    const int64_t t0 = table[cell], t1 = table[cell + 1];
    const int64_t v = t0 + (((t1 - t0) * frac) >> NT_FRAC_BITS);
    return (float)((double)v * scale);
}

static inline uint16_t f32_to_bf16_rne(float f)
{
    uint32_t b;
    memcpy(&b, &f, 4);
    return (uint16_t)((b + 0x7FFFu + ((b >> 16) & 1u)) >> 16);
}

/* rows[n_rows] (or NULL: rows row_begin .. row_begin + n_rows - 1) of a table with d columns; out is float32
 * (bf16 = 0) or uint16 bfloat16 bit patterns (bf16 = 1), n_rows x d; with as_f64 the same stored values widened to
 * double (exact), which is what the fp64 checker reads */
void synth_host_rows(uint64_t key, const int64_t *table, const int64_t *rows, int64_t row_begin, int64_t n_rows, int d,
                     double scale, int bf16, int as_f64, void *out)
{
#pragma omp parallel for schedule(static)
    for (int64_t k = 0; k < n_rows; ++k) {
        const int64_t r = rows ? rows[k] : row_begin + k;
        for (int c = 0; c < d; ++c) {
            const float f = draw(key, table, r * d + c, scale);
            if (as_f64) {
                float stored = f;
                if (bf16) {
                    const uint32_t b = (uint32_t)f32_to_bf16_rne(f) << 16;
                    memcpy(&stored, &b, 4);
                }
                ((double *)out)[k * d + c] = (double)stored;
            } else if (bf16) {
                ((uint16_t *)out)[k * d + c] = f32_to_bf16_rne(f);
            } else {
                ((float *)out)[k * d + c] = f;
            }
        }
    }
}
