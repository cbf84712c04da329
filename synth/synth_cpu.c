/*
 * Seeded synthetic-input generator (CPU).  Input generation only: nothing in this
 * file is part of the decoding method.  Both the CPU oracle and the CUDA library
 * receive the tensors produced here, so they see identical bits.
 *
 * Recipe for element `i` of tensor `tensor_id` under `seed`:
 *   group g = i / 8;  Philox4x32-10(counter = (g_lo, g_hi, tensor_id, TAG),
 *   key = (seed_lo, seed_hi)) gives four 32-bit words = eight 16-bit lanes;
 *   lane (i % 8) = word[(i%8)/2] low half (even lane) or high half (odd lane);
 *   value = (scale * Z[lane16]) * scale2, Z = inverse-normal table of 65536 fp32 entries
 *   handed in by the caller; two fp32 multiplies; bf16 output rounds to nearest even.
 *
 * Philox4x32-10 follows its published definition (Salmon, Moraes, Dror, Shaw,
 * "Parallel random numbers: as easy as 1, 2, 3", SC'11).
 */
#include <stdint.h>
#include <string.h>

#define SYNTH_TAG 0x53594E54u /* domain tag in counter word 3 */

static inline void philox4x32_10(uint32_t c[4], uint32_t k0, uint32_t k1)
{
    for (int r = 0; r < 10; ++r) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c[0];
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c[2];
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c[1] ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c[3] ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c[0] = n0; c[1] = n1; c[2] = n2; c[3] = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
}

static inline uint16_t f32_to_bf16_rne(float f)
{
    uint32_t u;
    memcpy(&u, &f, 4);
    u += 0x7FFFu + ((u >> 16) & 1u); /* finite inputs only */
    return (uint16_t)(u >> 16);
}

/* Raw Philox block, exported so the Python side can cross-check its scalar version. */
void synth_philox(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c[4] = {ctr[0], ctr[1], ctr[2], ctr[3]};
    philox4x32_10(c, key[0], key[1]);
    memcpy(out, c, 16);
}

/*
 * Fill `n` elements starting at flat index `first` of the tensor.
 * dtype: 0 = fp32 output, 1 = bf16 output (uint16 storage).
 */
void synth_fill(void* out, int64_t first, int64_t n, uint64_t seed, uint32_t tensor_id,
                float scale, float scale2, const float* Z, int dtype)
{
    const uint32_t k0 = (uint32_t)seed, k1 = (uint32_t)(seed >> 32);
    const int64_t g_begin = first / 8;
    const int64_t g_end = (first + n + 7) / 8;
    float* of = (float*)out;
    uint16_t* ob = (uint16_t*)out;
#pragma omp parallel for schedule(static)
    for (int64_t g = g_begin; g < g_end; ++g) {
        uint32_t c[4] = {(uint32_t)g, (uint32_t)((uint64_t)g >> 32), tensor_id, SYNTH_TAG};
        philox4x32_10(c, k0, k1);
        for (int lane = 0; lane < 8; ++lane) {
            int64_t i = g * 8 + lane;
            if (i < first || i >= first + n) continue;
            uint32_t w = c[lane >> 1];
            uint32_t h = (lane & 1) ? (w >> 16) : (w & 0xFFFFu);
            float v = (scale * Z[h]) * scale2; /* two fp32 multiplies, in this order */
            if (dtype == 0) of[i - first] = v;
            else ob[i - first] = f32_to_bf16_rne(v);
        }
    }
}
