/*
 * Seeded synthetic logit generator: the arithmetic shared by the host (C) and the
 * device (CUDA) builds of the generator.
 *
 * This is INPUT-GENERATION code only.  It holds none of the AdaSD method's
 * arithmetic (no softmax, entropy, divergence, sampling or threshold logic); it is
 * used by the test/bench harness to feed identical inputs to the CUDA library and
 * to the CPU oracle.
 *
 * Recipe (Zipf-offset Gaussian logits):
 *     zd32[v] = s * g1(v) - lnrank[v]            (draft row)
 *     zt32[v] = zd32[v] + tau * g2(v)            (target row on the same base)
 * with every multiply/add a separately rounded fp32 operation (no FMA contraction),
 * g1/g2 looked up in a 65536-entry table of standard-normal quantiles with a 16-bit
 * index taken from a 64-bit integer mix of (row key, v), and the result rounded
 * to bf16 (round-to-nearest-even) or kept as fp32.  Because every step is either an
 * integer operation, a table lookup or a single correctly rounded fp32 operation,
 * the host and the device produce bit-identical rows.
 */
#ifndef SYNTH_CORE_H
#define SYNTH_CORE_H

#include <stdint.h>

#if defined(__CUDACC__)
#define SYNTH_HD __host__ __device__ __forceinline__
#else
#define SYNTH_HD static inline
#endif

#define SYNTH_GAUSS_BITS 16
#define SYNTH_GAUSS_N (1u << SYNTH_GAUSS_BITS)

/* stream ids: which family of random numbers a key belongs to */
#define SYNTH_STREAM_LOGITS 1u   /* per-element Gaussian indices of a logit row */
#define SYNTH_STREAM_UNIFORM 2u  /* uniforms handed to the library / oracle */
#define SYNTH_STREAM_PARAM 3u    /* per-row scale s and noise tau */
#define SYNTH_STREAM_PERM 4u     /* vocabulary rank permutation */

/* splitmix64 finaliser: a bijective 64-bit mixer */
SYNTH_HD uint64_t synth_mix64(uint64_t x) {
    x ^= x >> 30;
    x *= 0xBF58476D1CE4E5B9ull;
    x ^= x >> 27;
    x *= 0x94D049BB133111EBull;
    x ^= x >> 31;
    return x;
}

/* key of one logit row / one family of draws: (seed, stream, round, b, k) */
SYNTH_HD uint64_t synth_row_key(uint64_t seed, uint32_t stream, uint32_t round,
                                uint32_t b, uint32_t k) {
    uint64_t h = synth_mix64(seed + 0x9E3779B97F4A7C15ull * (uint64_t)(stream + 1u));
    h = synth_mix64(h ^ ((uint64_t)round * 0xD1B54A32D192ED03ull + 0x2545F4914F6CDD1Dull));
    h = synth_mix64(h ^ ((uint64_t)b * 0x9E3779B97F4A7C15ull + 0x632BE59BD9B4E019ull));
    h = synth_mix64(h ^ ((uint64_t)k * 0xC2B2AE3D27D4EB4Full + 0x165667B19E3779F9ull));
    return h;
}

/* 64 mixed bits for element v of the row with this key */
SYNTH_HD uint64_t synth_elem_bits(uint64_t row_key, uint32_t v) {
    return synth_mix64(row_key + (uint64_t)v * 0x9E3779B97F4A7C15ull);
}

/* uniform in [0,1) with 24 random bits: exactly representable in fp32 */
SYNTH_HD float synth_uniform24(uint64_t bits) {
    return (float)(uint32_t)(bits >> 40) * (1.0f / 16777216.0f);
}

/* fp32 -> bf16 bits, round to nearest even (finite inputs; NaN kept quiet) */
SYNTH_HD uint16_t synth_f32_to_bf16_rne(float f) {
    union { float f; uint32_t u; } c;
    c.f = f;
    uint32_t u = c.u;
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) return (uint16_t)((u >> 16) | 0x0040u);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7FFFu + lsb;
    return (uint16_t)(u >> 16);
}

#if defined(__CUDA_ARCH__)
#define SYNTH_FMUL(a, b) __fmul_rn((a), (b))
#define SYNTH_FADD(a, b) __fadd_rn((a), (b))
#define SYNTH_FSUB(a, b) __fsub_rn((a), (b))
#else
/* the host build is compiled with -ffp-contract=off, so these stay separate ops */
#define SYNTH_FMUL(a, b) ((float)((float)(a) * (float)(b)))
#define SYNTH_FADD(a, b) ((float)((float)(a) + (float)(b)))
#define SYNTH_FSUB(a, b) ((float)((float)(a) - (float)(b)))
#endif

/* draft logit (fp32, before any bf16 rounding) */
SYNTH_HD float synth_draft_f32(uint64_t bits, float s, const float* gauss, float lnrank_v) {
    float g1 = gauss[bits & (SYNTH_GAUSS_N - 1u)];
    return SYNTH_FSUB(SYNTH_FMUL(s, g1), lnrank_v);
}

/* target logit (fp32): draft base + tau * independent Gaussian */
SYNTH_HD float synth_target_f32(uint64_t bits, float s, float tau, const float* gauss,
                                float lnrank_v) {
    float zd = synth_draft_f32(bits, s, gauss, lnrank_v);
    float g2 = gauss[(bits >> 16) & (SYNTH_GAUSS_N - 1u)];
    return SYNTH_FADD(zd, SYNTH_FMUL(tau, g2));
}

#endif /* SYNTH_CORE_H */
