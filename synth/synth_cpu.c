/*
 * Host build of the seeded synthetic generator (input generation only; see
 * synth_core.h).  Compiled with -ffp-contract=off so that every fp32 multiply/add
 * is rounded on its own, as on the device.
 */
#include <stddef.h>
#include <stdint.h>
#include <string.h>

#include "synth_core.h"

/* rank[v] in 1..V: a seeded Fisher-Yates shuffle of the identity */
void synth_permutation_rank(uint64_t seed, int32_t V, int32_t* rank_out) {
    for (int32_t v = 0; v < V; ++v) rank_out[v] = v + 1;
    uint64_t key = synth_row_key(seed, SYNTH_STREAM_PERM, 0u, 0u, 0u);
    for (int32_t i = V - 1; i > 0; --i) {
        uint64_t bits = synth_elem_bits(key, (uint32_t)i);
        /* multiply-shift reduction of the top 32 bits to [0, i] */
        uint32_t j = (uint32_t)(((bits >> 32) * (uint64_t)(i + 1)) >> 32);
        int32_t t = rank_out[i];
        rank_out[i] = rank_out[j];
        rank_out[j] = t;
    }
}

/*
 * Generate n_rows logit rows.  Row r is row (b[r], k[r]) of `round`.
 *   kind  : 0 = draft row, 1 = target row (same base + tau * second Gaussian)
 *   dtype : 0 = bf16 bits (uint16), 1 = fp32
 *   out   : row r starts at out + r * row_stride elements
 */
void synth_rows_cpu(int32_t kind, uint64_t seed, uint32_t round, int64_t n_rows,
                    const int32_t* b, const int32_t* k, const float* s, const float* tau,
                    int32_t V, const float* gauss, const float* lnrank, int32_t dtype,
                    void* out, int64_t row_stride) {
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t r = 0; r < n_rows; ++r) {
        uint64_t key = synth_row_key(seed, SYNTH_STREAM_LOGITS, round, (uint32_t)b[r],
                                     (uint32_t)k[r]);
        float sr = s[r];
        float tr = tau ? tau[r] : 0.0f;
        for (int32_t v = 0; v < V; ++v) {
            uint64_t bits = synth_elem_bits(key, (uint32_t)v);
            float z = kind == 0 ? synth_draft_f32(bits, sr, gauss, lnrank[v])
                                : synth_target_f32(bits, sr, tr, gauss, lnrank[v]);
            if (dtype == 0)
                ((uint16_t*)out)[r * row_stride + v] = synth_f32_to_bf16_rne(z);
            else
                ((float*)out)[r * row_stride + v] = z;
        }
    }
}

/* u[b * n + j] for b in [0,B), j in [0,n): uniforms in [0,1) with 24 random bits */
void synth_uniforms_cpu(uint64_t seed, uint32_t substream, uint32_t round, int32_t B,
                        int32_t n, float* out) {
    for (int32_t b = 0; b < B; ++b) {
        uint64_t key = synth_row_key(seed, SYNTH_STREAM_UNIFORM, round, (uint32_t)b, substream);
        for (int32_t j = 0; j < n; ++j)
            out[(size_t)b * n + j] = synth_uniform24(synth_elem_bits(key, (uint32_t)j));
    }
}

/* 64 raw parameter bits for (round, b, k, j): the Python side maps them to s and tau */
void synth_param_bits(uint64_t seed, uint32_t round, int32_t B, int32_t K, uint32_t j,
                      uint64_t* out) {
    for (int32_t b = 0; b < B; ++b)
        for (int32_t k = 0; k < K; ++k) {
            uint64_t key = synth_row_key(seed, SYNTH_STREAM_PARAM, round, (uint32_t)b, (uint32_t)k);
            out[(size_t)b * K + k] = synth_elem_bits(key, j);
        }
}
