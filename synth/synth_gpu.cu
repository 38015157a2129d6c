/*
 * Device build of the seeded synthetic generator (input generation only; see
 * synth_core.h).  Harness code: it feeds the library during tests and benchmarks
 * and is not part of the library itself.  Rows it writes are bit-identical to the
 * host generator's.
 */
#include <cuda_runtime.h>
#include <stdint.h>

#include "synth_core.h"

namespace {

template <int KIND, int DTYPE>
__global__ void synth_rows_kernel(uint64_t seed, uint32_t round, const uint32_t* round_dev,
                                  int32_t K, int32_t k0, const float* __restrict__ s_dev,
                                  const float* __restrict__ tau_dev, int64_t param_round_stride,
                                  int32_t param_row_stride, int32_t V,
                                  const float* __restrict__ gauss,
                                  const float* __restrict__ lnrank, void* out,
                                  int64_t seq_stride, int64_t row_stride) {
    const uint32_t b = blockIdx.z;
    const uint32_t kk = blockIdx.y;
    if (round_dev) round = *round_dev;
    const uint32_t k = (uint32_t)k0 + kk;
    const int64_t pidx = (int64_t)round * param_round_stride + (int64_t)b * param_row_stride + k;
    const float s = s_dev[pidx];
    const float tau = (KIND == 1) ? tau_dev[pidx] : 0.0f;
    const uint64_t key = synth_row_key(seed, SYNTH_STREAM_LOGITS, round, b, k);
    const int64_t row_off = (int64_t)b * seq_stride + (int64_t)kk * row_stride;
    const int32_t v0 = (blockIdx.x * blockDim.x + threadIdx.x) * 8;
    if (v0 >= V) return;
    if (DTYPE == 0) {
        uint16_t* o = (uint16_t*)out + row_off;
        uint16_t h[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            int32_t v = v0 + j;
            float z = 0.0f;
            if (v < V) {
                uint64_t bits = synth_elem_bits(key, (uint32_t)v);
                z = KIND == 0 ? synth_draft_f32(bits, s, gauss, lnrank[v])
                              : synth_target_f32(bits, s, tau, gauss, lnrank[v]);
            }
            h[j] = synth_f32_to_bf16_rne(z);
        }
        if (v0 + 8 <= V && ((((uintptr_t)(o + v0)) & 15u) == 0)) {
            uint4 pk;
            pk.x = h[0] | ((uint32_t)h[1] << 16);
            pk.y = h[2] | ((uint32_t)h[3] << 16);
            pk.z = h[4] | ((uint32_t)h[5] << 16);
            pk.w = h[6] | ((uint32_t)h[7] << 16);
            *(uint4*)(o + v0) = pk;
        } else {
            for (int j = 0; j < 8 && v0 + j < V; ++j) o[v0 + j] = h[j];
        }
    } else {
        float* o = (float*)out + row_off;
        for (int j = 0; j < 8 && v0 + j < V; ++j) {
            int32_t v = v0 + j;
            uint64_t bits = synth_elem_bits(key, (uint32_t)v);
            o[v] = KIND == 0 ? synth_draft_f32(bits, s, gauss, lnrank[v])
                             : synth_target_f32(bits, s, tau, gauss, lnrank[v]);
        }
    }
}

__global__ void synth_uniforms_kernel(uint64_t seed, uint32_t substream, uint32_t round,
                                      const uint32_t* round_dev, int32_t B, int32_t n,
                                      float* out) {
    if (round_dev) round = *round_dev;
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (int64_t)B * n) return;
    uint32_t b = (uint32_t)(i / n), j = (uint32_t)(i % n);
    uint64_t key = synth_row_key(seed, SYNTH_STREAM_UNIFORM, round, b, substream);
    out[i] = synth_uniform24(synth_elem_bits(key, j));
}

__global__ void synth_counter_add_kernel(uint32_t* counter, uint32_t inc) { *counter += inc; }

}  // namespace

extern "C" {

/*
 * Rows (b, k0..k0+K-1) for b in [0,B) of `round` (or *round_dev when non-null).
 * s_dev / tau_dev are indexed [round * param_round_stride + b * param_row_stride + k].
 * out row (b, kk) starts at b * seq_stride + kk * row_stride elements.
 * Returns the cudaError_t of the launch as an int.
 */
int synth_rows_gpu(int32_t kind, uint64_t seed, uint32_t round, const uint32_t* round_dev,
                   int32_t B, int32_t K, int32_t k0, const float* s_dev, const float* tau_dev,
                   int64_t param_round_stride, int32_t param_row_stride, int32_t V,
                   const float* gauss_dev, const float* lnrank_dev, int32_t dtype, void* out_dev,
                   int64_t seq_stride, int64_t row_stride, void* stream) {
    if (B <= 0 || K <= 0 || V <= 0) return 0;
    dim3 block(256);
    dim3 grid((unsigned)((V + 256 * 8 - 1) / (256 * 8)), (unsigned)K, (unsigned)B);
    cudaStream_t st = (cudaStream_t)stream;
#define LAUNCH(KIND, DT)                                                                      \
    synth_rows_kernel<KIND, DT><<<grid, block, 0, st>>>(                                      \
        seed, round, round_dev, K, k0, s_dev, tau_dev, param_round_stride, param_row_stride,  \
        V, gauss_dev, lnrank_dev, out_dev, seq_stride, row_stride)
    if (kind == 0 && dtype == 0) LAUNCH(0, 0);
    else if (kind == 0) LAUNCH(0, 1);
    else if (dtype == 0) LAUNCH(1, 0);
    else LAUNCH(1, 1);
#undef LAUNCH
    return (int)cudaGetLastError();
}

int synth_uniforms_gpu(uint64_t seed, uint32_t substream, uint32_t round,
                       const uint32_t* round_dev, int32_t B, int32_t n, float* out_dev,
                       void* stream) {
    int64_t total = (int64_t)B * n;
    if (total <= 0) return 0;
    synth_uniforms_kernel<<<(unsigned)((total + 255) / 256), 256, 0, (cudaStream_t)stream>>>(
        seed, substream, round, round_dev, B, n, out_dev);
    return (int)cudaGetLastError();
}

int synth_counter_add_gpu(uint32_t* counter_dev, uint32_t inc, void* stream) {
    synth_counter_add_kernel<<<1, 1, 0, (cudaStream_t)stream>>>(counter_dev, inc);
    return (int)cudaGetLastError();
}

}  // extern "C"
