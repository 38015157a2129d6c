// The adjusted distribution of Sec. 2.1.1 (temperature scaling, top-k sampling, top-p sampling).
//
// Temperature is a scale of the logits and costs the row passes nothing: they multiply by
// log2 e / temperature where they multiplied by log2 e.  Top-k and top-p cut the vocabulary, and
// both cuts are "keep the tokens whose logit is at least c" for one value c per row:
//   top-k: c = the k-th largest logit (tokens equal to it stay with it);
//   top-p: c = the smallest logit v such that the tokens STRICTLY above v hold less than top_p
//          of the mass of what top-k left (the smallest most-probable set whose mass reaches
//          top_p, ties at its edge included).
// row_cutoff_kernel finds c for every needed row; the row passes then read a logit below its
// row's c as -inf (apply_warp below), so entropy, JS distance, the accept ratio and every sample
// are those of the adjusted distribution.
//
// The search is a radix descent over the order-preserving integer image of the logits (16 bits
// for bf16, 32 for fp32), 8 bits a level, most significant first: a level histograms the
// weight (1 per token for top-k; 2^((z - max) log2 e / T) for top-p) of the tokens that match
// the digits fixed so far, and the bin where the weight counted from the top first reaches the
// threshold fixes the next digit.  Masses are formed in double precision and added as 2^-40
// fixed-point integers, so the sums do not depend on the order the atomics land in, the result
// is the same on every run, and a token's side of the cut is decided to about 1e-9 of the mass.
#pragma once

#include "adasd_device.cuh"

namespace adasd {

// One row's adjustment as the row passes apply it.
struct RowWarp {
    float inv_t;    // 1 / temperature
    float cut;      // logits below it are cut (-inf: none)
};
// -inf for a cut token, z / temperature for the others; NaN stays NaN (the row is unusable);
// {1, -inf} changes nothing, bit for bit.
__device__ __forceinline__ float apply_warp(float z, const RowWarp& w) {
    return (z < w.cut) ? -INFINITY : z * w.inv_t;
}
template <int N>
__device__ __forceinline__ void apply_warp(float (&x)[N], const RowWarp& w) {
#pragma unroll
    for (int j = 0; j < N; ++j) x[j] = apply_warp(x[j], w);
}

// load_unit with the row's adjustment applied
template <typename T, bool VEC>
__device__ __forceinline__ void load_unit_w(const T* __restrict__ row, int u, int V, float (&x)[Elt<T>::N],
                                            const RowWarp& w) {
    load_unit<T, VEC>(row, u, V, x);
    apply_warp(x, w);
}

struct CutParams {
    const void* z;
    long long seq_stride, row_stride;   // in elements
    const int32_t* draft_len;           // nullable: window K_b of sequence b (clamped to [0, R - extra])
    const uint8_t* active;              // nullable: sequences with 0 are skipped
    float* cut;                         // [B, R]
    uint32_t* status;
    int32_t B, R, V;
    int32_t extra;                      // 1: rows 0 .. K_b are needed (target rows, with the bonus row); 0: rows 0 .. K_b - 1
    double c1;                          // log2 e / temperature
    int32_t top_k;                      // <= 0 or >= V: off
    float top_p;                        // >= 1: off
};

constexpr int kCutThreads = 512;
constexpr int kCutWarps = kCutThreads / 32;
constexpr double kCutFix = 1099511627776.0;   // 2^40

template <typename T>
struct CutKey;
template <>
struct CutKey<__nv_bfloat16> {
    static constexpr int BITS = 16;
    __device__ static uint32_t of(float x) {
        uint32_t u = __float_as_uint(x) >> 16;
        if ((u & 0x7FFFu) == 0) u = 0;                       // -0 and +0 are one value
        return (u & 0x8000u) ? (~u & 0xFFFFu) : (u | 0x8000u);
    }
    __device__ static float value(uint32_t k) {
        const uint32_t u = (k & 0x8000u) ? (k & 0x7FFFu) : (~k & 0xFFFFu);
        return __uint_as_float(u << 16);
    }
};
template <>
struct CutKey<float> {
    static constexpr int BITS = 32;
    __device__ static uint32_t of(float x) {
        uint32_t u = __float_as_uint(x);
        if ((u & 0x7FFFFFFFu) == 0) u = 0;
        return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
    }
    __device__ static float value(uint32_t k) {
        return __uint_as_float((k & 0x80000000u) ? (k & 0x7FFFFFFFu) : ~k);
    }
};

struct CutShared {
    unsigned long long bins[kCutWarps][256];
    unsigned long long tot[256];
    float red[kCutWarps];
    int flag[kCutWarps];
    unsigned long long acc;       // weight above the digits fixed so far
    unsigned long long S;         // top-p: the mass of everything top-k left
    uint32_t prefix;
    int32_t found;
    float m;
    int32_t bad;
};

// One CTA per row at a time; rows are dealt round robin to a grid that fills the SMs.  The first
// pass reads the row from HBM, the later ones find it in L2.
template <typename T, bool VEC>
__global__ void __launch_bounds__(kCutThreads) row_cutoff_kernel(CutParams p) {
    constexpr int N = Elt<T>::N;
    constexpr int BITS = CutKey<T>::BITS;
    __shared__ CutShared sh;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int NU = (p.V + N - 1) / N;
    const int total = p.B * p.R;
    const bool use_k = p.top_k > 0 && p.top_k < p.V;
    const bool use_p = p.top_p < 1.f;

    for (int row = blockIdx.x; row < total; row += gridDim.x) {
        const int b = row / p.R, j = row - b * p.R;
        if (p.active && p.active[b] == 0) continue;
        if (p.draft_len) {
            const int kt = max(0, min(p.draft_len[b], p.R - p.extra));
            if (j >= kt + p.extra) continue;
        }
        const T* z = reinterpret_cast<const T*>(p.z) + (long long)b * p.seq_stride + (long long)j * p.row_stride;

        // largest logit and usability of the row
        float mx = -INFINITY;
        int bad = 0;
        for (int u = threadIdx.x; u < NU; u += kCutThreads) {
            float x[N];
            load_unit<T, VEC>(z, u, p.V, x);
#pragma unroll
            for (int q = 0; q < N; ++q) {
                bad |= (x[q] != x[q]);
                mx = fmaxf(mx, x[q]);
            }
        }
        mx = warp_max(mx);
        bad = __any_sync(0xFFFFFFFFu, bad);
        if (lane == 0) {
            sh.red[warp] = mx;
            sh.flag[warp] = bad;
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            float m = sh.red[0];
            int bd = sh.flag[0];
            for (int w = 1; w < kCutWarps; ++w) {
                m = fmaxf(m, sh.red[w]);
                bd |= sh.flag[w];
            }
            sh.m = m;
            sh.bad = bd || !(m > -INFINITY) || m == INFINITY;
        }
        __syncthreads();
        const float m = sh.m;
        if (sh.bad) {                       // an unusable row is not cut; the row pass reports it
            if (threadIdx.x == 0) p.cut[(size_t)b * p.R + j] = -INFINITY;
            __syncthreads();
            continue;
        }

        uint32_t lo_key = 0;                // tokens with a key below it are cut already
        for (int which = 0; which < 2; ++which) {
            const bool mass = (which == 1);
            if (mass ? !use_p : !use_k) continue;
            if (threadIdx.x == 0) {
                sh.acc = 0ull;
                sh.prefix = 0u;
                sh.found = 1;
            }
            __syncthreads();
            for (int shift = BITS - 8; shift >= 0; shift -= 8) {
                for (int i = threadIdx.x; i < kCutWarps * 256; i += kCutThreads) (&sh.bins[0][0])[i] = 0ull;
                __syncthreads();
                const uint32_t prefix = sh.prefix;
                const bool top_level = (shift == BITS - 8);
                for (int u = threadIdx.x; u < NU; u += kCutThreads) {
                    float x[N];
                    load_unit<T, VEC>(z, u, p.V, x);
#pragma unroll
                    for (int q = 0; q < N; ++q) {
                        if (u * N + q >= p.V) continue;
                        const uint32_t key = CutKey<T>::of(x[q]);
                        if (key < lo_key) continue;
                        if (!top_level && (key >> (shift + 8)) != prefix) continue;
                        unsigned long long w = 1ull;
                        if (mass) w = (unsigned long long)__double2ll_rn(exp2((double)(fmaxf(x[q], kFloor) - m) * p.c1) * kCutFix);
                        if (w) atomicAdd(&sh.bins[warp][(key >> shift) & 255u], w);
                    }
                }
                __syncthreads();
                if (threadIdx.x < 256) {
                    unsigned long long t = 0ull;
                    for (int w = 0; w < kCutWarps; ++w) t += sh.bins[w][threadIdx.x];
                    sh.tot[threadIdx.x] = t;
                }
                __syncthreads();
                if (threadIdx.x == 0 && sh.found) {
                    // threshold: k tokens, or top_p of the mass top-k left (the whole of it is in
                    // the top level's bins)
                    double thr;
                    if (!mass) {
                        thr = (double)p.top_k;
                    } else {
                        if (top_level) {
                            unsigned long long S = 0ull;
                            for (int d = 0; d < 256; ++d) S += sh.tot[d];
                            sh.S = S;
                        }
                        thr = (double)p.top_p * (double)sh.S;
                    }
                    unsigned long long acc = sh.acc;
                    int hit = -1;
                    for (int d = 255; d >= 0; --d) {
                        const unsigned long long w = sh.tot[d];
                        if (w == 0ull) continue;
                        if ((double)(acc + w) >= thr) {
                            hit = d;
                            break;
                        }
                        acc += w;
                    }
                    if (hit < 0) {
                        sh.found = 0;                   // the threshold is never reached: nothing is cut
                    } else {
                        sh.acc = acc;
                        sh.prefix = (prefix << 8) | (uint32_t)hit;
                    }
                }
                __syncthreads();
                if (!sh.found) break;
            }
            __syncthreads();
            if (sh.found) lo_key = max(lo_key, sh.prefix);
            __syncthreads();
        }
        if (threadIdx.x == 0) p.cut[(size_t)b * p.R + j] = lo_key ? CutKey<T>::value(lo_key) : -INFINITY;
        __syncthreads();
    }
}

}  // namespace adasd
