// Device-side building blocks shared by the AdaSD kernels: fast base-2 math, row
// loading, deterministic warp/CTA/cluster reductions and index-order inverse-CDF
// selection.  sm_100a only.
#pragma once

#include <cooperative_groups.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/adasd.h"

namespace adasd {

namespace cg = cooperative_groups;

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
// Finite stand-in for -inf logits: keeps 0 * (-inf) out of the sums.  Any logit at or
// below it has probability exactly 0.
constexpr float kFloor = -1.0e30f;
constexpr float kTiny = 1.0e-37f;

constexpr int kThreads = 512;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxCluster = 8;
constexpr int kMaxGW = kMaxCluster * kWarps;  // warps that can share one row

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float lg2(float x) {
    float y;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Per-sequence adaptive state (Algorithm 1, initialisation block), structure of arrays.
struct State {
    float* T_G;      // [B] generation threshold
    double* sumE;    // [B] sum of L_E^R
    int32_t* nE;     // [B]
    int32_t* nA;     // [B]
    int32_t* nR;     // [B]
    double* sumA;    // [B] sum and sum of squares of L_D^A / L_D^R: bandwidth without a list pass
    double* sumA2;
    double* sumR;
    double* sumR2;
    float* LE;       // [B,cap]
    float* LA;       // [B,cap]
    float* LR;       // [B,cap]
    int32_t cap;
    uint32_t* status;
};

template <typename T>
struct Elt;
template <>
struct Elt<__nv_bfloat16> {
    static constexpr int N = 8;  // elements per 16-byte unit
};
template <>
struct Elt<float> {
    static constexpr int N = 4;
};

__device__ __forceinline__ float to_f32(__nv_bfloat16 h) { return __bfloat162float(h); }
__device__ __forceinline__ float to_f32(float f) { return f; }

__device__ __forceinline__ void unpack16(const uint4& r, float (&x)[8]) {
    x[0] = __uint_as_float(r.x << 16);
    x[1] = __uint_as_float(r.x & 0xFFFF0000u);
    x[2] = __uint_as_float(r.y << 16);
    x[3] = __uint_as_float(r.y & 0xFFFF0000u);
    x[4] = __uint_as_float(r.z << 16);
    x[5] = __uint_as_float(r.z & 0xFFFF0000u);
    x[6] = __uint_as_float(r.w << 16);
    x[7] = __uint_as_float(r.w & 0xFFFF0000u);
}
__device__ __forceinline__ void unpack16(const uint4& r, float (&x)[4]) {
    x[0] = __uint_as_float(r.x);
    x[1] = __uint_as_float(r.y);
    x[2] = __uint_as_float(r.z);
    x[3] = __uint_as_float(r.w);
}

// Unit u of a row = elements [u*N, u*N+N).  Elements at or beyond V read as -inf.
// VEC: the row base and stride are 16-byte aligned, so full units take one 16-byte load.
template <typename T, bool VEC>
__device__ __forceinline__ void load_unit(const T* __restrict__ row, int u, int V,
                                          float (&x)[Elt<T>::N]) {
    constexpr int N = Elt<T>::N;
    const int v0 = u * N;
    if (VEC && v0 + N <= V) {
        uint4 r = __ldg(reinterpret_cast<const uint4*>(row + v0));
        unpack16(r, x);
    } else {
#pragma unroll
        for (int j = 0; j < N; ++j) x[j] = (v0 + j < V) ? to_f32(row[v0 + j]) : -INFINITY;
    }
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
    return v;
}

// All-reduce of N floats over every thread of the cluster, in a fixed order (so that
// the draft and the target row of a pair, and repeated runs, reduce identically).
// s_warp: [kWarps*N] scratch of this CTA; s_x: [kMaxCluster*N] exchange buffer of this
// CTA, one per call site (remote CTAs write their partial into slot [rank]).
template <int N, bool IS_MAX>
__device__ __forceinline__ void cluster_allreduce(float (&v)[N], float* s_warp, float* s_x,
                                                  int CS, int rank, cg::cluster_group& cluster) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int k = 0; k < N; ++k) v[k] = IS_MAX ? warp_max(v[k]) : warp_sum(v[k]);
    if (lane == 0) {
#pragma unroll
        for (int k = 0; k < N; ++k) s_warp[warp * N + k] = v[k];
    }
    __syncthreads();
    if (threadIdx.x < N) {
        float a = s_warp[threadIdx.x];
        for (int w = 1; w < kWarps; ++w) {
            float b = s_warp[w * N + threadIdx.x];
            a = IS_MAX ? fmaxf(a, b) : a + b;
        }
        for (int r = 0; r < CS; ++r) {
            float* dst = cluster.map_shared_rank(s_x, r);
            dst[rank * N + threadIdx.x] = a;
        }
    }
    cluster.sync();
#pragma unroll
    for (int k = 0; k < N; ++k) {
        float a = s_x[k];
        for (int r = 1; r < CS; ++r) {
            float b = s_x[r * N + k];
            a = IS_MAX ? fmaxf(a, b) : a + b;
        }
        v[k] = a;
    }
}

// Which warp's contiguous range holds the inverse-CDF crossing.  tab[g] is the weight
// total of cluster-wide warp g (index order).  Returns the chosen warp, the weight
// before it and the target u * total; if rounding leaves no crossing the last warp with
// mass is chosen and the target is +inf (the caller then takes its last element with
// mass).  total == 0 returns -1.
__device__ __forceinline__ int select_warp(const float* tab, int GW, float u, float& base,
                                           float& target) {
    float total = 0.f;
    for (int g = 0; g < GW; ++g) total += tab[g];
    if (!(total > 0.f)) return -1;
    target = u * total;
    float cum = 0.f;
    int chosen = -1, last_pos = -1;
    float last_base = 0.f;
    for (int g = 0; g < GW; ++g) {
        float w = tab[g];
        float nc = cum + w;
        if (w > 0.f) {
            last_pos = g;
            last_base = cum;
            if (chosen < 0 && nc > target) {
                chosen = g;
                base = cum;
            }
        }
        cum = nc;
    }
    if (chosen < 0) {
        chosen = last_pos;
        base = last_base;
        target = INFINITY;
    }
    return chosen;
}

// Run by one full warp over its unit range [u0,u1): the first element (index order)
// whose running weight exceeds target, else the last element with mass.
// weights(u, w) fills the N weights of unit u (0 beyond V).
template <int N, typename F>
__device__ __forceinline__ int warp_scan_select(int u0, int u1, int V, float base, float target,
                                                F weights) {
    const int lane = threadIdx.x & 31;
    float run = base;
    int found = -1;
    int last_pos = -1;
    for (int ub = u0; ub < u1 && found < 0; ub += 32) {
        const int u = ub + lane;
        float w[N];
        if (u < u1) {
            weights(u, w);
        } else {
#pragma unroll
            for (int j = 0; j < N; ++j) w[j] = 0.f;
        }
        float ls = 0.f;
#pragma unroll
        for (int j = 0; j < N; ++j) ls += w[j];
        float incl = ls;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            float t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= o) incl += t;
        }
        float excl = __shfl_up_sync(0xFFFFFFFFu, incl, 1);
        if (lane == 0) excl = 0.f;
        float c = run + excl;
        int hit = -1;
#pragma unroll
        for (int j = 0; j < N; ++j) {
            c += w[j];
            if (w[j] > 0.f) {
                if (u * N + j < V) last_pos = u * N + j;
                if (hit < 0 && c > target) hit = j;
            }
        }
        unsigned m = __ballot_sync(0xFFFFFFFFu, hit >= 0);
        if (m) {
            int src = __ffs(m) - 1;
            int tok = u * N + hit;
            found = __shfl_sync(0xFFFFFFFFu, tok, src);
        }
        run += __shfl_sync(0xFFFFFFFFu, incl, 31);
    }
    if (found < 0) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) last_pos = max(last_pos, __shfl_xor_sync(0xFFFFFFFFu, last_pos, o));
        found = last_pos;
    }
    return found;
}

}  // namespace adasd
