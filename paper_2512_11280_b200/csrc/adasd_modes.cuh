// Greedy decoding (Sec. 2.1.3) and the Gen-Only ablation variant (Sec. 5).
//
//  * row_argmax_kernel: the most probable token of every needed logit row, x = argmax_v z_v
//    (Sec. 2.1.1, deterministic selection), the lowest index among equal maxima.  One CTA per
//    row at a time, rows dealt round robin to a grid that fills the SMs; any V, dtype and
//    stride (16-byte loads where the row allows them).
//  * greedy_accept_kernel: candidate x_i is accepted only if it equals argmax p_i; the scan
//    stops at the first mismatch and the token after the accepted prefix is the target's own
//    choice there (the bonus row's after a full match).
//  * gen_only_update_kernel: the feedback of the generation component alone: the entropy of
//    the candidate that vanilla verification rejected joins L_E^R, T_G = mean(L_E^R).
#pragma once

#include "adasd_device.cuh"

namespace adasd {

struct ArgmaxParams {
    const void* z;
    long long seq_stride, row_stride;   // in elements
    const int32_t* draft_len;           // nullable: rows 0 .. min(draft_len[b], R - 1) of a sequence are needed
    const uint8_t* active;              // nullable: sequences with 0 are skipped
    int32_t* out;                       // [B, R]: the row's most probable token, -1 for an unusable row
    uint32_t* status;
    int32_t B, R, V;
};

constexpr int kAThreads = 256;

template <typename T, bool VEC>
__global__ void __launch_bounds__(kAThreads) row_argmax_kernel(ArgmaxParams p) {
    constexpr int N = Elt<T>::N;
    __shared__ float s_val[kAThreads / 32];
    __shared__ int s_idx[kAThreads / 32];
    __shared__ int s_bad[kAThreads / 32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int NU = (p.V + N - 1) / N;
    const int total = p.B * p.R;
    for (int row = blockIdx.x; row < total; row += gridDim.x) {
        const int b = row / p.R, j = row - b * p.R;
        if (p.active && p.active[b] == 0) continue;
        if (p.draft_len) {
            const int kt = max(0, min(p.draft_len[b], p.R - 1));
            if (j > kt) continue;
        }
        const T* z = reinterpret_cast<const T*>(p.z) + (long long)b * p.seq_stride + (long long)j * p.row_stride;
        // each thread walks its units in increasing index order: a later element replaces the
        // running maximum only if it is strictly larger, so the lowest index of equal maxima stays
        float best = -INFINITY;
        int bi = -1, bad = 0;
        for (int u = threadIdx.x; u < NU; u += kAThreads) {
            float x[N];
            load_unit<T, VEC>(z, u, p.V, x);
#pragma unroll
            for (int q = 0; q < N; ++q) {
                bad |= (x[q] != x[q]);
                if (x[q] > best) {
                    best = x[q];
                    bi = u * N + q;
                }
            }
        }
        // larger value wins, equal values go to the lower index
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float ov = __shfl_xor_sync(0xFFFFFFFFu, best, o);
            const int oi = __shfl_xor_sync(0xFFFFFFFFu, bi, o);
            if (ov > best || (ov == best && oi >= 0 && (bi < 0 || oi < bi))) {
                best = ov;
                bi = oi;
            }
        }
        bad = __any_sync(0xFFFFFFFFu, bad);
        if (lane == 0) {
            s_val[warp] = best;
            s_idx[warp] = bi;
            s_bad[warp] = bad;
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            for (int w = 1; w < kAThreads / 32; ++w) {
                const float ov = s_val[w];
                const int oi = s_idx[w];
                if (ov > best || (ov == best && oi >= 0 && (bi < 0 || oi < bi))) {
                    best = ov;
                    bi = oi;
                }
                bad |= s_bad[w];
            }
            const bool unusable = bad || !(best > -INFINITY) || best == INFINITY;
            if (unusable) atomicOr(p.status, ADASD_STATUS_NAN);
            p.out[(size_t)b * p.R + j] = unusable ? -1 : bi;
        }
        __syncthreads();
    }
}

// One thread per sequence: longest prefix of candidates that equal the target's choice.
__global__ void greedy_accept_kernel(const int32_t* __restrict__ x, const int32_t* __restrict__ am,
                                     const int32_t* __restrict__ draft_len, int32_t* accept_len,
                                     int32_t* next_token, int32_t* argmax_user, int B, int Kmax) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    const int K1 = Kmax + 1;
    int kt = draft_len ? draft_len[b] : Kmax;
    kt = max(0, min(kt, Kmax));
    int w = kt;
    for (int i = 0; i < kt; ++i) {
        if (x[(size_t)b * Kmax + i] != am[(size_t)b * K1 + i]) {
            w = i;
            break;
        }
    }
    accept_len[b] = w;
    next_token[b] = am[(size_t)b * K1 + w];
    if (argmax_user)
        for (int i = 0; i <= kt; ++i) argmax_user[(size_t)b * K1 + i] = am[(size_t)b * K1 + i];
}

// One thread per sequence: L_E^R += H(q) of the candidate vanilla verification rejected.
__global__ void gen_only_update_kernel(State st, const float* __restrict__ H_d, const int32_t* __restrict__ draft_len,
                                       const int32_t* __restrict__ accept_len, int B, int Kmax) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    int kt = draft_len ? draft_len[b] : Kmax;
    kt = max(0, min(kt, Kmax));
    const int w = accept_len[b];
    if (w < 0 || w >= kt) return;                     // nothing was rejected
    const float Hw = H_d[(size_t)b * Kmax + w];
    if (!(Hw == Hw) || !(fabsf(Hw) < INFINITY)) return;
    const int nE = st.nE[b];
    if (nE >= st.cap) {
        atomicOr(st.status, ADASD_STATUS_CAPACITY);
        return;
    }
    st.LE[(size_t)b * st.cap + nE] = Hw;
    const double sE = st.sumE[b] + (double)Hw;
    st.nE[b] = nE + 1;
    st.sumE[b] = sE;
    st.T_G[b] = (float)(sE / (double)(nE + 1));
}

}  // namespace adasd
