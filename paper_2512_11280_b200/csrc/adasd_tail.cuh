// The per-sequence tail of a verification round: KDE densities and the Bayes posterior
// P(A|d_i) for every candidate (Sec. 4.4), the first-rejection accept scan, the list
// appends and the T_G update (Algorithm 1, steps 2 and 3).  Run by ONE CTA per
// sequence, after every position of that sequence has published its scalars.
#pragma once

#include "adasd_device.cuh"

namespace adasd {

struct TailConfig {
    int32_t Kmax;
    int32_t min_samples;
    int32_t bw_rule;      // 0 Silverman, 1 Scott
    int32_t reject_rule;  // 0 Bernoulli, 1 threshold 1/2
    uint32_t update;      // append to the lists and refresh T_G
};

struct TailShared {
    float d[ADASD_KMAX_LIMIT];
    float H[ADASD_KMAX_LIMIT];
    float u[ADASD_KMAX_LIMIT];
    int32_t x[ADASD_KMAX_LIMIT];
    int32_t y[ADASD_KMAX_LIMIT + 1];
    float cA[ADASD_KMAX_LIMIT];    // -log2(e) / (2 h_A,i^2)
    float ihA[ADASD_KMAX_LIMIT];   // 1 / h_A,i
    float SA[ADASD_KMAX_LIMIT];    // sum of kernel terms over L_D^A (+ this round's prefix)
    float SR[ADASD_KMAX_LIMIT];
    float P[ADASD_KMAX_LIMIT];
    int32_t valid[ADASD_KMAX_LIMIT];
    float red[kWarps][8];
    float cR, ihR;
    int32_t validR;
};

// Bandwidth from running sums: h = sample_std * factor(n).  Returns 0 when undefined.
__device__ __forceinline__ double kde_bandwidth(double n, double sum, double sum2, int rule) {
    if (n < 2.0) return 0.0;
    double var = (sum2 - sum * sum / n) / (n - 1.0);
    // identical samples leave rounding noise instead of an exact zero
    if (!(var > 1e-13 * (sum2 / n))) return 0.0;
    double f = rule == 0 ? pow(0.75 * n, -0.2) : pow(n, -0.2);
    return sqrt(var) * f;
}

// Sum over a list of exp2(c_i * (d_i - x_j)^2) for up to 8 candidates at a time.
__device__ __forceinline__ void kde_sums(const float* __restrict__ list, int n, int K_t,
                                         const float* d, const float* c, bool per_candidate_c,
                                         float cR, float* S, TailShared& sh) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int i0 = 0; i0 < K_t; i0 += 8) {
        float acc[8], di[8], ci[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            acc[k] = 0.f;
            int i = min(i0 + k, K_t - 1);
            di[k] = d[i];
            ci[k] = per_candidate_c ? c[i] : cR;
        }
        for (int j = threadIdx.x; j < n; j += blockDim.x) {
            float xj = __ldcg(list + j);
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                float t = di[k] - xj;
                acc[k] += ex2(ci[k] * t * t);
            }
        }
#pragma unroll
        for (int k = 0; k < 8; ++k) acc[k] = warp_sum(acc[k]);
        __syncthreads();  // sh.red free again
        if (lane == 0) {
#pragma unroll
            for (int k = 0; k < 8; ++k) sh.red[warp][k] = acc[k];
        }
        __syncthreads();
        if (threadIdx.x < 8 && i0 + threadIdx.x < K_t) {
            float a = 0.f;
            const int nw = (int)(blockDim.x >> 5);     // the CTA running the tail may have fewer warps
            for (int w = 0; w < nw; ++w) a += sh.red[w][threadIdx.x];
            S[i0 + threadIdx.x] = a;
        }
    }
    __syncthreads();
}

struct TailIO {
    // per-position inputs of this round
    const float* H_d;       // [B,Kmax]
    const float* dist;      // [B,Kmax]
    const int32_t* y;       // [B,Kmax+1]
    const int32_t* x;       // [B,Kmax]
    const float* u_accept;  // [B,Kmax]
    const int32_t* draft_len;  // [B] or null
    // outputs
    float* p_acc;           // scratch record [B,Kmax]
    float* p_acc_user;      // nullable
    int32_t* accept_len;
    int32_t* next_token;
    int32_t* accept_len_rec;   // nullable record copies
    int32_t* rejected_rec;
    int32_t* draft_len_rec;
};

// Appends and threshold update of one sequence (Algorithm 1: the append lines of the
// verify loop and step 3).  One thread.
__device__ __forceinline__ void apply_update(State& st, int b, int w, bool rejected,
                                             const float* d, const float* H) {
    const int cap = st.cap;
    int nA = st.nA[b];
    double sA = st.sumA[b], sA2 = st.sumA2[b];
    for (int j = 0; j < w; ++j) {
        float dj = d[j];
        if (dj > 0.f && dj < 1.f) {
            if (nA < cap) {
                st.LA[(size_t)b * cap + nA] = dj;
                ++nA;
                sA += (double)dj;
                sA2 += (double)dj * (double)dj;
            } else {
                atomicOr(st.status, ADASD_STATUS_CAPACITY);
            }
        }
    }
    st.nA[b] = nA;
    st.sumA[b] = sA;
    st.sumA2[b] = sA2;
    if (rejected) {
        // The entropy of a row with NaN or no finite logit is NaN (the status word says so
        // already): recording it would leave T_G = NaN and switch the draft-stop check off for
        // good.  A full list skips the append whole, like the other two lists, so that T_G stays
        // the mean of the entries the list holds (what a checkpoint restores).
        const float Hw = H[w];
        int nE = st.nE[b];
        if (Hw == Hw && fabsf(Hw) < INFINITY) {
            if (nE < cap) {
                st.LE[(size_t)b * cap + nE] = Hw;
                double sE = st.sumE[b] + (double)Hw;
                ++nE;
                st.nE[b] = nE;
                st.sumE[b] = sE;
                st.T_G[b] = (float)(sE / (double)nE);  // T_G <- average(L_E^R)
            } else {
                atomicOr(st.status, ADASD_STATUS_CAPACITY);
            }
        }
        float dw = d[w];
        if (dw > 0.f && dw < 1.f) {
            int nR = st.nR[b];
            if (nR < cap) {
                st.LR[(size_t)b * cap + nR] = dw;
                st.nR[b] = nR + 1;
                st.sumR[b] += (double)dw;
                st.sumR2[b] += (double)dw * (double)dw;
            } else {
                atomicOr(st.status, ADASD_STATUS_CAPACITY);
            }
        }
    }
}

__device__ void verify_tail(const TailConfig& cfg, const TailIO& io, State& st, int b,
                            TailShared& sh) {
    const int Kmax = cfg.Kmax;
    int K_t = io.draft_len ? __ldcg(io.draft_len + b) : Kmax;
    K_t = max(0, min(K_t, Kmax));
    const int tid = threadIdx.x;
    if (tid <= K_t) sh.y[tid] = __ldcg(io.y + (size_t)b * (Kmax + 1) + tid);
    if (tid < K_t) {
        sh.d[tid] = __ldcg(io.dist + (size_t)b * Kmax + tid);
        sh.H[tid] = __ldcg(io.H_d + (size_t)b * Kmax + tid);
        sh.x[tid] = io.x[(size_t)b * Kmax + tid];
        sh.u[tid] = io.u_accept[(size_t)b * Kmax + tid];
    }
    __syncthreads();

    const int nA0 = st.nA[b], nR0 = st.nR[b];
    // bandwidths: candidate i sees L_D^A plus the distances d_1..d_{i-1} of this round
    // that lie strictly inside (0,1), i.e. the list "as it stands" if all of them were
    // accepted - which is the only case in which candidate i is reached at all.
    if (tid < K_t) {
        double n = (double)nA0, s = st.sumA[b], s2 = st.sumA2[b];
        for (int j = 0; j < tid; ++j) {
            float dj = sh.d[j];
            if (dj > 0.f && dj < 1.f) {
                n += 1.0;
                s += (double)dj;
                s2 += (double)dj * (double)dj;
            }
        }
        double h = kde_bandwidth(n, s, s2, cfg.bw_rule);
        int ok = (n >= (double)cfg.min_samples) && (h > 0.0);
        sh.valid[tid] = ok;
        sh.cA[tid] = ok ? (float)(-0.5 * 1.4426950408889634 / (h * h)) : 0.f;
        sh.ihA[tid] = ok ? (float)(1.0 / h) : 0.f;
    }
    if (tid == 0) {
        double h = kde_bandwidth((double)nR0, st.sumR[b], st.sumR2[b], cfg.bw_rule);
        int ok = (nR0 >= cfg.min_samples) && (h > 0.0);
        sh.validR = ok;
        sh.cR = ok ? (float)(-0.5 * 1.4426950408889634 / (h * h)) : 0.f;
        sh.ihR = ok ? (float)(1.0 / h) : 0.f;
    }
    __syncthreads();

    bool any_valid = false;
    for (int i = 0; i < K_t; ++i) any_valid |= (sh.valid[i] != 0);
    any_valid = any_valid && sh.validR;

    if (any_valid) {
        kde_sums(st.LA + (size_t)b * st.cap, nA0, K_t, sh.d, sh.cA, true, 0.f, sh.SA, sh);
        kde_sums(st.LR + (size_t)b * st.cap, nR0, K_t, sh.d, sh.cA, false, sh.cR, sh.SR, sh);
    }
    if (tid < K_t) {
        float P = 0.f;
        if (any_valid && sh.valid[tid]) {
            float SA = sh.SA[tid];
            const float di = sh.d[tid], ci = sh.cA[tid];
            for (int j = 0; j < tid; ++j) {
                float dj = sh.d[j];
                if (dj > 0.f && dj < 1.f) {
                    float t = di - dj;
                    SA += ex2(ci * t * t);
                }
            }
            // n_A f_A = SA / (h_A sqrt(2 pi)),  n_R f_R = SR / (h_R sqrt(2 pi))
            float a = SA * sh.ihA[tid];
            float r = sh.SR[tid] * sh.ihR;
            float den = a + r;
            if (den > 0.f && den < INFINITY) P = a / den;
        }
        sh.P[tid] = P;
        io.p_acc[(size_t)b * Kmax + tid] = P;
        if (io.p_acc_user) io.p_acc_user[(size_t)b * Kmax + tid] = P;
    }
    __syncthreads();

    if (tid == 0) {
        int w = K_t;
        bool rejected = false;
        for (int i = 0; i < K_t; ++i) {
            float P = sh.P[i];
            bool rej = cfg.reject_rule == 0 ? (sh.u[i] >= P) : (P < 0.5f);
            if (sh.x[i] != sh.y[i] && rej) {
                w = i;
                rejected = true;
                break;
            }
        }
        io.accept_len[b] = w;
        io.next_token[b] = sh.y[w];
        if (io.accept_len_rec) io.accept_len_rec[b] = w;
        if (io.rejected_rec) io.rejected_rec[b] = rejected ? 1 : 0;
        if (io.draft_len_rec) io.draft_len_rec[b] = K_t;
        if (cfg.update) apply_update(st, b, w, rejected, sh.d, sh.H);
    }
}

}  // namespace adasd
