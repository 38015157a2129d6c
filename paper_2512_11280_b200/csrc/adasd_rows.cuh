// Generic row kernels: one thread-block cluster per logit row (draft step) or per
// candidate position (verification).  Any V, any stride, bf16 or fp32; rows are read
// from global memory once per pass (later passes hit L2).  These kernels are the
// reference CUDA path and the fallback of the staged kernels.
#pragma once

#include "adasd_device.cuh"
#include "adasd_tail.cuh"
#include "adasd_warp.cuh"

namespace adasd {

constexpr int MODE_ADASD = 0;
constexpr int MODE_VANILLA = 1;

struct Scratch {            // context-owned per-round scratch, all [B,Kmax(+1)]
    float* H_d;
    float* H_t;
    float* lse_d;
    float* lse_t;
    float* jsd;
    float* dist;
    float* p_acc;
    int32_t* y;
    int32_t* van_flag;      // [B,Kmax] vanilla: 1 accept / 0 reject
    int32_t* van_tok;       // [B,Kmax+1] vanilla: resample (or bonus) candidate
    uint32_t* ticket;       // [B] arrival counter of a sequence's positions
    int32_t* only_pos;      // [B] vanilla: the position that is sampled (first rejection or bonus row)
    int32_t* q_items;       // [B] chip-wide queue of completed sequences awaiting their tail (-1: empty)
    uint32_t* q_ctl;        // [4] queue counters: pushed, drawn, workers gone (all 0 between launches)
};

struct VerifyParams {
    const void* zd;
    const void* zt;
    long long d_seq, d_row, t_seq, t_row;
    const int32_t* x;
    const int32_t* draft_len;
    const float* u_target;
    const float* u_accept;
    const float* u_resample;
    int32_t* accept_len;
    int32_t* next_token;
    float* alpha_out;
    adasd_round_record user;   // caller's record (entries may be null)
    Scratch sc;
    State st;
    TailConfig tail;
    int32_t B, V, Kmax;
    // adjusted distribution (Sec. 2.1.1): 1 / temperature and, per row, the logit below which
    // tokens are cut (null: no cut); the staged kernels fold the temperature into c1 = log2 e / T
    float inv_temp, c1;
    const float* cut_t;     // [B,Kmax+1]
    const float* cut_d;     // [B,Kmax]
};

struct DraftParams {
    const void* z;
    long long row_stride;
    const float* u;
    uint8_t* active;
    float* H_out;
    float* lse_out;
    int32_t* token_out;
    uint8_t* stop_out;
    int32_t* draft_len;
    State st;
    int32_t B, V;
    int32_t expire_row;     // self-test of the bounded waits: the row whose first copy is never asked for (-1: none)
    float inv_temp, c1;     // adjusted distribution: 1 / temperature, log2 e / temperature
    const float* cut;       // [B] logit below which a row's tokens are cut (null: no cut)
};

struct RowShared {
    float warp[kWarps * 4];
    float xA[kMaxCluster * 4];
    float xB[kMaxCluster * 2];
    float xC[kMaxCluster * 4];
    float wtab[kMaxGW];      // per-warp weight totals of the row being sampled
    float wtab2[kMaxGW];     // vanilla: per-warp residual totals
    int32_t token;           // sampled token, written by the chosen warp
    int32_t is_last;
};

// ------------------------------------------------------------------------------------
// Draft step: H(q), lse, x ~ q, stop = H > T_G   (Algorithm 1, generation loop body)
// ------------------------------------------------------------------------------------
template <typename T, bool VEC>
__global__ void __launch_bounds__(kThreads) draft_kernel(DraftParams p) {
    constexpr int N = Elt<T>::N;
    cg::cluster_group cluster = cg::this_cluster();
    const int CS = (int)cluster.num_blocks();
    const int rank = (int)cluster.block_rank();
    const int b = blockIdx.x / CS;
    if (p.active && p.active[b] == 0) return;   // same decision in every CTA of the cluster

    __shared__ RowShared sh;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int GW = CS * kWarps, gw = rank * kWarps + warp;
    const int NU = (p.V + N - 1) / N;
    const int u0 = (int)((long long)gw * NU / GW), u1 = (int)((long long)(gw + 1) * NU / GW);
    const T* row = reinterpret_cast<const T*>(p.z) + (long long)b * p.row_stride;
    const RowWarp wr = {p.inv_temp, p.cut ? p.cut[b] : -INFINITY};

    // pass A: max, NaN flag
    float vA[2] = {-INFINITY, 0.f};
    for (int u = u0 + lane; u < u1; u += 32) {
        float x[N];
        load_unit_w<T, VEC>(row, u, p.V, x, wr);
#pragma unroll
        for (int j = 0; j < N; ++j) {
            vA[1] = (x[j] != x[j]) ? 1.f : vA[1];
            vA[0] = fmaxf(vA[0], x[j]);
        }
    }
    cluster_allreduce<2, true>(vA, sh.warp, sh.xA, CS, rank, cluster);
    const bool bad = (vA[1] > 0.f) || !(vA[0] > kFloor) || (vA[0] == INFINITY);
    const float m = vA[0];

    // pass B: S = sum 2^t, T = sum 2^t t with t = (z - m) log2e (exactly 0 at the maximum, so
    // S >= 1 and a one-hot row has H == 0 exactly); per-warp S for sampling
    float vB[2] = {0.f, 0.f};
    for (int u = u0 + lane; u < u1; u += 32) {
        float x[N];
        load_unit_w<T, VEC>(row, u, p.V, x, wr);
#pragma unroll
        for (int j = 0; j < N; ++j) {
            float t = (fmaxf(x[j], kFloor) - m) * kLog2e;
            float e = ex2(t);
            vB[0] += e;
            vB[1] = fmaf(e, t, vB[1]);
        }
    }
    {
        float ws = warp_sum(vB[0]);
        if (lane == 0)
            for (int r = 0; r < CS; ++r) cluster.map_shared_rank(sh.wtab, r)[gw] = ws;
    }
    cluster_allreduce<2, false>(vB, sh.warp, sh.xB, CS, rank, cluster);

    const float S = vB[0];
    const float log2S = lg2(S);
    float H = kLn2 * (log2S - vB[1] / S);
    float lse = fmaf(kLn2, log2S, m);
    if (bad) H = lse = NAN;

    // x ~ q by inverse CDF in index order
    const bool sampling = (p.u != nullptr && p.token_out != nullptr);
    if (sampling && !bad) {
        float base = 0.f, target = 0.f;
        int chosen = select_warp(sh.wtab, GW, p.u[b], base, target);
        if (chosen == gw) {
            int tok = warp_scan_select<N>(u0, u1, p.V, base, target, [&](int u, float(&w)[N]) {
                float x[N];
                load_unit_w<T, VEC>(row, u, p.V, x, wr);
#pragma unroll
                for (int j = 0; j < N; ++j) w[j] = ex2((fmaxf(x[j], kFloor) - m) * kLog2e);
            });
            if (lane == 0) p.token_out[b] = tok;
        }
    } else if (sampling && rank == 0 && threadIdx.x == 0) {
        p.token_out[b] = -1;
    }
    if (rank == 0 && threadIdx.x == 0) {
        if (bad) atomicOr(p.st.status, ADASD_STATUS_NAN);
        p.H_out[b] = H;
        if (p.lse_out) p.lse_out[b] = lse;
        const bool stop = H > p.st.T_G[b];   // strict; NaN never stops
        if (p.stop_out) p.stop_out[b] = stop ? 1 : 0;
        if (p.draft_len) p.draft_len[b] += 1;
        if (p.active && stop) p.active[b] = 0;
    }
    cluster.sync();   // no CTA leaves while a peer may still address its shared memory
}

// ------------------------------------------------------------------------------------
// Verification position (b,i): softmax statistics of q_i and p_i, H, D_JS, d_i, y_i ~ p_i
// (AdaSD mode) or alpha_i and the residual sample (vanilla mode).  The cluster that
// publishes the last position of a sequence runs that sequence's tail.
// ------------------------------------------------------------------------------------
template <typename T, bool VEC, int MODE>
__global__ void __launch_bounds__(kThreads) verify_kernel(VerifyParams p) {
    constexpr int N = Elt<T>::N;
    cg::cluster_group cluster = cg::this_cluster();
    const int CS = (int)cluster.num_blocks();
    const int rank = (int)cluster.block_rank();
    const int pos = blockIdx.x / CS;
    const int Kmax = p.Kmax;
    const int b = pos / (Kmax + 1), i = pos % (Kmax + 1);
    int K_t = p.draft_len ? p.draft_len[b] : Kmax;
    K_t = max(0, min(K_t, Kmax));
    if (i > K_t) return;                       // same decision in every CTA of the cluster
    const bool bonus = (i == K_t);

    __shared__ RowShared sh;
    __shared__ TailShared tsh;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int GW = CS * kWarps, gw = rank * kWarps + warp;
    const int NU = (p.V + N - 1) / N;
    const int u0 = (int)((long long)gw * NU / GW), u1 = (int)((long long)(gw + 1) * NU / GW);
    const T* rt = reinterpret_cast<const T*>(p.zt) + (long long)b * p.t_seq + (long long)i * p.t_row;
    const T* rd = bonus ? rt
                        : reinterpret_cast<const T*>(p.zd) + (long long)b * p.d_seq + (long long)i * p.d_row;
    const RowWarp wt = {p.inv_temp, p.cut_t ? p.cut_t[(size_t)b * (Kmax + 1) + i] : -INFINITY};
    const RowWarp wd = {p.inv_temp, (p.cut_d && !bonus) ? p.cut_d[(size_t)b * Kmax + i] : -INFINITY};

    // pass A: maxima, NaN flag, "rows differ" flag
    float vA[4] = {-INFINITY, -INFINITY, 0.f, 0.f};
    for (int u = u0 + lane; u < u1; u += 32) {
        float xt[N], xd[N];
        load_unit_w<T, VEC>(rt, u, p.V, xt, wt);
        if (!bonus) load_unit_w<T, VEC>(rd, u, p.V, xd, wd);
#pragma unroll
        for (int j = 0; j < N; ++j) {
            if (bonus) xd[j] = xt[j];
            vA[2] = (xt[j] != xt[j] || xd[j] != xd[j]) ? 1.f : vA[2];
            vA[3] = (xt[j] != xd[j]) ? 1.f : vA[3];
            vA[0] = fmaxf(vA[0], xt[j]);
            vA[1] = fmaxf(vA[1], xd[j]);
        }
    }
    cluster_allreduce<4, true>(vA, sh.warp, sh.xA, CS, rank, cluster);
    const bool bad = (vA[2] > 0.f) || !(vA[0] > kFloor) || !(vA[1] > kFloor) ||
                     (vA[0] == INFINITY) || (vA[1] == INFINITY);
    const bool differ = vA[3] > 0.f;
    const float mt = vA[0], md = vA[1];

    // pass B: S_t, S_d; per-warp S_t for sampling y_i
    float vB[2] = {0.f, 0.f};
    for (int u = u0 + lane; u < u1; u += 32) {
        float xt[N], xd[N];
        load_unit_w<T, VEC>(rt, u, p.V, xt, wt);
        if (!bonus) load_unit_w<T, VEC>(rd, u, p.V, xd, wd);
#pragma unroll
        for (int j = 0; j < N; ++j) {
            vB[0] += ex2((fmaxf(xt[j], kFloor) - mt) * kLog2e);
            if (!bonus) vB[1] += ex2((fmaxf(xd[j], kFloor) - md) * kLog2e);
        }
    }
    {
        float ws = warp_sum(vB[0]);
        if (lane == 0)
            for (int r = 0; r < CS; ++r) cluster.map_shared_rank(sh.wtab, r)[gw] = ws;
    }
    cluster_allreduce<2, false>(vB, sh.warp, sh.xB, CS, rank, cluster);
    if (bonus) vB[1] = vB[0];
    // log2 p = (z - m) log2e - log2 S: exactly 0 for the only token of a one-hot row
    const float lSt = lg2(vB[0]), lSd = lg2(vB[1]);

    // vanilla: alpha_i at the draft token, known to every thread
    bool van_accept = true;
    float alpha = 1.f;
    if (MODE == MODE_VANILLA && !bonus && !bad) {
        const int xi = p.x[(size_t)b * Kmax + i];
        if (xi >= 0 && xi < p.V) {
            float a = fmaf(fmaxf(apply_warp(to_f32(rt[xi]), wt), kFloor) - mt, kLog2e, -lSt);
            float q = fmaf(fmaxf(apply_warp(to_f32(rd[xi]), wd), kFloor) - md, kLog2e, -lSd);
            alpha = fminf(1.f, ex2(a - q));
            if (!(ex2(q) > 0.f)) alpha = 1.f;   // q(x) = 0 cannot have been drafted
        } else {
            alpha = 0.f;
        }
        van_accept = p.u_accept[(size_t)b * Kmax + i] < alpha;
    }

    // pass C: sum p a', sum q b' (entropies: a' = log2 p, b' = log2 q), sum p q (== 0 means disjoint
    // supports, where D_JS is ln 2 exactly) and the divergence itself from non-negative terms,
    //   D_JS = 1/4 sum s phi(u),  s = p + q,  u = (q - p) / s,  phi(u) = (1-u) ln(1-u) + (1+u) ln(1+u):
    // for |u| < 1/2 the series u^2 + u^4/6 + u^6/15 + u^8/28 + u^10/45, else the two logarithms.
    // Nothing cancels however close the rows are (Sec. 2.2, first printed form, term by term).
    // vanilla on a rejected row: residual mass max(0, p - q), per warp and in total.
    float vC[4] = {0.f, 0.f, 0.f, 0.f};
    const bool need_resid = (MODE == MODE_VANILLA) && !bonus && !van_accept;
    if (MODE == MODE_ADASD || need_resid) {
        for (int u = u0 + lane; u < u1; u += 32) {
            float xt[N], xd[N];
            load_unit_w<T, VEC>(rt, u, p.V, xt, wt);
            if (!bonus) load_unit_w<T, VEC>(rd, u, p.V, xd, wd);
#pragma unroll
            for (int j = 0; j < N; ++j) {
                float a = fmaf(fmaxf(xt[j], kFloor) - mt, kLog2e, -lSt);
                float pp = ex2(a);
                if (MODE == MODE_ADASD) vC[0] = fmaf(pp, a, vC[0]);
                if (!bonus) {
                    float bq = fmaf(fmaxf(xd[j], kFloor) - md, kLog2e, -lSd);
                    float qq = ex2(bq);
                    if (MODE == MODE_ADASD) {
                        vC[1] = fmaf(qq, bq, vC[1]);
                        const float s = pp + qq;
                        if (s > 0.f) {
                            const float rs = __fdividef(1.f, s), uu = (qq - pp) * rs, w = uu * uu;
                            float ph;
                            if (w < 0.25f) {
                                ph = fmaf(w, 1.f / 45.f, 1.f / 28.f);
                                ph = fmaf(ph, w, 1.f / 15.f);
                                ph = fmaf(ph, w, 1.f / 6.f);
                                ph = fmaf(ph, w, 1.f);
                                ph *= w;
                            } else {
                                const float lo = 2.f * pp * rs, hi = 2.f * qq * rs;     // 1 - u and 1 + u, each to full relative accuracy
                                ph = kLn2 * ((lo > 0.f ? lo * lg2(lo) : 0.f) + (hi > 0.f ? hi * lg2(hi) : 0.f));
                            }
                            vC[2] = fmaf(s, ph, vC[2]);
                        }
                        vC[3] = fmaf(pp, qq, vC[3]);
                    } else {
                        vC[3] += fmaxf(pp - qq, 0.f);
                    }
                }
            }
        }
        if (MODE == MODE_VANILLA) {
            float ws = warp_sum(vC[3]);
            if (lane == 0)
                for (int r = 0; r < CS; ++r) cluster.map_shared_rank(sh.wtab2, r)[gw] = ws;
        }
    }
    cluster_allreduce<4, false>(vC, sh.warp, sh.xC, CS, rank, cluster);

    // sampling: y_i ~ p_i (AdaSD: every row; vanilla: bonus row, or residual-less fallback)
    const size_t it = (size_t)b * (Kmax + 1) + i;
    const size_t id = (size_t)b * Kmax + i;
    if (!bad) {
        bool from_resid = need_resid && (vC[3] > 0.f);
        bool do_sample = (MODE == MODE_ADASD) || bonus || need_resid;
        if (do_sample) {
            float uu = (MODE == MODE_ADASD) ? p.u_target[it] : p.u_resample[b];
            float base = 0.f, target = 0.f;
            int chosen = select_warp(from_resid ? sh.wtab2 : sh.wtab, GW, uu, base, target);
            if (chosen == gw) {
                int tok;
                if (from_resid) {
                    tok = warp_scan_select<N>(u0, u1, p.V, base, target, [&](int u, float(&w)[N]) {
                        float xt[N], xd[N];
                        load_unit_w<T, VEC>(rt, u, p.V, xt, wt);
                        load_unit_w<T, VEC>(rd, u, p.V, xd, wd);
#pragma unroll
                        for (int j = 0; j < N; ++j) {
                            float pp = ex2(fmaf(fmaxf(xt[j], kFloor) - mt, kLog2e, -lSt));
                            float qq = ex2(fmaf(fmaxf(xd[j], kFloor) - md, kLog2e, -lSd));
                            w[j] = fmaxf(pp - qq, 0.f);
                        }
                    });
                } else {
                    tok = warp_scan_select<N>(u0, u1, p.V, base, target, [&](int u, float(&w)[N]) {
                        float xt[N];
                        load_unit_w<T, VEC>(rt, u, p.V, xt, wt);
#pragma unroll
                        for (int j = 0; j < N; ++j)
                            w[j] = ex2((fmaxf(xt[j], kFloor) - mt) * kLog2e);
                    });
                }
                if (lane == 0) {
                    if (MODE == MODE_ADASD) {
                        p.sc.y[it] = tok;
                        if (p.user.y) p.user.y[it] = tok;
                    } else {
                        p.sc.van_tok[it] = tok;
                    }
                }
            }
        }
    }

    // publish this position's scalars
    if (rank == 0 && threadIdx.x == 0) {
        if (bad) atomicOr(p.st.status, ADASD_STATUS_NAN);
        if (MODE == MODE_ADASD) {
            float Ht = -kLn2 * vC[0], lse_t = fmaf(kLn2, lSt, mt);
            if (bad) {
                Ht = lse_t = NAN;
                p.sc.y[it] = -1;
                if (p.user.y) p.user.y[it] = -1;
            }
            p.sc.H_t[it] = Ht;
            p.sc.lse_t[it] = lse_t;
            if (p.user.H_t) p.user.H_t[it] = Ht;
            if (p.user.lse_t) p.user.lse_t[it] = lse_t;
            if (!bonus) {
                float Hd = -kLn2 * vC[1], lse_d = fmaf(kLn2, lSd, md);
                float jsd = 0.25f * vC[2];
                jsd = differ ? fminf(fmaxf(jsd, 0.f), kLn2) : 0.f;   // identical rows: exactly 0
                if (!(vC[3] > 0.f)) jsd = kLn2;                      // disjoint supports: exactly ln 2
                float dist = sqrtf(jsd / kLn2);
                dist = fminf(dist, 1.f);
                if (bad) Hd = lse_d = jsd = dist = NAN;
                p.sc.H_d[id] = Hd;
                p.sc.lse_d[id] = lse_d;
                p.sc.jsd[id] = jsd;
                p.sc.dist[id] = dist;
                if (p.user.H_d) p.user.H_d[id] = Hd;
                if (p.user.lse_d) p.user.lse_d[id] = lse_d;
                if (p.user.jsd) p.user.jsd[id] = jsd;
                if (p.user.dist) p.user.dist[id] = dist;
            }
        } else {
            if (!bonus) {
                p.sc.van_flag[id] = (van_accept && !bad) ? 1 : 0;
                if (p.alpha_out) p.alpha_out[id] = bad ? NAN : alpha;
            }
            if (bad) p.sc.van_tok[it] = -1;
        }
    }

    // all writes of this cluster are done once every CTA has passed this barrier
    cluster.sync();
    if (rank != 0) return;
    if (threadIdx.x == 0) {
        __threadfence();
        unsigned old = atomicAdd(p.sc.ticket + b, 1u);
        int last = (old == (unsigned)K_t);
        if (last) {
            p.sc.ticket[b] = 0u;    // ready for the next round
            __threadfence();
        }
        sh.is_last = last;
    }
    __syncthreads();
    if (!sh.is_last) return;

    if (MODE == MODE_ADASD) {
        TailIO io;
        io.H_d = p.sc.H_d;
        io.dist = p.sc.dist;
        io.y = p.sc.y;
        io.x = p.x;
        io.u_accept = p.u_accept;
        io.draft_len = p.draft_len;
        io.p_acc = p.sc.p_acc;
        io.p_acc_user = p.user.p_acc;
        io.accept_len = p.accept_len;
        io.next_token = p.next_token;
        io.accept_len_rec = p.user.accept_len;
        io.rejected_rec = p.user.rejected;
        io.draft_len_rec = p.user.draft_len;
        verify_tail(p.tail, io, p.st, b, tsh);
    } else if (threadIdx.x == 0) {
        int w = K_t;
        for (int j = 0; j < K_t; ++j) {
            if (__ldcg(p.sc.van_flag + (size_t)b * Kmax + j) == 0) {
                w = j;
                break;
            }
        }
        p.accept_len[b] = w;
        p.next_token[b] = __ldcg(p.sc.van_tok + (size_t)b * (Kmax + 1) + w);
    }
}

// ------------------------------------------------------------------------------------
// Stand-alone update from a record (for callers that do not fuse it into verify)
// ------------------------------------------------------------------------------------
__global__ void update_kernel(State st, adasd_round_record rec, int B, int Kmax) {
    int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    int K_t = max(0, min(rec.draft_len[b], Kmax));
    int w = max(0, min(rec.accept_len[b], K_t));
    bool rejected = rec.rejected[b] != 0 && w < K_t;
    apply_update(st, b, w, rejected, rec.dist + (size_t)b * Kmax, rec.H_d + (size_t)b * Kmax);
}

__global__ void reset_kernel(State st, const int32_t* ids, int n, int B) {
    int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= n) return;
    int b = ids ? ids[k] : k;
    if (b < 0 || b >= B) return;
    st.T_G[b] = 0.f;
    st.sumE[b] = 0.0;
    st.nE[b] = st.nA[b] = st.nR[b] = 0;
    st.sumA[b] = st.sumA2[b] = st.sumR[b] = st.sumR2[b] = 0.0;
}

__global__ void get_thresholds_kernel(State st, float* T_G, int32_t* nE, int32_t* nA, int32_t* nR,
                                      int B) {
    int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    if (T_G) T_G[b] = st.T_G[b];
    if (nE) nE[b] = st.nE[b];
    if (nA) nA[b] = st.nA[b];
    if (nR) nR[b] = st.nR[b];
}

}  // namespace adasd
