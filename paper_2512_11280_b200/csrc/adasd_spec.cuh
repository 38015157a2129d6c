// Warp-specialised verification kernel for sm_100a (AdaSD mode and vanilla speculative
// sampling mode).
//
// Persistent thread-block clusters; a position (b,i) = target row p_i + draft row q_i (bf16).
// The CTAs of a cluster split both rows into contiguous slices, the compute warps of a CTA
// split the CTA's slice into contiguous runs of "iterations" (one iteration = 32 lanes x 16
// bytes of each row).  Every logit row is read from HBM exactly once, by 1-D bulk copies
// (cp.async.bulk) into per-warp buffers that hold two whole positions; the copy of position
// n + 2 is issued the moment position n is done with, so HBM never waits for the arithmetic.
// Values live in the log2 domain: t = z log2 e - M, 2^t kept in registers for the first
// iterations and, for the rest, parked in the buffer over logits that have been used up.
//
//  * 12 COMPUTE warps per CTA (three per scheduler) do nothing but the passes over their share of a position
//    (A: maxima and flags; B: 2^t, S = sum 2^t and T = sum 2^t t; C: (p+q) log2 (p+q) in
//    AdaSD mode, the residual mass max(0, p - q) of a rejected row in vanilla mode), the
//    refill of their own buffers and, for the one warp that holds it, the inverse-CDF crossing.
//  * 1 CONTROL warp per CTA finds the cluster's positions, folds the warp partials into the
//    CTA's totals, exchanges them with the other CTAs of the cluster (st.async into their
//    shared memory, counted on their mbarriers: no cluster-wide barrier in the loop) and
//    turns the row totals into two small messages per compute warp: its scale factors (and,
//    vanilla, whether the row was accepted), then whether it holds the inverse-CDF crossing.
//  * 1 TAIL warp (leader CTA) finalises each position once the compute warps' sums are in,
//    draws the sequence's ticket and runs the tails (KDE/Bayes, accept scan, list appends,
//    T_G; vanilla: longest accepted prefix) of completed sequences, off everybody's critical
//    path; AdaSD tails are handed to the idle tail warps of the cluster's other CTAs.
//
// The CTA has 16 warps = four warpgroups.  All threads start with 128 registers; the warpgroup
// of service warps (control, tail and two idle warps) hands registers back with setmaxnreg and
// the three warpgroups of compute warps take them: 144 registers per compute thread, 80 per
// service thread.
//
// Every wait (buffer filled, partials in, totals in, message ready, sums in, queue) is bounded:
// a warp whose wait expires sets ADASD_STATUS_TIMEOUT, stops waiting and copying, and walks
// through the rest of the protocol, so the kernel always ends.
#pragma once

#include "adasd_cluster.cuh"

namespace adasd {

constexpr int kSW = 12;                          // compute warps per CTA
constexpr int kSCtl = kSW;                       // warp index of the control warp
constexpr int kSTail = kSW + 1;                  // warp index of the tail warp
constexpr int kSThreads = (kSW + 4) * 32;        // 512: three warpgroups of compute warps, one of service warps
constexpr int kSRegIter = 5;                     // iterations whose 2^t values stay in registers
constexpr int kSMaxIter = 10;                    // largest number of iterations per warp and row
// Iteration k >= kSRegIter parks its 2^t values in the buffer pieces of iterations 2 (k - kSRegIter)
// and 2 (k - kSRegIter) + 1, which must have been consumed before it: 2 (k - kSRegIter) + 1 < k.
static_assert(2 * (kSMaxIter - 1 - kSRegIter) + 1 <= kSMaxIter - 1, "parked 2^t values would overwrite unread logits");
static_assert(kSW <= kCW, "the exchange tables are sized for kCW warps");
constexpr int kSPosRing = 16;                    // positions the control warp keeps described
constexpr int kSWorkQ = 16;                      // tail work queue entries per CTA
constexpr int kSFinRing = 4;                     // positions whose sums may await finalisation
constexpr uint32_t kSPollSpins = 1u << 24;       // polls of a progress counter before giving up

// One position as the control warp describes it to the compute warps of its CTA.
struct __align__(16) PosCtx {
    unsigned long long src_t;     // global address of the CTA's slice of the target row
    unsigned long long src_d;     // ... of the draft row (unused for a bonus row)
    int32_t pos;                  // index into [B, Kmax+1]; >= total: none
    int32_t kt;                   // window K_t of its sequence
    int32_t bonus;                // 1: the sequence's bonus row (target row only)
    int32_t pad;
};

// What a compute warp needs after the exchange: p = 2^t_p * at, q = 2^t_q * ad; and, if it
// holds the inverse-CDF crossing (sel), the weight before its share and the target.
struct __align__(16) WarpMsg {
    float at, ad, ft;             // first part: ready when scal_bar completes
    int32_t act;                  // vanilla: 0 nothing left to do, 1 sample from p, 2 residual pass
    float target;                 // second part: ready when sel_bar completes
    int32_t sel;
    float base;
    int32_t pad1;
};

struct __align__(16) SpecShared {
    PosCtx pc[kSPosRing];
    RowPart wtab[2][kCW];             // this CTA's compute warps, by position parity
    RowPart ctab[2][kCMaxCluster];    // every CTA's totals (written over DSMEM), by parity
    WarpMsg wmsg[2][kCW];
    float4 tabC[kSFinRing][kCTab];    // leader: per-warp (sum s log2 s, sum 2^t_p 2^t_q, token or -1), by position
    float fin[kSFinRing][12];         // leader: row totals (and alpha, accept flag) kept for finalisation
    float rw[kCW];                    // vanilla: residual mass of each compute warp's share
    float4 rtab[kCMaxCluster];        // vanilla: every CTA's residual mass (written over DSMEM)
    unsigned long long entry_bar[2];  // one arrival per compute warp: wtab[par] complete
    unsigned long long ctab_bar[2];   // CS * 32 bytes from the control warps of the cluster: ctab[par] complete
    unsigned long long scal_bar[2];   // 1 arrival: first part of wmsg[par] ready
    unsigned long long sel_bar[2];    // 1 arrival: second part of wmsg[par] ready
    unsigned long long c_bar[kSFinRing];   // leader: 16 bytes from every compute warp of the cluster: tabC complete
    unsigned long long resid_bar;     // vanilla: one arrival per compute warp: rw complete
    unsigned long long r_bar;         // vanilla: CS * 16 bytes from the control warps of the cluster: rtab complete
    unsigned long long bar[kCW][2];   // per compute warp: "position buffer filled" barriers
    int32_t n_issued;                 // leader: positions whose messages have been sent
    int32_t n_final;                  // leader: number of positions of this cluster, -1 until known
    int32_t fin_done;                 // leader: positions finalised so far (written by the tail warp)
    int32_t wq[kSWorkQ];              // non-leader: sequences whose tail this CTA's tail warp must run (-1: stop)
    uint32_t wq_head, wq_tail;        // written by the leader's tail warp (remotely) / by this CTA's tail warp
    float td[ADASD_KMAX_LIMIT], tH[ADASD_KMAX_LIMIT];   // tail warp scratch
};

// ---- mbarrier helpers with explicit scopes -----------------------------------------------
__device__ __forceinline__ void mbar_arrive_cta(uint64_t* bar) {
    asm volatile("mbarrier.arrive.release.cta.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// shared::cluster address of `p` (an address in this CTA's shared memory) as seen in CTA `cta`
__device__ __forceinline__ uint32_t mapa_u32(const void* p, uint32_t cta) {
    uint32_t r;
    asm("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_u32(p)), "r"(cta));
    return r;
}
// 16 bytes into another CTA's shared memory; their arrival is counted (complete_tx) on a
// barrier of THAT CTA, so the receiver needs no fence and the sender no second message
__device__ __forceinline__ void st_async_v4(uint32_t remote_addr, float4 v, uint32_t remote_bar) {
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.f32 [%0], {%1, %2, %3, %4}, [%5];"
                 ::"r"(remote_addr), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w), "r"(remote_bar)
                 : "memory");
}

__device__ __forceinline__ void st_cluster_u32(uint32_t remote_addr, uint32_t v) {
    asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(remote_addr), "r"(v) : "memory");
}
__device__ __forceinline__ uint32_t ld_cluster_u32(uint32_t remote_addr) {
    uint32_t v;
    asm volatile("ld.volatile.shared::cluster.u32 %0, [%1];" : "=r"(v) : "r"(remote_addr) : "memory");
    return v;
}
__device__ __forceinline__ void fence_cluster() { asm volatile("fence.acq_rel.cluster;" ::: "memory"); }

// The per-sequence tail of a round, run by ONE warp: lane i owns candidate i.  Same
// arithmetic as verify_tail (KDE sums over L_D^A and L_D^R, Bayes posterior with the
// round's earlier distances counted as accepted, first-rejection scan, appends, T_G).
// sd/sH: 32-entry shared-memory scratch of this warp.
__device__ __forceinline__ void verify_tail_warp(const TailConfig& cfg, const TailIO& io, State& st, int b,
                                                 float* sd, float* sH) {
    const int lane = threadIdx.x & 31;
    const int Kmax = cfg.Kmax;
    int K_t = io.draft_len ? __ldcg(io.draft_len + b) : Kmax;
    K_t = max(0, min(K_t, Kmax));
    float d = 0.f, H = 0.f, u = 0.f;
    int x = 0, y = 0;
    if (lane < K_t) {
        d = __ldcg(io.dist + (size_t)b * Kmax + lane);
        H = __ldcg(io.H_d + (size_t)b * Kmax + lane);
        y = __ldcg(io.y + (size_t)b * (Kmax + 1) + lane);
        x = io.x[(size_t)b * Kmax + lane];
        u = io.u_accept[(size_t)b * Kmax + lane];
        sd[lane] = d;
        sH[lane] = H;
    }
    __syncwarp();
    const int nA0 = st.nA[b], nR0 = st.nR[b];
    const bool inside = d > 0.f && d < 1.f;          // enters the KDE lists when accepted

    // bandwidths: candidate i sees L_D^A plus the distances d_1..d_{i-1} of this round that
    // lie strictly inside (0,1): the list "as it stands" when candidate i is reached at all
    double n = (double)nA0, s = st.sumA[b], s2 = st.sumA2[b];
    for (int j = 0; j < K_t; ++j) {
        const float dj = __shfl_sync(0xFFFFFFFFu, d, j);
        if (j < lane && dj > 0.f && dj < 1.f) {
            n += 1.0;
            s += (double)dj;
            s2 += (double)dj * (double)dj;
        }
    }
    const double hA = kde_bandwidth(n, s, s2, cfg.bw_rule);
    const bool ok = lane < K_t && (n >= (double)cfg.min_samples) && (hA > 0.0);
    const float cA = ok ? (float)(-0.5 * 1.4426950408889634 / (hA * hA)) : 0.f;
    const float ihA = ok ? (float)(1.0 / hA) : 0.f;
    const double hR = kde_bandwidth((double)nR0, st.sumR[b], st.sumR2[b], cfg.bw_rule);
    const bool validR = (nR0 >= cfg.min_samples) && (hR > 0.0);
    const float cR = validR ? (float)(-0.5 * 1.4426950408889634 / (hR * hR)) : 0.f;
    const float ihR = validR ? (float)(1.0 / hR) : 0.f;
    const bool any_valid = (__ballot_sync(0xFFFFFFFFu, ok) != 0u) && validR;

    float SA = 0.f, SR = 0.f;
    if (any_valid) {
        const float* LA = st.LA + (size_t)b * st.cap;
        const float* LR = st.LR + (size_t)b * st.cap;
        for (int i0 = 0; i0 < K_t; i0 += 8) {
            float accA[8], accR[8], di[8], ci[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const int i = min(i0 + k, K_t - 1);
                accA[k] = accR[k] = 0.f;
                di[k] = __shfl_sync(0xFFFFFFFFu, d, i);
                ci[k] = __shfl_sync(0xFFFFFFFFu, cA, i);
            }
            for (int j = lane; j < nA0; j += 32) {
                const float xj = __ldcg(LA + j);
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const float t = di[k] - xj;
                    accA[k] += ex2(ci[k] * t * t);
                }
            }
            for (int j = lane; j < nR0; j += 32) {
                const float xj = __ldcg(LR + j);
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const float t = di[k] - xj;
                    accR[k] += ex2(cR * t * t);
                }
            }
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const float a = warp_sum(accA[k]), r = warp_sum(accR[k]);
                if (lane == i0 + k) {
                    SA = a;
                    SR = r;
                }
            }
        }
    }
    // kernel terms of this round's earlier distances, then the posterior
    float extra = 0.f;
    for (int j = 0; j < K_t; ++j) {
        const float dj = __shfl_sync(0xFFFFFFFFu, d, j);
        if (j < lane && dj > 0.f && dj < 1.f) {
            const float t = d - dj;
            extra += ex2(cA * t * t);
        }
    }
    float P = 0.f;
    if (any_valid && ok) {
        // n_A f_A = SA / (h_A sqrt(2 pi)),  n_R f_R = SR / (h_R sqrt(2 pi))
        const float a = (SA + extra) * ihA;
        const float r = SR * ihR;
        const float den = a + r;
        if (den > 0.f && den < INFINITY) P = a / den;
    }
    if (lane < K_t) {
        io.p_acc[(size_t)b * Kmax + lane] = P;
        if (io.p_acc_user) io.p_acc_user[(size_t)b * Kmax + lane] = P;
    }
    const bool rej = cfg.reject_rule == 0 ? (u >= P) : (P < 0.5f);
    const unsigned m = __ballot_sync(0xFFFFFFFFu, lane < K_t && x != y && rej);
    (void)inside;
    if (lane == 0) {
        const int w = m ? (__ffs(m) - 1) : K_t;
        const bool rejected = (m != 0u);
        io.accept_len[b] = w;
        io.next_token[b] = __ldcg(io.y + (size_t)b * (Kmax + 1) + w);
        if (io.accept_len_rec) io.accept_len_rec[b] = w;
        if (io.rejected_rec) io.rejected_rec[b] = rejected ? 1 : 0;
        if (io.draft_len_rec) io.draft_len_rec[b] = K_t;
        if (cfg.update) apply_update(st, b, w, rejected, sd, sH);
    }
    __syncwarp();
}

// ------------------------------------------------------------------------------------
template <int ITER, int MODE>
__global__ void __launch_bounds__(kSThreads, 1)
spec_verify_kernel(VerifyParams p, ClusterGeom gq) {
    constexpr int KR = ITER < kSRegIter ? ITER : kSRegIter;   // iterations kept in registers
    extern __shared__ __align__(128) unsigned char dyn_smem[];
    __shared__ SpecShared sh;

    cg::cluster_group cluster = cg::this_cluster();
    const int CS = (int)cluster.num_blocks();
    const int rank = (int)cluster.block_rank();
    const int cid = blockIdx.x / CS;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int Kmax = p.Kmax, K1 = Kmax + 1;
    const int total = p.B * K1;
    const int ncl = gq.ncl;
    const bool leader = (rank == 0);
    const int NU = p.V >> 3;                                   // 16-byte units per row
    const int cu0 = (int)((long long)rank * NU / CS), cu1 = (int)((long long)(rank + 1) * NU / CS);

    for (int q = threadIdx.x; q < kSFinRing * kCTab; q += kSThreads)
        reinterpret_cast<float4*>(sh.tabC)[q] = make_float4(0.f, 0.f, __int_as_float(-1), 0.f);
    if (threadIdx.x < kSPosRing) {
        sh.pc[threadIdx.x].pos = total;
        sh.pc[threadIdx.x].kt = 0;
        sh.pc[threadIdx.x].bonus = 0;
    }
    if (threadIdx.x == 0) {
        sh.n_issued = 0;
        sh.n_final = -1;
        sh.fin_done = 0;
        sh.wq_head = sh.wq_tail = 0u;
        for (int k = 0; k < 2; ++k) {
            mbar_init(reinterpret_cast<uint64_t*>(&sh.entry_bar[k]), kSW);
            mbar_init(reinterpret_cast<uint64_t*>(&sh.ctab_bar[k]), 1);
            mbar_init(reinterpret_cast<uint64_t*>(&sh.scal_bar[k]), 1);
            mbar_init(reinterpret_cast<uint64_t*>(&sh.sel_bar[k]), 1);
        }
        for (int k = 0; k < kSFinRing; ++k) mbar_init(reinterpret_cast<uint64_t*>(&sh.c_bar[k]), 1);
        mbar_init(reinterpret_cast<uint64_t*>(&sh.resid_bar), kSW);
        mbar_init(reinterpret_cast<uint64_t*>(&sh.r_bar), 1);
    }
    if (warp < kSW && lane == 0)
        for (int s = 0; s < 2; ++s) mbar_init(reinterpret_cast<uint64_t*>(&sh.bar[warp][s]), 1);
    __syncthreads();

    // first active position among start, start + ncl, ... (32 candidates per round)
    auto window = [&](int b) -> int {
        int kt = p.draft_len ? __ldg(p.draft_len + b) : Kmax;
        return max(0, min(kt, Kmax));
    };
    auto scan_from = [&](int start) -> PosRef {
        PosRef r;
        r.pos = total;
        r.kt = 0;
        for (int base = start; base < total; base += 32 * ncl) {
            const long long cl = (long long)base + (long long)lane * ncl;
            int kt = 0;
            bool ok = false;
            if (cl < total) {
                const int c = (int)cl, b = c / K1;
                kt = window(b);
                ok = (c - b * K1) <= kt;
            }
            const unsigned m = __ballot_sync(0xFFFFFFFFu, ok);
            if (m) {
                const int src = __ffs(m) - 1;
                r.pos = base + src * ncl;
                r.kt = __shfl_sync(0xFFFFFFFFu, kt, src);
                break;
            }
        }
        return r;
    };
    // control warp: describe position number n to the compute warps
    auto set_pos = [&](int n, const PosRef& r) {
        if (lane == 0) {
            PosCtx& c = sh.pc[n & (kSPosRing - 1)];
            c.pos = r.pos;
            c.kt = r.kt;
            if (r.pos < total) {
                const int b = r.pos / K1, i = r.pos - b * K1;
                c.bonus = (i == r.kt) ? 1 : 0;
                c.src_t = (unsigned long long)(reinterpret_cast<const __nv_bfloat16*>(p.zt) + (long long)b * p.t_seq +
                                               (long long)i * p.t_row + (size_t)cu0 * 8);
                c.src_d = (unsigned long long)(reinterpret_cast<const __nv_bfloat16*>(p.zd) + (long long)b * p.d_seq +
                                               (long long)i * p.d_row + (size_t)cu0 * 8);
            }
        }
        __syncwarp();
    };
    PosRef lastp;               // control warp: the latest position it has described
    lastp.pos = total;
    lastp.kt = 0;
    if (warp == kSCtl) {
        PosRef r = scan_from(cid);
        set_pos(0, r);
        for (int n = 1; n < 3; ++n) {
            if (r.pos < total) r = scan_from(r.pos + ncl);
            set_pos(n, r);
        }
        lastp = r;
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    cluster.sync();   // barriers and positions are set up in every CTA of the cluster

    // 512 threads start with 128 registers each.  The warpgroup of service warps (two of its four
    // warps have work) gives registers back, the three warpgroups of compute warps take them:
    // 12 x 32 x 144 + 4 x 32 x 80 = 65536.
    if (warp < kSW) asm volatile("setmaxnreg.inc.sync.aligned.u32 144;");
    else asm volatile("setmaxnreg.dec.sync.aligned.u32 80;");

    bool alive = true;         // false after a wait expired: this warp stops waiting and copying
    auto expired = [&]() {
        alive = false;
        if (lane == 0) atomicOr(p.st.status, ADASD_STATUS_TIMEOUT);
    };
    auto wait_cta = [&](unsigned long long* bar, uint32_t par) {
        if (!alive) return;
        bool ok = mbar_wait_bounded(reinterpret_cast<uint64_t*>(bar), par);
        ok = __all_sync(0xFFFFFFFFu, ok);
        if (!ok) expired();
    };

    if (warp < kSW) {
        // ============================== compute warp ======================================
        // Its share of a row: iterations [wi0, wi0 + I_w) of the CTA's slice; the host sizes
        // ITER so that every warp of every CTA gets ITER - 1 or ITER iterations.
        const int g = rank * kSW + warp;
        const int nwi = (cu1 - cu0 + 31) >> 5;                     // warp-iterations of this CTA
        // the first I_rem warps have one iteration more (every scheduler carries three compute warps)
        const int I_lo = nwi / kSW, I_rem = nwi % kSW;
        auto extra = [&](int w) -> int { return w < I_rem ? 1 : 0; };
        int wi0 = 0;
        for (int w = 0; w < warp; ++w) wi0 += I_lo + extra(w);
        const int I_w = min(ITER, I_lo + extra(warp));
        const bool full = (I_w == ITER);                           // the last iteration exists
        const int wu0 = cu0 + 32 * wi0;
        const int nwu = max(0, min(32 * I_w, cu1 - wu0));          // units of this warp (last one ragged)
        const uint32_t row_bytes = (uint32_t)nwu * 16u;            // this warp's share of one row
        const size_t woff = (size_t)wi0 * 512;                     // its byte offset in the CTA's slice

        // Two buffers per warp, one position each: [target share | draft share], ITER * 512 bytes
        // per row.  Position n lives in buffer n & 1 and is replaced by position n + 2 as soon as
        // pass C of position n is done, one whole position before it is needed.
        const int kRowB = I_w * 512;              // bytes of one row in this warp's buffers
        unsigned char* const bufs = dyn_smem + (size_t)wi0 * 2048;
        auto buf_of = [&](int n) -> unsigned char* { return bufs + (size_t)(n & 1) * (2 * kRowB) + (size_t)lane * 16; };
        auto bar_of = [&](int n) -> uint64_t* { return reinterpret_cast<uint64_t*>(&sh.bar[warp][n & 1]); };
        auto pcx = [&](int n) -> const PosCtx& { return sh.pc[n & (kSPosRing - 1)]; };

        // lanes 0 and 1 fetch the two rows of position n (lane 1 idles for a bonus row)
        auto issue_pos = [&](int n) {
            const PosCtx& c = pcx(n);
            if (!alive || nwu == 0 || c.pos >= total) return;
            const bool bonus = c.bonus != 0;
            uint64_t* bar = bar_of(n);
            unsigned char* dst = bufs + (size_t)(n & 1) * (2 * kRowB);
            // (the copies may complete before the expected byte count is posted: the phase cannot
            // end before this warp's one arrival, which comes with the count)
            if (lane == 0) mbar_expect_tx(bar, bonus ? row_bytes : 2u * row_bytes);
            if (lane < (bonus ? 1 : 2))
                bulk_g2s(dst + lane * kRowB,
                         reinterpret_cast<const unsigned char*>(lane ? c.src_d : c.src_t) + woff, row_bytes, bar);
        };
        issue_pos(0);
        issue_pos(1);

        // iteration k runs for this warp: all but the last always do
        auto k_on = [&](int k) -> bool { return (k < ITER - 1) || full; };
        // Only one of a warp's last two iterations can be ragged (the CTA's slice need not end
        // on a 32-unit boundary): lanes past the end take the clamp value, i.e. probability 0.
        auto mask_unit = [&](int k, uint4& w) {
            if (k >= ITER - 2 && !(lane + 32 * k < nwu))
                w = make_uint4(0xF149F149u, 0xF149F149u, 0xF149F149u, 0xF149F149u);
        };

        // ---- pass A: packed maxima and flags of one position ---------------------------------
        uint32_t a_mT = 0xFF80FF80u, a_mD = 0xFF80FF80u, a_df = 0u;   // -inf pairs
        bool a_done = false;
        // with blocking == false it gives up at once if the position has not landed yet
        auto pass_a = [&](auto bonus_c, int n, bool blocking) {
            constexpr bool BONUS = decltype(bonus_c)::value;
            if (!alive || a_done) return;
            if (nwu > 0) {
                const uint32_t par = (uint32_t)(n >> 1) & 1u;
                bool ok = blocking ? mbar_wait_bounded(bar_of(n), par) : (mbar_test_wait(bar_of(n), par) != 0);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) {
                    if (blocking) expired();     // the copy never landed
                    return;
                }
            }
            a_done = true;
            const unsigned char* sb = buf_of(n);
#pragma unroll
            for (int k = 0; k < ITER; ++k) {
                if (k_on(k)) {
                    uint4 T = *reinterpret_cast<const uint4*>(sb + k * 512);
                    mask_unit(k, T);
                    a_mT = bmax2(bmax2(a_mT, T.x), bmax2(T.y, bmax2(T.z, T.w)));
                    if (!BONUS) {
                        uint4 D = *reinterpret_cast<const uint4*>(sb + kRowB + k * 512);
                        mask_unit(k, D);
                        a_mD = bmax2(bmax2(a_mD, D.x), bmax2(D.y, bmax2(D.z, D.w)));
                        a_df |= (T.x ^ D.x) | (T.y ^ D.y) | (T.z ^ D.z) | (T.w ^ D.w);
                    }
                }
            }
        };
        auto pass_a_any = [&](bool bonus, int n, bool blocking) {
            if (bonus) pass_a(std::true_type{}, n, blocking);
            else pass_a(std::false_type{}, n, blocking);
        };

        // The warp's shifts and flags from the packed accumulators.  Every kept value is
        // 2^((z - max) log2 e) with the share's own largest logit, exactly 1 for that logit;
        // shares combine in the log2 domain through the differences of M = fl(max * log2 e).
        // A slice without a finite logit gets M = kFloorL and all-zero values.
        float nmt_w = 0.f, nmd_w = 0.f;           // addends of pass B (-max, or 0 for an empty slice)
        uint32_t flags_w = 0;
        auto finish_a = [&](bool bonus) {
            const float2 a = unpack2(a_mT), d = unpack2(a_mD);
            uint32_t bad = (a.x != a.x || a.y != a.y || d.x != d.x || d.y != d.y) ? 1u : 0u;
            const float vt = warp_max_f32(fmaxf(a.x, a.y));
            const float vd = bonus ? vt : warp_max_f32(fmaxf(d.x, d.y));
            if (vt == INFINITY || vd == INFINITY || !alive) bad = 1u;
            const bool has_t = vt > ADASD_FLOOR_BF, has_d = vd > ADASD_FLOOR_BF;
            nmt_w = has_t ? -vt : 0.f;
            nmd_w = has_d ? -vd : 0.f;
            // bits 4 and 8 (not published): the target / draft share has no finite logit
            flags_w = __reduce_or_sync(0xFFFFFFFFu, bad | (a_df ? 2u : 0u)) | (has_t ? 0u : 4u) | (has_d ? 0u : 8u);
            a_mT = a_mD = 0xFF80FF80u;
            a_df = 0u;
            a_done = false;
        };

        // 2^t values of one unit: 8 logits (four packed words) relative to the shift in `nm`
        // nv = -(largest logit of the share): t = (z - max) log2 e is exactly 0 for the largest
        // logit, so that a one-hot row gets S = 1, T = 0, p = 1 and H = 0 exactly.
        auto exps = [&](const uint4& W, const float2 nv, float (&e)[8], float2& S, float2& Tq) {
            const float2 L2 = make_float2(kLog2e, kLog2e);
            const uint32_t w[4] = {W.x, W.y, W.z, W.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float2 z = unpack2(bclamp2(w[j]));
                const float2 t = __fmul2_rn(__fadd2_rn(z, nv), L2);
                const float2 v = make_float2(ex2(t.x), ex2(t.y));
                e[2 * j] = v.x;
                e[2 * j + 1] = v.y;
                S = __fadd2_rn(S, v);
                Tq = __ffma2_rn(v, t, Tq);
            }
        };

        // ---- pass B: the warp's S and T; the 2^t values of the first KR iterations are kept ----
        float et[KR][8], ed[KR][8];
        float sB[4];                       // after pass_b: warp totals St, Tt, Sd, Td
        auto pass_b = [&](auto bonus_c, int n) {
            constexpr bool BONUS = decltype(bonus_c)::value;
            float2 St = make_float2(0.f, 0.f), Tt = St, Sd = St, Td = St;
            const float2 nmt = make_float2(nmt_w, nmt_w), nmd = make_float2(nmd_w, nmd_w);
            const unsigned char* sb = buf_of(n);
#pragma unroll
            for (int k = 0; k < ITER; ++k) {
                if (k_on(k)) {
                    float e1[8], e2[8];
                    uint4 T = *reinterpret_cast<const uint4*>(sb + k * 512);
                    mask_unit(k, T);
                    exps(T, nmt, e1, St, Tt);
                    if (!BONUS) {
                        uint4 D = *reinterpret_cast<const uint4*>(sb + kRowB + k * 512);
                        mask_unit(k, D);
                        exps(D, nmd, e2, Sd, Td);
                    } else {
#pragma unroll
                        for (int j = 0; j < 8; ++j) e2[j] = 0.f;
                    }
                    if (k < KR) {
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            et[k < KR ? k : 0][j] = e1[j];
                            ed[k < KR ? k : 0][j] = e2[j];
                        }
                    } else {
                        // no register left: the values go over logits this lane has already turned
                        // into 2^t values (two 512-byte pieces of each row per iteration)
                        float4* st = reinterpret_cast<float4*>(const_cast<unsigned char*>(sb) + (k - KR) * 1024);
                        st[0] = make_float4(e1[0], e1[1], e1[2], e1[3]);
                        st[32] = make_float4(e1[4], e1[5], e1[6], e1[7]);
                        if (!BONUS) {
                            float4* sd = reinterpret_cast<float4*>(const_cast<unsigned char*>(sb) + kRowB + (k - KR) * 1024);
                            sd[0] = make_float4(e2[0], e2[1], e2[2], e2[3]);
                            sd[32] = make_float4(e2[4], e2[5], e2[6], e2[7]);
                        }
                    }
                }
            }
            sB[0] = warp_sum(St.x + St.y);
            sB[1] = warp_sum(Tt.x + Tt.y);
            if (BONUS) {
                sB[2] = sB[0];
                sB[3] = sB[1];
            } else {
                sB[2] = warp_sum(Sd.x + Sd.y);
                sB[3] = warp_sum(Td.x + Td.y);
            }
        };
        // The 2^t values of iteration k (compile-time k after unrolling): from registers, or from
        // where pass B left them in the position's buffer.
        auto load_kept = [&](int k, int n, bool with_d, float (&a)[8], float (&b)[8]) {
            if (k < KR) {
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    a[j] = et[k < KR ? k : 0][j];
                    b[j] = ed[k < KR ? k : 0][j];
                }
            } else {
                const unsigned char* sb = buf_of(n);
                const float4* st = reinterpret_cast<const float4*>(sb + (k - KR) * 1024);
                const float4 a0 = st[0], a1 = st[32];
                a[0] = a0.x, a[1] = a0.y, a[2] = a0.z, a[3] = a0.w, a[4] = a1.x, a[5] = a1.y, a[6] = a1.z, a[7] = a1.w;
                if (with_d) {
                    const float4* sd = reinterpret_cast<const float4*>(sb + kRowB + (k - KR) * 1024);
                    const float4 b0 = sd[0], b1 = sd[32];
                    b[0] = b0.x, b[1] = b0.y, b[2] = b0.z, b[3] = b0.w, b[4] = b1.x, b[5] = b1.y, b[6] = b1.z, b[7] = b1.w;
                } else {
#pragma unroll
                    for (int j = 0; j < 8; ++j) b[j] = 0.f;
                }
            }
        };

        // Run by the warp that holds the crossing: first element (index order: iteration, lane,
        // element) where base + f * running weight exceeds target, else the last element with
        // weight.  vals(k, v) fills the 8 weights of this lane's unit of iteration k.
        auto select_kept = [&](float base, float f, float target, auto vals) -> int {
            float ls[ITER], tot[ITER];
#pragma unroll
            for (int k = 0; k < ITER; ++k) {
                ls[k] = 0.f;
                if (k_on(k)) {
                    float v[8];
                    vals(k, v);
                    ls[k] = ((v[0] + v[1]) + (v[2] + v[3])) + ((v[4] + v[5]) + (v[6] + v[7]));
                }
            }
#pragma unroll
            for (int k = 0; k < ITER; ++k) tot[k] = warp_sum(ls[k]);
            int ksel = -1, klast = -1;
            float run = 0.f, runsel = 0.f, runlast = 0.f;
#pragma unroll
            for (int k = 0; k < ITER; ++k) {
                if (tot[k] > 0.f) {
                    klast = k;
                    runlast = run;
                    if (ksel < 0 && fmaf(f, run + tot[k], base) > target) {
                        ksel = k;
                        runsel = run;
                    }
                }
                run += tot[k];
            }
            if (ksel < 0) {
                ksel = klast;
                runsel = runlast;
                target = INFINITY;
            }
            if (ksel < 0) return -1;
            float v[8], lsum = 0.f;
#pragma unroll
            for (int j = 0; j < 8; ++j) v[j] = 0.f;
#pragma unroll
            for (int k = 0; k < ITER; ++k) {
                if (k == ksel) {          // same for the whole warp
                    vals(k, v);
                    lsum = ls[k];
                }
            }
            float incl = lsum;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const float t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                if (lane >= o) incl += t;
            }
            float c = runsel + (incl - lsum);
            int hit = -1, lastp = -1;
            const int e0 = (wu0 + lane + 32 * ksel) * 8;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                c += v[j];
                if (v[j] > 0.f) {
                    lastp = e0 + j;
                    if (hit < 0 && fmaf(f, c, base) > target) hit = e0 + j;
                }
            }
            const unsigned mh = __ballot_sync(0xFFFFFFFFu, hit >= 0);
            if (mh) return __shfl_sync(0xFFFFFFFFu, hit, __ffs(mh) - 1);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) lastp = max(lastp, __shfl_xor_sync(0xFFFFFFFFu, lastp, o));
            return lastp;
        };

        // ---------------------------------- main loop ----------------------------------------
        int n = 0;                 // sequence number of the current position
        if (pcx(0).pos < total) {
            pass_a_any(pcx(0).bonus != 0, 0, true);
            finish_a(pcx(0).bonus != 0);
        }
        while (pcx(n).pos < total) {
            const int par = n & 1;
            const uint32_t ph = (uint32_t)(n >> 1) & 1u;
            const bool bonus = pcx(n).bonus != 0;
            const int npos = pcx(n + 1).pos;
            const bool nbonus = npos < total && pcx(n + 1).bonus != 0;

            if (bonus) pass_b(std::true_type{}, n);
            else pass_b(std::false_type{}, n);
            if (lane == 0) {
                float4* w = reinterpret_cast<float4*>(&sh.wtab[par][warp]);
                const float Mt_w = (flags_w & 4u) ? kFloorL : -nmt_w * kLog2e;
                const float Md_w = (flags_w & 8u) ? kFloorL : -nmd_w * kLog2e;
                w[0] = make_float4(Mt_w, sB[0], sB[1], Md_w);
                w[1] = make_float4(sB[2], sB[3], __uint_as_float(flags_w & 3u), 0.f);
                mbar_arrive_cta(reinterpret_cast<uint64_t*>(&sh.entry_bar[par]));
            }
            __syncwarp();
            // while the control warps exchange the totals: maxima of the next position, if it
            // has landed in the other buffer
            bool a_fin = false;        // the next position's shifts are worked out already
            if (npos < total) {
                pass_a_any(nbonus, n + 1, false);
                if (a_done) {          // nothing of position n needs this warp's shifts any more
                    finish_a(nbonus);
                    a_fin = true;
                }
            }
            wait_cta(&sh.scal_bar[par], ph);
            const float4 m0 = *reinterpret_cast<const float4*>(&sh.wmsg[par][warp]);       // at, ad, ft

            // the target row's 2^t values of iteration k (what y_i ~ p_i is drawn from)
            auto vals_p = [&](int k, float(&v)[8]) {
                float d[8];
                load_kept(k, n, false, v, d);
            };
            float A = 0.f, PQ = 0.f;
            int tok = -1;
            if (MODE == MODE_ADASD) {
                // pass C: sum (p+q) log2 (p+q) and the overlap indicator sum 2^t_p 2^t_q
                if (!bonus) {
                    float2 A2 = make_float2(0.f, 0.f), PQ2 = make_float2(0.f, 0.f);
                    const float2 at2 = make_float2(m0.x, m0.x), ad2 = make_float2(m0.y, m0.y);
                    const float2 tiny2 = make_float2(kTiny, kTiny);
#pragma unroll
                    for (int k = 0; k < ITER; ++k) {
                        if (k_on(k)) {
                            float a[8], d[8];
                            load_kept(k, n, true, a, d);
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                const float2 a2 = make_float2(a[2 * j], a[2 * j + 1]);
                                const float2 d2 = make_float2(d[2 * j], d[2 * j + 1]);
                                const float2 pp = __ffma2_rn(a2, at2, tiny2);
                                const float2 ss = __ffma2_rn(d2, ad2, pp);
                                const float2 ll = make_float2(lg2(ss.x), lg2(ss.y));
                                A2 = __ffma2_rn(ss, ll, A2);
                                PQ2 = __ffma2_rn(a2, d2, PQ2);
                            }
                        }
                    }
                    A = warp_sum(A2.x + A2.y);
                    PQ = warp_sum(PQ2.x + PQ2.y);
                }
                // y_i ~ p_i: the control warp says (a little later than the scale factors) whether
                // this warp holds the crossing
                wait_cta(&sh.sel_bar[par], ph);
                const float4 m1 = *reinterpret_cast<const float4*>(&sh.wmsg[par][warp].target);   // target, sel, base
                if (__float_as_int(m1.y) != 0) tok = select_kept(m1.z, m0.z, m1.x, vals_p);
            } else {
                // vanilla: an accepted row needs nothing more; the bonus row draws from p; a rejected
                // row draws from the residual max(0, p - q) / R, whose mass this warp now adds up
                const int act = __float_as_int(m0.w);
                const float at = m0.x, ad = m0.y;
                auto vals_r = [&](int k, float(&v)[8]) {
                    float a[8], d[8];
                    load_kept(k, n, true, a, d);
#pragma unroll
                    for (int j = 0; j < 8; ++j) v[j] = fmaxf(fmaf(a[j], at, -d[j] * ad), 0.f);
                };
                if (act == 2) {
                    float r = 0.f;
#pragma unroll
                    for (int k = 0; k < ITER; ++k) {
                        if (k_on(k)) {
                            float v[8];
                            vals_r(k, v);
                            r += ((v[0] + v[1]) + (v[2] + v[3])) + ((v[4] + v[5]) + (v[6] + v[7]));
                        }
                    }
                    r = warp_sum(r);
                    if (lane == 0) {
                        sh.rw[warp] = r;
                        mbar_arrive_cta(reinterpret_cast<uint64_t*>(&sh.resid_bar));
                    }
                    __syncwarp();
                }
                if (act != 0) {
                    wait_cta(&sh.sel_bar[par], ph);
                    const float4 m1 = *reinterpret_cast<const float4*>(&sh.wmsg[par][warp].target);   // target, sel, base
                    const int sel = __float_as_int(m1.y);
                    if (sel == 1) tok = select_kept(m1.z, m0.z, m1.x, vals_p);
                    else if (sel == 2) tok = select_kept(m1.z, 1.f, m1.x, vals_r);
                }
            }
            // the buffer of position n is free: fetch position n + 2 into it (the bulk copy belongs
            // to the async proxy and must come after this warp's own stores to the buffer)
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            issue_pos(n + 2);
            // this warp's sums (and the token, if it drew it) go to the leader CTA in one message
            if (lane == 0) {
                const int fr = n & (kSFinRing - 1);
                st_async_v4(mapa_u32(&sh.tabC[fr][g], 0u), make_float4(A, PQ, __int_as_float(tok), 0.f),
                            mapa_u32(&sh.c_bar[fr], 0u));
            }
            __syncwarp();

            // the next position's maxima, if its copy had not landed during the exchange
            if (npos < total && !a_fin) {
                pass_a_any(nbonus, n + 1, true);
                finish_a(nbonus);
            }
            ++n;
        }
        // a warp that gave up on a copy still waits (bounded) for whatever it had in flight
        if (!alive && nwu > 0) {
            mbar_wait_bounded(bar_of(n), (uint32_t)(n >> 1) & 1u);
            mbar_wait_bounded(bar_of(n + 1), (uint32_t)((n + 1) >> 1) & 1u);
        }
    } else if (warp == kSCtl) {
        // ============================== control warp ======================================
        auto sum8 = [&](float v) -> float {       // total of the first eight lanes, in every lane
            v += __shfl_xor_sync(0xFFFFFFFFu, v, 4);
            v += __shfl_xor_sync(0xFFFFFFFFu, v, 2);
            v += __shfl_xor_sync(0xFFFFFFFFu, v, 1);
            return __shfl_sync(0xFFFFFFFFu, v, 0);
        };
        int n = 0;
        uint32_t nres = 0;                        // residual exchanges so far (phase of their barriers)
        while (sh.pc[n & (kSPosRing - 1)].pos < total) {
            const int par = n & 1;
            const uint32_t ph = (uint32_t)(n >> 1) & 1u;
            // describe position n + 3 while the compute warps are busy with position n
            {
                PosRef r;
                r.pos = total;
                r.kt = 0;
                if (lastp.pos < total) r = scan_from(lastp.pos + ncl);
                set_pos(n + 3, r);
                lastp = r;
            }
            // per-position scalars, fetched before the wait so that they are there after it
            const PosCtx& pcn = sh.pc[n & (kSPosRing - 1)];
            const bool bonus = pcn.bonus != 0;
            float u_samp, u_acc = 0.f, ztx = 0.f, zdx = 0.f;
            bool x_ok = false;
            if (MODE == MODE_ADASD) {
                u_samp = __ldg(p.u_target + pcn.pos);
            } else {
                const int b = pcn.pos / K1, i = pcn.pos - b * K1;
                u_samp = __ldg(p.u_resample + b);
                if (!bonus) {
                    const size_t idd = (size_t)b * Kmax + i;
                    u_acc = __ldg(p.u_accept + idd);
                    const int xi = __ldg(p.x + idd);
                    x_ok = xi >= 0 && xi < p.V;
                    if (x_ok) {
                        ztx = __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p.zt)[(long long)b * p.t_seq + (long long)i * p.t_row + xi]);
                        zdx = __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p.zd)[(long long)b * p.d_seq + (long long)i * p.d_row + xi]);
                    }
                }
            }

            // the CTA's totals from its compute warps, sent to every CTA of the cluster
            wait_cta(&sh.entry_bar[par], ph);
            if (leader && lane == 0) {
                // before anybody can send sums of position n: the ring entry it reuses (position
                // n - kSFinRing) must have been finalised
                bool room = !alive;
                for (uint32_t it = 0; !room && it < kSPollSpins; ++it) {
                    room = *reinterpret_cast<volatile int32_t*>(&sh.fin_done) > n - kSFinRing;
                    if (!room) __nanosleep(100);
                }
                if (!room) atomicOr(p.st.status, ADASD_STATUS_TIMEOUT);
                // every compute warp of the cluster will send 16 bytes for position n
                mbar_expect_tx(reinterpret_cast<uint64_t*>(&sh.c_bar[n & (kSFinRing - 1)]), (uint32_t)(CS * kSW * 16));
            }
            __syncwarp();
            float4 w0 = make_float4(kFloorL, 0.f, 0.f, kFloorL), w1 = make_float4(0.f, 0.f, 0.f, 0.f);
            if (lane < kSW) {
                const float4* w = reinterpret_cast<const float4*>(&sh.wtab[par][lane]);
                w0 = w[0];
                w1 = w[1];
            }
            {
                const float Mt = warp_max_f32(w0.x), Md = warp_max_f32(w0.w);
                const float dt = w0.x - Mt, dd = w0.w - Md;
                const float ft = ex2(dt), fd = ex2(dd);
                const float St = warp_sum(ft * w0.y), Tt = warp_sum(ft * fmaf(dt, w0.y, w0.z));
                const float Sd = warp_sum(fd * w1.x), Td = warp_sum(fd * fmaf(dd, w1.x, w1.y));
                const uint32_t fl = __reduce_or_sync(0xFFFFFFFFu, __float_as_uint(w1.z));
                if (lane == 0) mbar_expect_tx(reinterpret_cast<uint64_t*>(&sh.ctab_bar[par]), (uint32_t)(CS * 32));
                if (lane < CS) {
                    const uint32_t dst = mapa_u32(&sh.ctab[par][rank], (uint32_t)lane);
                    const uint32_t bar = mapa_u32(&sh.ctab_bar[par], (uint32_t)lane);
                    st_async_v4(dst, make_float4(Mt, St, Tt, Md), bar);
                    st_async_v4(dst + 16, make_float4(Sd, Td, __uint_as_float(fl), 0.f), bar);
                }
            }
            // the row's totals from the CTA totals, lane c holding CTA c
            wait_cta(&sh.ctab_bar[par], ph);
            float4 e0 = make_float4(kFloorL, 0.f, 0.f, kFloorL), e1 = make_float4(0.f, 0.f, 0.f, 0.f);
            if (lane < CS) {
                const float4* e = reinterpret_cast<const float4*>(&sh.ctab[par][lane]);
                e0 = e[0];
                e1 = e[1];
            }
            const float Mt = warp_max_f32(e0.x), Md = warp_max_f32(e0.w);
            const float cdt = e0.x - Mt, cdd = e0.w - Md;
            const float cft = ex2(cdt), cfd = ex2(cdd);
            const float st_c = cft * e0.y;                    // CTA sums of the target row, scaled to Mt
            const float St = sum8(st_c), Sd = sum8(cfd * e1.x);

            // vanilla: alpha = min(1, p(x) / q(x)) at the draft token, and what is left to do
            const uint32_t fl = __reduce_or_sync(0xFFFFFFFFu, __float_as_uint(e1.z));
            const bool bad = (fl & 1u) || !(Mt > kFloorL) || !(Md > kFloorL);
            float alpha = 0.f;
            bool van_accept = true;
            int act = 1;                          // AdaSD: every row draws y_i ~ p_i
            if (MODE == MODE_VANILLA) {
                if (!bonus) {
                    if (x_ok) {
                        const float a = fmaf(fmaxf(ztx, ADASD_FLOOR_BF), kLog2e, -Mt) - lg2(St);
                        const float q = fmaf(fmaxf(zdx, ADASD_FLOOR_BF), kLog2e, -Md) - lg2(Sd);
                        alpha = fminf(1.f, ex2(a - q));
                        if (!(ex2(q) > 0.f)) alpha = 1.f;   // q(x) = 0 cannot have been drafted
                    }
                    van_accept = u_acc < alpha;
                }
                act = bad ? 0 : (bonus ? 1 : (van_accept ? 0 : 2));
            }

            // first message per compute warp (lane w): its scale factors; pass C starts on it
            const float ftw = ex2(w0.x - Mt), fdw = ex2(w0.w - Md);
            // correctly rounded quotients: a one-hot row must get p = 1 exactly, so that two rows
            // that are one-hot on the same token give p + q = 2 and a divergence of exactly 0
            const float at = __fdiv_rn(ftw, St), ad = __fdiv_rn(fdw, Sd);
            if (lane < kSW) *reinterpret_cast<float4*>(&sh.wmsg[par][lane]) = make_float4(at, ad, ftw, __int_as_float(act));
            __syncwarp();
            if (lane == 0) mbar_arrive_cta(reinterpret_cast<uint64_t*>(&sh.scal_bar[par]));

            // Off the critical path: T totals for the finaliser, then the second message.
            const float Tt = sum8(cft * fmaf(cdt, e0.y, e0.z)), Td = sum8(cfd * fmaf(cdd, e1.x, e1.y));
            // Which warp holds the crossing of `target`
            // in index order (CTA by CTA, then warp by warp), given the weight cw of CTA `lane` and
            // the weight ww of this CTA's compute warp `lane`; `kind` says what the warp scans.
            int sel = 0;
            float base = 0.f, target = 0.f;
            auto locate = [&](float cw, float ww, float tgt, int kind) {
                target = tgt;
                float incl = cw;
#pragma unroll
                for (int o = 1; o < 8; o <<= 1) {
                    const float t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                    if (lane >= o) incl += t;
                }
                const bool mass = lane < CS && cw > 0.f;
                int cstar = -1;
                const unsigned mc = __ballot_sync(0xFFFFFFFFu, mass && incl > target);
                if (mc) {
                    cstar = __ffs(mc) - 1;
                } else {
                    const unsigned ml = __ballot_sync(0xFFFFFFFFu, mass);
                    if (ml) cstar = 31 - __clz(ml);
                    target = INFINITY;
                }
                const float cbase = __shfl_sync(0xFFFFFFFFu, incl - cw, max(cstar, 0));
                if (cstar == rank) {
                    const float w = (lane < kSW) ? ww : 0.f;
                    float winc = w;
#pragma unroll
                    for (int o = 1; o < 16; o <<= 1) {
                        const float t = __shfl_up_sync(0xFFFFFFFFu, winc, o);
                        if (lane >= o) winc += t;
                    }
                    int wsel = -1;
                    const unsigned mh = __ballot_sync(0xFFFFFFFFu, w > 0.f && cbase + winc > target);
                    if (mh) {
                        wsel = __ffs(mh) - 1;
                    } else {
                        const unsigned ml = __ballot_sync(0xFFFFFFFFu, w > 0.f);
                        if (ml) wsel = 31 - __clz(ml);
                        target = INFINITY;
                    }
                    if (lane == wsel) {
                        sel = kind;
                        base = cbase + (winc - w);
                    }
                }
            };
            bool from_p = (act == 1);
            if (MODE == MODE_VANILLA && act == 2) {
                // residual mass: warp sums -> CTA sum -> every CTA of the cluster
                const uint32_t rph = nres & 1u;
                ++nres;
                wait_cta(&sh.resid_bar, rph);
                const float rwv = (lane < kSW) ? sh.rw[lane] : 0.f;
                const float r_cta = warp_sum(rwv);
                if (lane == 0) mbar_expect_tx(reinterpret_cast<uint64_t*>(&sh.r_bar), (uint32_t)(CS * 16));
                __syncwarp();
                if (lane < CS)
                    st_async_v4(mapa_u32(&sh.rtab[rank], (uint32_t)lane), make_float4(r_cta, 0.f, 0.f, 0.f),
                                mapa_u32(&sh.r_bar, (uint32_t)lane));
                wait_cta(&sh.r_bar, rph);
                const float rc = (lane < CS) ? sh.rtab[lane].x : 0.f;
                const float R = sum8(rc);
                if (R > 0.f && alive) locate(rc, rwv, u_samp * R, 2);
                else from_p = true;               // no residual mass: draw from p
            }
            if (from_p && !bad) locate(st_c, ftw * w0.y, u_samp * St, 1);
            if (lane < kSW)
                *reinterpret_cast<float4*>(&sh.wmsg[par][lane].target) = make_float4(target, __int_as_float(sel), base, 0.f);
            if (leader && lane == 0) {
                float* f = sh.fin[n & (kSFinRing - 1)];
                f[0] = Mt;
                f[1] = St;
                f[2] = Tt;
                f[3] = Md;
                f[4] = Sd;
                f[5] = Td;
                f[6] = __uint_as_float(fl | (alive ? 0u : 1u));
                f[7] = alpha;
                f[8] = van_accept ? 1.f : 0.f;
            }
            __syncwarp();
            if (lane == 0) {
                mbar_arrive_cta(reinterpret_cast<uint64_t*>(&sh.sel_bar[par]));
                if (leader) {
                    __threadfence_block();
                    *reinterpret_cast<volatile int32_t*>(&sh.n_issued) = n + 1;
                }
            }
            ++n;
        }
        if (leader && lane == 0) {
            __threadfence_block();
            *reinterpret_cast<volatile int32_t*>(&sh.n_final) = n;
        }
    } else if (warp == kSTail) {
        // ================================ tail warp =======================================
        // Leader CTA only: finalises every position of the cluster, in order, as soon as its sums
        // are in, and runs the tail of each sequence whose last position that was.
        if (leader) {
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
            // leader: the published scalars of position number m, once every compute warp of the
            // cluster has sent its pass-C sums (they did before publishing their next partials)
            auto finalize = [&](int m) -> int {
                const int par = m & (kSFinRing - 1);
                wait_cta(&sh.c_bar[par], (uint32_t)(m / kSFinRing) & 1u);
                const float4 c0 = sh.tabC[par][4 * lane], c1 = sh.tabC[par][4 * lane + 1];
                const float4 c2 = sh.tabC[par][4 * lane + 2], c3 = sh.tabC[par][4 * lane + 3];
                const float A = warp_sum(((c0.x + c1.x) + c2.x) + c3.x);
                const float PQ = warp_sum(((c0.y + c1.y) + c2.y) + c3.y);
                const int tok_all = __reduce_max_sync(0xFFFFFFFFu, max(max(__float_as_int(c0.z), __float_as_int(c1.z)),
                                                                       max(__float_as_int(c2.z), __float_as_int(c3.z))));
                int done_b = -1;
                if (lane == 0) {
                    const PosCtx& c = sh.pc[m & (kSPosRing - 1)];
                    const int b = c.pos / K1, i = c.pos - b * K1;
                    const bool bonus = c.bonus != 0;
                    const float Mt = sh.fin[par][0], St = sh.fin[par][1], Tt = sh.fin[par][2];
                    const float Md = sh.fin[par][3], Sd = sh.fin[par][4], Td = sh.fin[par][5];
                    const uint32_t fl = __float_as_uint(sh.fin[par][6]);
                    const bool bad = (fl & 1u) || !(Mt > kFloorL) || !(Md > kFloorL) || !alive;
                    const size_t idt = (size_t)b * K1 + i, idd = (size_t)b * Kmax + i;
                    int tok = tok_all;
                    if (bad) {
                        atomicOr(p.st.status, ADASD_STATUS_NAN);
                        tok = -1;
                    }
                    if (MODE == MODE_VANILLA) {
                        if (!bonus) {
                            p.sc.van_flag[idd] = (sh.fin[par][8] != 0.f && !bad) ? 1 : 0;
                            if (p.alpha_out) p.alpha_out[idd] = bad ? NAN : sh.fin[par][7];
                        }
                        p.sc.van_tok[idt] = tok;
                    } else {
                    const float lSt = lg2(St), lSd = lg2(Sd);
                    const float Hbt = lSt - Tt / St, Hbd = lSd - Td / Sd;      // entropies in bits
                    float Ht = kLn2 * Hbt, lse_t = kLn2 * (Mt + lSt);
                    if (bad) Ht = lse_t = NAN;
                    p.sc.H_t[idt] = Ht;
                    p.sc.lse_t[idt] = lse_t;
                    p.sc.y[idt] = tok;
                    if (p.user.H_t) p.user.H_t[idt] = Ht;
                    if (p.user.lse_t) p.user.lse_t[idt] = lse_t;
                    if (p.user.y) p.user.y[idt] = tok;
                    if (!bonus) {
                        float Hd = kLn2 * Hbd, lse_d = kLn2 * (Md + lSd);
                        // D_JS = H(m) - (H(p) + H(q)) / 2 with H(m) = (ln 2 / 2) (2 - sum s log2 s), s = p + q
                        float jsd = 0.5f * kLn2 * ((2.f - A) - (Hbt + Hbd));
                        jsd = (fl & 2u) ? fminf(fmaxf(jsd, 0.f), kLn2) : 0.f;   // identical rows: exactly 0
                        if (!(PQ > 0.f)) jsd = kLn2;                            // disjoint supports: ln 2
                        float dist = fminf(sqrtf(jsd / kLn2), 1.f);
                        if (bad) Hd = lse_d = jsd = dist = NAN;
                        p.sc.H_d[idd] = Hd;
                        p.sc.lse_d[idd] = lse_d;
                        p.sc.jsd[idd] = jsd;
                        p.sc.dist[idd] = dist;
                        if (p.user.H_d) p.user.H_d[idd] = Hd;
                        if (p.user.lse_d) p.user.lse_d[idd] = lse_d;
                        if (p.user.jsd) p.user.jsd[idd] = jsd;
                        if (p.user.dist) p.user.dist[idd] = dist;
                    }
                    }
                    __threadfence();
                    const unsigned ticket = atomicAdd(p.sc.ticket + b, 1u);
                    if (ticket == (unsigned)c.kt) {
                        p.sc.ticket[b] = 0u;          // ready for the next round
                        done_b = b;
                    }
                }
                return __shfl_sync(0xFFFFFFFFu, done_b, 0);
            };

            // tails go round robin to the tail warps of the other CTAs of the cluster, which have
            // nothing else to do: entry number k of CTA r's queue
            uint32_t ndisp = 0;
            auto send = [&](uint32_t r, uint32_t k, int b) {
                if (lane == 0) {
                    const uint32_t tail_addr = mapa_u32(&sh.wq_tail, r);
                    bool room = !alive;
                    for (uint32_t it = 0; !room && it < kSPollSpins; ++it) {
                        room = (k - ld_cluster_u32(tail_addr)) < (uint32_t)kSWorkQ;
                        if (!room) __nanosleep(100);
                    }
                    if (room) {
                        __threadfence();
                        st_cluster_u32(mapa_u32(&sh.wq[k % kSWorkQ], r), (uint32_t)b);
                        fence_cluster();
                        st_cluster_u32(mapa_u32(&sh.wq_head, r), k + 1u);
                    } else {
                        atomicOr(p.st.status, ADASD_STATUS_TIMEOUT);
                    }
                }
                __syncwarp();
            };
            auto dispatch = [&](int b) {
                const uint32_t nw = (uint32_t)(CS - 1);
                send(1u + ndisp % nw, ndisp / nw, b);
                ++ndisp;
            };
            for (int m = 0;; ++m) {
                // position m exists once its messages have gone out; the control warp says when
                // the cluster has no more
                int go = -1;
                if (lane == 0) {
                    for (uint32_t it = 0; it < kSPollSpins; ++it) {
                        if (*reinterpret_cast<volatile int32_t*>(&sh.n_issued) > m) {
                            go = 1;
                            break;
                        }
                        if (*reinterpret_cast<volatile int32_t*>(&sh.n_final) == m) {
                            go = 0;
                            break;
                        }
                        __nanosleep(100);
                    }
                    if (go < 0) atomicOr(p.st.status, ADASD_STATUS_TIMEOUT);
                }
                go = __shfl_sync(0xFFFFFFFFu, go, 0);
                if (go <= 0) break;
                const int done_b = finalize(m);
                if (done_b >= 0) {
                    if (MODE == MODE_VANILLA) {
                        // longest accepted prefix, then the token drawn at the first rejection
                        // (or the bonus token)
                        __threadfence();
                        const int kt = window(done_b);
                        const bool rej = lane < kt && __ldcg(p.sc.van_flag + (size_t)done_b * Kmax + lane) == 0;
                        const unsigned mr = __ballot_sync(0xFFFFFFFFu, rej);
                        if (lane == 0) {
                            const int w = mr ? (__ffs(mr) - 1) : kt;
                            p.accept_len[done_b] = w;
                            p.next_token[done_b] = __ldcg(p.sc.van_tok + (size_t)done_b * K1 + w);
                        }
                    } else if (CS > 1) {
                        dispatch(done_b);
                    } else {
                        __threadfence();
                        verify_tail_warp(p.tail, io, p.st, done_b, sh.td, sh.tH);
                    }
                }
                if (lane == 0) {
                    __threadfence_block();
                    *reinterpret_cast<volatile int32_t*>(&sh.fin_done) = m + 1;
                }
            }
            // stop marks: CTA r has received the entries ndisp' < ndisp with ndisp' % nw == r - 1
            for (uint32_t r = 1; r < (uint32_t)CS; ++r) {
                const uint32_t nw = (uint32_t)(CS - 1);
                const uint32_t sent = ndisp / nw + ((ndisp % nw) > (r - 1u) ? 1u : 0u);
                send(r, sent, -1);
            }
        } else {
            // worker: tails handed over by the leader's tail warp, in order, until the stop mark
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
            for (uint32_t k = 0;; ++k) {
                int b = -2;
                if (lane == 0) {
                    for (uint32_t it = 0; it < kSPollSpins; ++it) {
                        if (*reinterpret_cast<volatile uint32_t*>(&sh.wq_head) != k) {
                            fence_cluster();
                            b = *reinterpret_cast<volatile int32_t*>(&sh.wq[k % kSWorkQ]);
                            break;
                        }
                        __nanosleep(200);
                    }
                    if (b == -2) atomicOr(p.st.status, ADASD_STATUS_TIMEOUT);
                }
                b = __shfl_sync(0xFFFFFFFFu, b, 0);
                if (b < 0) break;            // stop mark, or nothing ever came
                __threadfence();
                verify_tail_warp(p.tail, io, p.st, b, sh.td, sh.tH);
                if (lane == 0) *reinterpret_cast<volatile uint32_t*>(&sh.wq_tail) = k + 1u;
            }
        }
    }
    cluster.sync();   // no CTA leaves while a peer may still address its shared memory
}

}  // namespace adasd
