// Warp-specialised verification kernel for sm_100a (AdaSD mode and vanilla speculative
// sampling mode).
//
// Persistent thread-block clusters; a position (b,i) = target row p_i + draft row q_i (bf16).
// The CTAs of a cluster split both rows into contiguous slices, the compute warps of a CTA
// split the CTA's slice into contiguous runs of "iterations" (one iteration = 32 lanes x 16
// bytes of each row).  Every logit row is read from HBM exactly once, by 1-D bulk copies
// (cp.async.bulk) into per-warp buffers that hold two whole positions; the copy of position
// n + 2 is issued the moment the logits of position n have been turned into 2^t values, so
// HBM never waits for the arithmetic.  Values live in the log2 domain: t = z log2 e - M.  The
// 2^t values of a position wait for the row totals in TENSOR MEMORY (the SM's 256 KB that the
// tensor cores would use as accumulators; nothing here is a contraction, so it is free): the
// first iterations of a warp's share go there (tcgen05.st), the rest stay in registers.
// That leaves room for the head of position n + 1 to be worked through while the totals of
// position n are exchanged: the special-function pipe does not idle during the exchange.
//
//  * 12 COMPUTE warps per CTA (three per scheduler) do nothing but the passes over their share of a position
//    (A: maxima and flags; B: 2^t, S = sum 2^t, T = sum 2^t t and the largest |z_t - z_d|;
//    C: (p+q) log2 (p+q) in AdaSD mode - or, when the two rows are nearly equal everywhere, the
//    well-conditioned sum of (p+q) phi((q-p)/(q+p)) - and the residual mass max(0, p - q) of a
//    rejected row in vanilla mode), the refill of their own buffers and, for the one warp that
//    holds it, the inverse-CDF crossing.  Per position: A(n+1), head of B(n+1) | wait for the
//    scale factors of n | C(n) | tail of B(n+1), publish its partials, refill.
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
// The CTA has 16 warps of 128 registers per thread: the whole register file (136 per compute
// thread and 104 per service thread after setmaxnreg).
//
// Tensor memory: 512 columns x 128 lanes of 32 bits, allocated once per CTA by the control warp.
// A warp may only touch the 32 lanes of its quarter (warp index mod 4), so the three compute
// warps of a quarter split the columns: 160 each = two halves (position parity) of kSHead
// slots of 16 columns; a slot holds one iteration's 8 target and 8 draft values per lane.
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
constexpr int kSHead = 5;                        // iterations whose 2^t values wait in tensor memory
constexpr int kSRegIter = 5;                     // ... and in registers, at most
constexpr int kSMaxIter = kSHead + kSRegIter;    // largest number of iterations per warp and row
constexpr int kSTmemCols = 512;                  // columns allocated (all of them: one CTA per SM)
constexpr int kSTmemHalf = kSHead * 16;          // columns of one position's head: 16 per iteration
constexpr int kSTmemWarp = 2 * kSTmemHalf;       // columns of one compute warp: two positions in flight
static_assert((kSW / 4) * kSTmemWarp <= kSTmemCols, "the compute warps of a lane quarter share its columns");
static_assert(kSW % 4 == 0, "compute warps are spread evenly over the four lane quarters");
static_assert(kSW <= kCW, "the exchange tables are sized for kCW warps");
constexpr float kSNearDz = 0.5f;                 // rows count as nearly equal when no logit differs by more
constexpr int kSPosRing = 16;                    // positions the control warp keeps described
constexpr int kSFinRing = 4;                     // positions whose sums may await finalisation
constexpr uint32_t kSPollSpins = 1u << 24;       // polls of a progress counter before giving up

// One position as the control warp describes it to the compute warps of its CTA.
struct __align__(16) PosCtx {
    unsigned long long src_t;     // global address of the CTA's slice of the target row
    unsigned long long src_d;     // ... of the draft row (unused for a bonus row)
    int32_t pos;                  // index into [B, Kmax+1]; >= total: none
    int32_t kt;                   // window K_t of its sequence
    int32_t bonus;                // 1: the sequence's bonus row (target row only)
    uint32_t cut_t;               // adjusted distribution: the target row's cutoff logit as a bf16 pair
    uint32_t cut_d;               // ... the draft row's (kNoCut2: nothing is cut)
    int32_t pad[3];
};

// What a compute warp needs after the exchange: p = 2^t_p * at, q = 2^t_q * ad; and, if it
// holds the inverse-CDF crossing (sel), the weight before its share and the target.
struct __align__(16) WarpMsg {
    float at, ad, ft;             // first part: ready when scal_bar completes
    int32_t act;                  // vanilla: 0 nothing left to do, 1 sample from p, 2 residual pass;
                                  // AdaSD: 1, plus 4 when the rows are nearly equal (pass C in its u form)
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
    RowPart finc[kSFinRing][kCMaxCluster];   // leader: every CTA's totals, kept for the float64 finalisation
    uint32_t tmem_base;               // tensor-memory address the allocation returned
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
    float td[3][ADASD_KMAX_LIMIT], tH[3][ADASD_KMAX_LIMIT];   // scratch of the three tail workers of a CTA
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

// ---- tensor memory as a scratchpad ---------------------------------------------------------
// Allocation and release are warp-wide; the address lands in shared memory.
__device__ __forceinline__ void tmem_alloc(uint32_t* smem_dst, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_dst)), "r"(ncols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// 16 consecutive columns of this thread's lane: a[0..7] then b[0..7]
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const float (&a)[8], const float (&b)[8]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "f"(a[0]), "f"(a[1]), "f"(a[2]), "f"(a[3]), "f"(a[4]), "f"(a[5]), "f"(a[6]), "f"(a[7]),
          "f"(b[0]), "f"(b[1]), "f"(b[2]), "f"(b[3]), "f"(b[4]), "f"(b[5]), "f"(b[6]), "f"(b[7])
        : "memory");
}
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const float (&a)[8]) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                 ::"r"(taddr), "f"(a[0]), "f"(a[1]), "f"(a[2]), "f"(a[3]), "f"(a[4]), "f"(a[5]), "f"(a[6]), "f"(a[7])
                 : "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// The loads are asynchronous: the registers hold the values only after tmem_wait_ld, which
// takes them as operands so that nothing that uses them can be scheduled ahead of the wait.
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&a)[8], float (&b)[8]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=f"(a[0]), "=f"(a[1]), "=f"(a[2]), "=f"(a[3]), "=f"(a[4]), "=f"(a[5]), "=f"(a[6]), "=f"(a[7]),
          "=f"(b[0]), "=f"(b[1]), "=f"(b[2]), "=f"(b[3]), "=f"(b[4]), "=f"(b[5]), "=f"(b[6]), "=f"(b[7])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, float (&a)[8]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=f"(a[0]), "=f"(a[1]), "=f"(a[2]), "=f"(a[3]), "=f"(a[4]), "=f"(a[5]), "=f"(a[6]), "=f"(a[7])
                 : "r"(taddr)
                 : "memory");
}
__device__ __forceinline__ void tmem_wait_ld(float (&a)[8], float (&b)[8]) {
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+f"(a[0]), "+f"(a[1]), "+f"(a[2]), "+f"(a[3]), "+f"(a[4]), "+f"(a[5]), "+f"(a[6]), "+f"(a[7]),
                   "+f"(b[0]), "+f"(b[1]), "+f"(b[2]), "+f"(b[3]), "+f"(b[4]), "+f"(b[5]), "+f"(b[6]), "+f"(b[7])
                 :
                 : "memory");
}
__device__ __forceinline__ void tmem_wait_ld(float (&a)[8]) {
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+f"(a[0]), "+f"(a[1]), "+f"(a[2]), "+f"(a[3]), "+f"(a[4]), "+f"(a[5]), "+f"(a[6]), "+f"(a[7])
                 :
                 : "memory");
}
__device__ __forceinline__ float rcp_approx(float x) {
    float y;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ double warp_sum_f64(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

// The published scalars of one position from the CTAs' statistics (lane c holds CTA c) and the
// warps' pass-C sums, worked out in float64 by the whole tail warp.  In fp32 the totals
// (entropies of up to 17 bits, log2 of sums of up to 2^17) carry errors of about 1e-6 each, which
// the difference H(m) - (H(p) + H(q)) / 2 keeps.
struct FinOut {
    float Ht, lse_t, Hd, lse_d, jsd, dist;
};
// Top-k / top-p cut of one lane's units of a position buffer, in place (iterations are 512 bytes
// apart; row_b: offset of the draft row, 0 for a bonus row).  Kept out of line: it runs only when
// an adjusted distribution is set, and must not cost the ordinary path registers.
__device__ __noinline__ void cut_buffer(unsigned char* sb, int iters, int row_b, uint32_t c2t, uint32_t c2d) {
    for (int k = 0; k < iters; ++k) {
        uint4 T = *reinterpret_cast<const uint4*>(sb + k * 512);
        bcut8(T, c2t);
        *reinterpret_cast<uint4*>(sb + k * 512) = T;
        if (row_b) {
            uint4 D = *reinterpret_cast<const uint4*>(sb + row_b + k * 512);
            bcut8(D, c2d);
            *reinterpret_cast<uint4*>(sb + row_b + k * 512) = D;
        }
    }
}

__device__ __forceinline__ FinOut finalize_math(const RowPart* finc, int CS, float Mt, float Md, double A, float PQ,
                                             uint32_t fl, bool near) {
    const int lane = threadIdx.x & 31;
    // row totals: S = sum f_c S_c, T = sum f_c (T_c + (M_c - M) S_c) with f_c = 2^(M_c - M)
    double St = 0.0, Tt = 0.0, Sd = 0.0, Td = 0.0;
    if (lane < CS) {
        const float4* fc = reinterpret_cast<const float4*>(finc + lane);
        const float4 e0 = fc[0], e1 = fc[1];
        const double dt = (double)e0.x - (double)Mt, dd = (double)e0.w - (double)Md;
        const double ft = e0.x > kFloorL ? exp2(dt) : 0.0, fd = e0.w > kFloorL ? exp2(dd) : 0.0;
        St = ft * (double)e0.y;
        Tt = ft * ((double)e0.z + dt * (double)e0.y);
        Sd = fd * (double)e1.x;
        Td = fd * ((double)e1.y + dd * (double)e1.x);
    }
    St = warp_sum_f64(St);
    Tt = warp_sum_f64(Tt);
    Sd = warp_sum_f64(Sd);
    Td = warp_sum_f64(Td);
    const double kLn2d = 0.69314718055994530942;
    const double lSt = log2(St), lSd = log2(Sd);
    const double Hbt = lSt - Tt / St, Hbd = lSd - Td / Sd;      // entropies in bits
    FinOut o;
    o.Ht = (float)(kLn2d * Hbt);
    o.lse_t = (float)(kLn2d * ((double)Mt + lSt));
    o.Hd = (float)(kLn2d * Hbd);
    o.lse_d = (float)(kLn2d * ((double)Md + lSd));
    // nearly equal rows: A is sum s phi(u), D_JS = A / 4 (nats), nothing cancels; else
    // D_JS = H(m) - (H(p) + H(q)) / 2 with H(m) = (ln 2 / 2) (2 - sum s log2 s), s = p + q
    const double jd = near ? 0.25 * A : 0.5 * kLn2d * ((2.0 - A) - (Hbt + Hbd));
    float jsd = (float)fmin(fmax(jd, 0.0), kLn2d);
    if (!(fl & 2u)) jsd = 0.f;                              // identical rows: exactly 0
    if (!(PQ > 0.f)) jsd = kLn2;                            // disjoint supports: ln 2
    o.jsd = jsd;
    o.dist = jsd >= kLn2 ? 1.f : fminf((float)sqrt((double)jsd / kLn2d), 1.f);
    return o;
}

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
            // four list entries per lane and trip, all four loads in flight together (the lists live
            // in L2 / HBM: one load per trip would leave the warp waiting on memory, not on the
            // special-function pipe); entries past the end sit far away, where the kernel is 0
            for (int j0 = 0; j0 < nA0; j0 += 128) {
                float xj[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int j = j0 + 32 * q + lane;
                    xj[q] = j < nA0 ? __ldcg(LA + j) : 1.0e9f;
                }
#pragma unroll
                for (int q = 0; q < 4; ++q) {
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        const float t = di[k] - xj[q];
                        accA[k] += ex2(ci[k] * t * t);
                    }
                }
            }
            for (int j0 = 0; j0 < nR0; j0 += 128) {
                float xj[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int j = j0 + 32 * q + lane;
                    xj[q] = j < nR0 ? __ldcg(LR + j) : 1.0e9f;
                }
#pragma unroll
                for (int q = 0; q < 4; ++q) {
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        const float t = di[k] - xj[q];
                        accR[k] += ex2(cR * t * t);
                    }
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
// WARPED: an adjusted distribution is set (Sec. 2.1.1); the ordinary instantiation carries none of its code.
template <int ITER, int MODE, bool WARPED = false>
__global__ void __launch_bounds__(kSThreads, 1)
spec_verify_kernel(VerifyParams p, ClusterGeom gq) {
    const float c1 = WARPED ? p.c1 : kLog2e;                   // log2 e / temperature
    const float inv_temp = WARPED ? p.inv_temp : 1.f;
    constexpr int KH = ITER < kSHead ? ITER : kSHead;          // head iterations: 2^t values in tensor memory
    constexpr int KR = ITER - KH;                              // tail iterations: 2^t values in registers
    static_assert(KR <= kSRegIter, "too many iterations for the register file");
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
                c.cut_t = (WARPED && p.cut_t) ? cut_pair(__ldg(p.cut_t + r.pos)) : kNoCut2;
                c.cut_d = (WARPED && p.cut_d && !c.bonus) ? cut_pair(__ldg(p.cut_d + (size_t)b * Kmax + i)) : kNoCut2;
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
        // all of the SM's tensor memory (this kernel runs one CTA per SM): the address comes back
        // in shared memory and is read by everybody after the barrier below
        tmem_alloc(&sh.tmem_base, (uint32_t)kSTmemCols);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    cluster.sync();   // barriers, positions and tensor memory are set up in every CTA of the cluster
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem0 = *reinterpret_cast<volatile uint32_t*>(&sh.tmem_base);

    // 512 threads x 128 registers fill the register file.  The service warpgroup hands 24 registers a
    // thread to the three compute warpgroups (8 each): setmaxnreg draws on what the CTA was launched
    // with, so what one side gains the other must have given up first.  With the head of a position
    // in tensor memory the compute warps keep at most 80 registers of 2^t values, and 136 leave
    // them without spills; the tail warp's float64 finalisation and the queue workers' KDE loop get
    // by on 104 (measured on one GPU: 144 / 80, 136 / 104, 128 / 128 and 152 / 56 give 0.4933,
    // 0.4898, 0.4937 and 0.4955 ms on the largest workload).
    if (warp < kSW) asm volatile("setmaxnreg.inc.sync.aligned.u32 136;");
    else asm volatile("setmaxnreg.dec.sync.aligned.u32 104;");
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
        // per row.  Position n lives in buffer n & 1; once pass B has turned its logits into 2^t
        // values the buffer is refilled with position n + 2, one whole position before that is
        // needed.
        const int kRowB = I_w * 512;              // bytes of one row in this warp's buffers
        unsigned char* const bufs = dyn_smem + (size_t)wi0 * 2048;
        auto buf_of = [&](int n) -> unsigned char* { return bufs + (size_t)(n & 1) * (2 * kRowB) + (size_t)lane * 16; };
        auto bar_of = [&](int n) -> uint64_t* { return reinterpret_cast<uint64_t*>(&sh.bar[warp][n & 1]); };
        auto pcx = [&](int n) -> const PosCtx& { return sh.pc[n & (kSPosRing - 1)]; };
        // This warp's tensor-memory columns: the lanes of its quarter, 160 columns of its own.
        // Head iteration k of position n sits in slot k of half n & 1.
        const uint32_t tm_warp = tmem0 + ((uint32_t)(32 * (warp & 3)) << 16) + (uint32_t)((warp >> 2) * kSTmemWarp);
        auto tm_of = [&](int n, int k) -> uint32_t { return tm_warp + (uint32_t)((n & 1) * kSTmemHalf + k * 16); };

        // lanes 0 and 1 fetch the two rows of position n (lane 1 idles for a bonus row)
        int n_issued = 0, n_landed = 0;           // positions asked for / seen to have landed (for the give-up path)
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
            n_issued = n + 1;
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
        // The warp's shifts and flags from the packed maxima.  Every kept value is
        // 2^((z - max) log2 e) with the share's own largest logit, exactly 1 for that logit;
        // shares combine in the log2 domain through the differences of M = fl(max * log2 e).
        // A slice without a finite logit gets M = kFloorL and all-zero values.
        float nmt_w = 0.f, nmd_w = 0.f;           // addends of pass B (-max, or 0 for an empty slice)
        uint32_t flags_w = 0;
        auto pass_a = [&](auto bonus_c, int n) {
            constexpr bool BONUS = decltype(bonus_c)::value;
            uint32_t a_mT = 0xFF80FF80u, a_mD = 0xFF80FF80u, a_df = 0u;   // -inf pairs
            if (alive && nwu > 0) {
                bool ok = mbar_wait_bounded(bar_of(n), (uint32_t)(n >> 1) & 1u);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) expired();                // the copy never landed
                else n_landed = n + 1;
            }
            if (alive) {
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
            }
            const float2 a = unpack2(a_mT), d = unpack2(a_mD);
            uint32_t bad = (a.x != a.x || a.y != a.y || d.x != d.x || d.y != d.y) ? 1u : 0u;
            const float vt = warp_max_f32(fmaxf(a.x, a.y));
            const float vd = BONUS ? vt : warp_max_f32(fmaxf(d.x, d.y));
            if (vt == INFINITY || vd == INFINITY || !alive) bad = 1u;
            const bool has_t = vt > ADASD_FLOOR_BF, has_d = vd > ADASD_FLOOR_BF;
            nmt_w = has_t ? -vt : 0.f;
            nmd_w = has_d ? -vd : 0.f;
            // bits 4 and 8 (not published): the target / draft share has no finite logit
            flags_w = __reduce_or_sync(0xFFFFFFFFu, bad | (a_df ? 2u : 0u)) | (has_t ? 0u : 4u) | (has_d ? 0u : 8u);
        };

        // Adjusted distribution with a top-k / top-p cut: before pass A, the logits below the row's
        // cutoff are overwritten with the clamp value in the buffer (probability 0), so that every
        // later pass sees the adjusted rows.  The largest logit always stays, and a NaN is not
        // below anything, so the maxima and the flags of pass A are those of the rows as given.
        const bool any_cut = WARPED && (p.cut_t != nullptr);      // the same for every position of the launch
        auto run_a = [&](bool bonus, int n) {
            if (any_cut && alive && nwu > 0) {
                bool ok = mbar_wait_bounded(bar_of(n), (uint32_t)(n >> 1) & 1u);
                ok = __all_sync(0xFFFFFFFFu, ok);
                // (an expired wait is dealt with by pass A)
                if (ok) cut_buffer(buf_of(n), full ? ITER : ITER - 1, bonus ? 0 : kRowB, pcx(n).cut_t, pcx(n).cut_d);
            }
            if (bonus) pass_a(std::true_type{}, n);
            else pass_a(std::false_type{}, n);
        };

        // ---- pass B: 2^t of every logit of the share, S = sum 2^t, T = sum 2^t t, max |z_t - z_d| --
        // Head iterations [0, KH) park their values in tensor memory, tail iterations [KH, ITER)
        // keep them in registers.  t = (z - max) log2 e is exactly 0 for the largest logit of the
        // share, so that a one-hot row gets S = 1, T = 0, p = 1 and H = 0 exactly.
        float et[KR > 0 ? KR : 1][8], ed[KR > 0 ? KR : 1][8];
        float2 bSt = make_float2(0.f, 0.f), bTt = bSt, bSd = bSt, bTd = bSt;   // lane partials of the position in pass B
        float bdz = 0.f;
        auto pass_b = [&](auto bonus_c, auto k0_c, auto k1_c, int n) {
            constexpr bool BONUS = decltype(bonus_c)::value;
            constexpr int K0 = decltype(k0_c)::value, K1 = decltype(k1_c)::value;
            if (K0 == 0) {
                bSt = bTt = bSd = bTd = make_float2(0.f, 0.f);
                bdz = 0.f;
            }
            const float2 nmt = make_float2(nmt_w, nmt_w), nmd = make_float2(nmd_w, nmd_w);
            const float2 L2 = make_float2(c1, c1), neg1 = make_float2(-1.f, -1.f);
            const unsigned char* sb = buf_of(n);
#pragma unroll
            for (int k = K0; k < K1; ++k) {
                if (k_on(k)) {
                    float e1[8], e2[8];
                    uint4 T = *reinterpret_cast<const uint4*>(sb + k * 512);
                    mask_unit(k, T);
                    uint4 D = make_uint4(0u, 0u, 0u, 0u);
                    if (!BONUS) {
                        D = *reinterpret_cast<const uint4*>(sb + kRowB + k * 512);
                        mask_unit(k, D);
                    }
                    const uint32_t tw[4] = {T.x, T.y, T.z, T.w}, dw[4] = {D.x, D.y, D.z, D.w};
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const float2 zt = unpack2(bclamp2(tw[j]));
                        const float2 tt = __fmul2_rn(__fadd2_rn(zt, nmt), L2);
                        const float2 vt = make_float2(ex2(tt.x), ex2(tt.y));
                        e1[2 * j] = vt.x;
                        e1[2 * j + 1] = vt.y;
                        bSt = __fadd2_rn(bSt, vt);
                        bTt = __ffma2_rn(vt, tt, bTt);
                        if (!BONUS) {
                            const float2 zd = unpack2(bclamp2(dw[j]));
                            const float2 td = __fmul2_rn(__fadd2_rn(zd, nmd), L2);
                            const float2 vd = make_float2(ex2(td.x), ex2(td.y));
                            e2[2 * j] = vd.x;
                            e2[2 * j + 1] = vd.y;
                            bSd = __fadd2_rn(bSd, vd);
                            bTd = __ffma2_rn(vd, td, bTd);
                            const float2 df = __ffma2_rn(zd, neg1, zt);        // exact: both are bf16 values
                            bdz = fmaxf(bdz, fmaxf(fabsf(df.x), fabsf(df.y)));
                        } else {
                            e2[2 * j] = 0.f;
                            e2[2 * j + 1] = 0.f;
                        }
                    }
                    if (k < KH) {
                        if (BONUS) tmem_st8(tm_of(n, k), e1);
                        else tmem_st16(tm_of(n, k), e1, e2);
                    } else {
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            et[k >= KH ? k - KH : 0][j] = e1[j];
                            ed[k >= KH ? k - KH : 0][j] = e2[j];
                        }
                    }
                }
            }
            if (K0 < KH) tmem_wait_st();            // the head is in tensor memory before anything reads it
        };
        // this warp's partial statistics of position n go to the control warp
        auto publish = [&](bool bonus, int n) {
            const float St = warp_sum(bSt.x + bSt.y), Tt = warp_sum(bTt.x + bTt.y);
            float Sd = St, Td = Tt;
            if (!bonus) {
                Sd = warp_sum(bSd.x + bSd.y);
                Td = warp_sum(bTd.x + bTd.y);
            }
            const float dz = warp_max_f32(bdz);
            if (lane == 0) {
                float4* w = reinterpret_cast<float4*>(&sh.wtab[n & 1][warp]);
                const float Mt_w = (flags_w & 4u) ? kFloorL : -nmt_w * c1;
                const float Md_w = (flags_w & 8u) ? kFloorL : -nmd_w * c1;
                w[0] = make_float4(Mt_w, St, Tt, Md_w);
                w[1] = make_float4(Sd, Td, __uint_as_float(flags_w & 3u), dz);
                mbar_arrive_cta(reinterpret_cast<uint64_t*>(&sh.entry_bar[n & 1]));
            }
            __syncwarp();
        };
        // all of pass B of one position, in two parts
        auto b_head = [&](bool bonus, int n) {
            if (bonus) pass_b(std::true_type{}, std::integral_constant<int, 0>{}, std::integral_constant<int, KH>{}, n);
            else pass_b(std::false_type{}, std::integral_constant<int, 0>{}, std::integral_constant<int, KH>{}, n);
        };
        auto b_tail = [&](bool bonus, int n) {
            if (bonus) pass_b(std::true_type{}, std::integral_constant<int, KH>{}, std::integral_constant<int, ITER>{}, n);
            else pass_b(std::false_type{}, std::integral_constant<int, KH>{}, std::integral_constant<int, ITER>{}, n);
        };

        // The 2^t values of iteration k (compile-time k after unrolling): out of tensor memory
        // (synchronously; the sampling scans and the vanilla residual use this) or from registers.
        auto load_kept = [&](int k, int n, bool with_d, float (&a)[8], float (&b)[8]) {
            if (k < KH) {
                if (with_d) {
                    tmem_ld16(tm_of(n, k), a, b);
                    tmem_wait_ld(a, b);
                } else {
                    tmem_ld8(tm_of(n, k), a);
                    tmem_wait_ld(a);
#pragma unroll
                    for (int j = 0; j < 8; ++j) b[j] = 0.f;
                }
            } else {
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    a[j] = et[k >= KH ? k - KH : 0][j];
                    b[j] = with_d ? ed[k >= KH ? k - KH : 0][j] : 0.f;
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

        // ---- pass C (AdaSD mode) over the kept values of position n ---------------------------
        // NEAR == false: A = sum (p+q) log2 (p+q) and the overlap indicator sum 2^t_p 2^t_q.
        // NEAR == true (no logit of the two rows differs by more than kSNearDz): the divergence
        // itself from non-negative terms, D_JS = 1/4 sum s phi(u) with s = p + q, u = (q - p) / s and
        // phi(u) = (1-u) ln(1-u) + (1+u) ln(1+u) = u^2 + u^4/6 + u^6/15 + u^8/28 + ...; |u| <= tanh(1/2)
        // there, so four terms are good to 5e-5 of phi, and nothing cancels however close the rows are.
        // The loads of head iteration k + 1 are in flight while iteration k is worked on.
        auto pass_c = [&](auto near_c, int n, float at, float ad, float& A, float& PQ) {
            constexpr bool NEAR = decltype(near_c)::value;
            float2 A2 = make_float2(0.f, 0.f), PQ2 = make_float2(0.f, 0.f);
            const float2 at2 = make_float2(at, at), ad2 = make_float2(ad, ad);
            const float2 tiny2 = make_float2(kTiny, kTiny), neg1 = make_float2(-1.f, -1.f);
            auto body = [&](const float (&a)[8], const float (&d)[8]) {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float2 a2 = make_float2(a[2 * j], a[2 * j + 1]);
                    const float2 d2 = make_float2(d[2 * j], d[2 * j + 1]);
                    const float2 pp = __ffma2_rn(a2, at2, tiny2);
                    const float2 ss = __ffma2_rn(d2, ad2, pp);
                    if (NEAR) {
                        const float2 qq = __fmul2_rn(d2, ad2);
                        const float2 df = __ffma2_rn(__fmul2_rn(a2, at2), neg1, qq);     // q - p
                        const float2 u = __fmul2_rn(df, make_float2(rcp_approx(ss.x), rcp_approx(ss.y)));
                        const float2 w = __fmul2_rn(u, u);
                        float2 ph = __ffma2_rn(w, make_float2(1.f / 28.f, 1.f / 28.f), make_float2(1.f / 15.f, 1.f / 15.f));
                        ph = __ffma2_rn(ph, w, make_float2(1.f / 6.f, 1.f / 6.f));
                        ph = __ffma2_rn(ph, w, make_float2(1.f, 1.f));
                        A2 = __ffma2_rn(__fmul2_rn(ss, w), ph, A2);
                    } else {
                        const float2 ll = make_float2(lg2(ss.x), lg2(ss.y));
                        A2 = __ffma2_rn(ss, ll, A2);
                        PQ2 = __ffma2_rn(a2, d2, PQ2);
                    }
                }
            };
            float xa[2][8], xd[2][8];              // head values in flight / in use
            if (KH > 0 && k_on(0)) tmem_ld16(tm_of(n, 0), xa[0], xd[0]);
#pragma unroll
            for (int k = 0; k < ITER; ++k) {
                if (k_on(k)) {
                    if (k < KH) {
                        tmem_wait_ld(xa[k & 1], xd[k & 1]);
                        if (k + 1 < KH && k_on(k + 1)) tmem_ld16(tm_of(n, k + 1), xa[(k + 1) & 1], xd[(k + 1) & 1]);
                        body(xa[k & 1], xd[k & 1]);
                    } else {
                        body(et[k >= KH ? k - KH : 0], ed[k >= KH ? k - KH : 0]);
                    }
                }
            }
            A = warp_sum(A2.x + A2.y);
            PQ = NEAR ? 1.f : warp_sum(PQ2.x + PQ2.y);
        };

        // ---------------------------------- main loop ----------------------------------------
        // Invariant at the top of the loop: pass B of position n is complete and its partial
        // statistics are with the control warp; the buffer of position n is being refilled.
        int n = 0;                 // sequence number of the current position
        if (pcx(0).pos < total) {
            const bool b0 = pcx(0).bonus != 0;
            run_a(b0, 0);
            b_head(b0, 0);
            b_tail(b0, 0);
            publish(b0, 0);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            issue_pos(2);
        }
        while (pcx(n).pos < total) {
            const int par = n & 1;
            const uint32_t ph = (uint32_t)(n >> 1) & 1u;
            const bool bonus = pcx(n).bonus != 0;
            const int npos = pcx(n + 1).pos;
            const bool nbonus = npos < total && pcx(n + 1).bonus != 0;

            // while the control warps exchange the totals of position n: maxima and the head of
            // pass B of position n + 1 (its 2^t values go to the other half of tensor memory)
            if (npos < total) {
                run_a(nbonus, n + 1);
                b_head(nbonus, n + 1);
            }
            wait_cta(&sh.scal_bar[par], ph);
            const float4 m0 = *reinterpret_cast<const float4*>(&sh.wmsg[par][warp]);       // at, ad, ft, act

            // the target row's 2^t values of iteration k (what y_i ~ p_i is drawn from)
            auto vals_p = [&](int k, float(&v)[8]) {
                float d[8];
                load_kept(k, n, false, v, d);
            };
            float A = 0.f, PQ = 0.f;
            int tok = -1;
            const int act = __float_as_int(m0.w);
            if (MODE == MODE_ADASD) {
                if (!bonus) {
                    if (act & 4) pass_c(std::true_type{}, n, m0.x, m0.y, A, PQ);
                    else pass_c(std::false_type{}, n, m0.x, m0.y, A, PQ);
                }
                // y_i ~ p_i: the control warp says (a little later than the scale factors) whether
                // this warp holds the crossing
                wait_cta(&sh.sel_bar[par], ph);
                const float4 m1 = *reinterpret_cast<const float4*>(&sh.wmsg[par][warp].target);   // target, sel, base
                if (__float_as_int(m1.y) != 0) tok = select_kept(m1.z, m0.z, m1.x, vals_p);
            } else {
                // vanilla: an accepted row needs nothing more; the bonus row draws from p; a rejected
                // row draws from the residual max(0, p - q) / R, whose mass this warp now adds up
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
            // this warp's sums (and the token, if it drew it) go to the leader CTA in one message
            if (lane == 0) {
                const int fr = n & (kSFinRing - 1);
                st_async_v4(mapa_u32(&sh.tabC[fr][g], 0u), make_float4(A, PQ, __int_as_float(tok), 0.f),
                            mapa_u32(&sh.c_bar[fr], 0u));
            }
            __syncwarp();

            // the rest of pass B of position n + 1 (its values stay in registers until pass C of
            // n + 1), its partials to the control warp, and its buffer refilled with position n + 3
            if (npos < total) {
                b_tail(nbonus, n + 1);
                publish(nbonus, n + 1);
                // (the bulk copy belongs to the async proxy: order it after this warp's reads of the buffer)
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                issue_pos(n + 3);
            }
            ++n;
        }
        // a warp that gave up on a copy still waits (bounded) for whatever it had in flight
        if (!alive && nwu > 0) {
            for (int m = n_landed; m < n_issued; ++m) mbar_wait_bounded(bar_of(m), (uint32_t)(m >> 1) & 1u);
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
                        // a candidate below its row's cutoff has probability 0 there
                        if (WARPED) {
                            if (ztx < unpack2(pcn.cut_t).x) ztx = -INFINITY;
                            if (zdx < unpack2(pcn.cut_d).x) zdx = -INFINITY;
                        }
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
                const float dz = warp_max_f32(w1.w);          // largest |z_t - z_d| of this CTA's slice (>= 0)
                if (lane == 0) mbar_expect_tx(reinterpret_cast<uint64_t*>(&sh.ctab_bar[par]), (uint32_t)(CS * 32));
                if (lane < CS) {
                    const uint32_t dst = mapa_u32(&sh.ctab[par][rank], (uint32_t)lane);
                    const uint32_t bar = mapa_u32(&sh.ctab_bar[par], (uint32_t)lane);
                    st_async_v4(dst, make_float4(Mt, St, Tt, Md), bar);
                    st_async_v4(dst + 16, make_float4(Sd, Td, __uint_as_float(fl), dz), bar);
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
            // AdaSD: the two rows are nearly equal everywhere -> pass C in its well-conditioned form
            const bool near = (MODE == MODE_ADASD) && !bonus && !bad && (fl & 2u) && warp_max_f32(e1.w) * inv_temp <= kSNearDz;
            float alpha = 0.f;
            bool van_accept = true;
            int act = near ? 5 : 1;               // AdaSD: every row draws y_i ~ p_i
            if (MODE == MODE_VANILLA) {
                if (!bonus) {
                    if (x_ok) {
                        const float a = fmaf(fmaxf(ztx, ADASD_FLOOR_BF), c1, -Mt) - lg2(St);
                        const float q = fmaf(fmaxf(zdx, ADASD_FLOOR_BF), c1, -Md) - lg2(Sd);
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
            bool from_p = ((act & 3) == 1);
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
                f[9] = near ? 1.f : 0.f;
            }
            // every CTA's totals, for the finaliser's float64 combination
            if (leader && lane < CS) {
                float4* fc = reinterpret_cast<float4*>(&sh.finc[n & (kSFinRing - 1)][lane]);
                fc[0] = e0;
                fc[1] = e1;
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
                // The warps' sums are small numbers (1/72 of the total each): added up in float64, as
                // are the CTAs' row statistics below.  In fp32 the totals (entropies of up to 17 bits)
                // carry an error of about 1e-6 each, which the difference H(m) - (H(p)+H(q))/2 keeps.
                const double A = warp_sum_f64(((double)c0.x + (double)c1.x) + ((double)c2.x + (double)c3.x));
                const float PQ = warp_sum(((c0.y + c1.y) + c2.y) + c3.y);
                const int tok_all = __reduce_max_sync(0xFFFFFFFFu, max(max(__float_as_int(c0.z), __float_as_int(c1.z)),
                                                                       max(__float_as_int(c2.z), __float_as_int(c3.z))));
                const float Mt = sh.fin[par][0], Md = sh.fin[par][3];
                FinOut fo = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
                if (MODE == MODE_ADASD)
                    fo = finalize_math(&sh.finc[par][0], CS, Mt, Md, A, PQ, __float_as_uint(sh.fin[par][6]),
                                       sh.fin[par][9] != 0.f);
                int done_b = -1;
                if (lane == 0) {
                    const PosCtx& c = sh.pc[m & (kSPosRing - 1)];
                    const int b = c.pos / K1, i = c.pos - b * K1;
                    const bool bonus = c.bonus != 0;
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
                    float Ht = fo.Ht, lse_t = fo.lse_t;
                    if (bad) Ht = lse_t = NAN;
                    p.sc.H_t[idt] = Ht;
                    p.sc.lse_t[idt] = lse_t;
                    p.sc.y[idt] = tok;
                    if (p.user.H_t) p.user.H_t[idt] = Ht;
                    if (p.user.lse_t) p.user.lse_t[idt] = lse_t;
                    if (p.user.y) p.user.y[idt] = tok;
                    if (!bonus) {
                        float Hd = fo.Hd, lse_d = fo.lse_d, jsd = fo.jsd, dist = fo.dist;
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

            // A completed sequence goes to the chip-wide queue of tails (device memory): whichever
            // worker warp on the chip is free takes it.  (Handing the tails to this cluster's own
            // workers would pile them up on the cluster that runs last, which draws most last tickets
            // and would fall back further.)
            auto push = [&](int b) {
                if (lane == 0) {
                    __threadfence();                      // this sequence's position scalars are out
                    const uint32_t idx = atomicAdd(p.sc.q_ctl + 0, 1u);
                    if (idx < (uint32_t)p.B) *reinterpret_cast<volatile int32_t*>(p.sc.q_items + idx) = b;
                }
                __syncwarp();
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
                    } else {
                        push(done_b);
                    }
                }
                if (lane == 0) {
                    __threadfence_block();
                    *reinterpret_cast<volatile int32_t*>(&sh.fin_done) = m + 1;
                }
            }
        }
    }
    // ============================== tail workers ==========================================
    // AdaSD mode: the tail warps of the non-leader CTAs and the two spare warps of every CTA take
    // completed sequences from the chip-wide queue and run their tails (KDE/Bayes, accept scan,
    // appends, T_G).  Every sequence has a bonus row, so exactly B tails are queued per launch: a
    // worker leaves when it draws a number >= B, and the last worker to leave puts the counters
    // back to zero for the next launch.
    if (MODE == MODE_ADASD && warp >= kSTail && !(leader && warp == kSTail)) {
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
        const int slot = warp - kSTail;           // this worker's scratch
        const uint32_t nworkers = (uint32_t)(gridDim.x / CS) * (uint32_t)(3 * CS - 1);
        for (;;) {
            int b = -2;
            if (lane == 0) {
                const uint32_t idx = atomicAdd(p.sc.q_ctl + 1, 1u);
                if (idx >= (uint32_t)p.B) {
                    b = -1;                       // no more tails this launch
                    if (atomicAdd(p.sc.q_ctl + 2, 1u) + 1u == nworkers) {
                        p.sc.q_ctl[0] = 0u;       // every worker has left: ready for the next launch
                        p.sc.q_ctl[1] = 0u;
                        p.sc.q_ctl[2] = 0u;
                    }
                } else {
                    volatile int32_t* item = p.sc.q_items + idx;
                    for (uint32_t it = 0; it < kSPollSpins; ++it) {
                        b = *item;
                        if (b >= 0) break;
                        __nanosleep(400);
                    }
                    if (b >= 0) *item = -1;       // the entry is free again
                    else {
                        b = -3;                   // nothing came: give this one up, go on
                        atomicOr(p.st.status, ADASD_STATUS_TIMEOUT);
                    }
                }
            }
            b = __shfl_sync(0xFFFFFFFFu, b, 0);
            if (b == -1) break;
            if (b < 0) continue;
            __threadfence();
            verify_tail_warp(p.tail, io, p.st, b, sh.td[slot], sh.tH[slot]);
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    cluster.sync();   // no CTA leaves while a peer may still address its shared memory
    if (warp == kSCtl) tmem_dealloc(tmem0, (uint32_t)kSTmemCols);   // by the warp that allocated it
}

}  // namespace adasd
