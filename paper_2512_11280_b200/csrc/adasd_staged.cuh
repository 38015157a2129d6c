// Staged verification kernel for sm_100a: persistent 8-CTA clusters, every logit row
// read from HBM exactly once.
//
//  * A position (b,i) = draft row q_i + target row p_i (bf16).  Each of the 128 warps of a
//    cluster owns a contiguous sub-slice of both rows.  Lane 0 of a warp brings its
//    sub-slices into the warp's own shared-memory region with 1-D bulk copies
//    (cp.async.bulk, completion on the warp's own mbarrier), two positions ahead, so HBM
//    stays busy while the cluster computes.  Every wait on a copy is bounded.
//  * Pass A (max) and pass B (sum of 2^t) use the warp's LOCAL maximum as the shift, so no
//    exchange is needed before pass B; one exchange of (m_w, S_w) per warp over DSMEM then
//    gives every warp the row's log-sum-exp.  The 2^t values of pass B stay in registers
//    (the "stash"), so pass C (entropies, JS divergence) needs one lg2 per pair and no ex2:
//    3 MUFU operations per logit pair in total.
//  * Two cluster barriers per position.  Pass B of the next position runs between the
//    arrive and the wait of barrier 2, pass A of the next position and the leader's
//    finalisation of the previous one between the arrive and the wait of barrier 1.
//  * The cluster that publishes the last position of a sequence runs that sequence's
//    tail (KDE/Bayes, accept scan, list appends, T_G) in the same launch.
#pragma once

#include "adasd_device.cuh"
#include "adasd_rows.cuh"
#include "adasd_tail.cuh"

namespace adasd {

constexpr int kSC = 8;                 // CTAs per cluster
constexpr int kSW = 16;                // warps per CTA
constexpr int kSG = kSC * kSW;         // warps per cluster
constexpr int kSThreads = kSW * 32;
constexpr int kStagedMaxIter = 5;      // 16-byte units per lane per row
constexpr uint32_t kWaitSpins = 1u << 22;
// bf16 value used to clamp -inf logits inside the staged kernels (0xF149 = -9.95e29), as fp32
#define ADASD_FLOOR_BF __uint_as_float(0xF1490000u)

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok;
}
// Bounded wait: false if the copy did not complete within the spin budget.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity) {
    for (uint32_t it = 0; it < kWaitSpins; ++it)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
// global -> this CTA's shared memory, completion counted in bytes on `bar`
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(dst)),
                 "l"(src), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}
// .aligned: every thread of the warp executes the barrier instruction together
__device__ __forceinline__ void cluster_arrive() {
    __syncwarp();
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
}
__device__ __forceinline__ void cluster_wait() {
    __syncwarp();
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void cta_bar(int id) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(kSThreads) : "memory");
}

__device__ __forceinline__ uint32_t bmax2(uint32_t a, uint32_t b) {   // NaN-propagating bf16x2 max
    uint32_t d;
    asm("max.NaN.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ uint32_t bclamp2(uint32_t a) {             // max(a, floor), NaN dropped
    uint32_t d;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(0xF149F149u));   // bf16(-9.98e29) twice
    return d;
}
__device__ __forceinline__ float2 unpack2(uint32_t w) {
    return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xFFFF0000u));
}

struct __align__(16) StagedShared {
    // exchange tables, double-buffered by position parity
    float tabB[2][5][kSG];     // m_t, S_t, m_d, S_d, flags of every warp of the cluster
    float tabC[2][4][kSG];     // leader only: sum p a', sum q b', sum s log2 s, sum p q | residual
    float fin[2][8];           // leader only: m_t, S_t, m_d, S_d, flags kept for finalisation
    int32_t token[2];          // leader only: sampled token of the position
    int32_t tail_seq;          // leader only: sequence whose tail must run (-1: none)
    unsigned long long bar[2][kSW];   // per-warp, per-buffer "copy landed" barriers
};

struct PosInfo {
    int pos, b, i, K_t;
    bool bonus;
};

// ------------------------------------------------------------------------------------
template <int ITER, int MODE>
__global__ void __launch_bounds__(kSThreads, 1)
staged_verify_kernel(VerifyParams p, int nclusters, int slice_pad_bytes) {
    extern __shared__ __align__(128) unsigned char dyn_smem[];
    __shared__ StagedShared sh;
    __shared__ TailShared tsh;

    cg::cluster_group cluster = cg::this_cluster();
    const int rank = (int)cluster.block_rank();
    const int cid = blockIdx.x / kSC;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = rank * kSW + warp;
    const int Kmax = p.Kmax;
    const int total = p.B * (Kmax + 1);
    const bool leader = (rank == 0);

    // this warp's units (16 bytes = 8 bf16) of a row
    const int NU = p.V >> 3;
    const int cu0 = (int)((long long)rank * NU / kSC), cu1 = (int)((long long)(rank + 1) * NU / kSC);
    const int ncu = cu1 - cu0;
    const int wu0 = cu0 + (int)((long long)warp * ncu / kSW), wu1 = cu0 + (int)((long long)(warp + 1) * ncu / kSW);
    const int nwu = wu1 - wu0;
    const uint32_t wbytes = (uint32_t)nwu * 16u;
    // shared-memory regions: [buffer][row (0 target, 1 draft)][slice]
    unsigned char* const wbase = dyn_smem + (size_t)(wu0 - cu0) * 16;
    auto buf = [&](int s, int row) -> unsigned char* {
        return wbase + (size_t)(s * 2 + row) * slice_pad_bytes;
    };

    if (threadIdx.x == 0) {
        for (int s = 0; s < 2; ++s)
            for (int w = 0; w < kSW; ++w) mbar_init(reinterpret_cast<uint64_t*>(&sh.bar[s][w]), 1);
        sh.tail_seq = -1;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    cluster.sync();   // every CTA of the cluster is running before any remote shared-memory access

    auto info = [&](int pos) -> PosInfo {
        PosInfo q;
        q.pos = pos;
        if (pos >= total) {
            q.b = q.i = q.K_t = 0;
            q.bonus = false;
            return q;
        }
        q.b = pos / (Kmax + 1);
        q.i = pos % (Kmax + 1);
        int K_t = p.draft_len ? __ldg(p.draft_len + q.b) : Kmax;
        q.K_t = max(0, min(K_t, Kmax));
        q.bonus = (q.i == q.K_t);
        return q;
    };
    // next active position of this cluster after `pos` (positions beyond a window are skipped)
    auto advance = [&](int pos) -> int {
        for (pos += nclusters; pos < total; pos += nclusters) {
            PosInfo q = info(pos);
            if (q.i <= q.K_t) return pos;
        }
        return total;
    };
    auto first = [&]() -> int {
        int pos = cid;
        if (pos < total) {
            PosInfo q = info(pos);
            if (q.i <= q.K_t) return pos;
            return advance(pos);
        }
        return total;
    };
    auto row_t = [&](const PosInfo& q) {
        return reinterpret_cast<const __nv_bfloat16*>(p.zt) + (long long)q.b * p.t_seq + (long long)q.i * p.t_row;
    };
    auto row_d = [&](const PosInfo& q) {
        return reinterpret_cast<const __nv_bfloat16*>(p.zd) + (long long)q.b * p.d_seq + (long long)q.i * p.d_row;
    };
    // lane 0: start the copies of this warp's sub-slices of position q into buffer s
    auto issue = [&](const PosInfo& q, int s) {
        if (lane == 0 && q.pos < total && nwu > 0) {
            uint64_t* bar = reinterpret_cast<uint64_t*>(&sh.bar[s][warp]);
            mbar_expect_tx(bar, q.bonus ? wbytes : 2u * wbytes);
            bulk_g2s(buf(s, 0), row_t(q) + (size_t)wu0 * 8, wbytes, bar);
            if (!q.bonus) bulk_g2s(buf(s, 1), row_d(q) + (size_t)wu0 * 8, wbytes, bar);
        }
    };

    uint32_t phase[2] = {0u, 0u};
    bool data_ok = true;
    auto wait_data = [&](int s) {
        data_ok = true;
        if (nwu > 0) {
            data_ok = mbar_wait_bounded(reinterpret_cast<uint64_t*>(&sh.bar[s][warp]), phase[s]);
            if (!data_ok && lane == 0) atomicOr(p.st.status, ADASD_STATUS_TIMEOUT);
        }
        phase[s] ^= 1u;
    };

    // ---- per-position registers -------------------------------------------------------
    float et[ITER][8], ed[ITER][8];     // stash: 2^t of pass B (target, draft)
    float mt_w = 0.f, md_w = 0.f;       // this warp's local maxima (pass A)
    uint32_t flags_w = 0;               // 1 NaN seen, 2 rows differ

    auto pass_a = [&](int s, bool bonus) {
        uint32_t mT = 0xFF80FF80u, mD = 0xFF80FF80u, df = 0u;   // -inf pairs
#pragma unroll
        for (int k = 0; k < ITER; ++k) {
            const int u = lane + 32 * k;
            if (u < nwu) {
                uint4 T = *reinterpret_cast<const uint4*>(buf(s, 0) + (size_t)u * 16);
                mT = bmax2(bmax2(mT, T.x), bmax2(T.y, bmax2(T.z, T.w)));
                if (!bonus) {
                    uint4 D = *reinterpret_cast<const uint4*>(buf(s, 1) + (size_t)u * 16);
                    mD = bmax2(bmax2(mD, D.x), bmax2(D.y, bmax2(D.z, D.w)));
                    df |= (T.x ^ D.x) | (T.y ^ D.y) | (T.z ^ D.z) | (T.w ^ D.w);
                }
            }
        }
        float2 a = unpack2(mT), d = unpack2(mD);
        float vt = (a.x != a.x || a.y != a.y) ? NAN : fmaxf(a.x, a.y);
        float vd = (d.x != d.x || d.y != d.y) ? NAN : fmaxf(d.x, d.y);
        if (bonus) vd = vt;
        uint32_t nan = (vt != vt || vd != vd) ? 1u : 0u;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            vt = fmaxf(vt, __shfl_xor_sync(0xFFFFFFFFu, vt, o));
            vd = fmaxf(vd, __shfl_xor_sync(0xFFFFFFFFu, vd, o));
            df |= __shfl_xor_sync(0xFFFFFFFFu, df, o);
            nan |= __shfl_xor_sync(0xFFFFFFFFu, nan, o);
        }
        // a warp whose sub-slice is all -inf (or empty) shifts by the clamp value: after the
        // rescaling to the row maximum its sums vanish
        mt_w = fmaxf(vt, ADASD_FLOOR_BF);
        md_w = fmaxf(vd, ADASD_FLOOR_BF);
        if (mt_w == INFINITY || md_w == INFINITY || !data_ok) nan = 1u;
        flags_w = nan | (df ? 2u : 0u);
    };

    // pass B: stash 2^((z - m_w) log2 e), publish (m_w, S_w) to every CTA of the cluster
    auto pass_b = [&](int s, bool bonus, int par) {
        float2 St = make_float2(0.f, 0.f), Sd = make_float2(0.f, 0.f);
        const float2 nmt = make_float2(-mt_w, -mt_w), nmd = make_float2(-md_w, -md_w);
        const float2 L2 = make_float2(kLog2e, kLog2e);
#pragma unroll
        for (int k = 0; k < ITER; ++k) {
            const int u = lane + 32 * k;
            if (u < nwu) {
                uint4 T = *reinterpret_cast<const uint4*>(buf(s, 0) + (size_t)u * 16);
                const uint32_t tw[4] = {T.x, T.y, T.z, T.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    float2 z = unpack2(bclamp2(tw[j]));
                    float2 t = __fmul2_rn(__fadd2_rn(z, nmt), L2);
                    float2 e = make_float2(ex2(t.x), ex2(t.y));
                    et[k][2 * j] = e.x;
                    et[k][2 * j + 1] = e.y;
                    St = __fadd2_rn(St, e);
                }
                if (!bonus) {
                    uint4 D = *reinterpret_cast<const uint4*>(buf(s, 1) + (size_t)u * 16);
                    const uint32_t dw[4] = {D.x, D.y, D.z, D.w};
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        float2 z = unpack2(bclamp2(dw[j]));
                        float2 t = __fmul2_rn(__fadd2_rn(z, nmd), L2);
                        float2 e = make_float2(ex2(t.x), ex2(t.y));
                        ed[k][2 * j] = e.x;
                        ed[k][2 * j + 1] = e.y;
                        Sd = __fadd2_rn(Sd, e);
                    }
                }
            } else {
#pragma unroll
                for (int j = 0; j < 8; ++j) et[k][j] = ed[k][j] = 0.f;
            }
        }
        float st = warp_sum(St.x + St.y);
        float sd = bonus ? st : warp_sum(Sd.x + Sd.y);
        if (lane < kSC) {
            StagedShared* r = cluster.map_shared_rank(&sh, lane);
            r->tabB[par][0][g] = mt_w;
            r->tabB[par][1][g] = st;
            r->tabB[par][2][g] = md_w;
            r->tabB[par][3][g] = sd;
            r->tabB[par][4][g] = __uint_as_float(flags_w);
        }
    };

    // Row statistics from the exchange table; every warp computes the same numbers.
    struct RowStat {
        float m, S;        // global max and sum relative to it
        float incl, excl;  // this lane's inclusive / exclusive prefix of scaled warp sums
        float4 sc;         // scaled sums of this lane's four entries
    };
    auto scan_row = [&](int par, int which) -> RowStat {
        RowStat r;
        float4 mv = *reinterpret_cast<const float4*>(&sh.tabB[par][2 * which][4 * lane]);
        float4 sv = *reinterpret_cast<const float4*>(&sh.tabB[par][2 * which + 1][4 * lane]);
        r.m = warp_max(fmaxf(fmaxf(mv.x, mv.y), fmaxf(mv.z, mv.w)));
        r.sc.x = sv.x * ex2((mv.x - r.m) * kLog2e);
        r.sc.y = sv.y * ex2((mv.y - r.m) * kLog2e);
        r.sc.z = sv.z * ex2((mv.z - r.m) * kLog2e);
        r.sc.w = sv.w * ex2((mv.w - r.m) * kLog2e);
        float ls = ((r.sc.x + r.sc.y) + r.sc.z) + r.sc.w;
        float incl = ls;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            float t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= o) incl += t;
        }
        r.incl = incl;
        r.excl = __shfl_up_sync(0xFFFFFFFFu, incl, 1);
        if (lane == 0) r.excl = 0.f;
        r.S = __shfl_sync(0xFFFFFFFFu, incl, 31);
        return r;
    };
    // Which cluster-warp holds the crossing of target = u * S in a scanned row: returns
    // (warp id, weight before it); if rounding leaves none, the last warp with mass and +inf.
    auto locate = [&](const RowStat& r, float u, int& gsel, float& base, float& target) {
        target = u * r.S;
        const float c[4] = {r.sc.x, r.sc.y, r.sc.z, r.sc.w};
        float run = r.excl;
        int hit = -1, lastp = -1;
        float hbase = 0.f, lbase = 0.f;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            float nr = run + c[k];
            if (c[k] > 0.f) {
                lastp = 4 * lane + k;
                lbase = run;
                if (hit < 0 && nr > target) {
                    hit = 4 * lane + k;
                    hbase = run;
                }
            }
            run = nr;
        }
        unsigned mh = __ballot_sync(0xFFFFFFFFu, hit >= 0);
        if (mh) {
            int src = __ffs(mh) - 1;
            gsel = __shfl_sync(0xFFFFFFFFu, hit, src);
            base = __shfl_sync(0xFFFFFFFFu, hbase, src);
        } else {
            unsigned ml = __ballot_sync(0xFFFFFFFFu, lastp >= 0);
            if (ml) {
                int src = 31 - __clz(ml);
                gsel = __shfl_sync(0xFFFFFFFFu, lastp, src);
                base = __shfl_sync(0xFFFFFFFFu, lbase, src);
            } else {
                gsel = -1;
                base = 0.f;
            }
            target = INFINITY;
        }
    };
    // Run by the chosen warp: first element (index order) where base + f * running weight
    // exceeds target; weights come from the stash through `wfun(k, j)`.
    auto stash_select = [&](float base, float f, float target, auto wfun) -> int {
        float run = 0.f;
        int found = -1, lastp = -1;
#pragma unroll
        for (int k = 0; k < ITER; ++k) {
            float w[8], ls = 0.f;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                w[j] = wfun(k, j);
                ls += w[j];
            }
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
            const int e0 = (wu0 + lane + 32 * k) * 8;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                c += w[j];
                if (w[j] > 0.f) {
                    lastp = e0 + j;
                    if (hit < 0 && fmaf(f, c, base) > target) hit = j;
                }
            }
            unsigned mh = __ballot_sync(0xFFFFFFFFu, hit >= 0);
            if (mh && found < 0) {
                int src = __ffs(mh) - 1;
                found = __shfl_sync(0xFFFFFFFFu, e0 + hit, src);
            }
            run += __shfl_sync(0xFFFFFFFFu, incl, 31);
        }
        if (found < 0) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) lastp = max(lastp, __shfl_xor_sync(0xFFFFFFFFu, lastp, o));
            found = lastp;
        }
        return found;
    };

    // Leader warp 0: turn the cluster's partial sums of position q into its published scalars.
    // Returns the ticket value (K_t means: this was the sequence's last position).
    auto finalize = [&](const PosInfo& q, int par) -> unsigned {
        float4 a = *reinterpret_cast<const float4*>(&sh.tabC[par][0][4 * lane]);
        float4 bq = *reinterpret_cast<const float4*>(&sh.tabC[par][1][4 * lane]);
        float4 c = *reinterpret_cast<const float4*>(&sh.tabC[par][2][4 * lane]);
        float4 d = *reinterpret_cast<const float4*>(&sh.tabC[par][3][4 * lane]);
        float spa = warp_sum(((a.x + a.y) + a.z) + a.w);
        float sqb = warp_sum(((bq.x + bq.y) + bq.z) + bq.w);
        float ssl = warp_sum(((c.x + c.y) + c.z) + c.w);
        float spq = warp_sum(((d.x + d.y) + d.z) + d.w);
        unsigned ticket = 0xFFFFFFFFu;
        if (lane == 0) {
            const float m_t = sh.fin[par][0], S_t = sh.fin[par][1], m_d = sh.fin[par][2], S_d = sh.fin[par][3];
            const uint32_t fl = __float_as_uint(sh.fin[par][4]);
            const bool bad = (fl & 1u) || !(m_t > ADASD_FLOOR_BF) || !(m_d > ADASD_FLOOR_BF);
            const size_t it = (size_t)q.b * (Kmax + 1) + q.i, id = (size_t)q.b * Kmax + q.i;
            int tok = sh.token[par];
            if (bad) {
                atomicOr(p.st.status, ADASD_STATUS_NAN);
                tok = -1;
            }
            if (MODE == MODE_ADASD) {
                float Ht = -kLn2 * spa, lse_t = fmaf(kLn2, lg2(S_t), m_t);
                if (bad) Ht = lse_t = NAN;
                p.sc.H_t[it] = Ht;
                p.sc.lse_t[it] = lse_t;
                p.sc.y[it] = tok;
                if (p.user.H_t) p.user.H_t[it] = Ht;
                if (p.user.lse_t) p.user.lse_t[it] = lse_t;
                if (p.user.y) p.user.y[it] = tok;
                if (!q.bonus) {
                    float Hd = -kLn2 * sqb, lse_d = fmaf(kLn2, lg2(S_d), m_d);
                    // sum s (1 - log2 s) with sum s = 2
                    float jsd = 0.5f * kLn2 * (spa + sqb + (2.f - ssl));
                    jsd = (fl & 2u) ? fminf(fmaxf(jsd, 0.f), kLn2) : 0.f;   // identical rows: exactly 0
                    if (!(spq > 0.f)) jsd = kLn2;                            // disjoint supports: ln 2
                    float dist = fminf(sqrtf(jsd / kLn2), 1.f);
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
                // vanilla: fin[5] = alpha, fin[6] = accept flag
                if (!q.bonus) {
                    p.sc.van_flag[id] = (sh.fin[par][6] != 0.f && !bad) ? 1 : 0;
                    if (p.alpha_out) p.alpha_out[id] = bad ? NAN : sh.fin[par][5];
                }
                p.sc.van_tok[it] = tok;
            }
            __threadfence();
            ticket = atomicAdd(p.sc.ticket + q.b, 1u);
        }
        return ticket;
    };

    // The sequence's tail, run by the whole leader CTA.
    auto run_tail = [&](int b) {
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
            int K_t = p.draft_len ? __ldcg(p.draft_len + b) : Kmax;
            K_t = max(0, min(K_t, Kmax));
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
    };

    // ================================== main loop ======================================
    PosInfo cur = info(first());
    PosInfo nxt = info(cur.pos < total ? advance(cur.pos) : total);
    if (cur.pos < total) issue(cur, 0);
    if (nxt.pos < total) issue(nxt, 1);
    int s = 0, par = 0;
    unsigned pending_ticket = 0xFFFFFFFFu;   // leader warp 0 lane 0: ticket of the previous position
    PosInfo prev = info(total);
    bool have_prev = false;

    if (cur.pos < total) {
        wait_data(0);
        pass_a(0, cur.bonus);
        pass_b(0, cur.bonus, 0);
    }
    while (cur.pos < total) {
        // per-position scalars needed after barrier 1, fetched early
        const size_t it = (size_t)cur.b * (Kmax + 1) + cur.i, id = (size_t)cur.b * Kmax + cur.i;
        float u_samp = 0.f, u_acc = 0.f, ztx = 0.f, zdx = 0.f;
        int xi = -1;
        if (MODE == MODE_ADASD) {
            u_samp = __ldg(p.u_target + it);
        } else {
            u_samp = __ldg(p.u_resample + cur.b);
            if (!cur.bonus) {
                u_acc = __ldg(p.u_accept + id);
                xi = __ldg(p.x + id);
                if (xi >= 0 && xi < p.V) {
                    ztx = __bfloat162float(row_t(cur)[xi]);
                    zdx = __bfloat162float(row_d(cur)[xi]);
                }
            }
        }

        cluster_arrive();                                    // ---- barrier 1: tabB[par] complete
        // shadow of barrier 1: pass A of the next position; leader warp 0 finalises the previous one
        const int sn = s ^ 1;
        if (nxt.pos < total) {
            wait_data(sn);
            pass_a(sn, nxt.bonus);
        }
        if (leader && warp == 0 && have_prev) pending_ticket = finalize(prev, par ^ 1);
        cluster_wait();

        RowStat rt_ = scan_row(par, 0);
        RowStat rd_ = scan_row(par, 1);
        uint32_t fl = __float_as_uint(sh.tabB[par][4][4 * lane]) | __float_as_uint(sh.tabB[par][4][4 * lane + 1]) |
                      __float_as_uint(sh.tabB[par][4][4 * lane + 2]) | __float_as_uint(sh.tabB[par][4][4 * lane + 3]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) fl |= __shfl_xor_sync(0xFFFFFFFFu, fl, o);
        // own scale factors: p = et * ct, log2 p = (z - my_mt) log2e - kt.
        // The stash of position `cur` was made with the maxima this warp had when pass B ran;
        // pass A of the next position has since overwritten mt_w/md_w, so they are re-read
        // from the exchange table (own entry).
        const float my_mt = sh.tabB[par][0][g], my_md = sh.tabB[par][2][g];
        const float lSt = lg2(rt_.S), lSd = lg2(rd_.S);
        const float dt = (my_mt - rt_.m) * kLog2e, dd = (my_md - rd_.m) * kLog2e;
        const float ft = ex2(dt), fd = ex2(dd);
        const float ct = ft / rt_.S, cd = fd / rd_.S;
        const float kt = lSt - dt, kd = lSd - dd;
        if (leader && warp == 0 && lane == 0) {
            sh.fin[par][0] = rt_.m;
            sh.fin[par][1] = rt_.S;
            sh.fin[par][2] = rd_.m;
            sh.fin[par][3] = rd_.S;
            sh.fin[par][4] = __uint_as_float(fl);
        }
        const bool bad = (fl & 1u) || !(rt_.m > ADASD_FLOOR_BF) || !(rd_.m > ADASD_FLOOR_BF);

        // vanilla: alpha at the draft token
        bool van_accept = true;
        if (MODE == MODE_VANILLA && !cur.bonus) {
            float alpha = 0.f;
            if (xi >= 0 && xi < p.V) {
                float a = fmaf(fmaxf(ztx, ADASD_FLOOR_BF) - rt_.m, kLog2e, -lSt);
                float q = fmaf(fmaxf(zdx, ADASD_FLOOR_BF) - rd_.m, kLog2e, -lSd);
                alpha = fminf(1.f, ex2(a - q));
                if (!(ex2(q) > 0.f)) alpha = 1.f;
            }
            van_accept = u_acc < alpha;
            if (leader && warp == 0 && lane == 0) {
                sh.fin[par][5] = alpha;
                sh.fin[par][6] = van_accept ? 1.f : 0.f;
            }
        }
        const bool need_resid = (MODE == MODE_VANILLA) && !cur.bonus && !van_accept && !bad;

        // sample from p (AdaSD: y_i for every row; vanilla: the bonus row)
        if ((MODE == MODE_ADASD || cur.bonus) && !bad) {
            int gsel;
            float base, target;
            locate(rt_, u_samp, gsel, base, target);
            if (gsel == g) {
                int tok = stash_select(base, ft, target, [&](int k, int j) { return et[k][j]; });
                if (lane == 0) cluster.map_shared_rank(&sh, 0)->token[par] = tok;
            }
        }

        // pass C
        float2 acc_pa = make_float2(0.f, 0.f), acc_qb = make_float2(0.f, 0.f);
        float2 acc_sl = make_float2(0.f, 0.f), acc_pq = make_float2(0.f, 0.f);
        if (MODE == MODE_ADASD) {
            const float2 L2 = make_float2(kLog2e, kLog2e);
            const float2 nmt = make_float2(-my_mt, -my_mt), nmd = make_float2(-my_md, -my_md);
            const float2 nkt = make_float2(-kt, -kt), nkd = make_float2(-kd, -kd);
            const float2 ct2 = make_float2(ct, ct), cd2 = make_float2(cd, cd);
            const float2 tiny2 = make_float2(kTiny, kTiny);
#pragma unroll
            for (int k = 0; k < ITER; ++k) {
                const int u = lane + 32 * k;
                if (u < nwu) {
                    uint4 T = *reinterpret_cast<const uint4*>(buf(s, 0) + (size_t)u * 16);
                    const uint32_t tw[4] = {T.x, T.y, T.z, T.w};
                    if (cur.bonus) {
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            float2 zt2 = unpack2(bclamp2(tw[j]));
                            float2 a = __ffma2_rn(__fadd2_rn(zt2, nmt), L2, nkt);
                            float2 pp = __fmul2_rn(make_float2(et[k][2 * j], et[k][2 * j + 1]), ct2);
                            acc_pa = __ffma2_rn(pp, a, acc_pa);
                        }
                    } else {
                        uint4 D = *reinterpret_cast<const uint4*>(buf(s, 1) + (size_t)u * 16);
                        const uint32_t dw[4] = {D.x, D.y, D.z, D.w};
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            float2 zt2 = unpack2(bclamp2(tw[j]));
                            float2 zd2 = unpack2(bclamp2(dw[j]));
                            float2 a = __ffma2_rn(__fadd2_rn(zt2, nmt), L2, nkt);
                            float2 bq = __ffma2_rn(__fadd2_rn(zd2, nmd), L2, nkd);
                            float2 pp = __fmul2_rn(make_float2(et[k][2 * j], et[k][2 * j + 1]), ct2);
                            float2 qq = __fmul2_rn(make_float2(ed[k][2 * j], ed[k][2 * j + 1]), cd2);
                            float2 ss = __fadd2_rn(pp, qq);
                            float2 sg = __fadd2_rn(ss, tiny2);
                            float2 ll = make_float2(lg2(sg.x), lg2(sg.y));
                            acc_pa = __ffma2_rn(pp, a, acc_pa);
                            acc_qb = __ffma2_rn(qq, bq, acc_qb);
                            acc_sl = __ffma2_rn(ss, ll, acc_sl);
                            acc_pq = __ffma2_rn(pp, qq, acc_pq);
                        }
                    }
                }
            }
        } else if (need_resid) {
            // vanilla, rejected row: residual mass max(0, p - q) of this warp
#pragma unroll
            for (int k = 0; k < ITER; ++k)
#pragma unroll
                for (int j = 0; j < 8; ++j) acc_pa.x += fmaxf(fmaf(et[k][j], ct, -ed[k][j] * cd), 0.f);
        }
        {
            float v0 = warp_sum(acc_pa.x + acc_pa.y), v1 = warp_sum(acc_qb.x + acc_qb.y);
            float v2 = warp_sum(acc_sl.x + acc_sl.y), v3 = warp_sum(acc_pq.x + acc_pq.y);
            if (lane == 0) {
                StagedShared* r0 = cluster.map_shared_rank(&sh, 0);
                r0->tabC[par][0][g] = v0;
                r0->tabC[par][1][g] = v1;
                r0->tabC[par][2][g] = v2;
                r0->tabC[par][3][g] = v3;
            }
        }

        // the raw slices of `cur` are dead for this warp: refill the buffer two positions ahead
        PosInfo nn = info(nxt.pos < total ? advance(nxt.pos) : total);
        __syncwarp();
        issue(nn, s);

        // leader CTA: the ticket drawn while finalising the previous position says whether its
        // sequence is complete; if so the whole CTA runs the tail now (the stash is dead here)
        if (leader) {
            if (warp == 0 && have_prev) {
                unsigned tk = __shfl_sync(0xFFFFFFFFu, pending_ticket, 0);
                if (lane == 0) {
                    int done = (tk == (unsigned)prev.K_t);
                    if (done) p.sc.ticket[prev.b] = 0u;
                    sh.tail_seq = done ? prev.b : -1;
                }
            }
            cta_bar(1);
            int tb = sh.tail_seq;
            if (tb >= 0) {
                __threadfence();
                run_tail(tb);
            }
        }

        cluster_arrive();                                    // ---- barrier 2: tabC[par], token complete
        if (need_resid) {
            // vanilla, rejected row: locate the residual sample; needs the whole tabC, i.e. barrier 2
            cluster_wait();
            StagedShared* r0 = cluster.map_shared_rank(&sh, 0);
            RowStat rr;
            {
                float4 sv = *reinterpret_cast<const float4*>(&r0->tabC[par][0][4 * lane]);
                rr.m = 0.f;
                rr.sc = sv;
                float ls = ((sv.x + sv.y) + sv.z) + sv.w;
                float incl = ls;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    float t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                    if (lane >= o) incl += t;
                }
                rr.incl = incl;
                rr.excl = __shfl_up_sync(0xFFFFFFFFu, incl, 1);
                if (lane == 0) rr.excl = 0.f;
                rr.S = __shfl_sync(0xFFFFFFFFu, incl, 31);
            }
            int gsel;
            float base, target;
            if (rr.S > 0.f) {
                locate(rr, u_samp, gsel, base, target);
                if (gsel == g) {
                    int tok = stash_select(base, 1.f, target, [&](int k, int j) {
                        return fmaxf(fmaf(et[k][j], ct, -ed[k][j] * cd), 0.f);
                    });
                    if (lane == 0) r0->token[par] = tok;
                }
            } else {   // no residual mass: sample from p
                locate(rt_, u_samp, gsel, base, target);
                if (gsel == g) {
                    int tok = stash_select(base, ft, target, [&](int k, int j) { return et[k][j]; });
                    if (lane == 0) r0->token[par] = tok;
                }
            }
            cluster_arrive();                                // ---- barrier 3 (rejected vanilla rows only)
        }
        // shadow of the last barrier: pass B of the next position
        if (nxt.pos < total) pass_b(sn, nxt.bonus, par ^ 1);
        cluster_wait();

        prev = cur;
        have_prev = true;
        cur = nxt;
        nxt = nn;
        s = sn;
        par ^= 1;
    }

    // drain: finalise the last position and run its tail if it completed a sequence
    if (leader && have_prev) {
        if (warp == 0) {
            unsigned tk = finalize(prev, par ^ 1);
            tk = __shfl_sync(0xFFFFFFFFu, tk, 0);
            if (lane == 0) {
                int done = (tk == (unsigned)prev.K_t);
                if (done) p.sc.ticket[prev.b] = 0u;
                sh.tail_seq = done ? prev.b : -1;
            }
        }
        cta_bar(1);
        int tb = sh.tail_seq;
        if (tb >= 0) {
            __threadfence();
            run_tail(tb);
        }
    }
}

}  // namespace adasd
