// Streaming verification kernel for sm_100a: persistent thread-block clusters, every logit
// row read from HBM exactly once, three SFU operations per logit pair.
//
//  * A position (b,i) = target row p_i + draft row q_i (bf16).  The CTAs of a cluster split
//    both rows into contiguous slices, the 16 warps of a CTA split the CTA's slice into
//    contiguous runs of "iterations" (one iteration = 32 lanes x 16 bytes of each row).
//  * Every warp owns a private ring of shared-memory slots (one slot = two iterations of
//    both rows).  Lane 0 fills a slot with two 1-D bulk copies (cp.async.bulk, completion
//    counted on the slot's own mbarrier) as soon as the warp has consumed it, so the ring
//    runs up to two positions ahead of the arithmetic and HBM never waits for it.  Every
//    wait on a copy is bounded; a warp whose wait expires reports it and stops copying.
//  * Pass A (row maxima, NaN and "rows differ" flags) of the NEXT position runs between the
//    arrive and the wait of the cluster barrier of the current one.  Pass B turns the slots
//    into 2^t values (t relative to the warp's own maximum) that stay on chip - the first
//    iterations in registers, the rest in shared memory - and into the warp's partial sums
//    S = sum 2^t and T = sum 2^t t.  One warp per CTA folds the 16 partials and sends the
//    CTA's totals to every CTA of the cluster over DSMEM; ONE cluster barrier per position.
//  * Pass C needs no logits and no ex2: with the row totals known it forms p + q from the
//    kept 2^t values and accumulates (p+q) log2(p+q); entropies come from S and T.
//  * The leader CTA finalises a position one barrier later and draws the per-sequence
//    ticket; the cluster that publishes the last position of a sequence runs that
//    sequence's tail (KDE/Bayes, accept scan, list appends, T_G) in the same launch.
#pragma once

#include "adasd_device.cuh"
#include "adasd_rows.cuh"
#include "adasd_tail.cuh"

namespace adasd {

constexpr int kCW = 12;                         // warps per CTA
constexpr int kCThreads = kCW * 32;
constexpr int kCMaxCluster = 8;
constexpr int kCMaxG = kCMaxCluster * kCW;      // warps per cluster, at most
constexpr int kCTab = 128;                      // entries of the per-warp tables (4 per lane)
static_assert(kCMaxG <= kCTab, "per-warp tables hold one entry per warp of the cluster");
constexpr int kCMaxSlots = 16;                  // ring slots per warp, at most
constexpr int kCSlotBytes = 2048;               // 2 iterations x (512 B target + 512 B draft)
constexpr int kCMaxIter = 10;                   // iterations per warp and row, at most
constexpr int kCRegIter = 5;                    // iterations whose 2^t values stay in registers
constexpr uint32_t kCWaitSpins = 1u << 22;
// bf16 value used to clamp -inf logits (0xF149 = -9.95e29), as fp32
#define ADASD_FLOOR_BF __uint_as_float(0xF1490000u)
// log2-domain shift of a slice (or row) without any finite logit; below floor * log2 e
constexpr float kFloorL = -2.0e30f;

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
__device__ __forceinline__ uint32_t mbar_test_wait(uint64_t* bar, uint32_t parity) {   // never blocks
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok;
}
// Bounded wait: false if the copy did not complete within the spin budget.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity) {
    for (uint32_t it = 0; it < kCWaitSpins; ++it)
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
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(kCThreads) : "memory");
}
__device__ __forceinline__ float warp_max_f32(float v) {   // NaN inputs are ignored
    float r;
    asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(r) : "f"(v));
    return r;
}
__device__ __forceinline__ uint32_t bmax2(uint32_t a, uint32_t b) {   // NaN-propagating bf16x2 max
    uint32_t d;
    asm("max.NaN.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ uint32_t bclamp2(uint32_t a) {             // max(a, floor), NaN dropped
    uint32_t d;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(0xF149F149u));
    return d;
}
__device__ __forceinline__ float2 unpack2(uint32_t w) {
    return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xFFFF0000u));
}

struct ClusterGeom {
    int32_t ncl;         // clusters in the grid
    int32_t NS;          // ring slots per warp (at least the slots of one position)
    int32_t stash_off;   // byte offset of the shared-memory part of the 2^t values (ring at 0)
};

// Partial (or total) softmax statistics of both rows over some slice of the vocabulary:
// maxima, S = sum 2^t, T = sum 2^t t with t = (z - max) log2 e.
struct __align__(16) RowPart {
    float mt, St, Tt, md;
    float Sd, Td;
    uint32_t flags;      // 1: NaN / +inf / expired wait, 2: the rows differ
    float pad;
};

struct __align__(16) ClusterShared {
    RowPart wtab[2][kCW];             // this CTA's warps, by position parity
    RowPart ctab[2][kCMaxCluster];    // every CTA's totals (written over DSMEM), by parity
    float2 tabC[2][kCTab];            // leader: per-warp (sum s log2 s, sum 2^t_p 2^t_q)
    float rtab[kCTab];                // vanilla: per-warp residual mass, every CTA holds all
    float fin[2][12];                 // leader: row totals kept for finalisation
    int32_t token[2];                 // leader: sampled token of the position
    int32_t tail_seq[2];              // leader: sequence whose tail must run (-1: none)
    uint32_t cnt[2];                  // warps of this CTA that have published wtab[par]
    unsigned long long bar[kCW][kCMaxSlots];   // "slot filled" barriers
};

struct PosRef {
    int pos;   // index into [B, Kmax+1]; >= total means "none"
    int kt;    // window K_t of its sequence
};

// ------------------------------------------------------------------------------------
template <int ITER, int MODE>
__global__ void __launch_bounds__(kCThreads, 1)
cluster_verify_kernel(VerifyParams p, ClusterGeom gq) {
    constexpr int KR = ITER < kCRegIter ? ITER : kCRegIter;   // iterations kept in registers
    extern __shared__ __align__(128) unsigned char dyn_smem[];
    __shared__ ClusterShared sh;
    __shared__ TailShared tsh;

    cg::cluster_group cluster = cg::this_cluster();
    const int CS = (int)cluster.num_blocks();
    const int rank = (int)cluster.block_rank();
    const int cid = blockIdx.x / CS;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = rank * kCW + warp;
    const int Kmax = p.Kmax, K1 = Kmax + 1;
    const int total = p.B * K1;
    const int ncl = gq.ncl;
    const bool leader = (rank == 0);

    // ---- this warp's share of a row: iterations [wi0, wi0 + I_w) of the CTA's slice -------
    const int NU = p.V >> 3;                                   // 16-byte units per row
    const int cu0 = (int)((long long)rank * NU / CS), cu1 = (int)((long long)(rank + 1) * NU / CS);
    const int nwi = (cu1 - cu0 + 31) >> 5;                     // warp-iterations of this CTA
    const int I_lo = nwi / kCW, I_rem = nwi % kCW;
    const int I_w = min(ITER, I_lo + (warp < I_rem ? 1 : 0));
    const int wu0 = cu0 + 32 * (warp * I_lo + min(warp, I_rem));
    const int nwu = max(0, min(32 * I_w, cu1 - wu0));          // units of this warp (last one ragged)
    const int n_stg = (I_w + 1) >> 1;                          // ring slots one position takes
    const int NSw = min(gq.NS, 2 * n_stg);                     // slots this warp cycles through

    unsigned char* const ring = dyn_smem + (size_t)warp * gq.NS * kCSlotBytes;
    unsigned char* const stash = dyn_smem + gq.stash_off + (size_t)warp * kCSlotBytes + (size_t)lane * 16;
    // shared-memory 2^t values of iteration k >= KR: slot (k-KR)*16 + warp, four 512-byte planes
    auto stash_ptr = [&](int k, int plane) -> float4* {
        return reinterpret_cast<float4*>(stash + (size_t)(k - KR) * (kCW * kCSlotBytes) + plane * 512);
    };

    for (int q = threadIdx.x; q < 4 * kCTab; q += kCThreads) reinterpret_cast<float*>(sh.tabC)[q] = 0.f;
    if (threadIdx.x < kCTab) sh.rtab[threadIdx.x] = 0.f;
    if (threadIdx.x == 0) {
        sh.tail_seq[0] = sh.tail_seq[1] = -1;
        sh.cnt[0] = sh.cnt[1] = 0u;
        sh.token[0] = sh.token[1] = -1;
    }
    if (lane == 0) {
        for (int s = 0; s < kCMaxSlots; ++s) mbar_init(reinterpret_cast<uint64_t*>(&sh.bar[warp][s]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    cluster.sync();   // every CTA of the cluster is running before any remote shared-memory access

    // ---- positions of this cluster: cid, cid + ncl, ... skipping those beyond a window ------
    auto window = [&](int b) -> int {
        int kt = p.draft_len ? __ldg(p.draft_len + b) : Kmax;
        return max(0, min(kt, Kmax));
    };
    // first active position among start, start + ncl, start + 2 ncl, ... (32 candidates per round)
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
    auto advance = [&](const PosRef& q) -> PosRef {
        if (q.pos >= total) return q;
        return scan_from(q.pos + ncl);
    };
    auto is_bonus = [&](const PosRef& q) -> bool { return (q.pos % K1) == q.kt; };

    PosRef cur = scan_from(cid), nxt = advance(cur), nn = advance(nxt);

    // ---- ring: fills are issued in position order, one slot at a time -----------------------
    uint32_t phase = 0;        // bit s: parity to wait for on slot s
    int cons_slot = 0;         // slot holding the next stage to be consumed
    int ip_which = 0;          // position the next fill belongs to: 0 cur, 1 nxt, 2 nn
    int ip_stage = 0;          // its next stage
    bool alive = true;         // false after a wait expired: no more copies, outputs flagged
    auto bar_of = [&](int s) -> uint64_t* { return reinterpret_cast<uint64_t*>(&sh.bar[warp][s]); };
    auto issue_one = [&](int slot) {
        if (!alive || n_stg == 0 || ip_which > 2) return;
        const PosRef q = ip_which == 0 ? cur : (ip_which == 1 ? nxt : nn);
        if (q.pos >= total) return;
        if (lane == 0) {
            const int b = q.pos / K1, i = q.pos - b * K1;
            const bool bonus = (i == q.kt);
            const int u0 = 64 * ip_stage;                               // first unit of the stage
            const uint32_t bytes = (uint32_t)min(64, nwu - u0) * 16u;
            const __nv_bfloat16* rt = reinterpret_cast<const __nv_bfloat16*>(p.zt) + (long long)b * p.t_seq +
                                      (long long)i * p.t_row + (size_t)(wu0 + u0) * 8;
            unsigned char* dst = ring + (size_t)slot * kCSlotBytes;
            uint64_t* bar = bar_of(slot);
            mbar_expect_tx(bar, bonus ? bytes : 2u * bytes);
            bulk_g2s(dst, rt, bytes, bar);
            if (!bonus) {
                const __nv_bfloat16* rd = reinterpret_cast<const __nv_bfloat16*>(p.zd) + (long long)b * p.d_seq +
                                          (long long)i * p.d_row + (size_t)(wu0 + u0) * 8;
                bulk_g2s(dst + 1024, rd, bytes, bar);
            }
        }
        if (++ip_stage == n_stg) {
            ip_stage = 0;
            ++ip_which;
        }
    };
    for (int s = 0; s < NSw; ++s) issue_one(s);

    // ---- pass A: packed maxima and flags of one position, slot by slot ----------------------
    uint32_t a_mT = 0xFF80FF80u, a_mD = 0xFF80FF80u, a_df = 0u;   // -inf pairs
    int a_next = 0;                                                 // first stage not yet scanned
    // scans stages [a_next, n_stg) of the position whose first slot is cons_slot; with
    // blocking == false it stops at the first slot that has not landed yet
    auto pass_a = [&](bool bonus, bool blocking) {
        if (!alive) return;
#pragma unroll
        for (int st = 0; st < (ITER + 1) / 2; ++st) {
            if (st >= a_next && st < n_stg) {
                int slot = cons_slot + st;
                if (slot >= NSw) slot -= NSw;
                const uint32_t par = (phase >> slot) & 1u;
                bool ok = blocking ? mbar_wait_bounded(bar_of(slot), par)
                                   : (mbar_test_wait(bar_of(slot), par) != 0);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) {
                    if (blocking) {          // the copy never landed: report it, stop copying
                        alive = false;
                        if (lane == 0) atomicOr(p.st.status, ADASD_STATUS_TIMEOUT);
                    }
                    break;
                }
                a_next = st + 1;
                const unsigned char* sb = ring + (size_t)slot * kCSlotBytes + (size_t)lane * 16;
#pragma unroll
                for (int kk = 0; kk < 2; ++kk) {
                    const int k = 2 * st + kk;
                    if (k < ITER && lane + 32 * k < nwu) {
                        const uint4 T = *reinterpret_cast<const uint4*>(sb + kk * 512);
                        a_mT = bmax2(bmax2(a_mT, T.x), bmax2(T.y, bmax2(T.z, T.w)));
                        if (!bonus) {
                            const uint4 D = *reinterpret_cast<const uint4*>(sb + 1024 + kk * 512);
                            a_mD = bmax2(bmax2(a_mD, D.x), bmax2(D.y, bmax2(D.z, D.w)));
                            a_df |= (T.x ^ D.x) | (T.y ^ D.y) | (T.z ^ D.z) | (T.w ^ D.w);
                        }
                    }
                }
            }
        }
    };
    // The warp's shifts and flags from the packed accumulators; resets them for the next
    // position.  Shifts live in the log2 domain: M = fl(max * log2 e), and every kept value is
    // 2^(z log2 e - M) with ONE rounding (an FMA), so sums of different warps combine through
    // the exact differences of their M.  A slice without a finite logit gets M = kFloorL and
    // all-zero values.
    float Mt_w = kFloorL, Md_w = kFloorL;     // published shifts
    float nmt_w = 0.f, nmd_w = 0.f;           // FMA addends of pass B (-M, or 0 for an empty slice)
    uint32_t flags_w = 0;
    auto finish_a = [&](bool bonus) {
        const float2 a = unpack2(a_mT), d = unpack2(a_mD);
        uint32_t bad = (a.x != a.x || a.y != a.y || d.x != d.x || d.y != d.y) ? 1u : 0u;
        const float vt = warp_max_f32(fmaxf(a.x, a.y));
        const float vd = bonus ? vt : warp_max_f32(fmaxf(d.x, d.y));
        if (vt == INFINITY || vd == INFINITY || !alive) bad = 1u;
        const bool has_t = vt > ADASD_FLOOR_BF, has_d = vd > ADASD_FLOOR_BF;
        Mt_w = has_t ? vt * kLog2e : kFloorL;
        Md_w = has_d ? vd * kLog2e : kFloorL;
        nmt_w = has_t ? -Mt_w : 0.f;
        nmd_w = has_d ? -Md_w : 0.f;
        flags_w = __reduce_or_sync(0xFFFFFFFFu, bad | (a_df ? 2u : 0u));
        a_mT = a_mD = 0xFF80FF80u;
        a_df = 0u;
        a_next = 0;
    };

    // ---- pass B: 2^t values (kept) and the warp's S and T ------------------------------------
    float et[KR][8], ed[KR][8];
    float sB[4];                       // after pass_b: warp totals St, Tt, Sd, Td
    auto pass_b = [&](bool bonus) {
        float2 St = make_float2(0.f, 0.f), Tt = St, Sd = St, Td = St;
        const float2 L2 = make_float2(kLog2e, kLog2e);
        const float2 nmt = make_float2(nmt_w, nmt_w);
        const float2 nmd = make_float2(nmd_w, nmd_w);
        const unsigned char* sb = ring;
#pragma unroll
        for (int k = 0; k < ITER; ++k) {
            if (k < I_w) {                                             // same for the whole warp
                if ((k & 1) == 0) sb = ring + (size_t)cons_slot * kCSlotBytes + (size_t)lane * 16;
                float e1[8], e2[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) e1[j] = e2[j] = 0.f;
                if (alive && lane + 32 * k < nwu) {
                    const uint4 T = *reinterpret_cast<const uint4*>(sb + (k & 1) * 512);
                    const uint32_t tw[4] = {T.x, T.y, T.z, T.w};
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const float2 z = unpack2(bclamp2(tw[j]));
                        const float2 t = __ffma2_rn(z, L2, nmt);
                        const float2 e = make_float2(ex2(t.x), ex2(t.y));
                        e1[2 * j] = e.x;
                        e1[2 * j + 1] = e.y;
                        St = __fadd2_rn(St, e);
                        Tt = __ffma2_rn(e, t, Tt);
                    }
                    if (!bonus) {
                        const uint4 D = *reinterpret_cast<const uint4*>(sb + 1024 + (k & 1) * 512);
                        const uint32_t dw[4] = {D.x, D.y, D.z, D.w};
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const float2 z = unpack2(bclamp2(dw[j]));
                            const float2 t = __ffma2_rn(z, L2, nmd);
                            const float2 e = make_float2(ex2(t.x), ex2(t.y));
                            e2[2 * j] = e.x;
                            e2[2 * j + 1] = e.y;
                            Sd = __fadd2_rn(Sd, e);
                            Td = __ffma2_rn(e, t, Td);
                        }
                    }
                }
                if (k < KR) {
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        et[k < KR ? k : 0][j] = e1[j];
                        ed[k < KR ? k : 0][j] = e2[j];
                    }
                } else {
                    *stash_ptr(k, 0) = make_float4(e1[0], e1[1], e1[2], e1[3]);
                    *stash_ptr(k, 1) = make_float4(e1[4], e1[5], e1[6], e1[7]);
                    *stash_ptr(k, 2) = make_float4(e2[0], e2[1], e2[2], e2[3]);
                    *stash_ptr(k, 3) = make_float4(e2[4], e2[5], e2[6], e2[7]);
                }
                if ((k & 1) == 1 || k == I_w - 1) {
                    // the slot is consumed: flip its parity and refill it with the next stage
                    __syncwarp();
                    phase ^= 1u << cons_slot;
                    issue_one(cons_slot);
                    if (++cons_slot == NSw) cons_slot = 0;
                }
            } else if (k < KR) {
#pragma unroll
                for (int j = 0; j < 8; ++j) et[k < KR ? k : 0][j] = ed[k < KR ? k : 0][j] = 0.f;
            }
        }
        sB[0] = warp_sum(St.x + St.y);
        sB[1] = warp_sum(Tt.x + Tt.y);
        if (bonus) {
            sB[2] = sB[0];
            sB[3] = sB[1];
        } else {
            sB[2] = warp_sum(Sd.x + Sd.y);
            sB[3] = warp_sum(Td.x + Td.y);
        }
    };
    // the 2^t values of iteration k (compile-time k after unrolling)
    auto load_stash = [&](int k, float (&a)[8], float (&b)[8]) {
        if (k < KR) {
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                a[j] = et[k < KR ? k : 0][j];
                b[j] = ed[k < KR ? k : 0][j];
            }
        } else {
            const float4 a0 = *stash_ptr(k, 0), a1 = *stash_ptr(k, 1), b0 = *stash_ptr(k, 2), b1 = *stash_ptr(k, 3);
            a[0] = a0.x, a[1] = a0.y, a[2] = a0.z, a[3] = a0.w, a[4] = a1.x, a[5] = a1.y, a[6] = a1.z, a[7] = a1.w;
            b[0] = b0.x, b[1] = b0.y, b[2] = b0.z, b[3] = b0.w, b[4] = b1.x, b[5] = b1.y, b[6] = b1.z, b[7] = b1.w;
        }
    };

    // ---- exchange: warp partials -> CTA totals -> every CTA of the cluster -------------------
    // The warp that publishes last (a shared-memory counter tells) folds the 16 partials.
    auto publish = [&](int par) {
        unsigned old = 0;
        if (lane == 0) {
            float4* w = reinterpret_cast<float4*>(&sh.wtab[par][warp]);
            w[0] = make_float4(Mt_w, sB[0], sB[1], Md_w);
            w[1] = make_float4(sB[2], sB[3], __uint_as_float(flags_w), 0.f);
            __threadfence_block();
            old = atomicAdd(&sh.cnt[par], 1u);
        }
        old = __shfl_sync(0xFFFFFFFFu, old, 0);
        if (old == kCW - 1) {
            if (lane == 0) sh.cnt[par] = 0u;
            __threadfence_block();
            float4 e0 = make_float4(kFloorL, 0.f, 0.f, kFloorL), e1 = make_float4(0.f, 0.f, 0.f, 0.f);
            if (lane < kCW) {
                const float4* w = reinterpret_cast<const float4*>(&sh.wtab[par][lane]);
                e0 = w[0];
                e1 = w[1];
            }
            const float Mt = warp_max_f32(e0.x), Md = warp_max_f32(e0.w);
            const float dt = e0.x - Mt, dd = e0.w - Md;
            const float ft = ex2(dt), fd = ex2(dd);
            const float St = warp_sum(ft * e0.y), Tt = warp_sum(ft * fmaf(dt, e0.y, e0.z));
            const float Sd = warp_sum(fd * e1.x), Td = warp_sum(fd * fmaf(dd, e1.x, e1.y));
            const uint32_t fl = __reduce_or_sync(0xFFFFFFFFu, __float_as_uint(e1.z));
            if (lane < CS) {
                float4* dst = reinterpret_cast<float4*>(&cluster.map_shared_rank(&sh, lane)->ctab[par][rank]);
                dst[0] = make_float4(Mt, St, Tt, Md);
                dst[1] = make_float4(Sd, Td, __uint_as_float(fl), 0.f);
            }
        }
    };

    struct Totals {
        float Mt, St, Tt, Md, Sd, Td;
        uint32_t fl;
    };
    // row totals from the CTA totals; every lane of every warp computes the same numbers
    auto totals = [&](int par) -> Totals {
        Totals r;
        r.Mt = r.Md = kFloorL;
        r.fl = 0u;
#pragma unroll
        for (int c = 0; c < kCMaxCluster; ++c) {
            if (c < CS) {
                const float4* e = reinterpret_cast<const float4*>(&sh.ctab[par][c]);
                const float4 e0 = e[0], e1 = e[1];
                r.Mt = fmaxf(r.Mt, e0.x);
                r.Md = fmaxf(r.Md, e0.w);
                r.fl |= __float_as_uint(e1.z);
            }
        }
        r.St = r.Tt = r.Sd = r.Td = 0.f;
#pragma unroll
        for (int c = 0; c < kCMaxCluster; ++c) {
            if (c < CS) {
                const float4* e = reinterpret_cast<const float4*>(&sh.ctab[par][c]);
                const float4 e0 = e[0], e1 = e[1];
                const float dt = e0.x - r.Mt, dd = e0.w - r.Md;
                const float ft = ex2(dt), fd = ex2(dd);
                r.St = fmaf(ft, e0.y, r.St);
                r.Tt = fmaf(ft, fmaf(dt, e0.y, e0.z), r.Tt);
                r.Sd = fmaf(fd, e1.x, r.Sd);
                r.Td = fmaf(fd, fmaf(dd, e1.x, e1.y), r.Td);
            }
        }
        return r;
    };

    // Which warp of THIS CTA holds the crossing of target = u * S_t of the target row, in index
    // order (CTA by CTA, then warp by warp).  Returns the warp (-1: another CTA, or no mass)
    // and the weight before it; if rounding leaves no crossing, the last warp with mass and
    // target = +inf (the caller then takes its last element with mass).
    auto locate_p = [&](int par, const Totals& tt, float u, float& base, float& target) -> int {
        target = u * tt.St;
        float cum = 0.f, cbase = 0.f, lbase = 0.f;
        int cstar = -1, clast = -1;
#pragma unroll
        for (int c = 0; c < kCMaxCluster; ++c) {
            if (c < CS) {
                const float4 e0 = *reinterpret_cast<const float4*>(&sh.ctab[par][c]);
                const float w = ex2(e0.x - tt.Mt) * e0.y;
                const float nc = cum + w;
                if (w > 0.f) {
                    clast = c;
                    lbase = cum;
                    if (cstar < 0 && nc > target) {
                        cstar = c;
                        cbase = cum;
                    }
                }
                cum = nc;
            }
        }
        if (cstar < 0) {
            cstar = clast;
            cbase = lbase;
            target = INFINITY;
        }
        if (cstar != rank) return -1;
        float w = 0.f;
        if (lane < kCW) {
            const float4 e0 = *reinterpret_cast<const float4*>(&sh.wtab[par][lane]);
            w = ex2(e0.x - tt.Mt) * e0.y;
        }
        float incl = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const float t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= o) incl += t;
        }
        const float excl = incl - w;
        const unsigned mh = __ballot_sync(0xFFFFFFFFu, w > 0.f && cbase + incl > target);
        int wsel;
        if (mh) {
            wsel = __ffs(mh) - 1;
        } else {
            const unsigned ml = __ballot_sync(0xFFFFFFFFu, w > 0.f);
            if (!ml) return -1;
            wsel = 31 - __clz(ml);
            target = INFINITY;
        }
        base = cbase + __shfl_sync(0xFFFFFFFFu, excl, wsel);
        return wsel;
    };

    // Run by the chosen warp: first element (index order: iteration, lane, element) where
    // base + f * running weight exceeds target, else the last element with weight.
    // vals(k, v) fills the 8 weights of this lane's unit of iteration k.
    auto select_kept = [&](float base, float f, float target, auto vals) -> int {
        float ls[ITER], tot[ITER];
#pragma unroll
        for (int k = 0; k < ITER; ++k) {
            ls[k] = 0.f;
            if (k < I_w) {
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

    // ---- leader warp 0: a position's published scalars, one barrier after its pass C ----------
    // Returns nothing; writes sh.tail_seq[tpar] (the sequence whose last position this was, or -1).
    auto finalize = [&](const PosRef& q, int par, int tpar) {
        const float2 c0 = sh.tabC[par][4 * lane], c1 = sh.tabC[par][4 * lane + 1];
        const float2 c2 = sh.tabC[par][4 * lane + 2], c3 = sh.tabC[par][4 * lane + 3];
        const float A = warp_sum(((c0.x + c1.x) + c2.x) + c3.x);
        const float PQ = warp_sum(((c0.y + c1.y) + c2.y) + c3.y);
        if (lane == 0) {
            const int b = q.pos / K1, i = q.pos - b * K1;
            const bool bonus = (i == q.kt);
            const float Mt = sh.fin[par][0], St = sh.fin[par][1], Tt = sh.fin[par][2];
            const float Md = sh.fin[par][3], Sd = sh.fin[par][4], Td = sh.fin[par][5];
            const uint32_t fl = __float_as_uint(sh.fin[par][6]);
            const bool bad = (fl & 1u) || !(Mt > kFloorL) || !(Md > kFloorL);
            const size_t it = (size_t)b * K1 + i, id = (size_t)b * Kmax + i;
            int tok = sh.token[par];
            if (bad) {
                atomicOr(p.st.status, ADASD_STATUS_NAN);
                tok = -1;
            }
            if (MODE == MODE_ADASD) {
                const float lSt = lg2(St), lSd = lg2(Sd);
                const float Hbt = lSt - Tt / St, Hbd = lSd - Td / Sd;      // entropies in bits
                float Ht = kLn2 * Hbt, lse_t = kLn2 * (Mt + lSt);
                if (bad) Ht = lse_t = NAN;
                p.sc.H_t[it] = Ht;
                p.sc.lse_t[it] = lse_t;
                p.sc.y[it] = tok;
                if (p.user.H_t) p.user.H_t[it] = Ht;
                if (p.user.lse_t) p.user.lse_t[it] = lse_t;
                if (p.user.y) p.user.y[it] = tok;
                if (!bonus) {
                    float Hd = kLn2 * Hbd, lse_d = kLn2 * (Md + lSd);
                    // D_JS = H(m) - (H(p) + H(q)) / 2 with H(m) = (ln 2 / 2) (2 - sum s log2 s), s = p + q
                    float jsd = 0.5f * kLn2 * ((2.f - A) - (Hbt + Hbd));
                    jsd = (fl & 2u) ? fminf(fmaxf(jsd, 0.f), kLn2) : 0.f;   // identical rows: exactly 0
                    if (!(PQ > 0.f)) jsd = kLn2;                            // disjoint supports: ln 2
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
                if (!bonus) {
                    p.sc.van_flag[id] = (sh.fin[par][8] != 0.f && !bad) ? 1 : 0;
                    if (p.alpha_out) p.alpha_out[id] = bad ? NAN : sh.fin[par][7];
                }
                p.sc.van_tok[it] = tok;
            }
            __threadfence();
            const unsigned ticket = atomicAdd(p.sc.ticket + b, 1u);
            const bool done = (ticket == (unsigned)q.kt);
            if (done) p.sc.ticket[b] = 0u;          // ready for the next round
            sh.tail_seq[tpar] = done ? b : -1;
        }
    };

    // The sequence's tail, run by the whole leader CTA.
    auto run_tail = [&](int b) {
        __threadfence();
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
            const int kt = window(b);
            int w = kt;
            for (int j = 0; j < kt; ++j) {
                if (__ldcg(p.sc.van_flag + (size_t)b * Kmax + j) == 0) {
                    w = j;
                    break;
                }
            }
            p.accept_len[b] = w;
            p.next_token[b] = __ldcg(p.sc.van_tok + (size_t)b * K1 + w);
        }
    };

    // ================================== main loop ======================================
    PosRef prev;
    prev.pos = total;
    prev.kt = 0;
    int it = 0;                                   // positions this cluster has started
    if (cur.pos < total) pass_a(is_bonus(cur), true);
    while (cur.pos < total) {
        const int par = it & 1;
        const int b = cur.pos / K1, i = cur.pos - b * K1;
        const bool bonus = (i == cur.kt);
        const size_t idt = (size_t)b * K1 + i, idd = (size_t)b * Kmax + i;

        finish_a(bonus);
        pass_b(bonus);
        publish(par);

        // per-position scalars needed after the barrier, fetched early
        float u_samp = 0.f, u_acc = 0.f, ztx = 0.f, zdx = 0.f;
        int xi = -1;
        if (MODE == MODE_ADASD) {
            u_samp = __ldg(p.u_target + idt);
        } else {
            u_samp = __ldg(p.u_resample + b);
            if (!bonus) {
                u_acc = __ldg(p.u_accept + idd);
                xi = __ldg(p.x + idd);
                if (xi >= 0 && xi < p.V) {
                    ztx = __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p.zt)[(long long)b * p.t_seq + (long long)i * p.t_row + xi]);
                    zdx = __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p.zd)[(long long)b * p.d_seq + (long long)i * p.d_row + xi]);
                }
            }
        }

        cluster_arrive();                                   // ---- the position's barrier
        // shadow of the barrier: maxima of the next position, as far as its slots have landed
        const bool nbonus = nxt.pos < total && is_bonus(nxt);
        if (nxt.pos < total) pass_a(nbonus, false);
        cluster_wait();

        // leader CTA: tail of the sequence completed one position ago, then this round's finalisation
        if (leader && it > 0) {
            const int tb = sh.tail_seq[par ^ 1];
            if (tb >= 0) run_tail(tb);
            if (warp == 0) finalize(prev, par ^ 1, par);
        }

        const Totals tt = totals(par);
        const bool bad = (tt.fl & 1u) || !(tt.Mt > kFloorL) || !(tt.Md > kFloorL);
        const float ft = ex2(Mt_w - tt.Mt), fd = ex2(Md_w - tt.Md);
        const float at = ft / tt.St, ad = fd / tt.Sd;           // p = 2^t_p * at, q = 2^t_q * ad
        ClusterShared* const lead = cluster.map_shared_rank(&sh, 0);

        // vanilla: alpha at the draft token
        bool van_accept = true;
        float alpha = 0.f;
        if (MODE == MODE_VANILLA && !bonus) {
            if (xi >= 0 && xi < p.V) {
                const float a = fmaf(fmaxf(ztx, ADASD_FLOOR_BF), kLog2e, -tt.Mt) - lg2(tt.St);
                const float q = fmaf(fmaxf(zdx, ADASD_FLOOR_BF), kLog2e, -tt.Md) - lg2(tt.Sd);
                alpha = fminf(1.f, ex2(a - q));
                if (!(ex2(q) > 0.f)) alpha = 1.f;   // q(x) = 0 cannot have been drafted
            }
            van_accept = u_acc < alpha;
        }
        if (leader && warp == 0 && lane == 0) {
            sh.fin[par][0] = tt.Mt;
            sh.fin[par][1] = tt.St;
            sh.fin[par][2] = tt.Tt;
            sh.fin[par][3] = tt.Md;
            sh.fin[par][4] = tt.Sd;
            sh.fin[par][5] = tt.Td;
            sh.fin[par][6] = __uint_as_float(tt.fl);
            sh.fin[par][7] = alpha;
            sh.fin[par][8] = van_accept ? 1.f : 0.f;
        }
        const bool need_resid = (MODE == MODE_VANILLA) && !bonus && !van_accept && !bad;

        // sample from p (AdaSD: y_i of every row; vanilla: the bonus row)
        auto sample_p = [&]() {
            float base = 0.f, target = 0.f;
            const int wsel = locate_p(par, tt, u_samp, base, target);
            if (wsel == warp) {
                const int tok = select_kept(base, ft, target, [&](int k, float(&v)[8]) {
                    float d[8];
                    load_stash(k, v, d);
                });
                if (lane == 0) lead->token[par] = tok;
            }
        };
        if ((MODE == MODE_ADASD || bonus) && !bad) sample_p();

        // pass C: sum (p+q) log2 (p+q) and the overlap indicator sum 2^t_p 2^t_q
        if (MODE == MODE_ADASD && !bonus) {
            float2 A2 = make_float2(0.f, 0.f), PQ2 = make_float2(0.f, 0.f);
            const float2 at2 = make_float2(at, at), ad2 = make_float2(ad, ad);
            const float2 tiny2 = make_float2(kTiny, kTiny);
#pragma unroll
            for (int k = 0; k < ITER; ++k) {
                if (k < I_w) {
                    float a[8], d[8];
                    load_stash(k, a, d);
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
            const float A = warp_sum(A2.x + A2.y), PQ = warp_sum(PQ2.x + PQ2.y);
            if (lane == 0) lead->tabC[par][g] = make_float2(A, PQ);
        }

        if (need_resid) {
            // vanilla, rejected row: residual mass max(0, p - q) per warp, then a second barrier
            // so that every warp can find the one holding the crossing
            auto resid = [&](int k, float(&v)[8]) {
                float a[8], d[8];
                load_stash(k, a, d);
#pragma unroll
                for (int j = 0; j < 8; ++j) v[j] = fmaxf(fmaf(a[j], at, -d[j] * ad), 0.f);
            };
            float r = 0.f;
#pragma unroll
            for (int k = 0; k < ITER; ++k) {
                if (k < I_w) {
                    float v[8];
                    resid(k, v);
                    r += ((v[0] + v[1]) + (v[2] + v[3])) + ((v[4] + v[5]) + (v[6] + v[7]));
                }
            }
            r = warp_sum(r);
            if (lane < CS) cluster.map_shared_rank(&sh, lane)->rtab[g] = r;
            cluster_arrive();
            cluster_wait();
            const float4 sv = *reinterpret_cast<const float4*>(&sh.rtab[4 * lane]);
            const float c4[4] = {sv.x, sv.y, sv.z, sv.w};
            const float lsum = ((sv.x + sv.y) + sv.z) + sv.w;
            float incl = lsum;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const float t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                if (lane >= o) incl += t;
            }
            const float R = __shfl_sync(0xFFFFFFFFu, incl, 31);
            if (R > 0.f) {
                float target = u_samp * R, run = incl - lsum;
                int hit = -1, lastp = -1;
                float hbase = 0.f, lbase = 0.f;
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const float nr = run + c4[k];
                    if (c4[k] > 0.f) {
                        lastp = 4 * lane + k;
                        lbase = run;
                        if (hit < 0 && nr > target) {
                            hit = 4 * lane + k;
                            hbase = run;
                        }
                    }
                    run = nr;
                }
                int gsel;
                float base;
                const unsigned mh = __ballot_sync(0xFFFFFFFFu, hit >= 0);
                if (mh) {
                    const int src = __ffs(mh) - 1;
                    gsel = __shfl_sync(0xFFFFFFFFu, hit, src);
                    base = __shfl_sync(0xFFFFFFFFu, hbase, src);
                } else {
                    const unsigned ml = __ballot_sync(0xFFFFFFFFu, lastp >= 0);
                    const int src = ml ? 31 - __clz(ml) : 0;
                    gsel = __shfl_sync(0xFFFFFFFFu, lastp, src);
                    base = __shfl_sync(0xFFFFFFFFu, lbase, src);
                    target = INFINITY;
                }
                if (gsel == g) {
                    const int tok = select_kept(base, 1.f, target, resid);
                    if (lane == 0) lead->token[par] = tok;
                }
            } else {
                sample_p();   // no residual mass: sample from p
            }
        }

        // the rest of the next position's maxima (waits for slots still in flight)
        if (nxt.pos < total) pass_a(nbonus, true);

        prev = cur;
        cur = nxt;
        nxt = nn;
        nn = advance(nn);
        --ip_which;
        ++it;
    }

    // ---- drain: one more barrier makes the last position's sums visible to the leader -------
    if (it > 0) {
        cluster_arrive();
        cluster_wait();
        if (leader) {
            const int par = it & 1;
            const int tb = sh.tail_seq[par ^ 1];
            if (tb >= 0) run_tail(tb);
            if (warp == 0) finalize(prev, par ^ 1, par);
            cta_bar(1);
            const int tb2 = sh.tail_seq[par];
            if (tb2 >= 0) run_tail(tb2);
        }
    }
    // a warp that gave up on a copy still waits (bounded) for whatever it had in flight
    if (!alive) {
        for (int s = 0; s < NSw; ++s) mbar_wait_bounded(bar_of(s), (phase >> s) & 1u);
    }
}

}  // namespace adasd
