// Streaming draft-step kernel for sm_100a (adasd_draft_entropy on bf16 rows of a multiple of 8
// logits): every row is read from HBM once.
//
//  * One cluster of P CTAs per row (P = 1, 2, 4 or 8, chosen so that the launch fills the SMs);
//    the 8 warps of a CTA split the CTA's part of the row into contiguous shares and stream
//    them through two 4 KB buffers each (1-D bulk copies, bounded mbarrier waits).
//  * Per chunk: packed bf16 maximum, then 2^(z log2 e - M) with the warp's running shift M
//    (raised, with the sums rescaled, only when a chunk exceeds it), accumulating S = sum 2^t
//    and T = sum 2^t t.  The chunk's own sum is kept in a small table for sampling.
//  * The CTAs send their totals and tables to rank 0 over DSMEM; after ONE cluster barrier
//    rank 0 forms H(q) = ln 2 (log2 S - T / S), the log-sum-exp and the stop flag H > T_G,
//    finds the chunk that holds the inverse-CDF crossing of u and rescans just that chunk
//    (4 KB, from L2) for the token x ~ q.
#pragma once

#include "adasd_cluster.cuh"

namespace adasd {

constexpr int kDW = 8;                         // warps per CTA when two CTAs share an SM
constexpr int kDWBig = 16;                     // warps per CTA when the grid has one CTA per SM at most
constexpr int kDChunkUnits = 256;              // 16-byte units per chunk: 8 iterations of a warp
constexpr int kDChunkBytes = kDChunkUnits * 16;
constexpr int kDMaxChunks = 12;                // chunks per warp, at most (V <= 8 * 8 * 12 * 2048)
constexpr int kDMaxP = 8;

constexpr int kDMaxEntries = 64;               // warps per cluster (P * NW), at most: two table entries per lane
template <int NW>
struct __align__(16) DraftShared {
    float cm[kDMaxEntries][kDMaxChunks];       // rank 0: shift in force when a chunk was summed, by (rank, warp)
    float cs[kDMaxEntries][kDMaxChunks];       // rank 0: the chunk's sum of 2^t under that shift
    float4 wpart[kDMaxEntries];                // rank 0: every warp's (M, S, T, flags)
    unsigned long long bar[NW][2];
};

// NW warps per CTA: 8 (two CTAs per SM) or 16 (one CTA per SM, for grids that do not fill the
// SMs twice); P * NW <= kDMaxEntries.
// WARPED: an adjusted distribution is set (Sec. 2.1.1); the ordinary instantiation carries none of its code.
template <int NW, bool WARPED = false>
__global__ void __launch_bounds__(NW * 32, NW == kDW ? 2 : 1) draft_stream_kernel(DraftParams p) {
    constexpr int kDW = NW;                    // (shadows the namespace constant: warps of THIS kernel)
    extern __shared__ __align__(128) unsigned char dyn_smem[];
    __shared__ DraftShared<NW> sh;
    cg::cluster_group cluster = cg::this_cluster();
    const int P = (int)cluster.num_blocks();
    const int rank = (int)cluster.block_rank();
    const int b = blockIdx.x / P;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // Launched with programmatic stream serialisation: the CTAs may be resident before the
    // kernel ahead in the stream has finished; nothing it wrote (the logits, the active mask, the
    // window lengths) is touched before this wait, which returns once that kernel is complete.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const bool active = !(p.active && p.active[b] == 0);      // same in every CTA of the cluster
    // what the last step of the row needs from global memory is asked for now, by the warp that
    // will need it, so that it is there after the stream: the uniform and the threshold
    float u_row = 0.f, tg_row = 0.f;
    int32_t len_row = 0;
    if (active && rank == 0 && warp == 0) {
        if (p.u != nullptr) u_row = __ldg(p.u + b);
        tg_row = p.st.T_G[b];
        if (p.draft_len) len_row = p.draft_len[b];          // (only this row's CTA ever writes it)
    }

    // this warp's share of the row, in 16-byte units
    const int NU = p.V >> 3;
    const int cu0 = (int)((long long)rank * NU / P), cu1 = (int)((long long)(rank + 1) * NU / P);
    const int wu0 = cu0 + (int)((long long)warp * (cu1 - cu0) / kDW);
    const int wu1 = cu0 + (int)((long long)(warp + 1) * (cu1 - cu0) / kDW);
    const int nwu = wu1 - wu0;
    const int nch = min(kDMaxChunks, (nwu + kDChunkUnits - 1) / kDChunkUnits);
    const unsigned char* const src =
        reinterpret_cast<const unsigned char*>(reinterpret_cast<const __nv_bfloat16*>(p.z) + (long long)b * p.row_stride) +
        (size_t)wu0 * 16;
    unsigned char* const bufs = dyn_smem + (size_t)warp * (2 * kDChunkBytes);

    if (lane == 0) {
        mbar_init(reinterpret_cast<uint64_t*>(&sh.bar[warp][0]), 1);
        mbar_init(reinterpret_cast<uint64_t*>(&sh.bar[warp][1]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    // every CTA of the cluster is running before anyone writes into rank 0 (a CTA on its own
    // writes to itself, and every warp waits on barriers it set up itself)
    if (P > 1) cluster.sync();
    bool alive = true;
    // self-test of the give-up path: this warp never asks for its first chunk and waits for it only
    // briefly, so the wait runs out with nothing in flight
    const bool expiring = (b == p.expire_row && rank == 0 && warp == 0);
    auto issue = [&](int c) {
        if (lane == 0 && c < nch && !(expiring && c == 0)) {
            const uint32_t bytes = (uint32_t)min(kDChunkUnits, nwu - c * kDChunkUnits) * 16u;
            uint64_t* bar = reinterpret_cast<uint64_t*>(&sh.bar[warp][c & 1]);
            mbar_expect_tx(bar, bytes);
            bulk_g2s(bufs + (size_t)(c & 1) * kDChunkBytes, src + (size_t)c * kDChunkBytes, bytes, bar);
        }
    };
    // adjusted distribution: t = (z - max) log2 e / T, logits below the row's cutoff count as -inf
    const float c1 = WARPED ? p.c1 : kLog2e;
    const uint32_t cut2 = (WARPED && p.cut) ? cut_pair(__ldg(p.cut + b)) : kNoCut2;
    float M = kFloorL;                                   // running shift (log2 domain)
    // the largest logit so far (0 while there is none): t = (z - vM) log2 e is exactly 0 for it,
    // so that a one-hot row gets S = 1, T = 0 and H = 0 exactly
    float vM = 0.f;
    float2 S2 = make_float2(0.f, 0.f), T2 = S2;          // lane partials under M
    uint32_t bad = 0u;
    if (active) {
        issue(0);
        issue(1);
        // table entries of chunks this warp does not have: no weight
        if (lane >= nch && lane < kDMaxChunks) {
            DraftShared<NW>* r0 = cluster.map_shared_rank(&sh, 0);
            r0->cm[rank * kDW + warp][lane] = kFloorL;
            r0->cs[rank * kDW + warp][lane] = 0.f;
        }
        int cfail = -1;                                      // chunk whose copy never landed
        for (int c = 0; c < nch; ++c) {
            bool ok = alive && mbar_wait_bounded(reinterpret_cast<uint64_t*>(&sh.bar[warp][c & 1]), (uint32_t)(c >> 1) & 1u,
                                                 expiring && c == 0 ? 64u : kCWaitSpins);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) {
                if (alive && lane == 0) atomicOr(p.st.status, ADASD_STATUS_TIMEOUT);
                alive = false;
                bad = 1u;
                cfail = c;
                break;
            }
            const unsigned char* sb = bufs + (size_t)(c & 1) * kDChunkBytes + (size_t)lane * 16;
            const int ubase = c * kDChunkUnits + lane;
            uint4 W[8];
            uint32_t mx = 0xFF80FF80u;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                W[i] = *reinterpret_cast<const uint4*>(sb + i * 512);
                if (!(ubase + 32 * i < nwu)) W[i] = make_uint4(0xF149F149u, 0xF149F149u, 0xF149F149u, 0xF149F149u);
                mx = bmax2(bmax2(mx, W[i].x), bmax2(W[i].y, bmax2(W[i].z, W[i].w)));
            }
            if (WARPED && cut2 != kNoCut2) {
#pragma unroll
                for (int i = 0; i < 8; ++i) bcut8(W[i], cut2);
            }
            // both buffers are in registers or free: fetch the chunk after the next
            __syncwarp();
            issue(c + 2);
            const float2 mm = unpack2(mx);
            if (mm.x != mm.x || mm.y != mm.y) bad = 1u;
            const float vmax = warp_max_f32(fmaxf(mm.x, mm.y));
            if (vmax == INFINITY) bad = 1u;
            const float Mc = vmax > ADASD_FLOOR_BF ? vmax * c1 : kFloorL;
            if (Mc > M) {                                 // raise the shift, rescale what is summed
                const float d = M > kFloorL ? (vM - vmax) * c1 : kFloorL, f = ex2(d);
                T2.x = f * fmaf(d, S2.x, T2.x);
                T2.y = f * fmaf(d, S2.y, T2.y);
                S2.x *= f;
                S2.y *= f;
                M = Mc;
                vM = vmax;
            }
            const float2 nv2 = make_float2(-vM, -vM), L2 = make_float2(c1, c1);
            float2 Sc = make_float2(0.f, 0.f);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const uint32_t w[4] = {W[i].x, W[i].y, W[i].z, W[i].w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float2 z = unpack2(bclamp2(w[j]));
                    const float2 t = __fmul2_rn(__fadd2_rn(z, nv2), L2);
                    const float2 e = make_float2(ex2(t.x), ex2(t.y));
                    Sc = __fadd2_rn(Sc, e);
                    T2 = __ffma2_rn(e, t, T2);
                }
            }
            S2 = __fadd2_rn(S2, Sc);
            const float cs = warp_sum(Sc.x + Sc.y);
            if (lane == 0) {
                DraftShared<NW>* r0 = cluster.map_shared_rank(&sh, 0);
                r0->cm[rank * kDW + warp][c] = M;
                r0->cs[rank * kDW + warp][c] = cs;
            }
        }
        // a warp that gave up still waits (bounded) for what it had asked for and not taken: the
        // chunk it gave up on and the one after it; nothing may land in this CTA after it has gone
        if (cfail >= 0) {
            for (int c = cfail; c < min(cfail + 2, nch); ++c)
                if (!(expiring && c == 0))
                    mbar_wait_bounded(reinterpret_cast<uint64_t*>(&sh.bar[warp][c & 1]), (uint32_t)(c >> 1) & 1u);
        }
        const float Sw = warp_sum(S2.x + S2.y), Tw = warp_sum(T2.x + T2.y);
        bad = __reduce_or_sync(0xFFFFFFFFu, bad);
        if (lane == 0)
            cluster.map_shared_rank(&sh, 0)->wpart[rank * kDW + warp] = make_float4(M, Sw, Tw, __uint_as_float(bad));
    }
    // totals and tables of every CTA are in rank 0's shared memory
    if (P > 1) cluster.sync();
    else __syncthreads();
    if (!active || rank != 0) return;
    // (rank 0 only reads its own shared memory from here on; nobody writes to it any more)

    if (warp == 0) {
        // row totals: lane l holds warp-entry l (and l + 32 when P * 8 > 32)
        const int NE = P * kDW;
        const float4* wp = &sh.wpart[0];
        float4 e0 = lane < NE ? wp[lane] : make_float4(kFloorL, 0.f, 0.f, 0.f);
        float4 e1 = lane + 32 < NE ? wp[lane + 32] : make_float4(kFloorL, 0.f, 0.f, 0.f);
        const float Mr = warp_max_f32(fmaxf(e0.x, e1.x));
        const float d0 = e0.x - Mr, d1 = e1.x - Mr;
        const float f0 = ex2(d0), f1 = ex2(d1);
        const float S = warp_sum(f0 * e0.y + f1 * e1.y);
        const float T = warp_sum(f0 * fmaf(d0, e0.y, e0.z) + f1 * fmaf(d1, e1.y, e1.z));
        const uint32_t fl = __reduce_or_sync(0xFFFFFFFFu, __float_as_uint(e0.w) | __float_as_uint(e1.w));
        const bool rowbad = (fl & 1u) || !(Mr > kFloorL);
        const float lS = lg2(S);
        float H = kLn2 * (lS - T / S), lse = kLn2 * (Mr + lS);
        if (rowbad) H = lse = NAN;

        // x ~ q: the crossing of u * S in index order (rank, warp, chunk): first the warp share
        // that holds it (entry l of the totals, and l + 32), then the chunk within that share
        int tok = -1;
        const bool sampling = (p.u != nullptr && p.token_out != nullptr);
        if (sampling && !rowbad) {
            float target = u_row * S;
            const float w0 = f0 * e0.y, w1 = f1 * e1.y;
            float i0 = w0, i1 = w1;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const float t0 = __shfl_up_sync(0xFFFFFFFFu, i0, o), t1 = __shfl_up_sync(0xFFFFFFFFu, i1, o);
                if (lane >= o) {
                    i0 += t0;
                    i1 += t1;
                }
            }
            const float tot0 = __shfl_sync(0xFFFFFFFFu, i0, 31);
            i1 += tot0;
            const unsigned h0 = __ballot_sync(0xFFFFFFFFu, w0 > 0.f && i0 > target);
            const unsigned h1 = __ballot_sync(0xFFFFFFFFu, w1 > 0.f && i1 > target);
            const unsigned m0 = __ballot_sync(0xFFFFFFFFu, w0 > 0.f), m1 = __ballot_sync(0xFFFFFFFFu, w1 > 0.f);
            int ent = -1;
            if (h0) ent = __ffs(h0) - 1;
            else if (h1) ent = 32 + __ffs(h1) - 1;
            else {                   // rounding left no crossing: last share with mass, last token with mass
                if (m1) ent = 32 + 31 - __clz(m1);
                else if (m0) ent = 31 - __clz(m0);
                target = INFINITY;
            }
            if (ent >= 0) {
                const float ebase = ent < 32 ? __shfl_sync(0xFFFFFFFFu, i0 - w0, ent)
                                             : __shfl_sync(0xFFFFFFFFu, i1 - w1, ent - 32);
                const float* cmf = &sh.cm[0][0] + ent * kDMaxChunks;
                const float* csf = &sh.cs[0][0] + ent * kDMaxChunks;
                const float v = lane < kDMaxChunks ? ex2(cmf[lane] - Mr) * csf[lane] : 0.f;
                float incl = v;
#pragma unroll
                for (int o = 1; o < 16; o <<= 1) {
                    const float t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                    if (lane >= o) incl += t;
                }
                const unsigned ch = __ballot_sync(0xFFFFFFFFu, v > 0.f && ebase + incl > target);
                const unsigned cl = __ballot_sync(0xFFFFFFFFu, v > 0.f);
                int c = -1;
                if (ch) c = __ffs(ch) - 1;
                else if (cl) {
                    c = 31 - __clz(cl);
                    target = INFINITY;
                }
                if (c >= 0) {
                    const float base = ebase + __shfl_sync(0xFFFFFFFFu, incl - v, c);
                    const int r = ent / kDW, w = ent % kDW;
                    const int cu0r = (int)((long long)r * NU / P), cu1r = (int)((long long)(r + 1) * NU / P);
                    const int a0 = cu0r + (int)((long long)w * (cu1r - cu0r) / kDW);
                    const int a1 = cu0r + (int)((long long)(w + 1) * (cu1r - cu0r) / kDW);
                    const int u0 = a0 + c * kDChunkUnits, u1 = min(a1, u0 + kDChunkUnits);
                    // the chunk again (4 KB, from L2), all of it in flight at once
                    const uint4* row = reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(p.z) +
                                                                      (long long)b * p.row_stride);
                    // Lane l takes the units u0 + 8 l .. u0 + 8 l + 7, so that index order is lane order: one
                    // prefix over the lanes' sums places the crossing in a lane, which walks its 64 tokens.
                    uint4 Wq[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const int u = u0 + lane * 8 + i;
                        Wq[i] = u < u1 ? __ldg(row + u) : make_uint4(0xF149F149u, 0xF149F149u, 0xF149F149u, 0xF149F149u);
                        if (WARPED) bcut8(Wq[i], cut2);
                    }
                    float wt[8][8];
                    float ls = 0.f;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const uint32_t qw[4] = {Wq[i].x, Wq[i].y, Wq[i].z, Wq[i].w};
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const float2 z = unpack2(bclamp2(qw[j]));
                            wt[i][2 * j] = ex2(fmaf(z.x, c1, -Mr));
                            wt[i][2 * j + 1] = ex2(fmaf(z.y, c1, -Mr));
                            ls += wt[i][2 * j] + wt[i][2 * j + 1];
                        }
                    }
                    float li = ls;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const float t = __shfl_up_sync(0xFFFFFFFFu, li, o);
                        if (lane >= o) li += t;
                    }
                    float cc = base + (li - ls);
                    int hit = -1, last_pos = -1;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            cc += wt[i][j];
                            if (wt[i][j] > 0.f) {
                                const int idx = (u0 + lane * 8 + i) * 8 + j;
                                last_pos = idx;
                                if (hit < 0 && cc > target) hit = idx;
                            }
                        }
                    }
                    const unsigned mh = __ballot_sync(0xFFFFFFFFu, hit >= 0);
                    if (mh) tok = __shfl_sync(0xFFFFFFFFu, hit, __ffs(mh) - 1);
                    if (tok < 0) {
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) last_pos = max(last_pos, __shfl_xor_sync(0xFFFFFFFFu, last_pos, o));
                        tok = last_pos;
                    }
                }
            }
        }
        if (lane == 0) {
            if (rowbad) atomicOr(p.st.status, ADASD_STATUS_NAN);
            p.H_out[b] = H;
            if (p.lse_out) p.lse_out[b] = lse;
            if (sampling) p.token_out[b] = tok;
            const bool stop = H > tg_row;   // strict; NaN never stops
            if (p.stop_out) p.stop_out[b] = stop ? 1 : 0;
            if (p.draft_len) p.draft_len[b] = len_row + 1;
            if (p.active && stop) p.active[b] = 0;
        }
    }
}

}  // namespace adasd
