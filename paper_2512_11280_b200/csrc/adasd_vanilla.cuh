// Vanilla speculative sampling in two light steps (bf16 rows of a multiple of 8 logits).
//
// The accept test of a candidate needs only two numbers of its two rows, the log-sum-exps:
// alpha = min(1, exp((z_t[x] - lse_t) - (z_d[x] - lse_d))).  Only ONE position of a sequence
// needs more than that: the first rejected one (its residual max(0, p - q) is sampled) or, if
// none is rejected, the bonus row.  So:
//
//  1. row_lse_kernel streams every row of the round once (one `ex2` per logit, no second pass,
//     nothing kept) and leaves lse_t, lse_d;
//  2. vanilla_accept_kernel (one warp per sequence) forms the alphas, finds the first rejection
//     and names the one position that still needs work;
//  3. the warp-specialised verification kernel runs in vanilla mode over just those positions
//     (it reads their row pairs a second time: B row pairs out of B (2K + 1) rows).
#pragma once

#include "adasd_cluster.cuh"

namespace adasd {

constexpr int kLW = 8;                         // warps per CTA of row_lse_kernel
constexpr int kLChunkUnits = 256;              // 16-byte units per chunk: 8 iterations of a warp
constexpr int kLChunkBytes = kLChunkUnits * 16;

struct LseParams {
    const void* zd;
    const void* zt;
    long long d_seq, d_row, t_seq, t_row;
    const int32_t* draft_len;                  // nullable: Kmax
    float* lse_d;                              // [B, Kmax]
    float* lse_t;                              // [B, Kmax + 1]
    uint32_t* status;
    int32_t B, V, Kmax;
};

struct __align__(16) LseShared {
    float2 wpart[2][kLW];                      // (M, S) of every warp, by row parity
    uint32_t wbad[2][kLW];
    unsigned long long bar[kLW][2];
};

// Every needed row of the round (target rows 0..K_t, draft rows 0..K_t-1 of every sequence),
// one CTA per row at a time, rows dealt round robin to the CTAs of a grid that fills the SMs
// twice.  The 8 warps of a CTA split the row into contiguous shares and stream them through
// two 4 KB buffers each (1-D bulk copies, bounded waits); a warp's copies run on into its share
// of the CTA's next row, so the pipeline never drains between rows.
__global__ void __launch_bounds__(kLW * 32, 2) row_lse_kernel(LseParams p) {
    extern __shared__ __align__(128) unsigned char dyn_smem[];
    __shared__ LseShared sh;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int K = p.Kmax, R = 2 * K + 1;
    const int total = p.B * R;

    // this warp's share of any row, in 16-byte units
    const int NU = p.V >> 3;
    const int wu0 = (int)((long long)warp * NU / kLW), wu1 = (int)((long long)(warp + 1) * NU / kLW);
    const int nwu = wu1 - wu0;
    const int nch = (nwu + kLChunkUnits - 1) / kLChunkUnits;
    unsigned char* const bufs = dyn_smem + (size_t)warp * (2 * kLChunkBytes);

    if (lane == 0) {
        mbar_init(reinterpret_cast<uint64_t*>(&sh.bar[warp][0]), 1);
        mbar_init(reinterpret_cast<uint64_t*>(&sh.bar[warp][1]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();

    auto needed = [&](int r) -> bool {
        const int b = r / R, j = r - b * R;
        int kt = p.draft_len ? __ldg(p.draft_len + b) : K;
        kt = max(0, min(kt, K));
        return j <= K ? (j <= kt) : (j - K - 1 < kt);
    };
    auto next_row = [&](int r) -> int {          // first needed row among r, r + grid, ...
        while (r < total && !needed(r)) r += (int)gridDim.x;
        return min(r, total);
    };
    auto row_ptr = [&](int r) -> const unsigned char* {
        const int b = r / R, j = r - b * R;
        const __nv_bfloat16* base =
            j <= K ? reinterpret_cast<const __nv_bfloat16*>(p.zt) + (long long)b * p.t_seq + (long long)j * p.t_row
                   : reinterpret_cast<const __nv_bfloat16*>(p.zd) + (long long)b * p.d_seq + (long long)(j - K - 1) * p.d_row;
        return reinterpret_cast<const unsigned char*>(base) + (size_t)wu0 * 16;
    };

    bool alive = true;
    uint32_t n_issued = 0;                        // chunks this warp has asked for so far
    int ir = next_row((int)blockIdx.x), ic = 0;   // the next chunk to ask for: row, chunk
    auto issue_next = [&]() {
        if (!alive || ir >= total) return;
        if (lane == 0) {
            const uint32_t bytes = (uint32_t)min(kLChunkUnits, nwu - ic * kLChunkUnits) * 16u;
            uint64_t* bar = reinterpret_cast<uint64_t*>(&sh.bar[warp][n_issued & 1]);
            mbar_expect_tx(bar, bytes);
            bulk_g2s(bufs + (size_t)(n_issued & 1) * kLChunkBytes, row_ptr(ir) + (size_t)ic * kLChunkBytes, bytes, bar);
        }
        ++n_issued;
        if (++ic == nch) {
            ic = 0;
            ir = next_row(ir + (int)gridDim.x);
        }
    };
    issue_next();
    issue_next();

    uint32_t n_done = 0;                          // chunks consumed
    int rows_done = 0;
    for (int r = next_row((int)blockIdx.x); r < total; r = next_row(r + (int)gridDim.x)) {
        float M = kFloorL, vM = 0.f;              // running shift (log2 domain) and the logit it belongs to
        float2 S2 = make_float2(0.f, 0.f);
        uint32_t bad = 0u;
        for (int c = 0; c < nch; ++c) {
            bool ok = alive && mbar_wait_bounded(reinterpret_cast<uint64_t*>(&sh.bar[warp][n_done & 1]), (n_done >> 1) & 1u);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) {
                if (alive && lane == 0) atomicOr(p.status, ADASD_STATUS_TIMEOUT);
                alive = false;
                bad = 1u;
                break;
            }
            const unsigned char* sb = bufs + (size_t)(n_done & 1) * kLChunkBytes + (size_t)lane * 16;
            ++n_done;
            const int ubase = c * kLChunkUnits + lane;
            uint4 W[8];
            uint32_t mx = 0xFF80FF80u;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                W[i] = *reinterpret_cast<const uint4*>(sb + i * 512);
                if (!(ubase + 32 * i < nwu)) W[i] = make_uint4(0xF149F149u, 0xF149F149u, 0xF149F149u, 0xF149F149u);
                mx = bmax2(bmax2(mx, W[i].x), bmax2(W[i].y, bmax2(W[i].z, W[i].w)));
            }
            __syncwarp();
            issue_next();                         // the chunk is in registers, its buffer free
            const float2 mm = unpack2(mx);
            if (mm.x != mm.x || mm.y != mm.y) bad = 1u;
            const float vmax = warp_max_f32(fmaxf(mm.x, mm.y));
            if (vmax == INFINITY) bad = 1u;
            const float Mc = vmax > ADASD_FLOOR_BF ? vmax * kLog2e : kFloorL;
            if (Mc > M) {                         // raise the shift, rescale what is summed
                const float f = ex2(M > kFloorL ? (vM - vmax) * kLog2e : kFloorL);
                S2.x *= f;
                S2.y *= f;
                M = Mc;
                vM = vmax;
            }
            const float2 nv2 = make_float2(-vM, -vM), L2 = make_float2(kLog2e, kLog2e);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const uint32_t w[4] = {W[i].x, W[i].y, W[i].z, W[i].w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float2 z = unpack2(bclamp2(w[j]));
                    const float2 t = __fmul2_rn(__fadd2_rn(z, nv2), L2);
                    S2 = __fadd2_rn(S2, make_float2(ex2(t.x), ex2(t.y)));
                }
            }
        }
        const float Sw = warp_sum(S2.x + S2.y);
        bad = __reduce_or_sync(0xFFFFFFFFu, bad);
        const int par = rows_done & 1;
        if (lane == 0) {
            sh.wpart[par][warp] = make_float2(M, Sw);
            sh.wbad[par][warp] = bad;
        }
        __syncthreads();                          // every warp has put its share of row r down
        if (warp == 0) {
            const float2 e = lane < kLW ? sh.wpart[par][lane] : make_float2(kFloorL, 0.f);
            const uint32_t fl = __reduce_or_sync(0xFFFFFFFFu, lane < kLW ? sh.wbad[par][lane] : 0u);
            const float Mr = warp_max_f32(e.x);
            const float S = warp_sum(ex2(e.x - Mr) * e.y);
            if (lane == 0) {
                const bool rowbad = (fl & 1u) || !(Mr > kFloorL);
                const float lse = rowbad ? NAN : kLn2 * (Mr + lg2(S));
                const int b = r / R, j = r - b * R;
                if (j <= K) p.lse_t[(size_t)b * (K + 1) + j] = lse;
                else p.lse_d[(size_t)b * K + (j - K - 1)] = lse;
            }
        }
        ++rows_done;
    }
    // a warp that gave up on a copy still waits (bounded) for whatever it had in flight
    if (!alive) {
        for (uint32_t q = n_done; q < n_issued; ++q)
            mbar_wait_bounded(reinterpret_cast<uint64_t*>(&sh.bar[warp][q & 1]), (q >> 1) & 1u);
    }
}

// One warp per sequence, lane i on candidate i: alpha_i = min(1, p_i(x_i) / q_i(x_i)) from the
// log-sum-exps, the accept flags, the accepted length, and the one position whose rows the
// sampling kernel still has to read (the first rejected one, or the bonus row).  A row with NaN
// or no finite logit has lse = NaN: it counts as rejected and raises the status flag.
__global__ void vanilla_accept_kernel(VerifyParams p, int32_t* only_pos) {
    const int b = (int)((blockIdx.x * blockDim.x + threadIdx.x) >> 5), i = threadIdx.x & 31;
    if (b >= p.B) return;
    const int K = p.Kmax;
    int kt = p.draft_len ? p.draft_len[b] : K;
    kt = max(0, min(kt, K));
    bool reject = false, bad = false;
    if (i < kt) {
        const size_t idd = (size_t)b * K + i;
        const float lt = p.sc.lse_t[(size_t)b * (K + 1) + i], ld = p.sc.lse_d[idd];
        bad = (lt != lt) || (ld != ld);
        const int xi = p.x[idd];
        float alpha = 0.f;
        if (xi >= 0 && xi < p.V) {
            // ln p(x) and ln q(x), -inf logits clamped; their difference is formed before any
            // scaling so that identical rows give exactly 0, alpha exactly 1
            const __nv_bfloat16* zt = reinterpret_cast<const __nv_bfloat16*>(p.zt) + (long long)b * p.t_seq;
            const __nv_bfloat16* zd = reinterpret_cast<const __nv_bfloat16*>(p.zd) + (long long)b * p.d_seq;
            const float lp = fmaxf(__bfloat162float(zt[(long long)i * p.t_row + xi]), ADASD_FLOOR_BF) - lt;
            const float lq = fmaxf(__bfloat162float(zd[(long long)i * p.d_row + xi]), ADASD_FLOOR_BF) - ld;
            alpha = fminf(1.f, ex2(__fmul_rn(__fsub_rn(lp, lq), kLog2e)));
            if (!(ex2(__fmul_rn(lq, kLog2e)) > 0.f)) alpha = 1.f;       // q(x) = 0 cannot have been drafted
        }
        const bool accept = !bad && (p.u_accept[idd] < alpha);
        reject = !accept;
        p.sc.van_flag[idd] = accept ? 1 : 0;
        if (p.alpha_out) p.alpha_out[idd] = bad ? NAN : alpha;
    } else if (i == kt) {
        const float lb = p.sc.lse_t[(size_t)b * (K + 1) + kt];     // the bonus row
        bad = (lb != lb);
    }
    const unsigned mr = __ballot_sync(0xFFFFFFFFu, reject);
    const unsigned mb = __ballot_sync(0xFFFFFFFFu, bad);
    if (i == 0) {
        // Kmax = 32 leaves no lane for the bonus row: look at it here
        if (kt == 32) {
            const float lb = p.sc.lse_t[(size_t)b * (K + 1) + kt];
            if (lb != lb) atomicOr(p.st.status, ADASD_STATUS_NAN);
        }
        if (mb) atomicOr(p.st.status, ADASD_STATUS_NAN);
        const int w = mr ? (__ffs(mr) - 1) : kt;
        p.accept_len[b] = w;
        only_pos[b] = w;
    }
}

}  // namespace adasd
