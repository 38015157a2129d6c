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
//  3. vanilla_sample_kernel (one CTA per sequence) streams the row pair of that one position:
//     with the log-sum-exps known, p and q are final as they are read, so per-chunk sums of the
//     residual max(0, p - q) locate the chunk of the inverse-CDF crossing, which is scanned again
//     (B row pairs are read a second time, out of B (2K + 1) rows).
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
    float c1;                                  // log2 e / temperature (adjusted distribution)
    const float* cut_t;                        // nullable [B, Kmax + 1]: logit below which a row's tokens are cut
    const float* cut_d;                        // nullable [B, Kmax]
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
template <bool WARPED>
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
    const float c1 = WARPED ? p.c1 : kLog2e;
    for (int r = next_row((int)blockIdx.x); r < total; r = next_row(r + (int)gridDim.x)) {
        uint32_t cut2 = kNoCut2;
        if (WARPED && p.cut_t) {
            const int b = r / R, j = r - b * R;
            cut2 = cut_pair(j <= K ? __ldg(p.cut_t + (size_t)b * (K + 1) + j) : __ldg(p.cut_d + (size_t)b * K + (j - K - 1)));
        }
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
            if (WARPED && cut2 != kNoCut2) {
#pragma unroll
                for (int i = 0; i < 8; ++i) bcut8(W[i], cut2);
            }
            const float2 mm = unpack2(mx);
            if (mm.x != mm.x || mm.y != mm.y) bad = 1u;
            const float vmax = warp_max_f32(fmaxf(mm.x, mm.y));
            if (vmax == INFINITY) bad = 1u;
            const float Mc = vmax > ADASD_FLOOR_BF ? vmax * c1 : kFloorL;
            if (Mc > M) {                         // raise the shift, rescale what is summed
                const float f = ex2(M > kFloorL ? (vM - vmax) * c1 : kFloorL);
                S2.x *= f;
                S2.y *= f;
                M = Mc;
                vM = vmax;
            }
            const float2 nv2 = make_float2(-vM, -vM), L2 = make_float2(c1, c1);
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
            // (logits of the adjusted distribution: scaled by 1 / T, -inf below the row's cutoff)
            const RowWarp wt = {p.inv_temp, p.cut_t ? p.cut_t[(size_t)b * (K + 1) + i] : -INFINITY};
            const RowWarp wd = {p.inv_temp, p.cut_d ? p.cut_d[idd] : -INFINITY};
            const float lp = fmaxf(apply_warp(__bfloat162float(zt[(long long)i * p.t_row + xi]), wt), ADASD_FLOOR_BF) - lt;
            const float lq = fmaxf(apply_warp(__bfloat162float(zd[(long long)i * p.d_row + xi]), wd), ADASD_FLOOR_BF) - ld;
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

namespace adasd {

// ---- step 3 for large batches: the one sampled position of every sequence ------------------
//
// With the log-sum-exps known, p = 2^((z_t - lse_t) log2 e) and q likewise are final as they
// are read: one CTA per sequence streams the row pair once, keeps per-chunk sums of the
// residual max(0, p - q) (and of p, for the bonus row and for a residual without mass), finds
// the chunk that holds the inverse-CDF crossing of u and scans just that chunk again.
constexpr int kVW = 16;                        // warps per CTA
constexpr int kVChunkUnits = 128;              // 16-byte units per chunk of one row: 4 iterations of a warp
constexpr int kVChunkBytes = kVChunkUnits * 16;
constexpr int kVMaxChunks = 16;                // chunks per warp, at most

struct __align__(16) SampleShared {
    float cr[kVW][kVMaxChunks];                // residual mass of every chunk
    float cp[kVW][kVMaxChunks];                // target mass of every chunk
    unsigned long long bar[kVW][2];
};

// largest V the chunk tables hold
constexpr int kVMaxV = kVW * kVMaxChunks * kVChunkUnits * 8;

__global__ void __launch_bounds__(kVW * 32, 1) vanilla_sample_kernel(VerifyParams p, const int32_t* only_pos) {
    extern __shared__ __align__(128) unsigned char dyn_smem[];
    __shared__ SampleShared sh;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int b = blockIdx.x;
    const int K = p.Kmax, K1 = K + 1;
    int kt = p.draft_len ? __ldg(p.draft_len + b) : K;
    kt = max(0, min(kt, K));
    const int i = __ldg(only_pos + b);
    const bool bonus = (i >= kt);
    const float lt = p.sc.lse_t[(size_t)b * K1 + i];
    const float ld = bonus ? 0.f : p.sc.lse_d[(size_t)b * K + i];
    const bool rowbad = (lt != lt) || (ld != ld);

    const int NU = p.V >> 3;
    const int wu0 = (int)((long long)warp * NU / kVW), wu1 = (int)((long long)(warp + 1) * NU / kVW);
    const int nwu = wu1 - wu0;
    const int nch = min(kVMaxChunks, (nwu + kVChunkUnits - 1) / kVChunkUnits);
    const unsigned char* const src_t = reinterpret_cast<const unsigned char*>(
        reinterpret_cast<const __nv_bfloat16*>(p.zt) + (long long)b * p.t_seq + (long long)i * p.t_row) + (size_t)wu0 * 16;
    const unsigned char* const src_d = reinterpret_cast<const unsigned char*>(
        reinterpret_cast<const __nv_bfloat16*>(p.zd) + (long long)b * p.d_seq + (long long)min(i, K - 1) * p.d_row) + (size_t)wu0 * 16;
    unsigned char* const bufs = dyn_smem + (size_t)warp * (4 * kVChunkBytes);   // [buffer][target | draft]

    if (lane == 0) {
        mbar_init(reinterpret_cast<uint64_t*>(&sh.bar[warp][0]), 1);
        mbar_init(reinterpret_cast<uint64_t*>(&sh.bar[warp][1]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (lane < kVMaxChunks) {
        sh.cr[warp][lane] = 0.f;
        sh.cp[warp][lane] = 0.f;
    }
    __syncwarp();

    // weights of one 16-byte unit of both rows: p and max(0, p - q)
    // (adjusted distribution: logits scaled by 1 / T, those below the row's cutoff cut)
    const float nlt = -lt * kLog2e, nld = -ld * kLog2e, c1 = p.c1;
    const uint32_t cut2t = p.cut_t ? cut_pair(__ldg(p.cut_t + (size_t)b * K1 + i)) : kNoCut2;
    const uint32_t cut2d = (p.cut_d && !bonus) ? cut_pair(__ldg(p.cut_d + (size_t)b * K + i)) : kNoCut2;
    auto weights = [&](const uint4& Tin, const uint4& Din, float (&pv)[8], float (&rv)[8]) {
        uint4 T = Tin, D = Din;
        bcut8(T, cut2t);
        bcut8(D, cut2d);
        const uint32_t tw[4] = {T.x, T.y, T.z, T.w}, dw[4] = {D.x, D.y, D.z, D.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float2 zt2 = unpack2(bclamp2(tw[j])), zd2 = unpack2(bclamp2(dw[j]));
            pv[2 * j] = ex2(fmaf(zt2.x, c1, nlt));
            pv[2 * j + 1] = ex2(fmaf(zt2.y, c1, nlt));
            const float q0 = bonus ? 0.f : ex2(fmaf(zd2.x, c1, nld));
            const float q1 = bonus ? 0.f : ex2(fmaf(zd2.y, c1, nld));
            rv[2 * j] = fmaxf(pv[2 * j] - q0, 0.f);
            rv[2 * j + 1] = fmaxf(pv[2 * j + 1] - q1, 0.f);
        }
    };

    bool alive = !rowbad;                         // an unusable row is neither copied nor sampled
    auto issue = [&](int c) {
        if (alive && lane == 0 && c < nch) {
            const uint32_t bytes = (uint32_t)min(kVChunkUnits, nwu - c * kVChunkUnits) * 16u;
            uint64_t* bar = reinterpret_cast<uint64_t*>(&sh.bar[warp][c & 1]);
            unsigned char* dst = bufs + (size_t)(c & 1) * (2 * kVChunkBytes);
            mbar_expect_tx(bar, bonus ? bytes : 2u * bytes);
            bulk_g2s(dst, src_t + (size_t)c * kVChunkBytes, bytes, bar);
            if (!bonus) bulk_g2s(dst + kVChunkBytes, src_d + (size_t)c * kVChunkBytes, bytes, bar);
        }
    };
    issue(0);
    issue(1);
    const uint4 floor4 = make_uint4(0xF149F149u, 0xF149F149u, 0xF149F149u, 0xF149F149u);
    int cfail = -1;                               // chunk whose copy never landed
    for (int c = 0; c < nch && alive; ++c) {
        bool ok = mbar_wait_bounded(reinterpret_cast<uint64_t*>(&sh.bar[warp][c & 1]), (uint32_t)(c >> 1) & 1u);
        ok = __all_sync(0xFFFFFFFFu, ok);
        if (!ok) {
            if (lane == 0) atomicOr(p.st.status, ADASD_STATUS_TIMEOUT);
            alive = false;
            cfail = c;
            break;
        }
        const unsigned char* sb = bufs + (size_t)(c & 1) * (2 * kVChunkBytes) + (size_t)lane * 16;
        uint4 T[4], D[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const bool in = c * kVChunkUnits + lane + 32 * k < nwu;
            T[k] = in ? *reinterpret_cast<const uint4*>(sb + k * 512) : floor4;
            D[k] = (in && !bonus) ? *reinterpret_cast<const uint4*>(sb + kVChunkBytes + k * 512) : floor4;
        }
        __syncwarp();
        issue(c + 2);                             // the chunk is in registers, its buffer free
        float ps = 0.f, rs = 0.f;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            float pv[8], rv[8];
            weights(T[k], D[k], pv, rv);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                ps += pv[j];
                rs += rv[j];
            }
        }
        ps = warp_sum(ps);
        rs = warp_sum(rs);
        if (lane == 0) {
            sh.cp[warp][c] = ps;
            sh.cr[warp][c] = rs;
        }
    }
    // a warp that gave up on a copy still waits (bounded) for whatever it had in flight
    if (cfail >= 0) {
        for (int c = cfail; c < min(cfail + 2, nch); ++c)
            mbar_wait_bounded(reinterpret_cast<uint64_t*>(&sh.bar[warp][c & 1]), (uint32_t)(c >> 1) & 1u);
    }
    const int timed_out = __syncthreads_or(cfail >= 0);   // the chunk tables are complete
    if (warp != 0) return;

    // warp 0: which chunk holds the crossing (index order: warp, chunk), then that chunk again
    int tok = -1;
    if (!rowbad && !timed_out) {
        constexpr int E = kVW * kVMaxChunks;      // 256 table entries, 8 per lane in index order
        const float* crf = &sh.cr[0][0];
        const float* cpf = &sh.cp[0][0];
        float r8[8], p8[8], rl = 0.f, pl = 0.f;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            r8[j] = crf[lane * 8 + j];
            p8[j] = cpf[lane * 8 + j];
            rl += r8[j];
            pl += p8[j];
        }
        const float R = warp_sum(rl), P = warp_sum(pl);
        const bool use_r = !bonus && R > 0.f;     // a residual without mass: draw from p
        float w8[8], wl = use_r ? rl : pl;
#pragma unroll
        for (int j = 0; j < 8; ++j) w8[j] = use_r ? r8[j] : p8[j];
        float target = __ldg(p.u_resample + b) * (use_r ? R : P);
        float incl = wl;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const float t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= o) incl += t;
        }
        float run = incl - wl;
        int hit = -1, last = -1;
        float hbase = 0.f, lbase = 0.f;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            if (w8[j] > 0.f) {
                last = lane * 8 + j;
                lbase = run;
                if (hit < 0 && run + w8[j] > target) {
                    hit = lane * 8 + j;
                    hbase = run;
                }
            }
            run += w8[j];
        }
        const unsigned mh = __ballot_sync(0xFFFFFFFFu, hit >= 0), ml = __ballot_sync(0xFFFFFFFFu, last >= 0);
        int ent = -1;
        float base = 0.f;
        if (mh) {
            const int l = __ffs(mh) - 1;
            ent = __shfl_sync(0xFFFFFFFFu, hit, l);
            base = __shfl_sync(0xFFFFFFFFu, hbase, l);
        } else if (ml) {          // rounding left no crossing: last chunk with mass, last token with mass
            const int l = 31 - __clz(ml);
            ent = __shfl_sync(0xFFFFFFFFu, last, l);
            base = __shfl_sync(0xFFFFFFFFu, lbase, l);
            target = INFINITY;
        }
        if (ent >= 0) {
            const int w = ent / kVMaxChunks, c = ent % kVMaxChunks;
            const int a0 = (int)((long long)w * NU / kVW), a1 = (int)((long long)(w + 1) * NU / kVW);
            const int u0 = a0 + c * kVChunkUnits, u1 = min(a1, u0 + kVChunkUnits);
            const uint4* rowt = reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(p.zt) +
                                                               (long long)b * p.t_seq + (long long)i * p.t_row);
            const uint4* rowd = reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(p.zd) +
                                                               (long long)b * p.d_seq + (long long)min(i, K - 1) * p.d_row);
            uint4 Tq[4], Dq[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int u = u0 + 32 * k + lane;
                Tq[k] = u < u1 ? __ldg(rowt + u) : floor4;
                Dq[k] = (u < u1 && !bonus) ? __ldg(rowd + u) : floor4;
            }
            float runw = base;
            int last_pos = -1;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                if (tok < 0 && u0 + 32 * k < u1) {          // same for the whole warp
                    const int u = u0 + 32 * k + lane;
                    float pv[8], rv[8], wt[8];
                    weights(Tq[k], Dq[k], pv, rv);
                    float ls = 0.f;
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        wt[j] = use_r ? rv[j] : pv[j];
                        ls += wt[j];
                    }
                    float li = ls;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const float t = __shfl_up_sync(0xFFFFFFFFu, li, o);
                        if (lane >= o) li += t;
                    }
                    float cc = runw + (li - ls);
                    int h = -1;
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        cc += wt[j];
                        if (wt[j] > 0.f) {
                            last_pos = u * 8 + j;
                            if (h < 0 && cc > target) h = u * 8 + j;
                        }
                    }
                    const unsigned m2 = __ballot_sync(0xFFFFFFFFu, h >= 0);
                    if (m2) tok = __shfl_sync(0xFFFFFFFFu, h, __ffs(m2) - 1);
                    runw += __shfl_sync(0xFFFFFFFFu, li, 31);
                }
            }
            if (tok < 0) {
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) last_pos = max(last_pos, __shfl_xor_sync(0xFFFFFFFFu, last_pos, o));
                tok = last_pos;
            }
        }
    }
    if (lane == 0) {
        p.sc.van_tok[(size_t)b * K1 + i] = tok;
        p.next_token[b] = tok;
    }
}

}  // namespace adasd
