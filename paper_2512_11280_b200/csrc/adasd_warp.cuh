// The adjusted distribution of Sec. 2.1.1 (temperature scaling, top-k sampling, top-p sampling).
//
// Temperature is a scale of the logits and costs the row passes nothing: they multiply by
// log2 e / temperature where they multiplied by log2 e.  Top-k and top-p cut the vocabulary, and
// both cuts are "keep the tokens whose logit is at least c" for one value c per row:
//   top-k: c = the k-th largest logit (tokens equal to it stay with it);
//   top-p: c = the smallest logit v such that the tokens STRICTLY above v hold less than top_p
//          of the mass of what top-k left (the smallest most-probable set whose mass reaches
//          top_p, ties at its edge included).
// row_cutoff_kernel finds c for every needed row; the row passes then read a logit below its
// row's c as -inf (apply_warp below), so entropy, JS distance, the accept ratio and every sample
// are those of the adjusted distribution.
//
// The search is a radix descent over the order-preserving integer image of the logits (16 bits
// for bf16, 32 for fp32), 8 bits a level, most significant first: a level histograms the
// weight (1 per token for top-k; 2^((z - max) log2 e / T) for top-p) of the tokens that match
// the digits fixed so far, and the bin where the weight counted from the top first reaches the
// threshold fixes the next digit.  Masses are formed in double precision and added as 2^-40
// fixed-point integers, so the sums do not depend on the order the atomics land in, the result
// is the same on every run, and a token's side of the cut is decided to about 1e-9 of the mass.
#pragma once

#include "adasd_device.cuh"

namespace adasd {

// One row's adjustment as the row passes apply it.
struct RowWarp {
    float inv_t;    // 1 / temperature
    float cut;      // logits below it are cut (-inf: none)
};
// -inf for a cut token, z / temperature for the others; NaN stays NaN (the row is unusable);
// {1, -inf} changes nothing, bit for bit.
__device__ __forceinline__ float apply_warp(float z, const RowWarp& w) {
    return (z < w.cut) ? -INFINITY : z * w.inv_t;
}
template <int N>
__device__ __forceinline__ void apply_warp(float (&x)[N], const RowWarp& w) {
#pragma unroll
    for (int j = 0; j < N; ++j) x[j] = apply_warp(x[j], w);
}

// load_unit with the row's adjustment applied
template <typename T, bool VEC>
__device__ __forceinline__ void load_unit_w(const T* __restrict__ row, int u, int V, float (&x)[Elt<T>::N],
                                            const RowWarp& w) {
    load_unit<T, VEC>(row, u, V, x);
    apply_warp(x, w);
}

struct CutParams {
    const void* z;
    long long seq_stride, row_stride;   // in elements
    const int32_t* draft_len;           // nullable: window K_b of sequence b (clamped to [0, R - extra])
    const uint8_t* active;              // nullable: sequences with 0 are skipped
    float* cut;                         // [B, R]
    uint32_t* status;
    int32_t B, R, V;
    int32_t extra;                      // 1: rows 0 .. K_b are needed (target rows, with the bonus row); 0: rows 0 .. K_b - 1
    double c1;                          // log2 e / temperature
    int32_t top_k;                      // <= 0 or >= V: off
    float top_p;                        // >= 1: off
    int32_t only_flagged;               // 1: only the rows whose cut entry is NaN (left over by row_cutoff_hist_kernel)
};

constexpr int kCutThreads = 512;
constexpr int kCutWarps = kCutThreads / 32;
constexpr double kCutFix = 1099511627776.0;   // 2^40

template <typename T>
struct CutKey;
template <>
struct CutKey<__nv_bfloat16> {
    static constexpr int BITS = 16;
    __device__ static uint32_t of(float x) {
        uint32_t u = __float_as_uint(x) >> 16;
        if ((u & 0x7FFFu) == 0) u = 0;                       // -0 and +0 are one value
        return (u & 0x8000u) ? (~u & 0xFFFFu) : (u | 0x8000u);
    }
    __device__ static float value(uint32_t k) {
        const uint32_t u = (k & 0x8000u) ? (k & 0x7FFFu) : (~k & 0xFFFFu);
        return __uint_as_float(u << 16);
    }
};
template <>
struct CutKey<float> {
    static constexpr int BITS = 32;
    __device__ static uint32_t of(float x) {
        uint32_t u = __float_as_uint(x);
        if ((u & 0x7FFFFFFFu) == 0) u = 0;
        return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
    }
    __device__ static float value(uint32_t k) {
        return __uint_as_float((k & 0x80000000u) ? (k & 0x7FFFFFFFu) : ~k);
    }
};

struct CutShared {
    unsigned long long bins[kCutWarps][256];
    unsigned long long tot[256];
    float red[kCutWarps];
    int flag[kCutWarps];
    unsigned long long acc;       // weight above the digits fixed so far
    unsigned long long S;         // top-p: the mass of everything top-k left
    uint32_t prefix;
    int32_t found;
    float m;
    int32_t bad;
};

// One CTA per row at a time; rows are dealt round robin to a grid that fills the SMs.  The first
// pass reads the row from HBM, the later ones find it in L2.
template <typename T, bool VEC>
__global__ void __launch_bounds__(kCutThreads) row_cutoff_kernel(CutParams p) {
    constexpr int N = Elt<T>::N;
    constexpr int BITS = CutKey<T>::BITS;
    __shared__ CutShared sh;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int NU = (p.V + N - 1) / N;
    const int total = p.B * p.R;
    const bool use_k = p.top_k > 0 && p.top_k < p.V;
    const bool use_p = p.top_p < 1.f;

    for (int row = blockIdx.x; row < total; row += gridDim.x) {
        const int b = row / p.R, j = row - b * p.R;
        if (p.active && p.active[b] == 0) continue;
        if (p.draft_len) {
            const int kt = max(0, min(p.draft_len[b], p.R - p.extra));
            if (j >= kt + p.extra) continue;
        }
        if (p.only_flagged) {
            const float c = p.cut[(size_t)b * p.R + j];
            if (c == c) continue;                            // (the same for every thread of the CTA)
        }
        const T* z = reinterpret_cast<const T*>(p.z) + (long long)b * p.seq_stride + (long long)j * p.row_stride;

        // largest logit and usability of the row
        float mx = -INFINITY;
        int bad = 0;
        for (int u = threadIdx.x; u < NU; u += kCutThreads) {
            float x[N];
            load_unit<T, VEC>(z, u, p.V, x);
#pragma unroll
            for (int q = 0; q < N; ++q) {
                bad |= (x[q] != x[q]);
                mx = fmaxf(mx, x[q]);
            }
        }
        mx = warp_max(mx);
        bad = __any_sync(0xFFFFFFFFu, bad);
        if (lane == 0) {
            sh.red[warp] = mx;
            sh.flag[warp] = bad;
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            float m = sh.red[0];
            int bd = sh.flag[0];
            for (int w = 1; w < kCutWarps; ++w) {
                m = fmaxf(m, sh.red[w]);
                bd |= sh.flag[w];
            }
            sh.m = m;
            sh.bad = bd || !(m > -INFINITY) || m == INFINITY;
        }
        __syncthreads();
        const float m = sh.m;
        if (sh.bad) {                       // an unusable row is not cut; the row pass reports it
            if (threadIdx.x == 0) p.cut[(size_t)b * p.R + j] = -INFINITY;
            __syncthreads();
            continue;
        }

        uint32_t lo_key = 0;                // tokens with a key below it are cut already
        for (int which = 0; which < 2; ++which) {
            const bool mass = (which == 1);
            if (mass ? !use_p : !use_k) continue;
            if (threadIdx.x == 0) {
                sh.acc = 0ull;
                sh.prefix = 0u;
                sh.found = 1;
            }
            __syncthreads();
            for (int shift = BITS - 8; shift >= 0; shift -= 8) {
                for (int i = threadIdx.x; i < kCutWarps * 256; i += kCutThreads) (&sh.bins[0][0])[i] = 0ull;
                __syncthreads();
                const uint32_t prefix = sh.prefix;
                const bool top_level = (shift == BITS - 8);
                for (int u = threadIdx.x; u < NU; u += kCutThreads) {
                    float x[N];
                    load_unit<T, VEC>(z, u, p.V, x);
#pragma unroll
                    for (int q = 0; q < N; ++q) {
                        if (u * N + q >= p.V) continue;
                        const uint32_t key = CutKey<T>::of(x[q]);
                        if (key < lo_key) continue;
                        if (!top_level && (key >> (shift + 8)) != prefix) continue;
                        unsigned long long w = 1ull;
                        if (mass) w = (unsigned long long)__double2ll_rn(exp2((double)(fmaxf(x[q], kFloor) - m) * p.c1) * kCutFix);
                        if (w) atomicAdd(&sh.bins[warp][(key >> shift) & 255u], w);
                    }
                }
                __syncthreads();
                if (threadIdx.x < 256) {
                    unsigned long long t = 0ull;
                    for (int w = 0; w < kCutWarps; ++w) t += sh.bins[w][threadIdx.x];
                    sh.tot[threadIdx.x] = t;
                }
                __syncthreads();
                if (threadIdx.x == 0 && sh.found) {
                    // threshold: k tokens, or top_p of the mass top-k left (the whole of it is in
                    // the top level's bins)
                    double thr;
                    if (!mass) {
                        thr = (double)p.top_k;
                    } else {
                        if (top_level) {
                            unsigned long long S = 0ull;
                            for (int d = 0; d < 256; ++d) S += sh.tot[d];
                            sh.S = S;
                        }
                        thr = (double)p.top_p * (double)sh.S;
                    }
                    unsigned long long acc = sh.acc;
                    int hit = -1;
                    for (int d = 255; d >= 0; --d) {
                        const unsigned long long w = sh.tot[d];
                        if (w == 0ull) continue;
                        if ((double)(acc + w) >= thr) {
                            hit = d;
                            break;
                        }
                        acc += w;
                    }
                    if (hit < 0) {
                        sh.found = 0;                   // the threshold is never reached: nothing is cut
                    } else {
                        sh.acc = acc;
                        sh.prefix = (prefix << 8) | (uint32_t)hit;
                    }
                }
                __syncthreads();
                if (!sh.found) break;
            }
            __syncthreads();
            if (sh.found) lo_key = max(lo_key, sh.prefix);
            __syncthreads();
        }
        if (threadIdx.x == 0) p.cut[(size_t)b * p.R + j] = lo_key ? CutKey<T>::value(lo_key) : -INFINITY;
        __syncthreads();
    }
}

// ---- bf16 rows that take 16-byte loads: one pass ---------------------------------------------
//
// A bf16 logit has 65536 possible values, so ONE pass over the row can count how often each
// occurs (a histogram in shared memory, two 16-bit counters to a word), and everything else
// follows from the counts: the k-th largest value, and - because all tokens of a bin have the same
// logit - the mass of a bin as count * 2^((value - max) log2 e / T).  A descending scan of the bins
// (64 per thread, then a prefix over the threads, in double precision and a fixed order) finds
// where the count reaches k and where the mass reaches top_p of what top-k left.
// A value that occurs 65536 times or more in one row wraps its counter; the total then no longer
// equals V, the row's entry is left NaN, and row_cutoff_kernel (only_flagged) does that row.
// The pass works on the packed bf16 pairs as they are loaded (the order-preserving key of a value
// is three integer operations on its 16 bits): the integer pipe is what bounds it.
constexpr int kHistThreads = 1024;
constexpr int kHistWarps = kHistThreads / 32;
constexpr int kHistWords = 32768;                  // 65536 counters of 16 bits
constexpr int kHistPerThread = 65536 / kHistThreads;
static_assert(kHistPerThread == 64, "a thread's keys share bits 6..15");

// Order-preserving key of a bf16 bit pattern (-0 and +0 get neighbouring keys; a cut between them
// keeps both, because the row passes compare values).
__device__ __forceinline__ uint32_t hist_key(uint32_t h) { return h ^ (((h >> 15) * 0x7FFFu) + 0x8000u); }
// Word of the histogram that holds a key's counter.  Two keys 32768 apart share a word (neighbouring
// values, which are busy together, do not); the low five bits are mixed with bits 6..10 so that the
// scan, in which the threads of a warp read keys 64 apart, finds them in 32 different banks.
__device__ __forceinline__ uint32_t hist_slot(uint32_t key) { return (key & 0x7FFFu) ^ ((key >> 6) & 31u); }
__device__ __forceinline__ void hist_add(uint32_t* hist, uint32_t h) {
    const uint32_t key = hist_key(h);
    atomicAdd(&hist[hist_slot(key)], 1u + (key >> 15) * 0xFFFFu);      // low or high half of the word
}
__device__ __forceinline__ uint32_t cut_bmax2(uint32_t a, uint32_t b) {   // NaN-propagating bf16x2 max
    uint32_t d;
    asm("max.NaN.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}

struct HistShared {
    float red[kHistWarps];
    int flag[kHistWarps];
    long long wcnt[kHistWarps];
    double wmass[kHistWarps];
    long long incl_c[kHistThreads];    // inclusive prefix of the counts over the threads (descending keys)
    double incl_m[kHistThreads];       // ... of the masses
    float m;
    int32_t bad;
    int32_t owner;                     // first thread whose inclusive prefix reaches the threshold
    uint32_t key_k, key_p;
};

__global__ void __launch_bounds__(kHistThreads, 1) row_cutoff_hist_kernel(CutParams p) {
    using KeyT = CutKey<__nv_bfloat16>;
    extern __shared__ __align__(16) uint32_t hist[];
    __shared__ HistShared sh;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, tid = threadIdx.x;
    const int NUF = p.V >> 3;                  // full 16-byte units of a row
    const int total = p.B * p.R;
    const bool use_k = p.top_k > 0 && p.top_k < p.V;
    const bool use_p = p.top_p < 1.f;

    for (int row = blockIdx.x; row < total; row += gridDim.x) {
        const int b = row / p.R, j = row - b * p.R;
        if (p.active && p.active[b] == 0) continue;
        if (p.draft_len) {
            const int kt = max(0, min(p.draft_len[b], p.R - p.extra));
            if (j >= kt + p.extra) continue;
        }
        float* const out = p.cut + (size_t)b * p.R + j;
        const __nv_bfloat16* z =
            reinterpret_cast<const __nv_bfloat16*>(p.z) + (long long)b * p.seq_stride + (long long)j * p.row_stride;

        for (int i = tid; i < kHistWords / 4; i += kHistThreads)
            reinterpret_cast<uint4*>(hist)[i] = make_uint4(0u, 0u, 0u, 0u);
        __syncthreads();

        // the pass over the row: counts, largest logit, usability.  Four units of a thread are asked
        // for before the first is used: a CTA alone on its SM has to keep enough loads in flight.
        uint32_t mxp = 0xFF80FF80u;            // (-inf, -inf)
        {
            const uint4* zq = reinterpret_cast<const uint4*>(z);
            for (int u0 = tid; u0 < NUF; u0 += 4 * kHistThreads) {
                uint4 r[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) r[i] = __ldg(zq + min(u0 + i * kHistThreads, NUF - 1));
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    if (u0 + i * kHistThreads < NUF) {
                        const uint32_t w[4] = {r[i].x, r[i].y, r[i].z, r[i].w};
                        mxp = cut_bmax2(cut_bmax2(mxp, cut_bmax2(w[0], w[1])), cut_bmax2(w[2], w[3]));
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            hist_add(hist, w[q] & 0xFFFFu);
                            hist_add(hist, w[q] >> 16);
                        }
                    }
                }
            }
            if (tid == 0)                       // the ragged end of a row whose length is no multiple of 8
                for (int v = NUF * 8; v < p.V; ++v) {
                    const uint32_t h = (uint32_t)__bfloat16_as_ushort(z[v]);
                    mxp = cut_bmax2(mxp, h | (h << 16));
                    hist_add(hist, h);
                }
        }
        const float m0 = __uint_as_float(mxp << 16), m1 = __uint_as_float(mxp & 0xFFFF0000u);
        int bad = (m0 != m0) || (m1 != m1);
        float mx = warp_max(fmaxf(m0, m1));
        bad = __any_sync(0xFFFFFFFFu, bad);
        if (lane == 0) {
            sh.red[warp] = mx;
            sh.flag[warp] = bad;
        }
        __syncthreads();
        if (tid == 0) {
            float m = sh.red[0];
            int bd = sh.flag[0];
            for (int w = 1; w < kHistWarps; ++w) {
                m = fmaxf(m, sh.red[w]);
                bd |= sh.flag[w];
            }
            sh.m = m;
            sh.bad = bd || !(m > -INFINITY) || m == INFINITY;
            sh.key_k = 0u;
            sh.key_p = 0u;
        }
        __syncthreads();
        const float m = sh.m;
        if (sh.bad) {                       // an unusable row is not cut; the row pass reports it
            if (tid == 0) *out = -INFINITY;
            __syncthreads();
            continue;
        }

        // Thread t owns the keys hi, hi - 1, ..., hi - 63 with hi = 65535 - 64 t: in thread order the
        // bins run from the largest logit down.  Its keys share bits 6..15, so their counters sit in
        // one half of 64 words that differ in a fixed mix of the low five bits.
        const uint32_t hi = 65535u - (uint32_t)tid * kHistPerThread;
        const uint32_t mix = (hi >> 6) & 31u, half_shift = (hi >> 15) * 16u;
        auto count_of = [&](uint32_t key) -> uint32_t {
            return (hist[(key & 0x7FFFu) ^ mix] >> half_shift) & 0xFFFFu;
        };
        // count * 2^((value - max) log2 e / T): the exponent in double, its integer part applied as a
        // power of two, 2^fraction from the special-function unit (to about 1e-7 of the bin's mass)
        auto mass_of = [&](uint32_t key, uint32_t c) -> double {
            const double t = (double)(fmaxf(KeyT::value(key), kFloor) - m) * p.c1;
            if (t < -1000.0) return 0.0;
            const double ti = floor(t);
            const double w = (double)ex2((float)(t - ti));
            return (double)c * __longlong_as_double((long long)(1023 + (int)ti) << 52) * w;
        };
        // inclusive prefixes over the threads (thread order = descending keys) into sh.incl_c / incl_m
        auto block_prefix = [&](long long c, double ms) {
            long long ci = c;
            double mi = ms;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const long long tc = __shfl_up_sync(0xFFFFFFFFu, ci, o);
                const double tm = __shfl_up_sync(0xFFFFFFFFu, mi, o);
                if (lane >= o) {
                    ci += tc;
                    mi += tm;
                }
            }
            __syncthreads();                // (whatever read the tables before is done)
            if (lane == 31) {
                sh.wcnt[warp] = ci;
                sh.wmass[warp] = mi;
            }
            if (tid == 0) sh.owner = kHistThreads;
            __syncthreads();
            long long cb = 0;
            double mb = 0.0;
            for (int w = 0; w < warp; ++w) {
                cb += sh.wcnt[w];
                mb += sh.wmass[w];
            }
            sh.incl_c[tid] = cb + ci;
            sh.incl_m[tid] = mb + mi;
            __syncthreads();
        };

        long long lc = 0;
        for (int q = 0; q < kHistPerThread; ++q) lc += count_of(hi - q);
        block_prefix(lc, 0.0);
        if (sh.incl_c[kHistThreads - 1] != (long long)p.V) {     // a counter wrapped: left to the radix kernel
            if (tid == 0) *out = __int_as_float(0x7FC00000);
            __syncthreads();
            continue;
        }
        if (use_k) {
            const long long c_ex = tid ? sh.incl_c[tid - 1] : 0;
            if (c_ex < p.top_k && sh.incl_c[tid] >= p.top_k) {   // exactly one thread: the counts are integers
                long long run = c_ex;
                for (int q = 0; q < kHistPerThread; ++q) {
                    run += count_of(hi - q);
                    if (run >= p.top_k) {
                        sh.key_k = hi - q;
                        break;
                    }
                }
            }
            __syncthreads();
        }
        const uint32_t key_k = sh.key_k;                 // 0: top-k is off
        uint32_t key_cut = key_k;
        if (use_p) {
            // masses of this thread's bins among what top-k left
            double lm = 0.0;
            if (lc && hi >= key_k)
                for (int q = 0; q < kHistPerThread; ++q) {
                    const uint32_t key = hi - q, c = count_of(key);
                    if (c && key >= key_k) lm += mass_of(key, c);
                }
            block_prefix(0, lm);
            // top_p of the mass top-k left; the first thread whose prefix reaches it holds the cut
            const double thr = (double)p.top_p * sh.incl_m[kHistThreads - 1];
            if (sh.incl_m[tid] >= thr) atomicMin(&sh.owner, tid);
            __syncthreads();
            if (tid == sh.owner) {
                double run = tid ? sh.incl_m[tid - 1] : 0.0;
                uint32_t found = 0u, last = 0u;
                for (int q = 0; q < kHistPerThread && !found; ++q) {
                    const uint32_t key = hi - q, c = count_of(key);
                    if (!c || key < key_k) continue;
                    last = key;
                    run += mass_of(key, c);
                    if (run >= thr) found = key;
                }
                // (rounding between the prefix and the walk: the last bin with mass, or, if this
                // thread has none, everything below the threads before it)
                sh.key_p = found ? found : (last ? last : hi);
            }
            __syncthreads();
            key_cut = max(key_k, sh.key_p);
        }
        if (tid == 0) *out = key_cut ? KeyT::value(key_cut) : -INFINITY;
        __syncthreads();
    }
}

}  // namespace adasd
