// Building blocks of the streaming kernels for sm_100a: mbarrier and bulk-copy (cp.async.bulk)
// wrappers with bounded waits, packed bf16 helpers, and the small records the warps of a
// cluster exchange (per-slice softmax statistics, position references).
#pragma once

#include "adasd_device.cuh"
#include "adasd_rows.cuh"
#include "adasd_tail.cuh"

namespace adasd {

constexpr int kCW = 12;                         // warps per CTA, at most (sizes the exchange tables)
constexpr int kCMaxCluster = 8;
constexpr int kCMaxG = kCMaxCluster * kCW;      // warps per cluster, at most
constexpr int kCTab = 128;                      // entries of the per-warp tables (4 per lane)
static_assert(kCMaxG <= kCTab, "per-warp tables hold one entry per warp of the cluster");
constexpr uint32_t kCWaitSpins = 1u << 22;      // polls of an mbarrier before a wait gives up
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
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, uint32_t spins = kCWaitSpins) {
    for (uint32_t it = 0; it < spins; ++it)
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
// Top-k / top-p cut of the adjusted distribution on a packed pair: a half below the row's cutoff
// (cut2: the cutoff in both halves) becomes the floor value, i.e. probability 0; a NaN is not
// below anything and stays.  kNoCut2 (-inf, -inf) cuts nothing.
constexpr uint32_t kNoCut2 = 0xFF80FF80u;
__device__ __forceinline__ uint32_t bcut2(uint32_t a, uint32_t cut2) {
    uint32_t m;
    asm("set.lt.u32.bf16x2 %0, %1, %2;" : "=r"(m) : "r"(a), "r"(cut2));   // 0xFFFF per half that is below
    return (a & ~m) | (0xF149F149u & m);
}
__device__ __forceinline__ void bcut8(uint4& w, uint32_t cut2) {
    w.x = bcut2(w.x, cut2);
    w.y = bcut2(w.y, cut2);
    w.z = bcut2(w.z, cut2);
    w.w = bcut2(w.w, cut2);
}
// the cutoff of a bf16 row (a bf16 value, or -inf) as a packed pair
__device__ __forceinline__ uint32_t cut_pair(float cut) {
    const uint32_t h = __float_as_uint(cut) >> 16;
    return h | (h << 16);
}
__device__ __forceinline__ float2 unpack2(uint32_t w) {
    return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xFFFF0000u));
}

struct ClusterGeom {
    int32_t ncl;         // clusters in the grid
};

// Partial (or total) softmax statistics of both rows over some slice of the vocabulary:
// maxima, S = sum 2^t, T = sum 2^t t with t = (z - max) log2 e.
struct __align__(16) RowPart {
    float mt, St, Tt, md;
    float Sd, Td;
    uint32_t flags;      // 1: NaN / +inf / expired wait, 2: the rows differ
    float pad;
};

struct PosRef {
    int pos;   // index into [B, Kmax+1]; >= total means "none"
    int kt;    // window K_t of its sequence
};

}  // namespace adasd
